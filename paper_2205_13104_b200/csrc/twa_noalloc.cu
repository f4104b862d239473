// Projection for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc at the point where they need a
// projection: code running between the start and end of a region in which the CUDA
// allocator is off limits (a caching allocator that owns all device memory, a real-time
// loop that forbids calls which may synchronise the device, a plug-in handed only its input
// and output buffers).  twa_project needs two things from an allocator: the context's status
// word (twa_create allocates it) and the caller's workspace.  twa_project_noalloc needs
// neither: its scratch -- the per-block partial sums, the completion counter and a status
// word -- lives in a fixed array in the library's device image.
#include <mutex>
#include <stdio.h>
#include <string.h>

#include "twa_common.cuh"

namespace {

constexpr int NOALLOC_MAX_GRID = 256;                       // blocks whose partials fit
constexpr size_t NOALLOC_PARTIALS_BYTES = sizeof(float) * NOALLOC_MAX_GRID * TWA_MAX_N;
constexpr size_t NOALLOC_STATUS_OFF = NOALLOC_PARTIALS_BYTES;          // int[2]
constexpr size_t NOALLOC_TICKET_OFF = NOALLOC_PARTIALS_BYTES + 128;    // unsigned
constexpr size_t NOALLOC_SCRATCH_BYTES = NOALLOC_PARTIALS_BYTES + 256; // 131,328 bytes

// Every GPU that loads the library holds this array until the process exits.  In host code
// the name below is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char twa_noalloc_scratch[NOALLOC_SCRATCH_BYTES];

struct DeviceSetup {
  bool ready;
  unsigned char* scratch;      // device address of twa_noalloc_scratch on this device
  int sm_count, smem_optin;
  twa_encode_tiled_fn encode_tiled;
};

constexpr int MAX_DEVICES = 64;
DeviceSetup g_setup[MAX_DEVICES];
std::mutex g_setup_lock;
// Text of the calling thread's last rejected call ("" after a call that was accepted).
thread_local char g_noalloc_error[256] = "";

int reject(int code, const char* why) {
  snprintf(g_noalloc_error, sizeof(g_noalloc_error), "%s", why);
  return code;
}

int fail(int code, const char* what, cudaError_t e) {
  snprintf(g_noalloc_error, sizeof(g_noalloc_error), "%s: %s", what, cudaGetErrorString(e));
  return code;
}

// Once per device, with that device current.
int setup_device(int device, DeviceSetup** out) {
  std::lock_guard<std::mutex> guard(g_setup_lock);
  DeviceSetup& s = g_setup[device];
  if (!s.ready) {
    void* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, twa_noalloc_scratch);
    if (e != cudaSuccess || !ptr) return fail(TWA_ERR_CUDA, "cudaGetSymbolAddress(scratch)", e);
    int major = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device);
    if (e != cudaSuccess) return fail(TWA_ERR_CUDA, "cudaDeviceGetAttribute", e);
    if (major != 10) {
      snprintf(g_noalloc_error, sizeof(g_noalloc_error), "device %d is not sm_100", device);
      return TWA_ERR_UNSUPPORTED;
    }
    e = cudaDeviceGetAttribute(&s.sm_count, cudaDevAttrMultiProcessorCount, device);
    if (e != cudaSuccess) return fail(TWA_ERR_CUDA, "cudaDeviceGetAttribute", e);
    e = cudaDeviceGetAttribute(&s.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
    if (e != cudaSuccess) return fail(TWA_ERR_CUDA, "cudaDeviceGetAttribute", e);
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
    if (e != cudaSuccess || !fn || q != cudaDriverEntryPointSuccess)
      return fail(TWA_ERR_CUDA, "cudaGetDriverEntryPoint(cuTensorMapEncodeTiled)", e);
    s.encode_tiled = reinterpret_cast<twa_encode_tiled_fn>(fn);
    s.scratch = static_cast<unsigned char*>(ptr);
    s.ready = true;
  }
  *out = &s;
  return TWA_OK;
}

}  // namespace

extern "C" {

int twa_project_noalloc(int device, void* cuda_stream, const twa_basis* P, const void* g,
                        twa_dtype g_dtype, float* c_out, int* status_out) {
  g_noalloc_error[0] = 0;
  if (!P || !g || !c_out) return reject(TWA_ERR_INVALID_ARG, "P, g and c_out must not be null");
  if (device < 0 || device >= MAX_DEVICES) return reject(TWA_ERR_INVALID_ARG, "device index out of range");
  if (g_dtype != TWA_F32 && g_dtype != TWA_BF16) return reject(TWA_ERR_INVALID_ARG, "g_dtype is neither TWA_F32 nor TWA_BF16");
  if (P->n > TWA_MAX_N) {
    snprintf(g_noalloc_error, sizeof(g_noalloc_error),
             "n = %d exceeds the %d columns the static scratch holds", P->n, TWA_MAX_N);
    return TWA_ERR_UNSUPPORTED;
  }
  int rc = twa_check_basis(P);
  if (rc) return reject(rc, "the basis descriptor is not valid (sizes, width, alignment)");
  if (reinterpret_cast<uintptr_t>(g) & 15) return reject(TWA_ERR_MISALIGNED, "g is not 16-byte aligned");
  cudaError_t e = cudaSetDevice(device);
  if (e != cudaSuccess) return fail(TWA_ERR_CUDA, "cudaSetDevice", e);
  DeviceSetup* s = nullptr;
  rc = setup_device(device, &s);
  if (rc) return rc;

  // A context that lives on this stack frame only; nothing in it is allocated.
  twa_ctx ctx;
  memset(&ctx, 0, sizeof(ctx));
  ctx.device = device;
  ctx.stream = static_cast<cudaStream_t>(cuda_stream);
  ctx.sm_count = s->sm_count < NOALLOC_MAX_GRID ? s->sm_count : NOALLOC_MAX_GRID;
  ctx.smem_optin = s->smem_optin;
  ctx.d_status = reinterpret_cast<int*>(s->scratch + NOALLOC_STATUS_OFF);
  ctx.d_ticket = reinterpret_cast<unsigned*>(s->scratch + NOALLOC_TICKET_OFF);
  ctx.encode_tiled = s->encode_tiled;
  ctx.wait_limit_ns = 2000ull * 1000ull * 1000ull;

  // The scratch keeps what the previous call left: the counter and the status must start at 0.
  e = cudaMemsetAsync(s->scratch + NOALLOC_STATUS_OFF, 0, 256, ctx.stream);
  if (e != cudaSuccess) return fail(TWA_ERR_CUDA, "cudaMemsetAsync(scratch)", e);
  twa_project_epilogue epi = {c_out, nullptr, 0.0f, 0.0f, -1};
  rc = twa_launch_project(&ctx, P, g, g_dtype, epi, s->scratch);
  if (rc) {
    snprintf(g_noalloc_error, sizeof(g_noalloc_error), "%s", ctx.last_error);
    return rc;
  }
  if (status_out) {
    e = cudaMemcpyAsync(status_out, ctx.d_status, 2 * sizeof(int), cudaMemcpyDeviceToDevice, ctx.stream);
    if (e != cudaSuccess) return fail(TWA_ERR_CUDA, "cudaMemcpyAsync(status)", e);
  }
  return TWA_OK;
}

const char* twa_noalloc_last_error(void) { return g_noalloc_error; }

size_t twa_noalloc_scratch_bytes(void) { return NOALLOC_SCRATCH_BYTES; }

}  // extern "C"
