// Shared declarations of the TWA CUDA library: context, workspace layout, device-side
// status reporting, and thin wrappers over the mbarrier / bulk-tensor-copy PTX used by the
// streaming kernels.  sm_100a only.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "twa.h"

// ------------------------------------------------------------------------------------------
// Host-side context
// ------------------------------------------------------------------------------------------
typedef CUresult (*twa_encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                        const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                        const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                        CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct twa_ctx {
  int device;
  cudaStream_t stream;
  int sm_count;
  int smem_optin;             // largest dynamic shared memory a block may request
  int* d_status;              // [0] first error code, [1] its detail
  unsigned int* d_ticket;     // block-completion counters, zero between kernels
  twa_encode_tiled_fn encode_tiled;
  unsigned long long wait_limit_ns;
  int tune_project_warps, tune_lift_warps, tune_stages;
  int tune_dequant_path;      // 0 = integer tensor-pipe dot products, 1 = float FMA
  int tune_tile_segments;     // tensor-pipe path: 512-byte segments per tile column (0 = choose)
  int tune_build_panel;       // resident basis build: 0 = panels of 8 columns, Gram form inside; 1 = column by column; 2 = panels, column sweeps inside
  int tune_lift_base_path;    // tensor-pipe lift, base / output vectors: 0 = choose, 1 = lanes, 2 = base through the ring, 3 = both
  int tune_slab_rows;         // stepping calls: rows per launch (0 = one launch up to TWA_MAX_LAUNCH_ROWS, slabs of 2^30 above)
  cudaEvent_t* prof_events;   // 3 per recorded step, or null
  int prof_cap, prof_count;   // steps
  // state of a row-chunked basis build (twa_build_begin .. twa_build_end_pass)
  long long build_D;
  int build_n;
  float* build_wbar;
  char* build_ws;
  // twa_step_host: a second stream for the host copies and the events that order it with `stream`
  // (created by the first call that needs them)
  cudaStream_t copy_stream;
  cudaEvent_t* copy_events;   // 2 * TWA_HOST_CHUNKS + 2
  char last_error[256];
};

#define TWA_CUDA_OK(ctx, expr)                                                              \
  do {                                                                                      \
    cudaError_t e__ = (expr);                                                               \
    if (e__ != cudaSuccess) {                                                               \
      snprintf((ctx)->last_error, sizeof((ctx)->last_error), "%s: %s", #expr,               \
               cudaGetErrorString(e__));                                                    \
      return TWA_ERR_CUDA;                                                                  \
    }                                                                                       \
  } while (0)

// ------------------------------------------------------------------------------------------
// Workspace layout (bytes from the start of `ws`)
// ------------------------------------------------------------------------------------------
constexpr int TWA_MAX_GRID = 1024;                       // upper bound on blocks of a reduction
constexpr size_t TWA_WS_PARTIALS = 0;                    // float [TWA_MAX_GRID][TWA_MAX_N]
constexpr size_t TWA_WS_COEF = TWA_WS_PARTIALS + sizeof(float) * TWA_MAX_GRID * TWA_MAX_N;
                                                         // float [TWA_MAX_N]  projection coefficients
constexpr size_t TWA_WS_NORMS = TWA_WS_COEF + sizeof(float) * TWA_MAX_N;
                                                         // double[4]: 0 = |a_j|^2, 1 = |v|^2
constexpr size_t TWA_WS_DPART = TWA_WS_NORMS + 64;       // double [TWA_MAX_GRID] partial sums
constexpr size_t TWA_WS_ABSMAX = TWA_WS_DPART + sizeof(double) * TWA_MAX_GRID;
                                                         // uint  [TWA_MAX_N]  bit patterns of column absmax
constexpr int TWA_HOST_CHUNKS = 16;                      // row chunks of twa_step_host at most
constexpr size_t TWA_WS_CHUNK_COEF = TWA_WS_ABSMAX + sizeof(unsigned) * TWA_MAX_N;
                                                         // float [TWA_HOST_CHUNKS][TWA_MAX_N]  per-chunk projections
constexpr int TWA_PANEL_SUMSQ_BLOCKS = 256;              // blocks of the panel projection at most
constexpr size_t TWA_WS_PANEL_SUMSQ = TWA_WS_CHUNK_COEF + sizeof(float) * TWA_HOST_CHUNKS * TWA_MAX_N;
                                                         // double [TWA_PANEL_SUMSQ_BLOCKS][8]  squared norms of a panel's columns
constexpr size_t TWA_WS_BYTES = TWA_WS_PANEL_SUMSQ + sizeof(double) * TWA_PANEL_SUMSQ_BLOCKS * 8;

// ------------------------------------------------------------------------------------------
// Streaming-kernel geometry
// ------------------------------------------------------------------------------------------
constexpr int TWA_TILE_COL_BYTES = 512;                  // bytes of one column inside one tile
constexpr int TWA_TILE_COL_WORDS = TWA_TILE_COL_BYTES / 4;
constexpr int TWA_MAX_STAGES = 16;
constexpr int TWA_MAX_CONSUMER_WARPS = 20;
constexpr int TWA_MAX_THREADS = (TWA_MAX_CONSUMER_WARPS + 1) * 32;
constexpr int TWA_PROJECT_CPW = 8;                       // columns one warp owns at most (project)
constexpr int TWA_LIFT_CPW = 16;                         // columns one warp owns at most (lift)
constexpr int TWA_SMEM_HEADER = 2048;                    // barriers + small arrays before the ring

// rows covered by one tile for a storage width
__host__ __device__ constexpr int twa_tile_rows(int bits) { return TWA_TILE_COL_BYTES * 8 / bits; }

// Storage order of 8- and 4-bit codes inside a column.  Every aligned 512-byte segment of a
// column holds its 32 chunks of 16 bytes permuted: logical chunk c sits in slot
// (c & 24) | ((c ^ j) & 7), j the column index.  In shared memory, where a tile is
// [n columns][512 bytes], the same chunk of eight neighbouring columns then falls into eight
// different bank groups, so 8 x 16-byte matrix loads across columns are conflict-free, while
// global memory and the TMA copies keep 512 contiguous bytes per column and tile.
__host__ __device__ __forceinline__ int twa_chunk_slot(int c, int j) { return (c & 24) | ((c ^ j) & 7); }

// First bytes of every streaming kernel's shared memory.
struct twa_smem_header {
  unsigned long long full[TWA_MAX_STAGES];    // stage filled by the producer's copies
  unsigned long long empty[TWA_MAX_STAGES];   // stage released by every consumer warp
  int abort_flag;                             // a bounded wait ran out somewhere in the block
  int last_flag;                              // this block finished last (project)
  int bad_flag;                               // non-finite input met
  unsigned amax_bits;                         // lift: bit pattern of max |coefficient|
  float digit_scale[4];                       // lift: weight of each coefficient digit
  int pad[54];
  float c_part[TWA_MAX_N];                    // project: this block's column sums
};
static_assert(sizeof(twa_smem_header) <= TWA_SMEM_HEADER, "header too large");

// ------------------------------------------------------------------------------------------
// Device helpers
// ------------------------------------------------------------------------------------------
#ifdef __CUDACC__

__device__ __forceinline__ void twa_set_status(int* status, int code, int detail) {
  if (atomicCAS(&status[0], 0, code) == 0) status[1] = detail;
}

__device__ __forceinline__ uint32_t twa_smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ unsigned long long twa_globaltimer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void twa_mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void twa_fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void twa_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}

__device__ __forceinline__ void twa_mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ uint32_t twa_mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}

// Waits for the phase `parity` of an mbarrier, for at most `limit_ns`.  Returns false when
// the wait ran out or another thread of the block already gave up (*abort_flag != 0); the
// caller then leaves its loop.  The first thread to give up raises the flag.
__device__ __forceinline__ bool twa_mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                              unsigned long long limit_ns) {
  for (int i = 0; i < 64; ++i)
    if (twa_mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = twa_globaltimer();
  for (;;) {
    for (int i = 0; i < 64; ++i)
      if (twa_mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (twa_globaltimer() - t0 > limit_ns) {
      *abort_flag = 1;
      return false;
    }
  }
}

// Called by the thread that filled a ring of `stages` stages `issued` times, once it has issued its
// last copy: waits (for at most `limit_ns` per stage) until the newest fill of every stage has
// landed, so that no bulk copy is still writing this block's shared memory when the block reuses the
// ring or exits -- also when the consumers gave up on a wait of their own.  Returns false if a
// fill did not land in time.
__device__ __forceinline__ bool twa_drain_ring(twa_smem_header* hdr, int issued, int stages,
                                               unsigned long long limit_ns) {
  bool landed = true;
  const int live = issued < stages ? issued : stages;
  for (int q = 0; q < live; ++q) {
    const int last = ((issued - 1 - q) / stages) * stages + q;   // newest fill of stage q
    const unsigned par = static_cast<unsigned>(last / stages) & 1u;
    const uint32_t bar = twa_smem_u32(&hdr->full[q]);
    if (twa_mbar_try_wait(bar, par)) continue;
    const unsigned long long t0 = twa_globaltimer();
    while (!twa_mbar_try_wait(bar, par)) {
      if (twa_globaltimer() - t0 > limit_ns) {
        landed = false;
        break;
      }
    }
  }
  return landed;
}

// Bulk tensor copies global -> this block's shared memory, completion counted on an mbarrier.
__device__ __forceinline__ void twa_tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y,
                                                uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void twa_tma_load_1d(uint32_t dst, const CUtensorMap* map, int x,
                                                uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.1d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2}], [%3];"
      ::"r"(dst), "l"(map), "r"(x), "r"(bar)
      : "memory");
}

// Bulk tensor store from this block's shared memory, clipped by the tensor map; completion is
// tracked by the issuing thread's bulk async-group.
__device__ __forceinline__ void twa_tma_store_1d(const CUtensorMap* map, int x, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.1d.global.shared::cta.bulk_group [%0, {%1}], [%2];"
               ::"l"(map), "r"(x), "r"(src)
               : "memory");
}

__device__ __forceinline__ void twa_bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }

// Waits until all but the newest N bulk groups of this thread have finished reading shared memory.
template <int N>
__device__ __forceinline__ void twa_bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}

// Orders this thread's earlier shared-memory writes before later reads by the bulk-copy engine.
__device__ __forceinline__ void twa_fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void twa_prefetch_tensormap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void twa_named_barrier(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// ---- code -> float ------------------------------------------------------------------------
// Float path: a two's-complement byte (nibble) becomes offset binary by flipping its top bit;
// a byte u in [0,255] placed in the low mantissa bits of 2^23 gives the float 2^23 + u exactly;
// subtracting 2^23 + bias leaves the signed code as a float.
__device__ __forceinline__ float twa_byte_to_float(uint32_t word, int byte, float magic) {
  const uint32_t sel = 0x7440u + static_cast<uint32_t>(byte);
  return __uint_as_float(__byte_perm(word, 0x4B000000u, sel)) - magic;
}
constexpr float TWA_MAGIC_I8 = 8388608.0f + 128.0f;
constexpr float TWA_MAGIC_I4 = 8388608.0f + 8.0f;

// One element of the quantiser: IEEE float32 quotient, round half to even, clamp to +-qmax.
// qmax is an integer, so clamping first gives the same code; adding 1.5 * 2^23 then rounds the clamped
// quotient to an integer, half to even, in the float adder and leaves the code in the low bits of the
// sum's pattern (the rounding and conversion instructions run at a quarter of the adder's rate, and
// three of them per element held the encoding pass at half the memory rate).  A NaN quotient clamps to
// -qmax either way.
__device__ __forceinline__ int twa_encode_one(float p, float s, float qmax) {
  if (s == 0.0f) return 0;
  const float q = fminf(fmaxf(__fdiv_rn(p, s), -qmax), qmax);
  return __float_as_int(q + 12582912.0f) - 0x4B400000;
}

__device__ __forceinline__ float twa_bf16_lo(uint32_t pair) { return __uint_as_float(pair << 16); }
__device__ __forceinline__ float twa_bf16_hi(uint32_t pair) { return __uint_as_float(pair & 0xFFFF0000u); }

#endif  // __CUDACC__

// Adam moments and constants for the coefficient update (m == null: plain gradient descent).
// bc1 = 1 - beta1^t and bc2 = 1 - beta2^t for the 1-based step t, computed on the host.
struct twa_adam_args {
  float* m;
  float* v;
  float beta1, beta2, eps, bc1, bc2;
};

#ifdef __CUDACC__
// The optimiser step on one coefficient after the projection gave its gradient c:
//   gradient descent  x <- (1 - lr*lambda) x - lr c                      (Section 4.2, Algorithm 1)
//   Adam, decoupled decay  m <- b1 m + (1-b1) c,  v <- b2 v + (1-b2) c^2,
//                          x <- (1 - lr*lambda) x - lr (m/bc1) / (sqrt(v/bc2) + eps)
// in float64 on float32 state; idx addresses the moments.
__device__ __forceinline__ float twa_coefficient_update(float x, double c, float lr, float lambda,
                                                        const twa_adam_args& ad, size_t idx) {
  const double decay = 1.0 - static_cast<double>(lr) * static_cast<double>(lambda);
  if (!ad.m) return static_cast<float>(decay * static_cast<double>(x) - static_cast<double>(lr) * c);
  const double b1 = ad.beta1, b2 = ad.beta2;
  const double m = b1 * static_cast<double>(ad.m[idx]) + (1.0 - b1) * c;
  const double v = b2 * static_cast<double>(ad.v[idx]) + (1.0 - b2) * c * c;
  ad.m[idx] = static_cast<float>(m);
  ad.v[idx] = static_cast<float>(v);
  const double step = (m / static_cast<double>(ad.bc1)) / (sqrt(v / static_cast<double>(ad.bc2)) + static_cast<double>(ad.eps));
  return static_cast<float>(decay * static_cast<double>(x) - static_cast<double>(lr) * step);
}
#endif

// ------------------------------------------------------------------------------------------
// Internal launchers (defined in the .cu files)
// ------------------------------------------------------------------------------------------
struct twa_project_epilogue {
  float* c_out;        // n floats or null
  float* alpha;        // when non-null: alpha <- (1 - lr*lambda) alpha - lr c, or the Adam step below
  float lr, lambda;
  int nonfinite_detail; // detail reported with TWA_ERR_NONFINITE; -1 = index of the coefficient
  twa_adam_args adam;  // m == null: plain gradient descent
};

int twa_launch_project(twa_ctx* ctx, const twa_basis* P, const void* g, twa_dtype g_dtype,
                       const twa_project_epilogue& epi, void* ws);
int twa_launch_lift(twa_ctx* ctx, const twa_basis* P, const float* alpha, float alpha_mult,
                    const float* base, float* out, bool reverse_tiles);
int twa_check_basis(const twa_basis* P);
// Panel steps of the blocked basis build on the float32 matrix W (columns of stride ldw):
// C = Q^T A_p into the workspace, then A_p <- A_p - Q C; Q = columns 0..nq-1, A_p = the next pb <= 8.
// sumsq_out (device, 8 doubles) or null: the squared norms of the panel's columns as the projection read them.
int twa_launch_panel_project(twa_ctx* ctx, float* W, long long D, long long ldw, int nq, int pb, void* ws,
                             double* sumsq_out);
// given (device, 8 doubles) or null: with it the update also takes the Gram matrix of the panel as stored
// and leaves the factor of the panel's own Gram-Schmidt for twa_launch_panel_apply (rank and finiteness
// tests against `given`, or against the Gram matrix's diagonal, which then replaces `given`).
int twa_launch_panel_lift(twa_ctx* ctx, float* W, long long D, long long ldw, int nq, int pb, void* ws, double* given,
                          bool given_from_diagonal);
// The same factor from a pass over the panel (for a panel the update did not just store).
int twa_launch_panel_gram(twa_ctx* ctx, float* W, long long D, long long ldw, int j0, int pb, void* ws, double* given,
                          bool given_from_diagonal);
// A_p <- A_p T; absmax (device, one word per panel column) or null: largest magnitudes stored, as bit patterns.
int twa_launch_panel_apply(twa_ctx* ctx, float* W, long long D, long long ldw, int j0, int pb, void* ws,
                           unsigned* absmax);
// Validates the optimiser constants and fills the kernel-side Adam arguments (bias corrections for opt->step).
int twa_adam_device_args(const twa_adam* opt, float* m, float* v, twa_adam_args* out);
// scales[j] = absmax_j / qmax from the bit patterns of the column maxima; flags NaN/Inf
int twa_launch_scales(twa_ctx* ctx, const unsigned* absmax, int n, int bits, float* scales);
// Variants of the two launchers for 8- and 4-bit storage that compute the integer dot
// products on the tensor pipe (twa_stream_mma.cu).
int twa_launch_project_mma(twa_ctx* ctx, const twa_basis* P, const void* g, twa_dtype g_dtype,
                           const twa_project_epilogue& epi, void* ws);
int twa_launch_lift_mma(twa_ctx* ctx, const twa_basis* P, const float* alpha, float alpha_mult,
                        const float* base, float* out, bool reverse_tiles);
// Sets the dynamic shared memory limit of a kernel only when it has to grow.
int twa_ensure_smem(twa_ctx* ctx, const void* kernel, int* current, int wanted);
