// C entry points: context, status, and the per-step calls (project, lift, step).
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "twa_common.cuh"
#include "twa_slabs.cuh"

namespace {

int check_ws(const void* ws, size_t ws_bytes) {
  if (!ws || ws_bytes < TWA_WS_BYTES) return TWA_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(ws) & 15) return TWA_ERR_MISALIGNED;
  return TWA_OK;
}

bool misaligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) != 0; }

}  // namespace

namespace {
// One block waits, with the library's bounded wait, for an mbarrier phase that nothing completes.
__global__ void wait_selftest_kernel(int* status, unsigned long long limit_ns) {
  __shared__ unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    twa_mbar_init(twa_smem_u32(&bar), 1);
    abort_flag = 0;
    twa_fence_barrier_init();
  }
  __syncthreads();
  if (!twa_mbar_wait(twa_smem_u32(&bar), 0, &abort_flag, limit_ns)) {
    if (threadIdx.x == 0) twa_set_status(status, TWA_ERR_TIMEOUT, -1);
  }
}
}  // namespace

namespace {
// twa_step_host and the row slabs of a basis of 2^31 rows or more: the coefficients' gradient is the
// sum of the chunks' projections (float64, chunk order); written to c_out when that is non-null,
// and followed by the update of Algorithm 1 (or the Adam step) when alpha is.  One block of
// TWA_MAX_N threads.
__global__ void chunk_combine_kernel(const float* __restrict__ chunk_c, int chunks, int n, float* c_out, float* alpha,
                                     float lr, float lambda, twa_adam_args adam, int* status) {
  const int j = threadIdx.x;
  double c = 0.0;
  if (j < n)
    for (int k = 0; k < chunks; ++k) c += static_cast<double>(chunk_c[static_cast<size_t>(k) * TWA_MAX_N + j]);
  if (j < n && !isfinite(c)) twa_set_status(status, TWA_ERR_NONFINITE, j);
  if (j < n && c_out) c_out[j] = static_cast<float>(c);
  // alpha stays as it was when the projection is unusable (see twa_step)
  const int unusable = __syncthreads_or(!isfinite(c)) | (__ldcg(status) == TWA_ERR_TIMEOUT);
  if (j < n && alpha && !unusable) alpha[j] = twa_coefficient_update(alpha[j], c, lr, lambda, adam, j);
}

// Projection of every slab into its slot of ws, then the combine (and the optimiser step, if any).
int project_slabs(twa_ctx* ctx, const twa_basis* P, const void* g, twa_dtype g_dtype, const twa_project_epilogue& epi,
                  void* ws) {
  const SlabPlan plan = slab_plan(ctx, P->D);
  const int slabs = plan.count;
  const size_t gsz = g_dtype == TWA_BF16 ? 2 : 4;
  float* slab_c = reinterpret_cast<float*>(static_cast<char*>(ws) + TWA_WS_CHUNK_COEF);
  for (int k = 0; k < slabs; ++k) {
    long long r0;
    const twa_basis v = slab_view(P, plan, k, &r0);
    twa_project_epilogue part = {slab_c + static_cast<size_t>(k) * TWA_MAX_N, nullptr, 0.0f, 0.0f, -1};
    int rc = twa_launch_project(ctx, &v, static_cast<const char*>(g) + r0 * gsz, g_dtype, part, ws);
    if (rc) return rc;
  }
  chunk_combine_kernel<<<1, TWA_MAX_N, 0, ctx->stream>>>(slab_c, slabs, P->n, epi.c_out, epi.alpha, epi.lr, epi.lambda,
                                                         epi.adam, ctx->d_status);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}

// Lift of every slab, last slab first when the projection has just run (its rows are the likeliest in L2).
int lift_slabs(twa_ctx* ctx, const twa_basis* P, const float* alpha, const float* base, float* out, bool reverse) {
  const SlabPlan plan = slab_plan(ctx, P->D);
  const int slabs = plan.count;
  for (int i = 0; i < slabs; ++i) {
    const int k = reverse ? slabs - 1 - i : i;
    long long r0;
    const twa_basis v = slab_view(P, plan, k, &r0);
    int rc = twa_launch_lift(ctx, &v, alpha, 1.0f, base ? base + r0 : nullptr, out + r0, reverse);
    if (rc) return rc;
  }
  return TWA_OK;
}
}  // namespace

int twa_adam_device_args(const twa_adam* opt, float* m, float* v, twa_adam_args* out) {
  if (!opt || !m || !v || !out) return TWA_ERR_INVALID_ARG;
  if (opt->step < 1 || !(opt->beta1 >= 0.0f && opt->beta1 < 1.0f) || !(opt->beta2 >= 0.0f && opt->beta2 < 1.0f) ||
      !(opt->eps >= 0.0f))
    return TWA_ERR_INVALID_ARG;
  out->m = m;
  out->v = v;
  out->beta1 = opt->beta1;
  out->beta2 = opt->beta2;
  out->eps = opt->eps;
  out->bc1 = static_cast<float>(1.0 - pow(static_cast<double>(opt->beta1), opt->step));
  out->bc2 = static_cast<float>(1.0 - pow(static_cast<double>(opt->beta2), opt->step));
  return TWA_OK;
}

extern "C" {

int twa_selftest_wait(twa_ctx* ctx) {
  if (!ctx) return TWA_ERR_INVALID_ARG;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  wait_selftest_kernel<<<1, 64, 0, ctx->stream>>>(ctx->d_status, ctx->wait_limit_ns);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}

int twa_create(twa_ctx** out, int device, void* cuda_stream) {
  if (!out) return TWA_ERR_INVALID_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count)
    return TWA_ERR_INVALID_ARG;
  twa_ctx* ctx = static_cast<twa_ctx*>(calloc(1, sizeof(twa_ctx)));
  if (!ctx) return TWA_ERR_INVALID_ARG;
  ctx->device = device;
  ctx->stream = static_cast<cudaStream_t>(cuda_stream);
  ctx->wait_limit_ns = 2000ull * 1000ull * 1000ull;
  int rc = [&]() -> int {
    TWA_CUDA_OK(ctx, cudaSetDevice(device));
    cudaDeviceProp prop;
    TWA_CUDA_OK(ctx, cudaGetDeviceProperties(&prop, device));
    if (prop.major != 10) {
      snprintf(ctx->last_error, sizeof(ctx->last_error),
               "device %d is compute capability %d.%d; this library is built for sm_100a only",
               device, prop.major, prop.minor);
      return TWA_ERR_UNSUPPORTED;
    }
    ctx->sm_count = prop.multiProcessorCount;
    ctx->smem_optin = static_cast<int>(prop.sharedMemPerBlockOptin);
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    TWA_CUDA_OK(ctx, cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
    if (!fn || qres != cudaDriverEntryPointSuccess) {
      snprintf(ctx->last_error, sizeof(ctx->last_error), "cuTensorMapEncodeTiled not found in the driver");
      return TWA_ERR_CUDA;
    }
    ctx->encode_tiled = reinterpret_cast<twa_encode_tiled_fn>(fn);
    void* d = nullptr;
    TWA_CUDA_OK(ctx, cudaMalloc(&d, 256));
    TWA_CUDA_OK(ctx, cudaMemset(d, 0, 256));
    ctx->d_status = static_cast<int*>(d);
    ctx->d_ticket = reinterpret_cast<unsigned*>(static_cast<char*>(d) + 128);
    return TWA_OK;
  }();
  if (rc != TWA_OK) {
    fprintf(stderr, "twa_create: %s\n", ctx->last_error);
    if (ctx->d_status) cudaFree(ctx->d_status);
    free(ctx);
    return rc;
  }
  *out = ctx;
  return TWA_OK;
}

void twa_destroy(twa_ctx* ctx) {
  if (!ctx) return;
  cudaSetDevice(ctx->device);
  cudaStreamSynchronize(ctx->stream);
  if (ctx->prof_events) {
    for (int i = 0; i < 3 * ctx->prof_cap; ++i) cudaEventDestroy(ctx->prof_events[i]);
    free(ctx->prof_events);
  }
  if (ctx->copy_events) {
    cudaStreamSynchronize(ctx->copy_stream);
    for (int i = 0; i < 2 * TWA_HOST_CHUNKS + 2; ++i) cudaEventDestroy(ctx->copy_events[i]);
    free(ctx->copy_events);
    cudaStreamDestroy(ctx->copy_stream);
  }
  if (ctx->d_status) cudaFree(ctx->d_status);
  free(ctx);
}

int twa_get_status(twa_ctx* ctx, int* code, int* detail) {
  if (!ctx || !code) return TWA_ERR_INVALID_ARG;
  int h[2] = {0, -1};
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  TWA_CUDA_OK(ctx, cudaMemcpyAsync(h, ctx->d_status, sizeof(h), cudaMemcpyDeviceToHost, ctx->stream));
  TWA_CUDA_OK(ctx, cudaStreamSynchronize(ctx->stream));
  *code = h[0];
  if (detail) *detail = h[0] ? h[1] : -1;
  return TWA_OK;
}

int twa_clear_status(twa_ctx* ctx) {
  if (!ctx) return TWA_ERR_INVALID_ARG;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  TWA_CUDA_OK(ctx, cudaMemsetAsync(ctx->d_status, 0, 256, ctx->stream));
  return TWA_OK;
}

const char* twa_strerror(int code) {
  switch (code) {
    case TWA_OK: return "ok";
    case TWA_ERR_INVALID_ARG: return "invalid argument";
    case TWA_ERR_MISALIGNED: return "pointer or stride not 16-byte aligned";
    case TWA_ERR_UNSUPPORTED: return "unsupported size, width or device";
    case TWA_ERR_RANK_DEFICIENT: return "candidates are linearly dependent";
    case TWA_ERR_NONFINITE: return "non-finite value in the input";
    case TWA_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case TWA_ERR_CUDA: return "CUDA call failed";
    case TWA_ERR_WORKSPACE: return "workspace missing or too small";
    default: return "unknown error";
  }
}

const char* twa_last_error(const twa_ctx* ctx) { return ctx ? ctx->last_error : ""; }

int twa_set_tuning(twa_ctx* ctx, int key, int value) {
  if (!ctx || value < 0) return TWA_ERR_INVALID_ARG;
  switch (key) {
    case TWA_TUNE_PROJECT_WARPS: ctx->tune_project_warps = value; return TWA_OK;
    case TWA_TUNE_LIFT_WARPS: ctx->tune_lift_warps = value; return TWA_OK;
    case TWA_TUNE_STAGES: ctx->tune_stages = value; return TWA_OK;
    case TWA_TUNE_TILE_SEGMENTS:
      if (value == 3 || value > 4) return TWA_ERR_INVALID_ARG;
      ctx->tune_tile_segments = value;
      return TWA_OK;
    case TWA_TUNE_BUILD_PANEL:
      if (value > 2) return TWA_ERR_INVALID_ARG;
      ctx->tune_build_panel = value;
      return TWA_OK;
    case TWA_TUNE_LIFT_VECTORS:
      if (value > 3) return TWA_ERR_INVALID_ARG;
      ctx->tune_lift_base_path = value;
      return TWA_OK;
    case TWA_TUNE_DEQUANT_PATH:
      if (value > 1) return TWA_ERR_INVALID_ARG;
      ctx->tune_dequant_path = value;
      return TWA_OK;
    case TWA_TUNE_SLAB_ROWS:
      if ((value & 65535) || static_cast<long long>(value) > TWA_SLAB_ROWS) return TWA_ERR_INVALID_ARG;
      ctx->tune_slab_rows = value;
      return TWA_OK;
    case TWA_TUNE_WAIT_LIMIT_MS:
      ctx->wait_limit_ns = (value ? static_cast<unsigned long long>(value) : 2000ull) * 1000000ull;
      return TWA_OK;
    default: return TWA_ERR_INVALID_ARG;
  }
}

int twa_project(twa_ctx* ctx, const twa_basis* P, const void* g, twa_dtype g_dtype, float* c_out,
                void* ws, size_t ws_bytes) {
  if (!ctx || !g || !c_out) return TWA_ERR_INVALID_ARG;
  if (g_dtype != TWA_F32 && g_dtype != TWA_BF16) return TWA_ERR_INVALID_ARG;
  int rc = check_basis_slabbed(ctx, P);
  if (rc) return rc;
  rc = check_ws(ws, ws_bytes);
  if (rc) return rc;
  if (misaligned16(g)) return TWA_ERR_MISALIGNED;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  twa_project_epilogue epi = {c_out, nullptr, 0.0f, 0.0f, -1};
  if (slab_plan(ctx, P->D).count > 1) return project_slabs(ctx, P, g, g_dtype, epi, ws);
  return twa_launch_project(ctx, P, g, g_dtype, epi, ws);
}

int twa_lift(twa_ctx* ctx, const twa_basis* P, const float* alpha, const float* base, float* w_out,
             void* ws, size_t ws_bytes) {
  if (!ctx || !alpha || !w_out) return TWA_ERR_INVALID_ARG;
  int rc = check_basis_slabbed(ctx, P);
  if (rc) return rc;
  rc = check_ws(ws, ws_bytes);
  if (rc) return rc;
  if (misaligned16(w_out) || (base && misaligned16(base))) return TWA_ERR_MISALIGNED;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  if (slab_plan(ctx, P->D).count > 1) return lift_slabs(ctx, P, alpha, base, w_out, false);
  return twa_launch_lift(ctx, P, alpha, 1.0f, base, w_out, false);
}

static int step_impl(twa_ctx* ctx, const twa_basis* P, const void* g, twa_dtype g_dtype, float lr, float lambda,
                     const twa_adam_args& adam, float* alpha, const float* wbar, float* w, float* c_out, void* ws,
                     size_t ws_bytes) {
  if (!ctx || !g || !alpha || !wbar || !w) return TWA_ERR_INVALID_ARG;
  if (g_dtype != TWA_F32 && g_dtype != TWA_BF16) return TWA_ERR_INVALID_ARG;
  int rc = check_basis_slabbed(ctx, P);
  if (rc) return rc;
  rc = check_ws(ws, ws_bytes);
  if (rc) return rc;
  if (misaligned16(g) || misaligned16(w) || misaligned16(wbar)) return TWA_ERR_MISALIGNED;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  twa_project_epilogue epi = {c_out, alpha, lr, lambda, -1, adam};
  const bool slabbed = slab_plan(ctx, P->D).count > 1;
  cudaEvent_t* ev = nullptr;
  if (ctx->prof_events && ctx->prof_count < ctx->prof_cap) ev = ctx->prof_events + 3 * ctx->prof_count;
  if (ev) TWA_CUDA_OK(ctx, cudaEventRecord(ev[0], ctx->stream));
  rc = slabbed ? project_slabs(ctx, P, g, g_dtype, epi, ws) : twa_launch_project(ctx, P, g, g_dtype, epi, ws);
  if (rc) return rc;
  if (ev) TWA_CUDA_OK(ctx, cudaEventRecord(ev[1], ctx->stream));
  // The lift walks the tiles backwards: the part of P~ the projection read last is the part
  // most likely still in L2.
  rc = slabbed ? lift_slabs(ctx, P, alpha, wbar, w, true) : twa_launch_lift(ctx, P, alpha, 1.0f, wbar, w, true);
  if (rc) return rc;
  if (ev) {
    TWA_CUDA_OK(ctx, cudaEventRecord(ev[2], ctx->stream));
    ctx->prof_count++;
  }
  return TWA_OK;
}

int twa_step(twa_ctx* ctx, const twa_basis* P, const void* g, twa_dtype g_dtype, float lr, float lambda,
             float* alpha, const float* wbar, float* w, float* c_out, void* ws, size_t ws_bytes) {
  return step_impl(ctx, P, g, g_dtype, lr, lambda, twa_adam_args{}, alpha, wbar, w, c_out, ws, ws_bytes);
}

int twa_step_adam(twa_ctx* ctx, const twa_basis* P, const void* g, twa_dtype g_dtype, const twa_adam* opt,
                  float* alpha, float* m, float* v, const float* wbar, float* w, float* c_out, void* ws,
                  size_t ws_bytes) {
  twa_adam_args ad;
  int rc = twa_adam_device_args(opt, m, v, &ad);
  if (rc) return rc;
  return step_impl(ctx, P, g, g_dtype, opt->lr, opt->weight_decay, ad, alpha, wbar, w, c_out, ws, ws_bytes);
}

float twa_cosine_lr(float base_lr, int step, int total_steps, float min_lr) {
  double x = total_steps > 0 ? static_cast<double>(step) / static_cast<double>(total_steps) : 1.0;
  x = x < 0.0 ? 0.0 : (x > 1.0 ? 1.0 : x);
  return static_cast<float>(static_cast<double>(min_lr) +
                            0.5 * (static_cast<double>(base_lr) - static_cast<double>(min_lr)) *
                                (1.0 + cos(3.14159265358979323846 * x)));
}

int twa_weighted_average(twa_ctx* ctx, const float* W, int64_t D, int n, int64_t ldw, const float* weights,
                         float* w_out, void* ws, size_t ws_bytes) {
  if (!W || !weights) return TWA_ERR_INVALID_ARG;
  const twa_basis cand = {const_cast<float*>(W), nullptr, D, 4 * ldw, n, 32};
  return twa_lift(ctx, &cand, weights, nullptr, w_out, ws, ws_bytes);
}

int twa_profile_enable(twa_ctx* ctx, int max_steps) {
  if (!ctx || max_steps < 0 || max_steps > 65536) return TWA_ERR_INVALID_ARG;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  if (ctx->prof_events) {
    TWA_CUDA_OK(ctx, cudaStreamSynchronize(ctx->stream));
    for (int i = 0; i < 3 * ctx->prof_cap; ++i) cudaEventDestroy(ctx->prof_events[i]);
    free(ctx->prof_events);
    ctx->prof_events = nullptr;
    ctx->prof_cap = ctx->prof_count = 0;
  }
  if (max_steps == 0) return TWA_OK;
  ctx->prof_events = static_cast<cudaEvent_t*>(calloc(3 * static_cast<size_t>(max_steps), sizeof(cudaEvent_t)));
  if (!ctx->prof_events) return TWA_ERR_INVALID_ARG;
  for (int i = 0; i < 3 * max_steps; ++i) TWA_CUDA_OK(ctx, cudaEventCreate(&ctx->prof_events[i]));
  ctx->prof_cap = max_steps;
  ctx->prof_count = 0;
  return TWA_OK;
}

int twa_profile_read(twa_ctx* ctx, double* project_ms, double* lift_ms, int* steps) {
  if (!ctx || !project_ms || !lift_ms || !steps) return TWA_ERR_INVALID_ARG;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  TWA_CUDA_OK(ctx, cudaStreamSynchronize(ctx->stream));
  double p = 0, l = 0;
  for (int i = 0; i < ctx->prof_count; ++i) {
    float a = 0, b = 0;
    TWA_CUDA_OK(ctx, cudaEventElapsedTime(&a, ctx->prof_events[3 * i], ctx->prof_events[3 * i + 1]));
    TWA_CUDA_OK(ctx, cudaEventElapsedTime(&b, ctx->prof_events[3 * i + 1], ctx->prof_events[3 * i + 2]));
    p += a;
    l += b;
  }
  *project_ms = p;
  *lift_ms = l;
  *steps = ctx->prof_count;
  ctx->prof_count = 0;
  return TWA_OK;
}

int twa_step_host(twa_ctx* ctx, const twa_basis* P, const void* g_host, twa_dtype g_dtype, float lr,
                  float lambda, float* alpha, const float* wbar, float* w, float* w_host, void* g_stage,
                  void* ws, size_t ws_bytes) {
  if (!ctx || !g_host || !w_host || !g_stage || !P) return TWA_ERR_INVALID_ARG;
  if (g_dtype != TWA_F32 && g_dtype != TWA_BF16) return TWA_ERR_INVALID_ARG;
  if (P->D < 1) return TWA_ERR_INVALID_ARG;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  const size_t gsz = g_dtype == TWA_BF16 ? 2 : 4;
  const long long D = P->D;
  // Row chunks: multiples of 2^16 rows (whole tiles of every storage width), at most TWA_HOST_CHUNKS.
  // Below 2^22 rows the copies are too short to be worth splitting.
  long long chunk_rows = (D + TWA_HOST_CHUNKS - 1) / TWA_HOST_CHUNKS;
  chunk_rows = (chunk_rows + 65535) / 65536 * 65536;
  const int chunks = static_cast<int>((D + chunk_rows - 1) / chunk_rows);
  if (D < (1LL << 22) || chunks < 2) {
    TWA_CUDA_OK(ctx, cudaMemcpyAsync(g_stage, g_host, static_cast<size_t>(D) * gsz, cudaMemcpyHostToDevice, ctx->stream));
    int rc = twa_step(ctx, P, g_stage, g_dtype, lr, lambda, alpha, wbar, w, nullptr, ws, ws_bytes);
    if (rc) return rc;
    TWA_CUDA_OK(ctx, cudaMemcpyAsync(w_host, w, static_cast<size_t>(D) * 4, cudaMemcpyDeviceToHost, ctx->stream));
    return TWA_OK;
  }
  if (!alpha || !wbar || !w) return TWA_ERR_INVALID_ARG;
  int rc = check_basis_slabbed(ctx, P);
  if (rc) return rc;
  rc = check_ws(ws, ws_bytes);
  if (rc) return rc;
  if (misaligned16(g_stage) || misaligned16(w) || misaligned16(wbar)) return TWA_ERR_MISALIGNED;
  if (!ctx->copy_events) {
    TWA_CUDA_OK(ctx, cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking));
    const int count = 2 * TWA_HOST_CHUNKS + 2;
    cudaEvent_t* ev = static_cast<cudaEvent_t*>(calloc(count, sizeof(cudaEvent_t)));
    if (!ev) return TWA_ERR_INVALID_ARG;
    for (int i = 0; i < count; ++i) TWA_CUDA_OK(ctx, cudaEventCreateWithFlags(&ev[i], cudaEventDisableTiming));
    ctx->copy_events = ev;
  }
  cudaEvent_t* ev_up = ctx->copy_events;                       // gradient chunk k is on the device
  cudaEvent_t* ev_lift = ctx->copy_events + TWA_HOST_CHUNKS;   // rows of chunk k of w are final
  cudaEvent_t ev_begin = ctx->copy_events[2 * TWA_HOST_CHUNKS], ev_end = ctx->copy_events[2 * TWA_HOST_CHUNKS + 1];
  float* chunk_c = reinterpret_cast<float*>(static_cast<char*>(ws) + TWA_WS_CHUNK_COEF);
  const char* gh = static_cast<const char*>(g_host);
  char* gs = static_cast<char*>(g_stage);
  auto view = [&](int k, twa_basis* v, long long* r0) {
    *r0 = static_cast<long long>(k) * chunk_rows;
    const long long rows = (*r0 + chunk_rows < D) ? chunk_rows : D - *r0;
    *v = *P;
    v->data = static_cast<char*>(P->data) + (*r0 * P->bits) / 8;
    v->D = rows;
  };
  // the copies wait for everything enqueued on the context's stream so far (g_stage and w may be in use)
  TWA_CUDA_OK(ctx, cudaEventRecord(ev_begin, ctx->stream));
  TWA_CUDA_OK(ctx, cudaStreamWaitEvent(ctx->copy_stream, ev_begin, 0));
  for (int k = 0; k < chunks; ++k) {
    twa_basis v;
    long long r0;
    view(k, &v, &r0);
    TWA_CUDA_OK(ctx, cudaMemcpyAsync(gs + r0 * gsz, gh + r0 * gsz, static_cast<size_t>(v.D) * gsz, cudaMemcpyHostToDevice,
                                     ctx->copy_stream));
    TWA_CUDA_OK(ctx, cudaEventRecord(ev_up[k], ctx->copy_stream));
  }
  // projection of every chunk as soon as its rows of g have arrived
  for (int k = 0; k < chunks; ++k) {
    twa_basis v;
    long long r0;
    view(k, &v, &r0);
    TWA_CUDA_OK(ctx, cudaStreamWaitEvent(ctx->stream, ev_up[k], 0));
    twa_project_epilogue epi = {chunk_c + static_cast<size_t>(k) * TWA_MAX_N, nullptr, 0.0f, 0.0f, -1};
    rc = twa_launch_project(ctx, &v, gs + r0 * gsz, g_dtype, epi, ws);
    if (rc) return rc;
  }
  chunk_combine_kernel<<<1, TWA_MAX_N, 0, ctx->stream>>>(chunk_c, chunks, P->n, nullptr, alpha, lr, lambda,
                                                         twa_adam_args{}, ctx->d_status);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  // lift chunk by chunk; every chunk of w leaves for the host while the next one is computed
  for (int k = 0; k < chunks; ++k) {
    twa_basis v;
    long long r0;
    view(k, &v, &r0);
    rc = twa_launch_lift(ctx, &v, alpha, 1.0f, wbar + r0, w + r0, false);
    if (rc) return rc;
    TWA_CUDA_OK(ctx, cudaEventRecord(ev_lift[k], ctx->stream));
    TWA_CUDA_OK(ctx, cudaStreamWaitEvent(ctx->copy_stream, ev_lift[k], 0));
    TWA_CUDA_OK(ctx, cudaMemcpyAsync(w_host + r0, w + r0, static_cast<size_t>(v.D) * 4, cudaMemcpyDeviceToHost,
                                     ctx->copy_stream));
  }
  // later work on the context's stream (and a caller waiting for it) sees w_host complete
  TWA_CUDA_OK(ctx, cudaEventRecord(ev_end, ctx->copy_stream));
  TWA_CUDA_OK(ctx, cudaStreamWaitEvent(ctx->stream, ev_end, 0));
  return TWA_OK;
}

}  // extern "C"
