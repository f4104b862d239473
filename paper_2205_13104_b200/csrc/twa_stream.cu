// Streaming kernels of the TWA subspace step: project (c = P~^T g) and lift
// (w = base + P~ alpha).  Section 4.2 / 4.3 of the paper; loop body of Algorithm 1.
//
// Both kernels are persistent (one block per SM) and warp-specialised: one producer lane
// issues bulk tensor copies (TMA) of [n columns x 512 bytes] tiles of P~ into a ring of
// shared-memory stages guarded by full/empty mbarriers; the consumer warps dequantise from
// shared memory and accumulate in float32 registers.  P~ is read exactly once per kernel.
// Every wait is bounded; a wait that runs out raises the status word and the block leaves.
#include <mutex>
#include <stdio.h>

#include "twa_common.cuh"

namespace {

struct ProjectArgs {
  long long D;
  int n, warps, stages, tiles;
  unsigned stage_bytes, g_off, tx_bytes;
  const float* scales;
  float* partials;
  unsigned* ticket;
  int* status;
  float* c_out;
  float* alpha;
  float lr, lambda;
  twa_adam_args adam;
  int nonfinite_detail;
  unsigned long long wait_limit_ns;
};

struct LiftArgs {
  long long D;
  int n, warps, stages, tiles;
  unsigned stage_bytes, red_bytes;
  const float* scales;
  const float* alpha;
  float alpha_mult;
  const float* base;
  float* out;
  int reverse;
  int* status;
  unsigned long long wait_limit_ns;
};

using SmemHeader = twa_smem_header;

// Producer loop shared by both kernels.  G_BOXES 1-D boxes of the gradient follow the tile
// of P~ in the same stage (project only).
template <int ROWS, int G_BOXES, int G_BOX_ELEMS, int G_ELEM_BYTES, int KT = 1>
__device__ __forceinline__ void producer_loop(SmemHeader* hdr, unsigned char* ring,
                                              const CUtensorMap* map_p, const CUtensorMap* map_g,
                                              int tiles, int stages, unsigned stage_bytes,
                                              unsigned g_off, unsigned tx_bytes, bool reverse,
                                              int* status, unsigned long long limit) {
  twa_prefetch_tensormap(map_p);
  if (G_BOXES > 0) twa_prefetch_tensormap(map_g);
  volatile int* abort_flag = &hdr->abort_flag;
  int s = 0;
  unsigned phase = 0;          // parity of the consumers' release this stage waits for next
  int issued = 0;
  bool ok = true;
  for (int t = blockIdx.x; t < tiles; t += gridDim.x) {
    if (issued >= stages) {
      if (!twa_mbar_wait(twa_smem_u32(&hdr->empty[s]), phase, abort_flag, limit)) {
        ok = false;
        break;
      }
    }
    const int tile = reverse ? (tiles - 1 - t) : t;
    const uint32_t fb = twa_smem_u32(&hdr->full[s]);
    const uint32_t dst = twa_smem_u32(ring + static_cast<size_t>(s) * stage_bytes);
    twa_mbar_expect_tx(fb, tx_bytes);
    twa_tma_load_2d(dst, map_p, tile * (KT == 4 ? TWA_TILE_COL_BYTES / 8 * KT : TWA_TILE_COL_WORDS * KT), 0, fb);
#pragma unroll
    for (int b = 0; b < G_BOXES; ++b)
      twa_tma_load_1d(dst + g_off + b * G_BOX_ELEMS * G_ELEM_BYTES, map_g,
                      tile * ROWS + b * G_BOX_ELEMS, fb);
    ++issued;
    if (++s == stages) {
      s = 0;
      if (issued > stages) phase ^= 1u;
    }
  }
  // every copy issued has landed before this lane leaves, whatever the consumers did meanwhile
  if (!twa_drain_ring(hdr, issued, stages, limit)) ok = false;
  if (!ok) twa_set_status(status, TWA_ERR_TIMEOUT, -1);
}

// ---- project ------------------------------------------------------------------------------
// Dot product of the lane's 16 bytes of one column with the lane's gradient values.
template <int BITS>
__device__ __forceinline__ float lane_dot(const unsigned char* col16, const float* g) {
  const uint4 c = *reinterpret_cast<const uint4*>(col16);
  const uint32_t flip = BITS == 8 ? 0x80808080u : (BITS == 4 ? 0x88888888u : 0u);   // code -> offset binary
  const uint32_t w[4] = {c.x ^ flip, c.y ^ flip, c.z ^ flip, c.w ^ flip};
  float t;
  if (BITS == 32) {
    t = __uint_as_float(w[0]) * g[0];
    t = fmaf(__uint_as_float(w[1]), g[1], t);
    t = fmaf(__uint_as_float(w[2]), g[2], t);
    t = fmaf(__uint_as_float(w[3]), g[3], t);
  } else if (BITS == 8) {
    float t0 = twa_byte_to_float(w[0], 0, TWA_MAGIC_I8) * g[0];
    float t1 = twa_byte_to_float(w[1], 0, TWA_MAGIC_I8) * g[4];
    float t2 = twa_byte_to_float(w[2], 0, TWA_MAGIC_I8) * g[8];
    float t3 = twa_byte_to_float(w[3], 0, TWA_MAGIC_I8) * g[12];
#pragma unroll
    for (int b = 1; b < 4; ++b) {
      t0 = fmaf(twa_byte_to_float(w[0], b, TWA_MAGIC_I8), g[b], t0);
      t1 = fmaf(twa_byte_to_float(w[1], b, TWA_MAGIC_I8), g[4 + b], t1);
      t2 = fmaf(twa_byte_to_float(w[2], b, TWA_MAGIC_I8), g[8 + b], t2);
      t3 = fmaf(twa_byte_to_float(w[3], b, TWA_MAGIC_I8), g[12 + b], t3);
    }
    t = (t0 + t1) + (t2 + t3);
  } else {
    float tt[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t lo = w[k] & 0x0F0F0F0Fu;          // rows 8k + 0,2,4,6
      const uint32_t hi = (w[k] >> 4) & 0x0F0F0F0Fu;   // rows 8k + 1,3,5,7
      float u = twa_byte_to_float(lo, 0, TWA_MAGIC_I4) * g[8 * k];
      u = fmaf(twa_byte_to_float(hi, 0, TWA_MAGIC_I4), g[8 * k + 1], u);
#pragma unroll
      for (int b = 1; b < 4; ++b) {
        u = fmaf(twa_byte_to_float(lo, b, TWA_MAGIC_I4), g[8 * k + 2 * b], u);
        u = fmaf(twa_byte_to_float(hi, b, TWA_MAGIC_I4), g[8 * k + 2 * b + 1], u);
      }
      tt[k] = u;
    }
    t = (tt[0] + tt[1]) + (tt[2] + tt[3]);
  }
  return t;
}

// KT: 512-byte segments of every column per tile (a float32 basis with few columns: tiles of 128 rows
// are a few KB, and the per-tile hand-over then bounds the kernel, not the memory).
template <int BITS, bool GBF16, int KT = 1>
__global__ void __launch_bounds__(TWA_MAX_THREADS, 1)
twa_project_kernel(const __grid_constant__ CUtensorMap map_p,
                   const __grid_constant__ CUtensorMap map_g, const ProjectArgs a) {
  extern __shared__ __align__(1024) unsigned char smem[];
  constexpr int SROWS = twa_tile_rows(BITS);           // rows behind one segment
  constexpr int ROWS = SROWS * KT;
  constexpr int LROWS = SROWS / 32;                    // gradient values one lane needs per segment
  constexpr int GSZ = GBF16 ? 2 : 4;
  constexpr int GBOX = ROWS < 256 ? ROWS : 256;
  SmemHeader* hdr = reinterpret_cast<SmemHeader*>(smem);
  unsigned char* ring = smem + TWA_SMEM_HEADER;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int W = a.warps;

  if (threadIdx.x == 0) {
    for (int s = 0; s < a.stages; ++s) {
      twa_mbar_init(twa_smem_u32(&hdr->full[s]), 1);
      twa_mbar_init(twa_smem_u32(&hdr->empty[s]), W);
    }
    hdr->abort_flag = 0;
    hdr->last_flag = 0;
    twa_fence_barrier_init();
  }
  if (threadIdx.x < TWA_MAX_N) hdr->c_part[threadIdx.x] = 0.0f;
  __syncthreads();

  if (warp == W) {
    if (lane == 0)
      producer_loop<ROWS, ROWS / GBOX, GBOX, GSZ, KT>(hdr, ring, &map_p, &map_g, a.tiles, a.stages,
                                                      a.stage_bytes, a.g_off, a.tx_bytes, false,
                                                      a.status, a.wait_limit_ns);
  } else {
    // warp owns columns warp, warp + W, ...
    const int cpw = warp < a.n ? (a.n - warp + W - 1) / W : 0;
    float acc[TWA_PROJECT_CPW];
#pragma unroll
    for (int k = 0; k < TWA_PROJECT_CPW; ++k) acc[k] = 0.0f;
    volatile int* abort_flag = &hdr->abort_flag;
    int s = 0;
    unsigned phase = 0;
    for (int t = blockIdx.x; t < a.tiles; t += gridDim.x) {
      if (!twa_mbar_wait(twa_smem_u32(&hdr->full[s]), phase, abort_flag, a.wait_limit_ns)) {
        twa_set_status(a.status, TWA_ERR_TIMEOUT, -1);
        break;
      }
      const unsigned char* st = ring + static_cast<size_t>(s) * a.stage_bytes;
#pragma unroll
      for (int u = 0; u < KT; ++u) {
        // the lane's LROWS rows of segment u: rows u * SROWS + lane * LROWS ...
        const unsigned char* gseg = st + a.g_off + (u * SROWS + lane * LROWS) * GSZ;
        float g[LROWS];
        if (GBF16) {
          const uint4* gp = reinterpret_cast<const uint4*>(gseg);
#pragma unroll
          for (int q = 0; q < LROWS / 8; ++q) {
            const uint4 v = gp[q];
            g[8 * q + 0] = twa_bf16_lo(v.x); g[8 * q + 1] = twa_bf16_hi(v.x);
            g[8 * q + 2] = twa_bf16_lo(v.y); g[8 * q + 3] = twa_bf16_hi(v.y);
            g[8 * q + 4] = twa_bf16_lo(v.z); g[8 * q + 5] = twa_bf16_hi(v.z);
            g[8 * q + 6] = twa_bf16_lo(v.w); g[8 * q + 7] = twa_bf16_hi(v.w);
          }
          if (LROWS == 4) {                                // float32 basis: 4 rows = 8 bytes
            const uint2 v = *reinterpret_cast<const uint2*>(gseg);
            g[0] = twa_bf16_lo(v.x); g[1] = twa_bf16_hi(v.x);
            g[2] = twa_bf16_lo(v.y); g[3] = twa_bf16_hi(v.y);
          }
        } else {
          const float4* gp = reinterpret_cast<const float4*>(gseg);
#pragma unroll
          for (int q = 0; q < LROWS / 4; ++q) {
            const float4 v = gp[q];
            g[4 * q + 0] = v.x; g[4 * q + 1] = v.y; g[4 * q + 2] = v.z; g[4 * q + 3] = v.w;
          }
        }
#pragma unroll
        for (int k = 0; k < TWA_PROJECT_CPW; ++k) {
          if (k < cpw) {
            const int j = warp + k * W;
            const int slot = BITS == 32 ? lane : twa_chunk_slot(lane, j);
            acc[k] += lane_dot<BITS>(st + (j * KT + u) * TWA_TILE_COL_BYTES + slot * 16, g);
          }
        }
      }
      __syncwarp();
      if (lane == 0) twa_mbar_arrive(twa_smem_u32(&hdr->empty[s]));
      if (++s == a.stages) {
        s = 0;
        phase ^= 1u;
      }
    }
#pragma unroll
    for (int k = 0; k < TWA_PROJECT_CPW; ++k) {
      if (k < cpw) {
        float v = acc[k];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
        if (lane == 0) hdr->c_part[warp + k * W] = v;
      }
    }
  }
  __syncthreads();

  // Per-block partials, then the last block to finish combines them in block order.
  const int tid = threadIdx.x;
  if (tid < a.n) a.partials[static_cast<size_t>(blockIdx.x) * a.n + tid] = hdr->c_part[tid];
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const unsigned ticket = atomicAdd(a.ticket, 1u);
    hdr->last_flag = (ticket == gridDim.x - 1) ? 1 : 0;
  }
  __syncthreads();
  if (hdr->last_flag) {
    __threadfence();
    double c = 0.0;
    if (tid < a.n) {
      double sum = 0.0;
      for (unsigned b = 0; b < gridDim.x; ++b)
        sum += static_cast<double>(__ldcg(&a.partials[static_cast<size_t>(b) * a.n + tid]));
      c = (BITS == 32) ? sum : sum * static_cast<double>(a.scales[tid]);
      if (!isfinite(c))
        twa_set_status(a.status, TWA_ERR_NONFINITE, a.nonfinite_detail >= 0 ? a.nonfinite_detail : tid);
      if (a.c_out) a.c_out[tid] = static_cast<float>(c);
    }
    // The coefficients are state that outlives the call: they are left as they were when any c is not
    // finite or a wait ran out in some block (whose partial sums are then incomplete), so that the
    // caller can clear the status and repeat the step.
    const int unusable = __syncthreads_or(!isfinite(c)) | (__ldcg(a.status) == TWA_ERR_TIMEOUT);
    if (tid < a.n && a.alpha && !unusable)
      a.alpha[tid] = twa_coefficient_update(a.alpha[tid], c, a.lr, a.lambda, a.adam, tid);
    if (tid == 0) *a.ticket = 0u;
  }
}

// ---- lift ---------------------------------------------------------------------------------
// acc[i] += coef * code for the lane's 8 bytes of one column.
template <int BITS, int LR>
__device__ __forceinline__ void lane_axpy(const unsigned char* col8, float coef, float* acc) {
  uint2 c = *reinterpret_cast<const uint2*>(col8);
  if (BITS == 8) { c.x ^= 0x80808080u; c.y ^= 0x80808080u; }      // code -> offset binary
  if (BITS == 4) { c.x ^= 0x88888888u; c.y ^= 0x88888888u; }
  if (BITS == 32) {
    acc[0] = fmaf(__uint_as_float(c.x), coef, acc[0]);
    acc[1] = fmaf(__uint_as_float(c.y), coef, acc[1]);
  } else if (BITS == 8) {
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      acc[b] = fmaf(twa_byte_to_float(c.x, b, TWA_MAGIC_I8), coef, acc[b]);
      acc[4 + b] = fmaf(twa_byte_to_float(c.y, b, TWA_MAGIC_I8), coef, acc[4 + b]);
    }
  } else {
    const uint32_t w[2] = {c.x, c.y};
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const uint32_t lo = w[k] & 0x0F0F0F0Fu;
      const uint32_t hi = (w[k] >> 4) & 0x0F0F0F0Fu;
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        acc[8 * k + 2 * b] = fmaf(twa_byte_to_float(lo, b, TWA_MAGIC_I4), coef, acc[8 * k + 2 * b]);
        acc[8 * k + 2 * b + 1] =
            fmaf(twa_byte_to_float(hi, b, TWA_MAGIC_I4), coef, acc[8 * k + 2 * b + 1]);
      }
    }
  }
}

template <int BITS>
__global__ void __launch_bounds__(TWA_MAX_THREADS, 1)
twa_lift_kernel(const __grid_constant__ CUtensorMap map_p, const LiftArgs a) {
  extern __shared__ __align__(1024) unsigned char smem[];
  constexpr int ROWS = twa_tile_rows(BITS);            // 128 / 512 / 1024
  constexpr int LR = ROWS / 64;                        // rows behind a lane's 8 bytes: 2 / 8 / 16
  SmemHeader* hdr = reinterpret_cast<SmemHeader*>(smem);
  float* red = reinterpret_cast<float*>(smem + TWA_SMEM_HEADER);     // [CG][ROWS]
  unsigned char* ring = smem + TWA_SMEM_HEADER + a.red_bytes;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int W = a.warps, CG = W >> 1, NT = W * 32;

  if (threadIdx.x == 0) {
    for (int s = 0; s < a.stages; ++s) {
      twa_mbar_init(twa_smem_u32(&hdr->full[s]), 1);
      twa_mbar_init(twa_smem_u32(&hdr->empty[s]), W);
    }
    hdr->abort_flag = 0;
    twa_fence_barrier_init();
  }
  __syncthreads();

  if (warp == W) {
    if (lane == 0)
      producer_loop<ROWS, 0, 1, 1>(hdr, ring, &map_p, nullptr, a.tiles, a.stages, a.stage_bytes, 0,
                                   a.stage_bytes, a.reverse != 0, a.status, a.wait_limit_ns);
    return;
  }

  // warp = (column group cg, half h of the tile's rows); the group owns columns cg, cg + CG, ...
  const int h = warp & 1, cg = warp >> 1;
  const int cpw = cg < a.n ? (a.n - cg + CG - 1) / CG : 0;
  float coef[TWA_LIFT_CPW];
#pragma unroll
  for (int k = 0; k < TWA_LIFT_CPW; ++k) {
    const int j = cg + k * CG;
    float v = 0.0f;
    if (k < cpw) {
      v = a.alpha[j] * a.alpha_mult;
      if (BITS != 32) v *= a.scales[j];
    }
    coef[k] = v;
  }
  const int byte_off = h * 256 + lane * 8;             // lane's bytes inside a column of the tile
  const int row_off = byte_off * 8 / BITS;             // first of the lane's LR rows in the tile
  const int tid = threadIdx.x;
  volatile int* abort_flag = &hdr->abort_flag;
  int s = 0;
  unsigned phase = 0;
  for (int t = blockIdx.x; t < a.tiles; t += gridDim.x) {
    const int tile = a.reverse ? (a.tiles - 1 - t) : t;
    const long long row0 = static_cast<long long>(tile) * ROWS;
    // the rows this thread will finish: tid and tid + NT
    float bv[2] = {0.0f, 0.0f};
    if (a.base) {
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const int r = tid + q * NT;
        if (r < ROWS && row0 + r < a.D) bv[q] = a.base[row0 + r];
      }
    }
    float acc[LR];
#pragma unroll
    for (int i = 0; i < LR; ++i) acc[i] = 0.0f;
    const bool ok = twa_mbar_wait(twa_smem_u32(&hdr->full[s]), phase, abort_flag, a.wait_limit_ns);
    if (ok) {
      const unsigned char* st = ring + static_cast<size_t>(s) * a.stage_bytes;
#pragma unroll
      for (int k = 0; k < TWA_LIFT_CPW; ++k) {
        if (k < cpw) {
          const int j = cg + k * CG;
          const int off = BITS == 32 ? byte_off : (twa_chunk_slot(byte_off >> 4, j) << 4) | (byte_off & 15);
          lane_axpy<BITS, LR>(st + j * TWA_TILE_COL_BYTES + off, coef[k], acc);
        }
      }
      __syncwarp();
      if (lane == 0) twa_mbar_arrive(twa_smem_u32(&hdr->empty[s]));
    }
    float* dst = red + cg * ROWS + row_off;
#pragma unroll
    for (int i = 0; i < LR; i += 2) *reinterpret_cast<float2*>(dst + i) = make_float2(acc[i], acc[i + 1]);
    twa_named_barrier(1, NT);
    if (*abort_flag) break;                            // same value for every consumer thread
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      const int r = tid + q * NT;
      if (r < ROWS && row0 + r < a.D) {
        float sum = 0.0f;
        for (int c = 0; c < CG; ++c) sum += red[c * ROWS + r];
        a.out[row0 + r] = bv[q] + sum;
      }
    }
    twa_named_barrier(1, NT);
    if (++s == a.stages) {
      s = 0;
      phase ^= 1u;
    }
  }
  if (*abort_flag && tid == 0) twa_set_status(a.status, TWA_ERR_TIMEOUT, -1);
}

// ---- lift on a float32 basis ---------------------------------------------------------------------
// out[r] = base[r] + sum_j (alpha_j * mult) P_j[r]: a thread owns four consecutive rows and walks the
// columns in index order, eight columns per float32 partial sum, the partial sums added in float64 (the
// total is rounded once).  No shared-memory
// staging: every byte is used once and consecutive threads read consecutive 16-byte pieces of a column.
constexpr int LIFT32_BLOCK = 256;

__global__ void __launch_bounds__(LIFT32_BLOCK)
twa_lift32_kernel(const float* __restrict__ P, long long ld, int n, const float* __restrict__ alpha, float mult,
                  const float* base, float* out, long long D, int* status) {
  __shared__ float coef[TWA_MAX_N];
  if (threadIdx.x < n) {
    const float c = alpha[threadIdx.x] * mult;
    if (!isfinite(c) && blockIdx.x == 0) twa_set_status(status, TWA_ERR_NONFINITE, -1);
    coef[threadIdx.x] = c;
  }
  __syncthreads();
  const long long nvec = D >> 2;
  for (long long v = blockIdx.x * static_cast<long long>(LIFT32_BLOCK) + threadIdx.x; v < nvec;
       v += static_cast<long long>(gridDim.x) * LIFT32_BLOCK) {
    double s0 = 0, s1 = 0, s2 = 0, s3 = 0;
    if (base) {
      const float4 b = reinterpret_cast<const float4*>(base)[v];
      s0 = b.x; s1 = b.y; s2 = b.z; s3 = b.w;
    }
    // Eight columns at a time: their loads are issued together, their products are summed with float32
    // FMAs (eight terms: a few 1e-7 relative), and the group's sum joins the float64 total -- one
    // conversion per row and group instead of one per element, which kept the conversion pipe busy for
    // 40 % of the kernel's time.
    int j = 0;
    for (; j + 8 <= n; j += 8) {
      float4 x[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) x[q] = __ldcs(reinterpret_cast<const float4*>(P + (j + q) * ld) + v);
      float f0 = 0.0f, f1 = 0.0f, f2 = 0.0f, f3 = 0.0f;
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const float c = coef[j + q];
        f0 = fmaf(c, x[q].x, f0); f1 = fmaf(c, x[q].y, f1); f2 = fmaf(c, x[q].z, f2); f3 = fmaf(c, x[q].w, f3);
      }
      s0 += static_cast<double>(f0); s1 += static_cast<double>(f1);
      s2 += static_cast<double>(f2); s3 += static_cast<double>(f3);
    }
    for (; j < n; ++j) {
      const float4 x = __ldcs(reinterpret_cast<const float4*>(P + j * ld) + v);
      const double c = coef[j];
      s0 = fma(c, static_cast<double>(x.x), s0); s1 = fma(c, static_cast<double>(x.y), s1);
      s2 = fma(c, static_cast<double>(x.z), s2); s3 = fma(c, static_cast<double>(x.w), s3);
    }
    reinterpret_cast<float4*>(out)[v] = make_float4(static_cast<float>(s0), static_cast<float>(s1),
                                                    static_cast<float>(s2), static_cast<float>(s3));
  }
  if (blockIdx.x == 0 && threadIdx.x < (D & 3)) {
    const long long r = (nvec << 2) + threadIdx.x;
    double s = base ? static_cast<double>(base[r]) : 0.0;
    for (int j = 0; j < n; ++j) s = fma(static_cast<double>(coef[j]), static_cast<double>(P[j * ld + r]), s);
    out[r] = static_cast<float>(s);
  }
}

// ---- host side ----------------------------------------------------------------------------
int round_up(int x, int m) { return (x + m - 1) / m * m; }

int encode_basis_map(twa_ctx* ctx, const twa_basis* P, CUtensorMap* map, int kt = 1) {
  long long row_bytes = (P->D * P->bits + 7) / 8;
  // quantised columns are stored in whole, internally permuted 512-byte segments
  if (P->bits != 32) row_bytes = (row_bytes + 511) / 512 * 512;
  cuuint64_t dims[2] = {static_cast<cuuint64_t>((row_bytes + 3) / 4), static_cast<cuuint64_t>(P->n)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(P->col_stride)};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(TWA_TILE_COL_WORDS * kt), static_cast<cuuint32_t>(P->n)};
  if (kt == 4) {
    // a box dimension is limited to 256 elements: four segments are 256 elements of 8 bytes (the caller
    // has checked that a column's bytes are a multiple of 8, so no element reaches past row D - 1)
    dims[0] = static_cast<cuuint64_t>(row_bytes / 8);
    box[0] = TWA_TILE_COL_BYTES / 8 * 4;
  }
  cuuint32_t es[2] = {1, 1};
  CUresult r = ctx->encode_tiled(map, kt == 4 ? CU_TENSOR_MAP_DATA_TYPE_UINT64 : CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, P->data, dims, strides, box,
                                 es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(ctx->last_error, sizeof(ctx->last_error), "cuTensorMapEncodeTiled(P) failed: %d",
             static_cast<int>(r));
    return TWA_ERR_CUDA;
  }
  return TWA_OK;
}

int encode_vector_map(twa_ctx* ctx, const void* g, long long D, bool bf16, int box_elems,
                      CUtensorMap* map) {
  cuuint64_t dims[1] = {static_cast<cuuint64_t>(D)};
  cuuint64_t strides[1] = {0};
  cuuint32_t box[1] = {static_cast<cuuint32_t>(box_elems)};
  cuuint32_t es[1] = {1};
  CUresult r = ctx->encode_tiled(
      map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 1,
      const_cast<void*>(g), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
      CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(ctx->last_error, sizeof(ctx->last_error), "cuTensorMapEncodeTiled(g) failed: %d",
             static_cast<int>(r));
    return TWA_ERR_CUDA;
  }
  return TWA_OK;
}

// Consumer warps for project: cover n columns with at most TWA_PROJECT_CPW per warp, little
// idle capacity, and prefer more warps.
int choose_project_warps(int n, int tune) {
  if (tune >= 8 && tune <= TWA_MAX_CONSUMER_WARPS && (n + tune - 1) / tune <= TWA_PROJECT_CPW)
    return tune;
  int best = TWA_MAX_CONSUMER_WARPS;
  double best_score = 1e30;
  for (int w = 8; w <= TWA_MAX_CONSUMER_WARPS; ++w) {
    const int cpw = (n + w - 1) / w;
    if (cpw > TWA_PROJECT_CPW) continue;
    const double waste = static_cast<double>(cpw * w - n) / n;
    const double score = waste * 100.0 - 0.3 * w;
    if (score < best_score) {
      best_score = score;
      best = w;
    }
  }
  return best;
}

int choose_lift_warps(int n, int tune) {
  if (tune >= 16 && tune <= TWA_MAX_CONSUMER_WARPS && tune % 2 == 0 &&
      (n + tune / 2 - 1) / (tune / 2) <= TWA_LIFT_CPW)
    return tune;
  int best = TWA_MAX_CONSUMER_WARPS;
  double best_score = 1e30;
  for (int w = 16; w <= TWA_MAX_CONSUMER_WARPS; w += 2) {
    const int cg = w / 2;
    const int cpw = (n + cg - 1) / cg;
    if (cpw > TWA_LIFT_CPW) continue;
    const double waste = static_cast<double>(cpw * cg - n) / n;
    const double score = waste * 100.0 - 0.3 * w;
    if (score < best_score) {
      best_score = score;
      best = w;
    }
  }
  return best;
}

int choose_stages(const twa_ctx* ctx, int fixed_bytes, int stage_bytes) {
  int s = (ctx->smem_optin - fixed_bytes) / stage_bytes;
  if (s > TWA_MAX_STAGES) s = TWA_MAX_STAGES;
  if (ctx->tune_stages >= 2 && ctx->tune_stages < s) s = ctx->tune_stages;
  return s;
}

template <int BITS, bool GBF16, int KT = 1>
int launch_project_t(twa_ctx* ctx, const CUtensorMap& mp, const CUtensorMap& mg, const ProjectArgs& a,
                     int grid, int smem) {
  auto kern = twa_project_kernel<BITS, GBF16, KT>;
  static int smem_limit[64] = {0};   // per device
  int rc = twa_ensure_smem(ctx, reinterpret_cast<const void*>(kern), &smem_limit[ctx->device & 63], smem);
  if (rc) return rc;
  kern<<<grid, (a.warps + 1) * 32, smem, ctx->stream>>>(mp, mg, a);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}

template <int BITS>
int launch_lift_t(twa_ctx* ctx, const CUtensorMap& mp, const LiftArgs& a, int grid, int smem) {
  auto kern = twa_lift_kernel<BITS>;
  static int smem_limit[64] = {0};   // per device
  int rc = twa_ensure_smem(ctx, reinterpret_cast<const void*>(kern), &smem_limit[ctx->device & 63], smem);
  if (rc) return rc;
  kern<<<grid, (a.warps + 1) * 32, smem, ctx->stream>>>(mp, a);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}

}  // namespace

// The limit is an attribute of the kernel on a device, shared by every context of the process: the
// value reached so far is cached per kernel and device (`current`), and the cache is read and
// raised under one lock so that contexts driven from several host threads do not race on it.
int twa_ensure_smem(twa_ctx* ctx, const void* kernel, int* current, int wanted) {
  static std::mutex lock;
  std::lock_guard<std::mutex> guard(lock);
  if (wanted > *current) {
    TWA_CUDA_OK(ctx, cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, wanted));
    *current = wanted;
  }
  return TWA_OK;
}

int twa_check_basis(const twa_basis* P) {
  if (!P || !P->data) return TWA_ERR_INVALID_ARG;
  if (P->bits != 32 && P->bits != 8 && P->bits != 4) return TWA_ERR_UNSUPPORTED;
  if (P->n < 1 || P->D < 1 || P->D > TWA_MAX_LAUNCH_ROWS) return TWA_ERR_INVALID_ARG;
  if (P->n > TWA_MAX_N) return TWA_ERR_UNSUPPORTED;
  if (P->bits != 32 && !P->scales) return TWA_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(P->data) & 15) || (P->col_stride & 15)) return TWA_ERR_MISALIGNED;
  if (P->col_stride < (P->D * P->bits + 7) / 8) return TWA_ERR_INVALID_ARG;
  if (P->bits != 32 && (P->col_stride & 511)) return TWA_ERR_MISALIGNED;   // whole 512-byte segments
  return TWA_OK;
}

int twa_launch_project(twa_ctx* ctx, const twa_basis* P, const void* g, twa_dtype g_dtype,
                       const twa_project_epilogue& epi, void* ws) {
  if (P->bits != 32 && ctx->tune_dequant_path == 0)
    return twa_launch_project_mma(ctx, P, g, g_dtype, epi, ws);
  const bool bf16 = g_dtype == TWA_BF16;
  // a float32 basis of few columns takes tiles of two or four segments (256 or 512 rows): see
  // twa_project_kernel; four need the tensor map of 8-byte elements, i.e. an even number of rows
  int kt = 1;
  if (P->bits == 32) {
    kt = P->n <= 32 ? 4 : (P->n <= 64 ? 2 : 1);
    if (ctx->tune_tile_segments == 1 || ctx->tune_tile_segments == 2 || ctx->tune_tile_segments == 4)
      kt = ctx->tune_tile_segments;
    if (kt == 4 && (P->D & 1)) kt = 2;
    while (kt > 1 && (ctx->smem_optin - TWA_SMEM_HEADER) / (P->n * TWA_TILE_COL_BYTES * kt + twa_tile_rows(32) * kt * 4 + 128) < 3) kt >>= 1;
  }
  const int rows = twa_tile_rows(P->bits) * kt;
  const int gsz = bf16 ? 2 : 4;
  CUtensorMap mp, mg;
  int rc = encode_basis_map(ctx, P, &mp, kt);
  if (rc) return rc;
  rc = encode_vector_map(ctx, g, P->D, bf16, rows < 256 ? rows : 256, &mg);
  if (rc) return rc;

  ProjectArgs a;
  a.D = P->D;
  a.n = P->n;
  a.warps = choose_project_warps(P->n, ctx->tune_project_warps);
  a.tiles = static_cast<int>((P->D + rows - 1) / rows);
  a.g_off = static_cast<unsigned>(P->n) * TWA_TILE_COL_BYTES * kt;
  a.tx_bytes = a.g_off + static_cast<unsigned>(rows * gsz);
  a.stage_bytes = static_cast<unsigned>(round_up(static_cast<int>(a.tx_bytes), 128));
  a.stages = choose_stages(ctx, TWA_SMEM_HEADER, static_cast<int>(a.stage_bytes));
  if (a.stages < 2) return TWA_ERR_UNSUPPORTED;
  a.scales = P->scales;
  a.partials = reinterpret_cast<float*>(static_cast<char*>(ws) + TWA_WS_PARTIALS);
  a.ticket = ctx->d_ticket;
  a.status = ctx->d_status;
  a.c_out = epi.c_out;
  a.alpha = epi.alpha;
  a.lr = epi.lr;
  a.lambda = epi.lambda;
  a.adam = epi.adam;
  a.nonfinite_detail = epi.nonfinite_detail;
  a.wait_limit_ns = ctx->wait_limit_ns;
  int grid = ctx->sm_count < a.tiles ? ctx->sm_count : a.tiles;
  if (grid > TWA_MAX_GRID) grid = TWA_MAX_GRID;
  const int smem = TWA_SMEM_HEADER + a.stages * static_cast<int>(a.stage_bytes);

  switch (P->bits) {
    case 32:
      if (kt == 4)
        return bf16 ? launch_project_t<32, true, 4>(ctx, mp, mg, a, grid, smem)
                    : launch_project_t<32, false, 4>(ctx, mp, mg, a, grid, smem);
      if (kt == 2)
        return bf16 ? launch_project_t<32, true, 2>(ctx, mp, mg, a, grid, smem)
                    : launch_project_t<32, false, 2>(ctx, mp, mg, a, grid, smem);
      return bf16 ? launch_project_t<32, true>(ctx, mp, mg, a, grid, smem)
                  : launch_project_t<32, false>(ctx, mp, mg, a, grid, smem);
    case 8:
      return bf16 ? launch_project_t<8, true>(ctx, mp, mg, a, grid, smem)
                  : launch_project_t<8, false>(ctx, mp, mg, a, grid, smem);
    default:
      return bf16 ? launch_project_t<4, true>(ctx, mp, mg, a, grid, smem)
                  : launch_project_t<4, false>(ctx, mp, mg, a, grid, smem);
  }
}

int twa_launch_lift(twa_ctx* ctx, const twa_basis* P, const float* alpha, float alpha_mult,
                    const float* base, float* out, bool reverse_tiles) {
  if (P->bits != 32 && ctx->tune_dequant_path == 0)
    return twa_launch_lift_mma(ctx, P, alpha, alpha_mult, base, out, reverse_tiles);
  if (P->bits == 32) {
    const long long nvec = P->D >> 2;
    long long g = (nvec + LIFT32_BLOCK - 1) / LIFT32_BLOCK;
    const long long cap = static_cast<long long>(ctx->sm_count) * 8;
    if (g > cap) g = cap;
    if (g < 1) g = 1;
    twa_lift32_kernel<<<static_cast<int>(g), LIFT32_BLOCK, 0, ctx->stream>>>(
        static_cast<const float*>(P->data), P->col_stride / 4, P->n, alpha, alpha_mult, base, out, P->D, ctx->d_status);
    TWA_CUDA_OK(ctx, cudaGetLastError());
    return TWA_OK;
  }
  const int rows = twa_tile_rows(P->bits);
  CUtensorMap mp;
  int rc = encode_basis_map(ctx, P, &mp);
  if (rc) return rc;
  LiftArgs a;
  a.D = P->D;
  a.n = P->n;
  a.warps = choose_lift_warps(P->n, ctx->tune_lift_warps);
  a.tiles = static_cast<int>((P->D + rows - 1) / rows);
  a.stage_bytes = static_cast<unsigned>(P->n) * TWA_TILE_COL_BYTES;
  a.red_bytes = static_cast<unsigned>(round_up((a.warps / 2) * rows * 4, 128));
  a.stages = choose_stages(ctx, TWA_SMEM_HEADER + static_cast<int>(a.red_bytes),
                           static_cast<int>(a.stage_bytes));
  if (a.stages < 2) return TWA_ERR_UNSUPPORTED;
  a.scales = P->scales;
  a.alpha = alpha;
  a.alpha_mult = alpha_mult;
  a.base = base;
  a.out = out;
  a.reverse = reverse_tiles ? 1 : 0;
  a.status = ctx->d_status;
  a.wait_limit_ns = ctx->wait_limit_ns;
  int grid = ctx->sm_count < a.tiles ? ctx->sm_count : a.tiles;
  const int smem = TWA_SMEM_HEADER + static_cast<int>(a.red_bytes) +
                   a.stages * static_cast<int>(a.stage_bytes);
  switch (P->bits) {
    case 32: return launch_lift_t<32>(ctx, mp, a, grid, smem);
    case 8: return launch_lift_t<8>(ctx, mp, a, grid, smem);
    default: return launch_lift_t<4>(ctx, mp, a, grid, smem);
  }
}
