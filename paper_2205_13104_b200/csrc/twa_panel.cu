// Panel steps of the blocked Gram-Schmidt build (Section 4.1 of the paper: Schmidt
// orthogonalisation of {w_i}): a panel of up to 8 candidate columns is orthogonalised against all
// earlier basis vectors at once, so the earlier vectors are read once per panel instead of once
// per column.
//     C = Q^T A_p        (twa_launch_panel_project)   Q: columns 0 .. nq-1, A_p: columns nq .. nq+pb-1
//     A_p <- A_p - Q C   (twa_launch_panel_lift)
// The projection streams tiles of 128 rows x (nq + pb) columns of the float32 matrix through a TMA
// ring (one box per stage: the panel's columns are simply the last columns of the tile).
//  * projection: warp w of 15 owns columns w, w+15, ...; a lane owns 4 rows; up to 8 x 8 accumulators per lane;
//    lanes -> block -> last block to finish, float64 over blocks in block order.
//  * update: a lane owns two rows of a block of 1024 rows and walks all nq columns as they stream past
//    in chunks of 8, so there is no reduction at all.
//  * inside the panel: the Gram-Schmidt coefficients from the panel's Gram matrix, the new columns as
//    A_p T (one pass).  The Gram matrix is taken by the update kernel from the values it stores (float64
//    products on the tensor pipe), the squared norms of the panel's columns as given by the projection
//    kernel from the tiles it streams anyway; only the first panel, which has nothing before it, takes
//    its Gram matrix in a pass of its own.
#include <stdio.h>

#include "twa_common.cuh"

namespace {

constexpr int PANEL = 8;                         // columns per panel at most
constexpr int PROWS = 128;                       // rows per tile of the projection
constexpr int PCOL_BYTES = PROWS * 4;
constexpr int PWARPS = 16;                       // consumer warps
constexpr int PTHREADS = (PWARPS + 1) * 32;
// The projection runs 15 consumer warps and the producer: 16 warps, four per scheduler, leave 128
// registers per thread for up to 8 x 8 accumulators (with 17 warps one scheduler holds five and the
// limit is 96: the kernels for six and more columns per warp spilled).
constexpr int PJWARPS = 15;
constexpr int PJTHREADS = (PJWARPS + 1) * 32;
constexpr int CPART_BYTES = 4096;                // block's sums / coefficients: TWA_MAX_N x PANEL floats

struct PanelArgs {
  long long D, ldw;
  int nq, pb, tiles, stages, detail;
  unsigned stage_bytes, tx_bytes;
  float* panel;                // first column of the panel
  float* partials;             // [grid][nq * PANEL]
  float* C;                    // [nq][PANEL]
  double* sumsq_part;          // [grid][PANEL] squared norms of the panel's columns, or null
  double* sumsq;               // [PANEL]
  unsigned* ticket;
  int* status;
  unsigned long long wait_limit_ns;
};

__device__ __forceinline__ void panel_producer(twa_smem_header* hdr, unsigned char* ring, const CUtensorMap* map,
                                               const PanelArgs& a) {
  twa_prefetch_tensormap(map);
  volatile int* abort_flag = &hdr->abort_flag;
  int issued = 0;
  bool ok = true;
  for (int tile = blockIdx.x; tile < a.tiles; tile += gridDim.x, ++issued) {
    const int s = issued % a.stages, use = issued / a.stages;
    if (use > 0 && !twa_mbar_wait(twa_smem_u32(&hdr->empty[s]), static_cast<unsigned>(use - 1) & 1u, abort_flag,
                                  a.wait_limit_ns)) {
      ok = false;
      break;
    }
    const uint32_t fb = twa_smem_u32(&hdr->full[s]);
    twa_mbar_expect_tx(fb, a.tx_bytes);
    twa_tma_load_2d(twa_smem_u32(ring + static_cast<size_t>(s) * a.stage_bytes), map, tile * PROWS, 0, fb);
  }
  // every copy issued has landed before this lane leaves, whatever the consumers did meanwhile
  if (!twa_drain_ring(hdr, issued, a.stages, a.wait_limit_ns)) ok = false;
  if (!ok) twa_set_status(a.status, TWA_ERR_TIMEOUT, -1);
}

// CPW = columns of Q a warp owns at most, ceil(nq / 15): a compile-time constant, so that the loops
// over a warp's columns carry no guards (a warp with fewer columns repeats column 0 and drops the
// result).  With run-time bounds the same kernel spent four times the instructions at nq = 16.
template <int CPW>
__global__ void __launch_bounds__(PJTHREADS, 1)
panel_project_kernel(const __grid_constant__ CUtensorMap map, const PanelArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (twa_smem_u32(smem_raw) & 1023u)) & 1023u);
  twa_smem_header* hdr = reinterpret_cast<twa_smem_header*>(smem);
  float* cpart = reinterpret_cast<float*>(smem + TWA_SMEM_HEADER);
  unsigned char* ring = smem + TWA_SMEM_HEADER + CPART_BYTES;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < a.stages; ++s) {
      twa_mbar_init(twa_smem_u32(&hdr->full[s]), 1);
      twa_mbar_init(twa_smem_u32(&hdr->empty[s]), PJWARPS);
    }
    hdr->abort_flag = 0;
    hdr->last_flag = 0;
    twa_fence_barrier_init();
  }
  __syncthreads();

  if (warp == PJWARPS) {
    if (lane == 0) panel_producer(hdr, ring, &map, a);
  } else {
    // columns warp, warp + 15, ...: byte offset of this lane's four rows of each inside a tile
    // (all but the last always exist, at a constant stride; the last may not: it then repeats column 0)
    const int qbase = warp * PCOL_BYTES + lane * 16;
    const int qlast = (warp + (CPW - 1) * PJWARPS < a.nq ? warp + (CPW - 1) * PJWARPS : 0) * PCOL_BYTES + lane * 16;
    const int goff = a.nq * PCOL_BYTES + lane * 16;
    float acc[CPW][PANEL];
#pragma unroll
    for (int k = 0; k < CPW; ++k)
#pragma unroll
      for (int q = 0; q < PANEL; ++q) acc[k][q] = 0.0f;
    volatile int* abort_flag = &hdr->abort_flag;
    int s = 0;
    unsigned phase = 0;
    // warp q < pb also sums the squares of panel column q (float64), rows beyond D being zero in the tile
    const bool norm_warp = a.sumsq_part != nullptr && warp < a.pb;
    double ss = 0.0;
    for (int tile = blockIdx.x; tile < a.tiles; tile += gridDim.x) {
      if (!twa_mbar_wait(twa_smem_u32(&hdr->full[s]), phase, abort_flag, a.wait_limit_ns)) {
        twa_set_status(a.status, TWA_ERR_TIMEOUT, -1);
        break;
      }
      const unsigned char* st = ring + static_cast<size_t>(s) * a.stage_bytes;
      if (norm_warp) {
        const float4 v = *reinterpret_cast<const float4*>(st + goff + warp * PCOL_BYTES);
        ss = fma(static_cast<double>(v.x), static_cast<double>(v.x), ss);
        ss = fma(static_cast<double>(v.y), static_cast<double>(v.y), ss);
        ss = fma(static_cast<double>(v.z), static_cast<double>(v.z), ss);
        ss = fma(static_cast<double>(v.w), static_cast<double>(v.w), ss);
      }
      constexpr int GQ = 4;                               // panel columns in registers at a time
#pragma unroll
      for (int part = 0; part < PANEL / GQ; ++part) {
        float4 g[GQ];
#pragma unroll
        for (int q = 0; q < GQ; ++q)
          g[q] = part * GQ + q < a.pb ? *reinterpret_cast<const float4*>(st + goff + (part * GQ + q) * PCOL_BYTES)
                                      : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int k = 0; k < CPW; ++k) {
          const float4 p = *reinterpret_cast<const float4*>(st + (k < CPW - 1 ? qbase + k * PJWARPS * PCOL_BYTES : qlast));
#pragma unroll
          for (int q = 0; q < GQ; ++q)
            acc[k][part * GQ + q] =
                fmaf(p.x, g[q].x, fmaf(p.y, g[q].y, fmaf(p.z, g[q].z, fmaf(p.w, g[q].w, acc[k][part * GQ + q]))));
        }
      }
      __syncwarp();
      if (lane == 0) twa_mbar_arrive(twa_smem_u32(&hdr->empty[s]));
      if (++s == a.stages) {
        s = 0;
        phase ^= 1u;
      }
    }
    // lanes -> one value per (column, panel column); every pair belongs to exactly one warp
#pragma unroll
    for (int k = 0; k < CPW; ++k) {
#pragma unroll
      for (int q = 0; q < PANEL; ++q) {
        float v = acc[k][q];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
        if (lane == 0 && warp + k * PJWARPS < a.nq) cpart[(warp + k * PJWARPS) * PANEL + q] = v;
      }
    }
    if (norm_warp) {
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, off);
      if (lane == 0) a.sumsq_part[static_cast<size_t>(blockIdx.x) * PANEL + warp] = ss;
    }
  }
  __syncthreads();
  const int tid = threadIdx.x, outs = a.nq * PANEL;
  for (int i = tid; i < outs; i += blockDim.x) a.partials[static_cast<size_t>(blockIdx.x) * outs + i] = cpart[i];
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const unsigned ticket = atomicAdd(a.ticket, 1u);
    hdr->last_flag = (ticket == gridDim.x - 1) ? 1 : 0;
  }
  __syncthreads();
  if (hdr->last_flag) {
    __threadfence();
    for (int i = tid; i < outs; i += blockDim.x) {
      double sum = 0.0;
      for (unsigned b = 0; b < gridDim.x; ++b) sum += static_cast<double>(__ldcg(&a.partials[static_cast<size_t>(b) * outs + i]));
      if (!isfinite(sum)) twa_set_status(a.status, TWA_ERR_NONFINITE, a.detail + (i % PANEL));
      a.C[i] = static_cast<float>(sum);
    }
    if (a.sumsq_part && tid < a.pb) {
      double sum = 0.0;
      for (unsigned b = 0; b < gridDim.x; ++b) sum += __ldcg(&a.sumsq_part[static_cast<size_t>(b) * PANEL + tid]);
      a.sumsq[tid] = sum;
    }
    if (tid == 0) *a.ticket = 0u;
  }
}

constexpr int NPAIR = PANEL * (PANEL + 1) / 2;                     // 36
__host__ __device__ constexpr int pair_index(int i, int j) { return j * (j + 1) / 2 + i; }   // i <= j

// One thread: from the panel's Gram matrix G (upper triangle, G[pair_index(i, j)] = <a_i, a_j>) the
// Gram-Schmidt coefficients R (the Cholesky factor of G) with the rank and finiteness tests of the
// column-by-column schedule, and T = R^-1 ([column j][row i] at T[j * 8 + i]; a column found dependent
// or non-finite becomes zero and is reported).  `given`: the squared norms the rank test compares
// against; with given_from_diagonal they are G's diagonal, which is then also written there.
__device__ __noinline__ void panel_factor(const double* G, int pb, double* given, int given_from_diagonal, double* T, int* status,
                             int col0) {
  double r[NPAIR], tm[PANEL][PANEL];
  bool dead[PANEL];
  for (int j = 0; j < PANEL; ++j)
    for (int i = 0; i < PANEL; ++i) tm[i][j] = 0.0;
  for (int j = 0; j < pb; ++j) {
    double d = G[pair_index(j, j)];
    const double na = given_from_diagonal ? d : given[j];
    for (int k = 0; k < j; ++k) {
      double c = 0.0;
      if (!dead[k]) {
        c = G[pair_index(k, j)];
        for (int i = 0; i < k; ++i) c -= r[pair_index(i, k)] * r[pair_index(i, j)];
        c /= r[pair_index(k, k)];
      }
      r[pair_index(k, j)] = c;
      d -= c * c;
    }
    const double rjj = d > 0.0 ? sqrt(d) : 0.0;
    dead[j] = false;
    if (!isfinite(na) || !isfinite(d)) {
      twa_set_status(status, TWA_ERR_NONFINITE, col0 + j);
      dead[j] = true;
    } else if (!(rjj > 1e-5 * sqrt(na))) {
      twa_set_status(status, TWA_ERR_RANK_DEFICIENT, col0 + j);
      dead[j] = true;
    }
    r[pair_index(j, j)] = dead[j] ? 1.0 : rjj;
    if (!dead[j]) {
      // T[:, j] = (e_j - sum_{k<j} r_kj T[:, k]) / r_jj
      for (int i = 0; i <= j; ++i) {
        double v = i == j ? 1.0 : 0.0;
        for (int k = i; k < j; ++k) v -= r[pair_index(k, j)] * tm[i][k];
        tm[i][j] = v / rjj;
      }
    }
    if (given_from_diagonal) given[j] = na;
  }
  for (int j = 0; j < PANEL; ++j)
    for (int i = 0; i < PANEL; ++i) T[j * PANEL + i] = tm[i][j];
}

// Update kernel.  A block walks blocks of 1024 rows; a lane owns two neighbouring rows of the block
// (16 warps x 32 lanes x 2) and accumulates its 2 x 8 results while the columns of Q stream past in
// chunks of 8 (one stage = 1024 rows x 8 columns, four boxes of 256 rows); the chunk after the last
// one of Q is the panel itself, whose old values the lane then updates and stores.  Every consumer
// warp consumes every stage, in order: the plain ring protocol, no reduction anywhere.  Two rows
// per lane halve the shared-memory reads of the coefficients per product (with one row the kernel
// ran at 69 % issue utilisation, a third of it those reads).
//
// With a.gpart set the kernel also leaves the Gram matrix of the panel as it stores it, and the factor
// T of panel_factor: a warp writes its 64 rows x 8 columns of new values back into the stage, reads
// them as operands of 16 float64 tensor-pipe products (4 rows each; the 8 x 8 matrix in two registers
// per lane), the warps' matrices are added in warp order, the blocks' in block order by the block that
// finishes last, which factorises.  That is the panel's Gram pass without reading the panel again.
constexpr int LROWS_LANE = 2;
constexpr int LROWS_BLOCK = PWARPS * 32 * LROWS_LANE;        // 1024 rows per row block
constexpr int LCHUNK = PANEL;                                // columns per stage
constexpr unsigned LSTAGE_BYTES = LROWS_BLOCK * LCHUNK * 4;  // 32 KB
constexpr unsigned LBOX_BYTES = 256 * LCHUNK * 4;            // one box: 256 rows x 8 columns

struct PanelLiftArgs {
  long long D, ldw;
  int nq, pb, row_blocks, stages;
  float* panel;
  const float* C;
  int* status;
  unsigned long long wait_limit_ns;
  // Gram matrix of the stored panel and its factor (gpart == null: not wanted)
  double* gpart;               // [grid][64]
  double* given;
  int given_from_diagonal, col0;
  double* T;
  unsigned* ticket;
};

// d += a (8 x 4, row-major) * b (4 x 8, column-major) in float64 on the tensor pipe: lane l holds
// a[l >> 2][l & 3], b[l & 3][l >> 2] and d[l >> 2][2 * (l & 3) + {0, 1}].
__device__ __forceinline__ void panel_dmma(double (&d)[2], double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
               : "+d"(d[0]), "+d"(d[1])
               : "d"(a), "d"(b));
}

__global__ void __launch_bounds__(PTHREADS, 1)
panel_lift_kernel(const __grid_constant__ CUtensorMap map, const PanelLiftArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (twa_smem_u32(smem_raw) & 1023u)) & 1023u);
  twa_smem_header* hdr = reinterpret_cast<twa_smem_header*>(smem);
  float* Cs = reinterpret_cast<float*>(smem + TWA_SMEM_HEADER);        // [nq][PANEL]
  unsigned char* ring = smem + TWA_SMEM_HEADER + CPART_BYTES;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < a.stages; ++s) {
      twa_mbar_init(twa_smem_u32(&hdr->full[s]), 1);
      twa_mbar_init(twa_smem_u32(&hdr->empty[s]), PWARPS);
    }
    hdr->abort_flag = 0;
    twa_fence_barrier_init();
  }
  for (int i = threadIdx.x; i < a.nq * PANEL; i += blockDim.x) Cs[i] = a.C[i];
  __syncthreads();
  volatile int* abort_flag = &hdr->abort_flag;
  const int chunks = a.nq / LCHUNK + 1;                                // chunks of Q, then the panel
  if (warp == PWARPS) {
    if (lane != 0) return;
    twa_prefetch_tensormap(&map);
    int it = 0;
    bool ok = true;
    for (int rb = blockIdx.x; rb < a.row_blocks && ok; rb += gridDim.x) {
      for (int c = 0; c < chunks; ++c, ++it) {
        const int s = it % a.stages, use = it / a.stages;
        if (use > 0 && !twa_mbar_wait(twa_smem_u32(&hdr->empty[s]), static_cast<unsigned>(use - 1) & 1u, abort_flag,
                                      a.wait_limit_ns)) {
          ok = false;
          break;
        }
        const uint32_t fb = twa_smem_u32(&hdr->full[s]);
        const uint32_t dst = twa_smem_u32(ring + static_cast<size_t>(s) * LSTAGE_BYTES);
        twa_mbar_expect_tx(fb, LSTAGE_BYTES);
#pragma unroll
        for (int b = 0; b < LROWS_BLOCK / 256; ++b)
          twa_tma_load_2d(dst + b * LBOX_BYTES, &map, rb * LROWS_BLOCK + b * 256, c * LCHUNK, fb);
      }
    }
    // every copy issued has landed before this lane leaves, whatever the consumers did meanwhile
    if (!twa_drain_ring(hdr, it, a.stages, a.wait_limit_ns)) ok = false;
    if (!ok) twa_set_status(a.status, TWA_ERR_TIMEOUT, -1);
    return;
  }
  // element (column c of the chunk, row r of the block) sits at ((r >> 8) * 8 + c) * 256 + (r & 255)
  const int r = (warp * 32 + lane) * LROWS_LANE;
  const int base = (r >> 8) * LCHUNK * 256 + (r & 255);
  // Gram operands: lane (column c = lane >> 2, k = lane & 3) takes rows 16 t + 4 k .. + 3 of the warp's 64
  const int gram_base = ((warp * 64) >> 8) * LCHUNK * 256 + ((warp * 64) & 255) + (lane >> 2) * 256 + (lane & 3) * 4;
  const bool want_gram = a.gpart != nullptr;
  double gacc[2] = {0.0, 0.0};
  int it = 0;
  bool alive = true;
  for (int rb = blockIdx.x; rb < a.row_blocks && alive; rb += gridDim.x) {
    float acc0[PANEL], acc1[PANEL];
#pragma unroll
    for (int q = 0; q < PANEL; ++q) acc0[q] = acc1[q] = 0.0f;
    for (int c = 0; c < chunks; ++c, ++it) {
      const int s = it % a.stages;
      if (!twa_mbar_wait(twa_smem_u32(&hdr->full[s]), static_cast<unsigned>(it / a.stages) & 1u, abort_flag,
                         a.wait_limit_ns)) {
        twa_set_status(a.status, TWA_ERR_TIMEOUT, -1);
        alive = false;
        break;
      }
      const float* st = reinterpret_cast<const float*>(ring + static_cast<size_t>(s) * LSTAGE_BYTES) + base;
      if (c < chunks - 1) {
#pragma unroll
        for (int u = 0; u < LCHUNK; ++u) {
          const float2 x = *reinterpret_cast<const float2*>(st + u * 256);
          const float4 c0 = *reinterpret_cast<const float4*>(Cs + (c * LCHUNK + u) * PANEL);
          const float4 c1 = *reinterpret_cast<const float4*>(Cs + (c * LCHUNK + u) * PANEL + 4);
          acc0[0] = fmaf(x.x, c0.x, acc0[0]); acc0[1] = fmaf(x.x, c0.y, acc0[1]);
          acc0[2] = fmaf(x.x, c0.z, acc0[2]); acc0[3] = fmaf(x.x, c0.w, acc0[3]);
          acc0[4] = fmaf(x.x, c1.x, acc0[4]); acc0[5] = fmaf(x.x, c1.y, acc0[5]);
          acc0[6] = fmaf(x.x, c1.z, acc0[6]); acc0[7] = fmaf(x.x, c1.w, acc0[7]);
          acc1[0] = fmaf(x.y, c0.x, acc1[0]); acc1[1] = fmaf(x.y, c0.y, acc1[1]);
          acc1[2] = fmaf(x.y, c0.z, acc1[2]); acc1[3] = fmaf(x.y, c0.w, acc1[3]);
          acc1[4] = fmaf(x.y, c1.x, acc1[4]); acc1[5] = fmaf(x.y, c1.y, acc1[5]);
          acc1[6] = fmaf(x.y, c1.z, acc1[6]); acc1[7] = fmaf(x.y, c1.w, acc1[7]);
        }
        __syncwarp();
        if (lane == 0) twa_mbar_arrive(twa_smem_u32(&hdr->empty[s]));
      } else {
        float2 old[PANEL];
#pragma unroll
        for (int q = 0; q < PANEL; ++q) {
          old[q] = *reinterpret_cast<const float2*>(st + q * 256);
          old[q].x -= acc0[q];
          old[q].y -= acc1[q];
        }
        if (want_gram) {
          // the new values (zero in rows beyond D and in columns beyond pb, where everything read was
          // zero) go back to the lane's own places; the warp's 64 x 8 patch is its alone
          float* stw = const_cast<float*>(st);
#pragma unroll
          for (int q = 0; q < PANEL; ++q) *reinterpret_cast<float2*>(stw + q * 256) = old[q];
        }
        const long long row = static_cast<long long>(rb) * LROWS_BLOCK + r;
        if (row + 1 < a.D) {
#pragma unroll
          for (int q = 0; q < PANEL; ++q)
            if (q < a.pb) *reinterpret_cast<float2*>(a.panel + q * a.ldw + row) = old[q];
        } else if (row < a.D) {
#pragma unroll
          for (int q = 0; q < PANEL; ++q)
            if (q < a.pb) a.panel[q * a.ldw + row] = old[q].x;
        }
        if (want_gram) {
          __syncwarp();
          const float* gp = reinterpret_cast<const float*>(ring + static_cast<size_t>(s) * LSTAGE_BYTES) + gram_base;
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            const float4 gv = *reinterpret_cast<const float4*>(gp + 16 * t);
            const double x0 = gv.x, x1 = gv.y, x2 = gv.z, x3 = gv.w;
            panel_dmma(gacc, x0, x0);
            panel_dmma(gacc, x1, x1);
            panel_dmma(gacc, x2, x2);
            panel_dmma(gacc, x3, x3);
          }
          twa_fence_proxy_async();       // the writes above before the copy that refills the stage
        }
        __syncwarp();
        if (lane == 0) twa_mbar_arrive(twa_smem_u32(&hdr->empty[s]));
      }
    }
  }
  if (!want_gram) return;
  // The 16 consumer warps only from here on (the producer warp has left): barrier 1, 512 threads.
  // Every stage this block was sent has been consumed, so the ring is free to hold the warps' matrices.
  constexpr int CONSUMERS = PWARPS * 32;
  double* wsum = reinterpret_cast<double*>(ring);                       // [PWARPS][64]
  __shared__ double Gs[NPAIR];
  __shared__ int last;
  twa_named_barrier(1, CONSUMERS);                                      // the slowest warp has read its last stage
  wsum[warp * 64 + (lane >> 2) * 8 + 2 * (lane & 3)] = gacc[0];
  wsum[warp * 64 + (lane >> 2) * 8 + 2 * (lane & 3) + 1] = gacc[1];
  twa_named_barrier(1, CONSUMERS);
  if (threadIdx.x < 64) {
    double t = 0.0;
    for (int w = 0; w < PWARPS; ++w) t += wsum[w * 64 + threadIdx.x];
    a.gpart[static_cast<size_t>(blockIdx.x) * 64 + threadIdx.x] = t;
  }
  __threadfence();
  twa_named_barrier(1, CONSUMERS);
  if (threadIdx.x == 0) last = (atomicAdd(a.ticket, 1u) == gridDim.x - 1);
  twa_named_barrier(1, CONSUMERS);
  if (!last) return;
  __threadfence();
  if (threadIdx.x < 64) {
    const int i = threadIdx.x >> 3, j = threadIdx.x & 7;
    if (i <= j) {
      double t = 0.0;
      for (unsigned b = 0; b < gridDim.x; ++b) t += __ldcg(&a.gpart[static_cast<size_t>(b) * 64 + threadIdx.x]);
      Gs[pair_index(i, j)] = t;
    }
  }
  twa_named_barrier(1, CONSUMERS);
  if (threadIdx.x != 0) return;
  *a.ticket = 0u;
  panel_factor(Gs, a.pb, a.given, a.given_from_diagonal, a.T, a.status, a.col0);
}

// ------------------------------------------------------------------------------------------------
// Gram form of the sweeps inside a panel.  Gram-Schmidt on the panel's columns a_0 .. a_{pb-1} gives
// q_j = (a_j - sum_{k<j} r_kj q_k) / r_jj with r_kj = <q_k, a_j>; every q_k is a combination of the
// a's, so all r_kj follow from the panel's Gram matrix G = A_p^T A_p: they are the entries of its
// Cholesky factor, and Q_p = A_p T with T = R^-1 upper triangular.  One pass takes the 36 dot
// products <a_i, a_j> (float64 products and sums, warp shuffles, blocks combined in block order);
// the block that finishes last factorises G in float64, applies the rank and finiteness tests of
// the column-by-column schedule (r_jj <= 1e-5 |a_j| as given: the column becomes zero and is
// reported) and leaves T; a second pass writes A_p T.  Twelve column passes per panel and round
// instead of the 52 of the column sweeps.
constexpr int GRAM_BLOCK = 256;

__global__ void __launch_bounds__(GRAM_BLOCK, 2) panel_gram_kernel(const float* __restrict__ A0, long long ld, int pb,
                                                               long long D, double* __restrict__ gpart,
                                                               double* __restrict__ given, int given_from_diagonal,
                                                               double* __restrict__ T, unsigned* __restrict__ ticket,
                                                               int* status, int col0) {
  __shared__ double sh[NPAIR][GRAM_BLOCK / 32];
  __shared__ double G[NPAIR];
  __shared__ int last;
  double s[NPAIR];
#pragma unroll
  for (int p = 0; p < NPAIR; ++p) s[p] = 0.0;
  const long long nvec = D >> 2;
  for (long long t = blockIdx.x * static_cast<long long>(GRAM_BLOCK) + threadIdx.x; t < nvec;
       t += static_cast<long long>(gridDim.x) * GRAM_BLOCK) {
    float4 x[PANEL];
#pragma unroll
    for (int j = 0; j < PANEL; ++j)
      x[j] = j < pb ? __ldcs(reinterpret_cast<const float4*>(A0 + j * ld) + t) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int comp = 0; comp < 4; ++comp) {
      double v[PANEL];
#pragma unroll
      for (int j = 0; j < PANEL; ++j)
        v[j] = static_cast<double>(comp == 0 ? x[j].x : comp == 1 ? x[j].y : comp == 2 ? x[j].z : x[j].w);
#pragma unroll
      for (int j = 0; j < PANEL; ++j)
#pragma unroll
        for (int i = 0; i <= j; ++i) s[pair_index(i, j)] = fma(v[i], v[j], s[pair_index(i, j)]);
    }
  }
  if (blockIdx.x == 0 && threadIdx.x < (D & 3)) {
    const long long r = (nvec << 2) + threadIdx.x;
    double v[PANEL];
#pragma unroll
    for (int j = 0; j < PANEL; ++j) v[j] = j < pb ? static_cast<double>(A0[j * ld + r]) : 0.0;
#pragma unroll
    for (int j = 0; j < PANEL; ++j)
#pragma unroll
      for (int i = 0; i <= j; ++i) s[pair_index(i, j)] = fma(v[i], v[j], s[pair_index(i, j)]);
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
  for (int p = 0; p < NPAIR; ++p) {
    double t = s[p];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, off);
    if (lane == 0) sh[p][warp] = t;
  }
  __syncthreads();
  if (threadIdx.x < NPAIR) {
    double t = 0;
    for (int w = 0; w < GRAM_BLOCK / 32; ++w) t += sh[threadIdx.x][w];
    gpart[static_cast<size_t>(blockIdx.x) * NPAIR + threadIdx.x] = t;
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
  __syncthreads();
  if (!last) return;
  __threadfence();
  if (threadIdx.x < NPAIR) {
    double t = 0;
    for (unsigned b = 0; b < gridDim.x; ++b) t += __ldcg(&gpart[static_cast<size_t>(b) * NPAIR + threadIdx.x]);
    G[threadIdx.x] = t;
  }
  __syncthreads();
  if (threadIdx.x != 0) return;
  *ticket = 0u;
  panel_factor(G, pb, given, given_from_diagonal, T, status, col0);
}

// A_p <- A_p T (T upper triangular, [column j][row i] at T[j * 8 + i]); float64 sums, one rounding per stored
// value.  Column j needs columns 0 .. j only, so the columns are replaced from the last to the first in
// the registers that hold them.  With `absmax` the largest magnitude stored in each column is folded
// into absmax[j] (bit patterns of |x|: NaN and Inf compare above every finite value).
__global__ void __launch_bounds__(GRAM_BLOCK, 2) panel_apply_kernel(float* __restrict__ A0, long long ld, int pb, long long D,
                                                                   const double* __restrict__ T,
                                                                   unsigned* __restrict__ absmax) {
  __shared__ double Ts[PANEL * PANEL];
  __shared__ unsigned mx[PANEL];
  if (threadIdx.x < PANEL * PANEL) Ts[threadIdx.x] = T[threadIdx.x];
  if (threadIdx.x < PANEL) mx[threadIdx.x] = 0u;
  __syncthreads();
  unsigned m[PANEL];
#pragma unroll
  for (int j = 0; j < PANEL; ++j) m[j] = 0u;
  const long long nvec = D >> 2;
  for (long long t = blockIdx.x * static_cast<long long>(GRAM_BLOCK) + threadIdx.x; t < nvec;
       t += static_cast<long long>(gridDim.x) * GRAM_BLOCK) {
    float4 x[PANEL];
#pragma unroll
    for (int j = 0; j < PANEL; ++j)
      x[j] = j < pb ? __ldcs(reinterpret_cast<const float4*>(A0 + j * ld) + t) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int j = PANEL - 1; j >= 0; --j) {
      double a = 0.0, b = 0.0, c = 0.0, d = 0.0;
#pragma unroll
      for (int i = 0; i <= j; ++i) {
        const double w = Ts[j * PANEL + i];
        a = fma(static_cast<double>(x[i].x), w, a);
        b = fma(static_cast<double>(x[i].y), w, b);
        c = fma(static_cast<double>(x[i].z), w, c);
        d = fma(static_cast<double>(x[i].w), w, d);
      }
      x[j] = make_float4(static_cast<float>(a), static_cast<float>(b), static_cast<float>(c), static_cast<float>(d));
      if (j < pb) {
        __stcs(reinterpret_cast<float4*>(A0 + j * ld) + t, x[j]);
        m[j] = max(max(m[j], __float_as_uint(x[j].x) & 0x7FFFFFFFu), max(__float_as_uint(x[j].y) & 0x7FFFFFFFu,
                   max(__float_as_uint(x[j].z) & 0x7FFFFFFFu, __float_as_uint(x[j].w) & 0x7FFFFFFFu)));
      }
    }
  }
  if (blockIdx.x == 0 && threadIdx.x < (D & 3)) {
    const long long r = (nvec << 2) + threadIdx.x;
    double x[PANEL];
#pragma unroll
    for (int j = 0; j < PANEL; ++j) x[j] = j < pb ? static_cast<double>(A0[j * ld + r]) : 0.0;
#pragma unroll
    for (int j = 0; j < PANEL; ++j) {
      double a = 0.0;
#pragma unroll
      for (int i = 0; i <= j; ++i) a = fma(x[i], Ts[j * PANEL + i], a);
      const float y = static_cast<float>(a);
      if (j < pb) {
        A0[j * ld + r] = y;
        m[j] = max(m[j], __float_as_uint(y) & 0x7FFFFFFFu);
      }
    }
  }
  if (!absmax) return;
#pragma unroll
  for (int j = 0; j < PANEL; ++j) {
    unsigned v = m[j];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v = max(v, __shfl_xor_sync(0xFFFFFFFFu, v, off));
    if ((threadIdx.x & 31) == 0 && j < pb) atomicMax(&mx[j], v);
  }
  __syncthreads();
  if (threadIdx.x < pb) atomicMax(&absmax[threadIdx.x], mx[threadIdx.x]);
}

int encode_panel_map(twa_ctx* ctx, const float* W, long long D, long long ldw, int cols, CUtensorMap* map) {
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(cols)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(ldw * 4)};
  cuuint32_t box[2] = {PROWS, static_cast<cuuint32_t>(cols)};
  cuuint32_t es[2] = {1, 1};
  CUresult r = ctx->encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(W), dims, strides, box, es,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(ctx->last_error, sizeof(ctx->last_error), "cuTensorMapEncodeTiled(panel) failed: %d", static_cast<int>(r));
    return TWA_ERR_CUDA;
  }
  return TWA_OK;
}

int fill_args(twa_ctx* ctx, float* W, long long D, long long ldw, int nq, int pb, void* ws, PanelArgs* a, int* grid,
              int* smem) {
  if (nq < 1 || pb < 1 || pb > PANEL || nq + pb > TWA_MAX_N) return TWA_ERR_INVALID_ARG;
  a->D = D;
  a->ldw = ldw;
  a->nq = nq;
  a->pb = pb;
  a->detail = nq;
  a->tiles = static_cast<int>((D + PROWS - 1) / PROWS);
  a->tx_bytes = static_cast<unsigned>(nq + pb) * PCOL_BYTES;
  a->stage_bytes = (a->tx_bytes + 1023) / 1024 * 1024;
  const int fixed = TWA_SMEM_HEADER + CPART_BYTES + 1024;
  int stages = (ctx->smem_optin - fixed) / static_cast<int>(a->stage_bytes);
  if (stages > TWA_MAX_STAGES) stages = TWA_MAX_STAGES;
  if (stages < 2) return TWA_ERR_UNSUPPORTED;
  a->stages = stages;
  a->panel = W + static_cast<long long>(nq) * ldw;
  // the float region of the workspace: per-block sums, then the coefficients (1024 floats), then
  // 16 floats the caller keeps for itself
  float* region = reinterpret_cast<float*>(static_cast<char*>(ws) + TWA_WS_PARTIALS);
  const size_t region_floats = static_cast<size_t>(TWA_MAX_GRID) * TWA_MAX_N;
  a->partials = region;
  a->C = region + region_floats - 1040;
  a->sumsq_part = nullptr;
  a->sumsq = nullptr;
  a->ticket = ctx->d_ticket;
  a->status = ctx->d_status;
  a->wait_limit_ns = ctx->wait_limit_ns;
  int g = ctx->sm_count < a->tiles ? ctx->sm_count : a->tiles;
  if (g > TWA_PANEL_SUMSQ_BLOCKS) g = TWA_PANEL_SUMSQ_BLOCKS;
  const size_t per_block = static_cast<size_t>(nq) * PANEL;
  if (static_cast<size_t>(g) * per_block > region_floats - 1040) g = static_cast<int>((region_floats - 1040) / per_block);
  *grid = g;
  *smem = fixed + stages * static_cast<int>(a->stage_bytes);
  return TWA_OK;
}

template <int CPW>
int launch_panel_project(twa_ctx* ctx, const CUtensorMap& map, const PanelArgs& a, int grid, int smem) {
  static int smem_limit[64] = {0};
  int rc = twa_ensure_smem(ctx, reinterpret_cast<const void*>(panel_project_kernel<CPW>), &smem_limit[ctx->device & 63], smem);
  if (rc) return rc;
  panel_project_kernel<CPW><<<grid, PJTHREADS, smem, ctx->stream>>>(map, a);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}

}  // namespace

int twa_launch_panel_project(twa_ctx* ctx, float* W, long long D, long long ldw, int nq, int pb, void* ws,
                             double* sumsq_out) {
  PanelArgs a;
  int grid, smem;
  int rc = fill_args(ctx, W, D, ldw, nq, pb, ws, &a, &grid, &smem);
  if (rc) return rc;
  if (sumsq_out) {
    a.sumsq_part = reinterpret_cast<double*>(static_cast<char*>(ws) + TWA_WS_PANEL_SUMSQ);
    a.sumsq = sumsq_out;
  }
  CUtensorMap map;
  rc = encode_panel_map(ctx, W, D, ldw, nq + pb, &map);
  if (rc) return rc;
  const int cpw = (nq + PJWARPS - 1) / PJWARPS;
  switch (cpw) {
    case 1: return launch_panel_project<1>(ctx, map, a, grid, smem);
    case 2: return launch_panel_project<2>(ctx, map, a, grid, smem);
    case 3: return launch_panel_project<3>(ctx, map, a, grid, smem);
    case 4: return launch_panel_project<4>(ctx, map, a, grid, smem);
    case 5: return launch_panel_project<5>(ctx, map, a, grid, smem);
    case 6: return launch_panel_project<6>(ctx, map, a, grid, smem);
    case 7: return launch_panel_project<7>(ctx, map, a, grid, smem);
    default: return launch_panel_project<8>(ctx, map, a, grid, smem);
  }
}

int twa_launch_panel_lift(twa_ctx* ctx, float* W, long long D, long long ldw, int nq, int pb, void* ws, double* given,
                          bool given_from_diagonal) {
  if (nq < LCHUNK || (nq % LCHUNK) != 0 || pb < 1 || pb > PANEL || nq + pb > TWA_MAX_N) return TWA_ERR_INVALID_ARG;
  PanelLiftArgs a;
  a.D = D;
  a.ldw = ldw;
  a.nq = nq;
  a.pb = pb;
  a.row_blocks = static_cast<int>((D + LROWS_BLOCK - 1) / LROWS_BLOCK);
  const int fixed = TWA_SMEM_HEADER + CPART_BYTES + 1024;
  int stages = (ctx->smem_optin - fixed) / static_cast<int>(LSTAGE_BYTES);
  if (stages > TWA_MAX_STAGES) stages = TWA_MAX_STAGES;
  if (stages < 2) return TWA_ERR_UNSUPPORTED;
  a.stages = stages;
  a.panel = W + static_cast<long long>(nq) * ldw;
  const float* region = reinterpret_cast<const float*>(static_cast<const char*>(ws) + TWA_WS_PARTIALS);
  a.C = region + static_cast<size_t>(TWA_MAX_GRID) * TWA_MAX_N - 1040;      // where the projection left it
  a.status = ctx->d_status;
  a.wait_limit_ns = ctx->wait_limit_ns;
  // with `given`: the Gram matrix of the stored panel, per block at the start of the float region (the
  // coefficients this kernel reads sit at its end), and its factor where twa_launch_panel_apply reads it
  a.gpart = given ? reinterpret_cast<double*>(static_cast<char*>(ws) + TWA_WS_PARTIALS) : nullptr;
  a.given = given;
  a.given_from_diagonal = given_from_diagonal ? 1 : 0;
  a.col0 = nq;
  a.T = reinterpret_cast<double*>(static_cast<char*>(ws) + TWA_WS_COEF);
  a.ticket = ctx->d_ticket;
  // boxes of 256 rows x 8 columns over the matrix's first nq + pb columns (columns past them read as zero)
  CUtensorMap map;
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(nq + pb)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(ldw * 4)};
  cuuint32_t box[2] = {256, LCHUNK};
  cuuint32_t es[2] = {1, 1};
  CUresult r = ctx->encode_tiled(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, W, dims, strides, box, es,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(ctx->last_error, sizeof(ctx->last_error), "cuTensorMapEncodeTiled(panel update) failed: %d",
             static_cast<int>(r));
    return TWA_ERR_CUDA;
  }
  const int grid = ctx->sm_count < a.row_blocks ? ctx->sm_count : a.row_blocks;
  const int smem = fixed + stages * static_cast<int>(LSTAGE_BYTES);
  static int smem_limit[64] = {0};
  int rc = twa_ensure_smem(ctx, reinterpret_cast<const void*>(panel_lift_kernel), &smem_limit[ctx->device & 63], smem);
  if (rc) return rc;
  panel_lift_kernel<<<grid, PTHREADS, smem, ctx->stream>>>(map, a);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}

namespace {
int apply_grid(const twa_ctx* ctx, long long D) {
  long long g = (D / 4 + GRAM_BLOCK - 1) / GRAM_BLOCK;
  const long long cap = static_cast<long long>(ctx->sm_count) * 4;
  if (g > cap) g = cap;
  if (g > TWA_MAX_GRID) g = TWA_MAX_GRID;
  if (g < 1) g = 1;
  return static_cast<int>(g);
}
}  // namespace

// A_p <- A_p T with the factor twa_launch_panel_lift or the Gram pass left in the workspace; with `absmax`
// (device, one word per column of the panel) the largest magnitudes stored are folded into it.
int twa_launch_panel_apply(twa_ctx* ctx, float* W, long long D, long long ldw, int j0, int pb, void* ws,
                           unsigned* absmax) {
  if (pb < 1 || pb > PANEL) return TWA_ERR_INVALID_ARG;
  const double* T = reinterpret_cast<const double*>(static_cast<const char*>(ws) + TWA_WS_COEF);
  panel_apply_kernel<<<apply_grid(ctx, D), GRAM_BLOCK, 0, ctx->stream>>>(W + static_cast<long long>(j0) * ldw, ldw, pb, D, T,
                                                                        absmax);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}

// The Gram pass of a panel that was not just stored by twa_launch_panel_lift (see panel_gram_kernel):
// leaves the factor for twa_launch_panel_apply.  `given`: device array of 8 doubles, the squared norms the
// rank test compares against; with given_from_diagonal they are taken from (and written as) the diagonal
// of this pass's Gram matrix.
int twa_launch_panel_gram(twa_ctx* ctx, float* W, long long D, long long ldw, int j0, int pb, void* ws, double* given,
                          bool given_from_diagonal) {
  if (pb < 1 || pb > PANEL) return TWA_ERR_INVALID_ARG;
  char* w = static_cast<char*>(ws);
  double* gpart = reinterpret_cast<double*>(w + TWA_WS_PARTIALS);           // [grid][36], start of the float region
  double* T = reinterpret_cast<double*>(w + TWA_WS_COEF);                    // 64 doubles
  static_assert(sizeof(float) * TWA_MAX_N >= sizeof(double) * PANEL * PANEL, "coefficient area too small for T");
  float* A0 = W + static_cast<long long>(j0) * ldw;
  panel_gram_kernel<<<apply_grid(ctx, D), GRAM_BLOCK, 0, ctx->stream>>>(A0, ldw, pb, D, gpart, given,
                                                                       given_from_diagonal ? 1 : 0, T, ctx->d_ticket,
                                                                       ctx->d_status, j0);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}
