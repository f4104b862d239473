// Row-chunked construction of the orthonormal basis for candidate sets that do not fit in
// device memory at once (Section 4.1 of the paper: Schmidt orthogonalisation of {w_i};
// Section 4.6 for the storage).
//
// The orthonormal basis with span{q_1..q_j} = span{w_1..w_j} and positive diagonal is unique
// (A = Q R), so it can be computed from row chunks without ever holding A: two rounds of
// "orthogonalise, then re-orthogonalise" in Gram form,
//     G1 = A^T A,  R1 = chol(G1),  Q1 = A R1^-1,   G2 = Q1^T Q1,  R2 = chol(G2),  Q = A (R1^-1 R2^-1),
// with every n x n quantity and every accumulation in float64.  The caller feeds each row chunk
// of the candidates once per pass:
//     pass 0: mean, G1      pass 1: G2      pass 2: column absmax of Q (and float32 Q if wanted)
//     pass 3: codes of Q
// Passes 2 and 3 evaluate Q with identical arithmetic, so the codes are exactly the quantiser
// applied to the float32 Q of pass 2.
#include <math.h>
#include <stdio.h>

#include "twa_common.cuh"
#include "twa_quant.cuh"

namespace {

constexpr int RT = 128;                 // rows per tile = threads per block
constexpr int ASTR = RT + 1;            // padded strides: conflict-free column-strided reads
constexpr int DSTR = RT + 4;            // stride of the float64 tile: the matrix-fragment loads below are conflict-free
constexpr int MAX_BLOCKS = 1024;
constexpr int BUILD_MAX_N = 64;

struct ChunkArgs {
  const float* A;
  long long ld, rows, rows_padded, row0, D;
  int n;
  const double* M;          // n x n upper triangular, stride NP (modes 1..3)
  double* partials;         // [grid][NP*NP]  (modes 0, 1)
  float* wbar;              // mode 0
  unsigned* absmax;         // mode 2
  float* q32;               // modes 2, 3, optional: q32[j * ldq + row inside the chunk]
  long long ldq;
  // mode 3: the quantised bases that receive the codes of this chunk's rows (one or two widths)
  struct CodeTarget {
    unsigned char* codes;
    long long stride, rows_padded;   // bytes between columns; rows of the chunk incl. the zero fill of the last segment
    const float* scales;
    int bits;
  } target[2];
  int targets;
};

// workspace layout for padded size NP
struct BuildLayout {
  size_t g, r1inv, rinv, absmax, partials, total;
};
BuildLayout layout_for(int np) {
  BuildLayout l;
  const size_t m = sizeof(double) * np * np;
  l.g = 0;
  l.r1inv = m;
  l.rinv = 2 * m;
  l.absmax = 3 * m;
  l.partials = 3 * m + 512;
  l.total = l.partials + static_cast<size_t>(MAX_BLOCKS) * m;
  return l;
}
int padded_n(int n) { return (n + 15) / 16 * 16; }

// d += a (8 x 4, row-major) * b (4 x 8, column-major) in float64 on the tensor pipe: lane l holds
// a[l >> 2][l & 3], b[l & 3][l >> 2] and d[l >> 2][2 * (l & 3) + {0, 1}].
__device__ __forceinline__ void dmma_8x8x4(double (&d)[2], double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
               : "+d"(d[0]), "+d"(d[1])
               : "d"(a), "d"(b));
}

// Gram matrix of a tile held column by column in float64 (T[c * DSTR + r], RT rows, NP columns):
// warp w takes the 8-row bands w, w + 4, ... of G and all NP / 8 column blocks of each; one
// tensor-pipe product per 8 x 8 block and 4 rows, the rows in order.  With scalar float64 FMAs this
// loop issued seven times the instructions and the Gram passes ran at a quarter of the float64 rate.
template <int NP>
__device__ __forceinline__ void gram_accumulate(const double* T, double (&acc)[(NP / 8 + 3) / 4][NP / 8][2], int warp,
                                                int lane) {
  constexpr int NB = NP / 8, IBW = (NB + 3) / 4;
  const int off = (lane >> 2) * DSTR + (lane & 3);
#pragma unroll 2
  for (int k0 = 0; k0 < RT; k0 += 4) {
    double b[NB];
#pragma unroll
    for (int jb = 0; jb < NB; ++jb) b[jb] = T[jb * 8 * DSTR + off + k0];
#pragma unroll
    for (int u = 0; u < IBW; ++u) {
      const int ib = warp + 4 * u;
      if (ib < NB) {
        const double av = T[ib * 8 * DSTR + off + k0];
#pragma unroll
        for (int jb = 0; jb < NB; ++jb) dmma_8x8x4(acc[u][jb], av, b[jb]);
      }
    }
  }
}

// The same for 32 columns (four 8 x 8 blocks a side) with the symmetry used: only the ten blocks on and
// above the diagonal are formed, three or two per warp (`pairs`), ten tensor-pipe products per four rows
// instead of sixteen; the factorisation reads the upper triangle only, and sym4_store writes zeros below.
struct Sym4Pairs {
  int ib[3], jb[3], count;
};
__device__ __forceinline__ Sym4Pairs sym4_pairs(int warp) {
  switch (warp) {
    case 0: return {{0, 0, 0}, {0, 1, 2}, 3};
    case 1: return {{0, 1, 3}, {3, 3, 3}, 3};
    case 2: return {{1, 1, 1}, {1, 2, 2}, 2};
    default: return {{2, 2, 2}, {2, 3, 3}, 2};
  }
}
__device__ __forceinline__ void gram_accumulate_sym4(const double* T, double (&acc)[1][4][2], int warp, int lane) {
  const Sym4Pairs p = sym4_pairs(warp);
  const int off = (lane >> 2) * DSTR + (lane & 3);
  const int oa0 = p.ib[0] * 8 * DSTR + off, oa1 = p.ib[1] * 8 * DSTR + off, oa2 = p.ib[2] * 8 * DSTR + off;
  const int ob0 = p.jb[0] * 8 * DSTR + off, ob1 = p.jb[1] * 8 * DSTR + off, ob2 = p.jb[2] * 8 * DSTR + off;
  const bool three = p.count == 3;
#pragma unroll 2
  for (int k0 = 0; k0 < RT; k0 += 4) {
    dmma_8x8x4(acc[0][0], T[oa0 + k0], T[ob0 + k0]);
    dmma_8x8x4(acc[0][1], T[oa1 + k0], T[ob1 + k0]);
    if (three) dmma_8x8x4(acc[0][2], T[oa2 + k0], T[ob2 + k0]);
  }
}
// This warp's blocks of the block's Gram matrix (row-major [32][32]) and zeros in their mirror images.
__device__ __forceinline__ void sym4_store(double* out, const double (&acc)[1][4][2], int warp, int lane) {
  const Sym4Pairs p = sym4_pairs(warp);
  for (int s = 0; s < p.count; ++s) {
    double* at = out + (p.ib[s] * 8 + (lane >> 2)) * 32 + p.jb[s] * 8 + 2 * (lane & 3);
    at[0] = acc[0][s][0];
    at[1] = acc[0][s][1];
    if (p.ib[s] != p.jb[s]) {
      double* mirror = out + (p.jb[s] * 8 + (lane >> 2)) * 32 + p.ib[s] * 8 + 2 * (lane & 3);
      mirror[0] = 0.0;
      mirror[1] = 0.0;
    }
  }
}

// MODE 0: mean rows + Gram of A.  MODE 1: Gram of A*M.  MODE 2: absmax (and float32 copy) of A*M.
// MODE 3: codes of A*M.
template <int NP, int MODE>
__global__ void __launch_bounds__(RT) chunk_kernel(const ChunkArgs a) {
  extern __shared__ __align__(16) unsigned char sm[];
  float* As = reinterpret_cast<float*>(sm);                                   // [NP][ASTR]
  double* Ms = reinterpret_cast<double*>(sm + sizeof(float) * NP * ASTR + 8); // [NP][NP]
  double* T = Ms + NP * NP;                                                   // [NP][DSTR] (mode 1; mode 0 keeps its copy at Ms)
  float* Tq = reinterpret_cast<float*>(T);                                    // [NP][ASTR] (modes 2, 3)
  __shared__ unsigned smax[NP];
  const int tid = threadIdx.x;
  constexpr int NB = NP / 8, IBW = (NB + 3) / 4;   // Gram: 8 x 8 blocks; bands of G per warp
  const int warp = tid >> 5, lane = tid & 31;

  if (MODE >= 1)
    for (int i = tid; i < NP * NP; i += RT) Ms[i] = a.M[i];
  if (MODE == 2 && tid < NP) smax[tid] = 0u;
  // Fragment (kb, jb) of M for the products below: M[4 kb + (lane & 3)][8 jb + (lane >> 2)]; kept in
  // registers for NP <= 32 (20 values), read from shared memory for wider bases.
  constexpr bool MREG = NP <= 32;
  double mreg[MREG ? NB * (NP / 4) : 1] = {0.0};
  auto mfrag = [&](int kb, int jb) -> double {
    return MREG ? mreg[jb * (NP / 4) + kb] : Ms[(kb * 4 + (lane & 3)) * NP + jb * 8 + (lane >> 2)];
  };
  double acc[IBW][NB][2];
#pragma unroll
  for (int x = 0; x < IBW; ++x)
#pragma unroll
    for (int y = 0; y < NB; ++y) acc[x][y][0] = acc[x][y][1] = 0.0;
  __syncthreads();
  if (MODE >= 1 && MREG) {
#pragma unroll
    for (int jb = 0; jb < NB; ++jb)
#pragma unroll
      for (int kb = 0; kb < NP / 4; ++kb)
        mreg[jb * (NP / 4) + kb] = kb <= 2 * jb + 1 ? Ms[(kb * 4 + (lane & 3)) * NP + jb * 8 + (lane >> 2)] : 0.0;
  }

  const long long ntiles = (a.rows_padded + RT - 1) / RT;
  for (long long tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
    const long long r = tile * RT + tid;            // row inside the chunk
    const bool valid = r < a.rows;
    // all of the row's loads are issued before the first is used: with four in flight per thread the
    // passes ran at a tenth of the memory rate
    float row[NP];
#pragma unroll
    for (int j = 0; j < NP; ++j) row[j] = (j < a.n && valid) ? __ldcs(a.A + j * a.ld + r) : 0.0f;
#pragma unroll
    for (int j = 0; j < NP; ++j) As[j * ASTR + tid] = row[j];
    __syncthreads();

    if (MODE == 0) {
      if (valid) {
        double s = 0.0;
        for (int j = 0; j < a.n; ++j) s += As[j * ASTR + tid];
        a.wbar[a.row0 + r] = static_cast<float>(s / static_cast<double>(a.n));
      }
      // the tile once more as float64 (Ms is free in this mode)
      double* T0 = Ms;
#pragma unroll
      for (int j = 0; j < NP; ++j) T0[j * DSTR + tid] = static_cast<double>(row[j]);
      __syncthreads();
      if constexpr (NP == 32) gram_accumulate_sym4(T0, acc, warp, lane);
      else gram_accumulate<NP>(T0, acc, warp, lane);
    } else {
      // the tile's rows of A*M, q[r][j] = sum_{i <= j} a[r][i] M[i][j], as float64 tensor-pipe products:
      // warp w takes the 8-row bands 4w .. 4w+3 of the tile; a band's fragment of A serves all column
      // blocks; blocks of M below the diagonal are skipped.  (One thread per row with scalar FMAs
      // took 528 shared-memory reads and as many FMAs per row at n = 32.)
#pragma unroll 1
      for (int u = 0; u < RT / 32; ++u) {
        const int r0 = (warp * (RT / 32) + u) * 8;
        double c[NB][2];
#pragma unroll
        for (int jb = 0; jb < NB; ++jb) c[jb][0] = c[jb][1] = 0.0;
#pragma unroll
        for (int kb = 0; kb < NP / 4; ++kb) {
          const double av = static_cast<double>(As[(kb * 4 + (lane & 3)) * ASTR + r0 + (lane >> 2)]);
#pragma unroll
          for (int jb = kb >> 1; jb < NB; ++jb) dmma_8x8x4(c[jb], av, mfrag(kb, jb));
        }
#pragma unroll
        for (int jb = 0; jb < NB; ++jb) {
          const int col = jb * 8 + 2 * (lane & 3), rr = r0 + (lane >> 2);
          if (MODE == 1) {
            T[col * DSTR + rr] = c[jb][0];
            T[(col + 1) * DSTR + rr] = c[jb][1];
          } else {
            Tq[col * ASTR + rr] = static_cast<float>(c[jb][0]);
            Tq[(col + 1) * ASTR + rr] = static_cast<float>(c[jb][1]);
          }
        }
      }
      __syncthreads();
      if (MODE == 1) {
        if constexpr (NP == 32) gram_accumulate_sym4(T, acc, warp, lane);
        else gram_accumulate<NP>(T, acc, warp, lane);
      } else {
#pragma unroll
        for (int j = 0; j < NP; ++j) {
          const float qf = Tq[j * ASTR + tid];
          if (a.q32 && valid && j < a.n) a.q32[j * a.ldq + r] = qf;
          if (MODE == 2) {
            const unsigned m = __reduce_max_sync(0xFFFFFFFFu, __float_as_uint(qf) & 0x7FFFFFFFu);
            if ((tid & 31) == 0 && j < a.n) atomicMax(&smax[j], m);
          }
        }
        if (MODE == 3) {
          // 16 output bytes per task: 16 rows (8-bit) or 32 rows (4-bit) of one column; the tile of Q just
          // formed serves every target in turn
          for (int tg = 0; tg < a.targets; ++tg) {
            const ChunkArgs::CodeTarget& t = a.target[tg];
            const int rows_per_chunk = 128 / t.bits;
            const int chunks_per_col = RT / rows_per_chunk;
            const float qmax = t.bits == 8 ? 127.0f : 7.0f;
            for (int task = tid; task < a.n * chunks_per_col; task += RT) {
              const int j = task / chunks_per_col, c = task - j * chunks_per_col;
              if (tile * RT + c * rows_per_chunk >= t.rows_padded) continue;   // past this width's last segment
              const float s = t.scales[j];
              const float recip = encode_reciprocal(s);
              const float* src = Tq + j * ASTR + c * rows_per_chunk;
              uint32_t w[4] = {0, 0, 0, 0};
              // by the reciprocal first; the whole group again by the IEEE division if an element came
              // too close to a half-integer (or the scale has no usable reciprocal)
              bool hard = recip == 0.0f;
              if (!hard) {
                if (t.bits == 8) {
#pragma unroll
                  for (int k = 0; k < 16; ++k) {
                    bool h;
                    w[k >> 2] |= (static_cast<uint32_t>(encode_by_reciprocal(src[k], recip, qmax, &h)) & 0xFFu) << (8 * (k & 3));
                    hard |= h;
                  }
                } else {
#pragma unroll
                  for (int k = 0; k < 32; ++k) {
                    bool h;
                    w[k >> 3] |= (static_cast<uint32_t>(encode_by_reciprocal(src[k], recip, qmax, &h)) & 0xFu) << (4 * (k & 7));
                    hard |= h;
                  }
                }
              }
              if (hard) {
                w[0] = w[1] = w[2] = w[3] = 0u;
                if (t.bits == 8) {
#pragma unroll
                  for (int k = 0; k < 16; ++k)
                    w[k >> 2] |= (static_cast<uint32_t>(twa_encode_one(src[k], s, qmax)) & 0xFFu) << (8 * (k & 3));
                } else {
#pragma unroll
                  for (int k = 0; k < 32; ++k)
                    w[k >> 3] |= (static_cast<uint32_t>(twa_encode_one(src[k], s, qmax)) & 0xFu) << (4 * (k & 7));
                }
              }
              const long long qidx = (a.row0 + tile * RT) / rows_per_chunk + c;   // logical 16-byte chunk of the column
              const long long slot = (qidx & ~31LL) | twa_chunk_slot(static_cast<int>(qidx & 31), j);
              reinterpret_cast<uint4*>(t.codes + j * t.stride)[slot] = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
        }
      }
    }
    __syncthreads();
  }

  if (MODE <= 1 && NP == 32) {
    if constexpr (NP == 32) sym4_store(a.partials + static_cast<size_t>(blockIdx.x) * NP * NP, acc, warp, lane);
  } else if (MODE <= 1) {
    double* out = a.partials + static_cast<size_t>(blockIdx.x) * NP * NP;
#pragma unroll
    for (int u = 0; u < IBW; ++u) {
      const int ib = warp + 4 * u;
      if (ib < NB) {
#pragma unroll
        for (int jb = 0; jb < NB; ++jb) {
          double* at = out + (ib * 8 + (lane >> 2)) * NP + jb * 8 + 2 * (lane & 3);
          at[0] = acc[u][jb][0];
          at[1] = acc[u][jb][1];
        }
      }
    }
  }
  if (MODE == 2) {
    __syncthreads();
    if (tid < a.n) atomicMax(&a.absmax[tid], smax[tid]);
  }
}

// G[idx] += sum over blocks of partials[b][idx], in block order
__global__ void gram_combine_kernel(double* G, const double* partials, int blocks, int count) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= count) return;
  double s = 0.0;
  for (int b = 0; b < blocks; ++b) s += partials[static_cast<size_t>(b) * count + idx];
  G[idx] += s;
}

// One block.  R = chol(G) (upper, R^T R = G), X = R^-1; out = X (first) or prev * X (second).
__global__ void factor_kernel(const double* G, const double* prev, double* out, int n, int np,
                              int second, int* status) {
  extern __shared__ double fs[];
  double* R = fs;                  // [np][np]
  double* X = fs + np * np;        // [np][np]
  __shared__ int flag;
  const int t = threadIdx.x;       // blockDim.x == np
  if (t == 0) flag = 0;
  for (int i = 0; i < np; ++i) {
    R[i * np + t] = 0.0;
    X[i * np + t] = 0.0;
  }
  __syncthreads();
  for (int k = 0; k < n; ++k) {
    if (t == 0) {
      double d = G[k * np + k];
      for (int m = 0; m < k; ++m) d -= R[m * np + k] * R[m * np + k];
      const double ref = second ? 1.0 : G[k * np + k];
      if (!isfinite(d) || !isfinite(ref)) {
        if (!flag) { flag = 1; twa_set_status(status, TWA_ERR_NONFINITE, k); }
        d = 1.0;
      } else if (!(d > 1e-10 * ref)) {     // remainder below 1e-5 of the column's length
        if (!flag) { flag = 1; twa_set_status(status, TWA_ERR_RANK_DEFICIENT, k); }
        d = 1.0;
      }
      R[k * np + k] = sqrt(d);
    }
    __syncthreads();
    if (t > k && t < n) {
      double v = G[k * np + t];
      for (int m = 0; m < k; ++m) v -= R[m * np + k] * R[m * np + t];
      R[k * np + t] = v / R[k * np + k];
    }
    __syncthreads();
  }
  if (t < n) {                      // column t of X = R^-1 by back substitution
    X[t * np + t] = 1.0 / R[t * np + t];
    for (int i = t - 1; i >= 0; --i) {
      double v = 0.0;
      for (int m = i + 1; m <= t; ++m) v += R[i * np + m] * X[m * np + t];
      X[i * np + t] = -v / R[i * np + i];
    }
  }
  __syncthreads();
  for (int i = 0; i < np; ++i) {
    double v = 0.0;
    if (i < n && t < n && i <= t) {
      if (second) {
        for (int m = i; m <= t; ++m) v += prev[i * np + m] * X[m * np + t];
      } else {
        v = X[i * np + t];
      }
    }
    out[i * np + t] = v;
  }
}

template <int NP, int MODE>
int launch_chunk(twa_ctx* ctx, const ChunkArgs& a, int grid, int* grid_used) {
  size_t smem = sizeof(float) * NP * ASTR + 8;
  if (MODE >= 1) smem += sizeof(double) * NP * NP;
  if (MODE <= 1) smem += sizeof(double) * NP * DSTR;      // the tile (mode 0) or A*M (mode 1) as float64
  if (MODE >= 2) smem += sizeof(float) * NP * ASTR;        // A*M as float32
  auto kern = chunk_kernel<NP, MODE>;
  static int smem_limit[64] = {0};
  if (smem > 48 * 1024) {
    int rc = twa_ensure_smem(ctx, reinterpret_cast<const void*>(kern), &smem_limit[ctx->device & 63],
                             static_cast<int>(smem));
    if (rc) return rc;
  }
  // as many blocks as are resident at once (three to five per SM, by shared memory): one wave, and the
  // warps of the other blocks cover a block's load and barrier phases
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, RT, smem) != cudaSuccess || per_sm < 1) per_sm = 1;
  const int fit = per_sm * ctx->sm_count;
  if (grid > fit) grid = fit;
  kern<<<grid, RT, smem, ctx->stream>>>(a);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  *grid_used = grid;
  return TWA_OK;
}

template <int MODE>
int launch_chunk_np(twa_ctx* ctx, int np, const ChunkArgs& a, int grid, int* grid_used) {
  switch (np) {
    case 16: return launch_chunk<16, MODE>(ctx, a, grid, grid_used);
    case 32: return launch_chunk<32, MODE>(ctx, a, grid, grid_used);
    case 48: return launch_chunk<48, MODE>(ctx, a, grid, grid_used);
    default: return launch_chunk<64, MODE>(ctx, a, grid, grid_used);
  }
}

}  // namespace

extern "C" {

size_t twa_build_workspace_bytes(int n) {
  if (n < 1 || n > BUILD_MAX_N) return 0;
  return layout_for(padded_n(n)).total;
}

int twa_build_begin(twa_ctx* ctx, int64_t D, int n, float* wbar_out, void* bws, size_t bws_bytes) {
  if (!ctx || !wbar_out || D < 1 || D > TWA_MAX_ROWS || n < 1) return TWA_ERR_INVALID_ARG;
  if (n > BUILD_MAX_N) return TWA_ERR_UNSUPPORTED;
  const BuildLayout l = layout_for(padded_n(n));
  if (!bws || bws_bytes < l.total) return TWA_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(bws) & 15) return TWA_ERR_MISALIGNED;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  TWA_CUDA_OK(ctx, cudaMemsetAsync(bws, 0, l.partials, ctx->stream));
  ctx->build_D = D;
  ctx->build_n = n;
  ctx->build_wbar = wbar_out;
  ctx->build_ws = static_cast<char*>(bws);
  return TWA_OK;
}

}  // extern "C"

namespace {

// twa_build_feed; in pass 3 `Pq` is a host array of `widths` (1 or 2) quantised bases.
int build_feed(twa_ctx* ctx, int pass, const float* chunk, int64_t ldc, int64_t row0, int64_t rows,
               const twa_basis* Pq, int widths, float* q32_out, int64_t ldq) {
  if (!ctx || !ctx->build_ws || !chunk || pass < 0 || pass > 3) return TWA_ERR_INVALID_ARG;
  const long long D = ctx->build_D;
  const int n = ctx->build_n, np = padded_n(n);
  if (rows < 1 || row0 < 0 || row0 + rows > D || ldc < rows) return TWA_ERR_INVALID_ARG;
  // chunks start and (except the last) end on whole code segments
  if (row0 % 1024 != 0 || (row0 + rows != D && rows % 1024 != 0)) return TWA_ERR_MISALIGNED;
  if (q32_out && ldq < rows) return TWA_ERR_INVALID_ARG;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  const BuildLayout l = layout_for(np);
  char* ws = ctx->build_ws;
  ChunkArgs a;
  a.A = chunk;
  a.ld = ldc;
  a.rows = rows;
  a.rows_padded = rows;
  a.row0 = row0;
  a.D = D;
  a.n = n;
  a.M = reinterpret_cast<const double*>(ws + (pass == 1 ? l.r1inv : l.rinv));
  a.partials = reinterpret_cast<double*>(ws + l.partials);
  a.wbar = ctx->build_wbar;
  a.absmax = reinterpret_cast<unsigned*>(ws + l.absmax);
  a.q32 = (pass >= 2) ? q32_out : nullptr;
  a.ldq = ldq;
  a.targets = 0;
  if (pass == 3) {
    if (!Pq || widths < 1 || widths > 2) return TWA_ERR_INVALID_ARG;
    for (int k = 0; k < widths; ++k) {
      const twa_basis& q = Pq[k];
      if (!q.data || !q.scales || (q.bits != 8 && q.bits != 4) || q.D != D || q.n != n) return TWA_ERR_INVALID_ARG;
      ChunkArgs::CodeTarget& t = a.target[k];
      t.codes = static_cast<unsigned char*>(q.data);
      t.stride = q.col_stride;
      t.scales = q.scales;
      t.bits = q.bits;
      t.rows_padded = rows;
      if (row0 + rows == D) {
        // the last chunk also fills the rest of the width's last 512-byte segment with the code 0
        const long long seg_rows = 512LL * 8 / q.bits;
        t.rows_padded = (D + seg_rows - 1) / seg_rows * seg_rows - row0;
      }
      if (t.rows_padded > a.rows_padded) a.rows_padded = t.rows_padded;
    }
    a.targets = widths;
  }
  long long tiles = (a.rows_padded + RT - 1) / RT;
  int grid = static_cast<int>(tiles < MAX_BLOCKS ? tiles : MAX_BLOCKS);     // cut to one resident wave at the launch
  int rc;
  switch (pass) {
    case 0: rc = launch_chunk_np<0>(ctx, np, a, grid, &grid); break;
    case 1: rc = launch_chunk_np<1>(ctx, np, a, grid, &grid); break;
    case 2: rc = launch_chunk_np<2>(ctx, np, a, grid, &grid); break;
    default: rc = launch_chunk_np<3>(ctx, np, a, grid, &grid); break;
  }
  if (rc) return rc;
  if (pass <= 1) {
    const int count = np * np;
    gram_combine_kernel<<<(count + 255) / 256, 256, 0, ctx->stream>>>(
        reinterpret_cast<double*>(ws + l.g), a.partials, grid, count);
    TWA_CUDA_OK(ctx, cudaGetLastError());
  }
  return TWA_OK;
}

}  // namespace

extern "C" {

int twa_build_feed(twa_ctx* ctx, int pass, const float* chunk, int64_t ldc, int64_t row0, int64_t rows,
                   const twa_basis* Pq, float* q32_out, int64_t ldq) {
  return build_feed(ctx, pass, chunk, ldc, row0, rows, Pq, 1, q32_out, ldq);
}

int twa_build_feed_codes(twa_ctx* ctx, const float* chunk, int64_t ldc, int64_t row0, int64_t rows,
                         const twa_basis* Pq, int widths, float* q32_out, int64_t ldq) {
  return build_feed(ctx, 3, chunk, ldc, row0, rows, Pq, widths, q32_out, ldq);
}

int twa_build_end_pass(twa_ctx* ctx, int pass, int bits, twa_basis* Pq) {
  if (!ctx || !ctx->build_ws || pass < 0 || pass > 3) return TWA_ERR_INVALID_ARG;
  const int n = ctx->build_n, np = padded_n(n);
  const BuildLayout l = layout_for(np);
  char* ws = ctx->build_ws;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  double* G = reinterpret_cast<double*>(ws + l.g);
  const size_t fsmem = 2 * sizeof(double) * np * np;
  if (pass <= 1) {
    static int smem_limit[64] = {0};
    if (fsmem > 48 * 1024) {
      int rc = twa_ensure_smem(ctx, reinterpret_cast<const void*>(factor_kernel),
                               &smem_limit[ctx->device & 63], static_cast<int>(fsmem));
      if (rc) return rc;
    }
    factor_kernel<<<1, np, fsmem, ctx->stream>>>(
        G, reinterpret_cast<const double*>(ws + l.r1inv),
        reinterpret_cast<double*>(ws + (pass == 0 ? l.r1inv : l.rinv)), n, np, pass, ctx->d_status);
    TWA_CUDA_OK(ctx, cudaGetLastError());
    TWA_CUDA_OK(ctx, cudaMemsetAsync(G, 0, sizeof(double) * np * np, ctx->stream));
    return TWA_OK;
  }
  if (pass == 2) {
    if (bits == 32) return TWA_OK;
    if (bits != 8 && bits != 4) return TWA_ERR_UNSUPPORTED;
    if (!Pq || !Pq->data || !Pq->scales) return TWA_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(Pq->data) & 15) return TWA_ERR_MISALIGNED;
    int rc = twa_launch_scales(ctx, reinterpret_cast<const unsigned*>(ws + l.absmax), n, bits, Pq->scales);
    if (rc) return rc;
    Pq->D = ctx->build_D;
    Pq->col_stride = twa_basis_col_stride(ctx->build_D, bits);
    Pq->n = n;
    Pq->bits = bits;
    return TWA_OK;
  }
  ctx->build_ws = nullptr;      // pass 3 done: the build is over
  return TWA_OK;
}

}  // extern "C"
