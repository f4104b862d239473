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

namespace {

constexpr int RT = 128;                 // rows per tile = threads per block
constexpr int ASTR = RT + 1;            // padded strides: conflict-free column-strided reads
constexpr int MAX_BLOCKS = 512;
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
  unsigned char* codes;     // mode 3
  long long code_stride;
  const float* scales;
  int bits;
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

// MODE 0: mean rows + Gram of A.  MODE 1: Gram of A*M.  MODE 2: absmax (and float32 copy) of A*M.
// MODE 3: codes of A*M.
template <int NP, int MODE>
__global__ void __launch_bounds__(RT) chunk_kernel(const ChunkArgs a) {
  extern __shared__ __align__(16) unsigned char sm[];
  float* As = reinterpret_cast<float*>(sm);                                   // [NP][ASTR]
  double* Ms = reinterpret_cast<double*>(sm + sizeof(float) * NP * ASTR + 8); // [NP][NP]
  double* T = Ms + NP * NP;                                                   // [NP][ASTR] (mode 1; mode 0 keeps its copy at Ms)
  float* Tq = reinterpret_cast<float*>(T);                                    // [NP][ASTR] (mode 3)
  __shared__ unsigned smax[NP];
  const int tid = threadIdx.x;
  constexpr int IB = NP / 8, JB = NP / 16;
  const int ti = tid >> 4, tj = tid & 15;          // Gram: rows ti + 8a, columns tj + 16b

  if (MODE >= 1)
    for (int i = tid; i < NP * NP; i += RT) Ms[i] = a.M[i];
  if (MODE == 2 && tid < NP) smax[tid] = 0u;
  double acc[IB][JB];
#pragma unroll
  for (int x = 0; x < IB; ++x)
#pragma unroll
    for (int y = 0; y < JB; ++y) acc[x][y] = 0.0;
  __syncthreads();

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
      // the tile once more as float64 (Ms is free in this mode): one conversion per element instead
      // of six per product group in the loop below, which made this pass the slowest of the four
      double* T0 = Ms;
#pragma unroll
      for (int j = 0; j < NP; ++j) T0[j * ASTR + tid] = static_cast<double>(row[j]);
      __syncthreads();
#pragma unroll 2
      for (int k = 0; k < RT; ++k) {
        double x[IB], y[JB];
#pragma unroll
        for (int u = 0; u < IB; ++u) x[u] = T0[(ti + 8 * u) * ASTR + k];
#pragma unroll
        for (int v = 0; v < JB; ++v) y[v] = T0[(tj + 16 * v) * ASTR + k];
#pragma unroll
        for (int u = 0; u < IB; ++u)
#pragma unroll
          for (int v = 0; v < JB; ++v) acc[u][v] = fma(x[u], y[v], acc[u][v]);
      }
    } else {
      // this thread's row of A*M: q[j] = sum_{i <= j} a_i M[i][j]
      double q[NP];
#pragma unroll
      for (int j = 0; j < NP; ++j) q[j] = 0.0;
#pragma unroll
      for (int i = 0; i < NP; ++i) {
        const double ai = As[i * ASTR + tid];
#pragma unroll
        for (int j = i; j < NP; ++j) q[j] = fma(ai, Ms[i * NP + j], q[j]);
      }
      if (MODE == 1) {
#pragma unroll
        for (int j = 0; j < NP; ++j) T[j * ASTR + tid] = q[j];
        __syncthreads();
#pragma unroll 2
        for (int k = 0; k < RT; ++k) {
          double x[IB], y[JB];
#pragma unroll
          for (int u = 0; u < IB; ++u) x[u] = T[(ti + 8 * u) * ASTR + k];
#pragma unroll
          for (int v = 0; v < JB; ++v) y[v] = T[(tj + 16 * v) * ASTR + k];
#pragma unroll
          for (int u = 0; u < IB; ++u)
#pragma unroll
            for (int v = 0; v < JB; ++v) acc[u][v] = fma(x[u], y[v], acc[u][v]);
        }
      } else {
#pragma unroll
        for (int j = 0; j < NP; ++j) {
          const float qf = static_cast<float>(q[j]);
          if (a.q32 && valid && j < a.n) a.q32[j * a.ldq + r] = qf;
          if (MODE == 2) {
            const unsigned m = __reduce_max_sync(0xFFFFFFFFu, __float_as_uint(qf) & 0x7FFFFFFFu);
            if ((tid & 31) == 0 && j < a.n) atomicMax(&smax[j], m);
          } else {
            Tq[j * ASTR + tid] = qf;
          }
        }
        if (MODE == 3) {
          __syncthreads();
          // 16 output bytes per task: 16 rows (8-bit) or 32 rows (4-bit) of one column
          const int rows_per_chunk = 128 / a.bits;
          const int chunks_per_col = RT / rows_per_chunk;
          const float qmax = a.bits == 8 ? 127.0f : 7.0f;
          for (int task = tid; task < a.n * chunks_per_col; task += RT) {
            const int j = task / chunks_per_col, c = task - j * chunks_per_col;
            const float s = a.scales[j];
            const float* src = Tq + j * ASTR + c * rows_per_chunk;
            uint32_t w[4] = {0, 0, 0, 0};
            if (a.bits == 8) {
#pragma unroll
              for (int k = 0; k < 16; ++k)
                w[k >> 2] |= (static_cast<uint32_t>(twa_encode_one(src[k], s, qmax)) & 0xFFu) << (8 * (k & 3));
            } else {
#pragma unroll
              for (int k = 0; k < 32; ++k)
                w[k >> 3] |= (static_cast<uint32_t>(twa_encode_one(src[k], s, qmax)) & 0xFu) << (4 * (k & 7));
            }
            const long long qidx = (a.row0 + tile * RT) / rows_per_chunk + c;   // logical 16-byte chunk of the column
            const long long slot = (qidx & ~31LL) | twa_chunk_slot(static_cast<int>(qidx & 31), j);
            reinterpret_cast<uint4*>(a.codes + j * a.code_stride)[slot] = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
    }
    __syncthreads();
  }

  if (MODE <= 1) {
    double* out = a.partials + static_cast<size_t>(blockIdx.x) * NP * NP;
#pragma unroll
    for (int u = 0; u < IB; ++u)
#pragma unroll
      for (int v = 0; v < JB; ++v) out[(ti + 8 * u) * NP + tj + 16 * v] = acc[u][v];
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
int launch_chunk(twa_ctx* ctx, const ChunkArgs& a, int grid) {
  size_t smem = sizeof(float) * NP * ASTR + 8;
  if (MODE >= 1) smem += sizeof(double) * NP * NP;
  if (MODE <= 1) smem += sizeof(double) * NP * ASTR;      // the tile (mode 0) or A*M (mode 1) as float64
  if (MODE == 3) smem += sizeof(float) * NP * ASTR;
  auto kern = chunk_kernel<NP, MODE>;
  static int smem_limit[64] = {0};
  if (smem > 48 * 1024) {
    int rc = twa_ensure_smem(ctx, reinterpret_cast<const void*>(kern), &smem_limit[ctx->device & 63],
                             static_cast<int>(smem));
    if (rc) return rc;
  }
  kern<<<grid, RT, smem, ctx->stream>>>(a);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}

template <int MODE>
int launch_chunk_np(twa_ctx* ctx, int np, const ChunkArgs& a, int grid) {
  switch (np) {
    case 16: return launch_chunk<16, MODE>(ctx, a, grid);
    case 32: return launch_chunk<32, MODE>(ctx, a, grid);
    case 48: return launch_chunk<48, MODE>(ctx, a, grid);
    default: return launch_chunk<64, MODE>(ctx, a, grid);
  }
}

}  // namespace

extern "C" {

size_t twa_build_workspace_bytes(int n) {
  if (n < 1 || n > BUILD_MAX_N) return 0;
  return layout_for(padded_n(n)).total;
}

int twa_build_begin(twa_ctx* ctx, int64_t D, int n, float* wbar_out, void* bws, size_t bws_bytes) {
  if (!ctx || !wbar_out || D < 1 || D >= (1LL << 31) || n < 1) return TWA_ERR_INVALID_ARG;
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

int twa_build_feed(twa_ctx* ctx, int pass, const float* chunk, int64_t ldc, int64_t row0, int64_t rows,
                   const twa_basis* Pq, float* q32_out, int64_t ldq) {
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
  a.codes = nullptr;
  a.code_stride = 0;
  a.scales = nullptr;
  a.bits = 8;
  if (pass == 3) {
    if (!Pq || !Pq->data || !Pq->scales || (Pq->bits != 8 && Pq->bits != 4) || Pq->D != D || Pq->n != n)
      return TWA_ERR_INVALID_ARG;
    a.codes = static_cast<unsigned char*>(Pq->data);
    a.code_stride = Pq->col_stride;
    a.scales = Pq->scales;
    a.bits = Pq->bits;
    if (row0 + rows == D) {
      // the last chunk also fills the rest of the last 512-byte segment with the code 0
      const long long seg_rows = 512LL * 8 / Pq->bits;
      a.rows_padded = (D + seg_rows - 1) / seg_rows * seg_rows - row0;
    }
  }
  long long tiles = (a.rows_padded + RT - 1) / RT;
  int grid = static_cast<int>(tiles < MAX_BLOCKS ? tiles : MAX_BLOCKS);
  const int cap = ctx->sm_count * 3;
  if (grid > cap) grid = cap;
  if (grid > MAX_BLOCKS) grid = MAX_BLOCKS;
  int rc;
  switch (pass) {
    case 0: rc = launch_chunk_np<0>(ctx, np, a, grid); break;
    case 1: rc = launch_chunk_np<1>(ctx, np, a, grid); break;
    case 2: rc = launch_chunk_np<2>(ctx, np, a, grid); break;
    default: rc = launch_chunk_np<3>(ctx, np, a, grid); break;
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
