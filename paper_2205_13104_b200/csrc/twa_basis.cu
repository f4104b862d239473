// Subspace construction and low-bit storage: mean of the candidates, classical Gram-Schmidt
// with re-orthogonalisation (Section 4.1 of the paper), per-column absmax quantisation
// (the symmetric per-column variant of Section 4.6) and the canonical export / import.
#include <math.h>
#include <stdio.h>

#include "twa_common.cuh"
#include "twa_quant.cuh"

namespace {

constexpr int BLOCK = 256;

// ---- mean ---------------------------------------------------------------------------------
// One thread owns four consecutive rows and walks the n columns in index order.
__global__ void __launch_bounds__(BLOCK) mean_kernel(const float* __restrict__ W, long long D, int n,
                                                     long long ldw, float* __restrict__ out) {
  const long long nvec = D >> 2;
  const double dn = static_cast<double>(n);
  for (long long v = blockIdx.x * static_cast<long long>(BLOCK) + threadIdx.x; v < nvec;
       v += static_cast<long long>(gridDim.x) * BLOCK) {
    double s0 = 0, s1 = 0, s2 = 0, s3 = 0;
#pragma unroll 8
    for (int i = 0; i < n; ++i) {
      const float4 x = __ldcs(reinterpret_cast<const float4*>(W + i * ldw) + v);
      s0 += x.x; s1 += x.y; s2 += x.z; s3 += x.w;
    }
    out[4 * v + 0] = static_cast<float>(s0 / dn);
    out[4 * v + 1] = static_cast<float>(s1 / dn);
    out[4 * v + 2] = static_cast<float>(s2 / dn);
    out[4 * v + 3] = static_cast<float>(s3 / dn);
  }
  if (blockIdx.x == 0 && threadIdx.x < (D & 3)) {
    const long long r = (nvec << 2) + threadIdx.x;
    double s = 0;
    for (int i = 0; i < n; ++i) s += W[i * ldw + r];
    out[r] = static_cast<float>(s / dn);
  }
}

// ---- squared norm of a column ----------------------------------------------------------------
__device__ __forceinline__ double block_sum(double v, double* sh) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) sh[warp] = v;
  __syncthreads();
  double t = 0;
  if (threadIdx.x == 0)
    for (int w = 0; w < BLOCK / 32; ++w) t += sh[w];
  return t;   // valid in thread 0
}

__global__ void __launch_bounds__(BLOCK) sumsq_kernel(const float* __restrict__ v, long long D,
                                                      double* __restrict__ dpart,
                                                      double* __restrict__ result,
                                                      unsigned* __restrict__ ticket) {
  __shared__ double sh[BLOCK / 32];
  __shared__ int last;
  const long long nvec = D >> 2;
  double s = 0;
  for (long long i = blockIdx.x * static_cast<long long>(BLOCK) + threadIdx.x; i < nvec;
       i += static_cast<long long>(gridDim.x) * BLOCK) {
    const float4 x = reinterpret_cast<const float4*>(v)[i];
    s += static_cast<double>(x.x) * x.x + static_cast<double>(x.y) * x.y +
         static_cast<double>(x.z) * x.z + static_cast<double>(x.w) * x.w;
  }
  if (blockIdx.x == 0 && threadIdx.x < (D & 3)) {
    const double x = v[(nvec << 2) + threadIdx.x];
    s += x * x;
  }
  const double bs = block_sum(s, sh);
  if (threadIdx.x == 0) {
    dpart[blockIdx.x] = bs;
    __threadfence();
    last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
  }
  __syncthreads();
  if (last && threadIdx.x == 0) {
    __threadfence();
    double t = 0;
    for (unsigned b = 0; b < gridDim.x; ++b) t += __ldcg(&dpart[b]);
    *result = t;
    *ticket = 0u;
  }
}

// ---- sweeps inside a panel: a column against at most 7 earlier columns -------------------------
constexpr int INPANEL = 7;

// coef[i] = sum_r Q_i[r] v[r], i < cnt: products and sums in float64, blocks combined in block order.
__global__ void __launch_bounds__(BLOCK) inpanel_dots_kernel(const float* __restrict__ Q0, long long ld, int cnt,
                                                             const float* __restrict__ v, long long D,
                                                             double* __restrict__ dpart, float* __restrict__ coef,
                                                             unsigned* __restrict__ ticket, int* status, int detail) {
  __shared__ double sh[INPANEL][BLOCK / 32];
  __shared__ int last;
  const long long nvec = D >> 2;
  double s[INPANEL];
#pragma unroll
  for (int i = 0; i < INPANEL; ++i) s[i] = 0.0;
  for (long long t = blockIdx.x * static_cast<long long>(BLOCK) + threadIdx.x; t < nvec;
       t += static_cast<long long>(gridDim.x) * BLOCK) {
    const float4 x = reinterpret_cast<const float4*>(v)[t];
#pragma unroll
    for (int i = 0; i < INPANEL; ++i) {
      if (i < cnt) {
        const float4 q = __ldcs(reinterpret_cast<const float4*>(Q0 + i * ld) + t);
        s[i] += static_cast<double>(x.x) * q.x + static_cast<double>(x.y) * q.y + static_cast<double>(x.z) * q.z +
                static_cast<double>(x.w) * q.w;
      }
    }
  }
  if (blockIdx.x == 0 && threadIdx.x < (D & 3)) {
    const long long r = (nvec << 2) + threadIdx.x;
    for (int i = 0; i < cnt; ++i) s[i] += static_cast<double>(v[r]) * Q0[i * ld + r];
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
  for (int i = 0; i < INPANEL; ++i) {
    double t = s[i];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, off);
    if (lane == 0) sh[i][warp] = t;
  }
  __syncthreads();
  if (threadIdx.x < INPANEL) {
    double t = 0;
    for (int w = 0; w < BLOCK / 32; ++w) t += sh[threadIdx.x][w];
    dpart[static_cast<size_t>(blockIdx.x) * 8 + threadIdx.x] = t;
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
  __syncthreads();
  if (last) {
    __threadfence();
    if (threadIdx.x < cnt) {
      double t = 0;
      for (unsigned b = 0; b < gridDim.x; ++b) t += __ldcg(&dpart[static_cast<size_t>(b) * 8 + threadIdx.x]);
      if (!isfinite(t)) twa_set_status(status, TWA_ERR_NONFINITE, detail);
      coef[threadIdx.x] = static_cast<float>(t);
    }
    if (threadIdx.x == 0) *ticket = 0u;
  }
}

// v <- v - sum_i coef[i] Q_i (float32, the coefficients applied in index order), and
// *result = sum of the squares of the stored values (float64).
__global__ void __launch_bounds__(BLOCK) inpanel_update_kernel(const float* __restrict__ Q0, long long ld, int cnt,
                                                               float* __restrict__ v, long long D,
                                                               const float* __restrict__ coef,
                                                               double* __restrict__ dpart, double* __restrict__ result,
                                                               unsigned* __restrict__ ticket) {
  __shared__ double sh[BLOCK / 32];
  __shared__ int last;
  float c[INPANEL];
#pragma unroll
  for (int i = 0; i < INPANEL; ++i) c[i] = i < cnt ? coef[i] : 0.0f;
  const long long nvec = D >> 2;
  double s = 0;
  for (long long t = blockIdx.x * static_cast<long long>(BLOCK) + threadIdx.x; t < nvec;
       t += static_cast<long long>(gridDim.x) * BLOCK) {
    float4 x = reinterpret_cast<const float4*>(v)[t];
#pragma unroll
    for (int i = 0; i < INPANEL; ++i) {
      if (i < cnt) {
        const float4 q = __ldcs(reinterpret_cast<const float4*>(Q0 + i * ld) + t);
        x.x = fmaf(-c[i], q.x, x.x); x.y = fmaf(-c[i], q.y, x.y);
        x.z = fmaf(-c[i], q.z, x.z); x.w = fmaf(-c[i], q.w, x.w);
      }
    }
    reinterpret_cast<float4*>(v)[t] = x;
    s += static_cast<double>(x.x) * x.x + static_cast<double>(x.y) * x.y + static_cast<double>(x.z) * x.z +
         static_cast<double>(x.w) * x.w;
  }
  if (blockIdx.x == 0 && threadIdx.x < (D & 3)) {
    const long long r = (nvec << 2) + threadIdx.x;
    float x = v[r];
    for (int i = 0; i < cnt; ++i) x = fmaf(-c[i], Q0[i * ld + r], x);
    v[r] = x;
    s += static_cast<double>(x) * x;
  }
  const double bs = block_sum(s, sh);
  if (threadIdx.x == 0) {
    dpart[blockIdx.x] = bs;
    __threadfence();
    last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
  }
  __syncthreads();
  if (last && threadIdx.x == 0) {
    __threadfence();
    double t = 0;
    for (unsigned b = 0; b < gridDim.x; ++b) t += __ldcg(&dpart[b]);
    *result = t;
    *ticket = 0u;
  }
}

// ---- normalise a column: v <- v / |v|, with the rank and finiteness checks -------------------
__global__ void __launch_bounds__(BLOCK) normalise_kernel(float* __restrict__ v, long long D,
                                                          const double* __restrict__ norm_before,
                                                          const double* __restrict__ norm_after, int column,
                                                          int* status) {
  const double na = *norm_before, nv = *norm_after;
  double f;
  if (!isfinite(na) || !isfinite(nv)) {
    if (blockIdx.x == 0 && threadIdx.x == 0) twa_set_status(status, TWA_ERR_NONFINITE, column);
    f = 0.0;
  } else if (!(sqrt(nv) > 1e-5 * sqrt(na))) {
    if (blockIdx.x == 0 && threadIdx.x == 0) twa_set_status(status, TWA_ERR_RANK_DEFICIENT, column);
    f = 0.0;
  } else {
    f = 1.0 / sqrt(nv);
  }
  const long long nvec = D >> 2;
  for (long long i = blockIdx.x * static_cast<long long>(BLOCK) + threadIdx.x; i < nvec;
       i += static_cast<long long>(gridDim.x) * BLOCK) {
    float4 x = reinterpret_cast<float4*>(v)[i];
    x.x = static_cast<float>(x.x * f); x.y = static_cast<float>(x.y * f);
    x.z = static_cast<float>(x.z * f); x.w = static_cast<float>(x.w * f);
    reinterpret_cast<float4*>(v)[i] = x;
  }
  if (blockIdx.x == 0 && threadIdx.x < (D & 3)) {
    const long long r = (nvec << 2) + threadIdx.x;
    v[r] = static_cast<float>(v[r] * f);
  }
}

// ---- quantiser -------------------------------------------------------------------------------
// Bit pattern of |x|: ordering as unsigned integers equals ordering of the magnitudes, and
// every NaN or Inf compares above every finite value, so non-finite input surfaces in the max.
__global__ void __launch_bounds__(BLOCK) absmax_kernel(const float* __restrict__ P, long long D,
                                                       long long ld, unsigned* __restrict__ absmax) {
  __shared__ unsigned sh[BLOCK / 32];
  const float* col = P + blockIdx.y * ld;
  const long long nvec = D >> 2;
  unsigned m = 0;
  for (long long i = blockIdx.x * static_cast<long long>(BLOCK) + threadIdx.x; i < nvec;
       i += static_cast<long long>(gridDim.x) * BLOCK) {
    const uint4 x = reinterpret_cast<const uint4*>(col)[i];
    m = max(m, x.x & 0x7FFFFFFFu); m = max(m, x.y & 0x7FFFFFFFu);
    m = max(m, x.z & 0x7FFFFFFFu); m = max(m, x.w & 0x7FFFFFFFu);
  }
  if (blockIdx.x == 0 && threadIdx.x < (D & 3))
    m = max(m, __float_as_uint(col[(nvec << 2) + threadIdx.x]) & 0x7FFFFFFFu);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, off));
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < BLOCK / 32; ++w) m = max(m, sh[w]);
    atomicMax(&absmax[blockIdx.y], m);
  }
}

__global__ void scales_kernel(const unsigned* __restrict__ absmax, int n, float qmax,
                              float* __restrict__ scales, int* status) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= n) return;
  const unsigned b = absmax[j];
  if (b >= 0x7F800000u) {
    twa_set_status(status, TWA_ERR_NONFINITE, j);
    scales[j] = 0.0f;
  } else {
    scales[j] = __fdiv_rn(__uint_as_float(b), qmax);
  }
}

// Rows r .. r + 3 of a column; rows from D on read as zero.
__device__ __forceinline__ float4 load_four(const float* __restrict__ col, long long r, long long D) {
  if (r + 3 < D) return __ldcs(reinterpret_cast<const float4*>(col + r));
  float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
  if (r < D) x.x = col[r];
  if (r + 1 < D) x.y = col[r + 1];
  if (r + 2 < D) x.z = col[r + 2];
  return x;
}

// Four codes as the low bytes (BITS == 8) or nibbles (BITS == 4) of a word, x.x first.  `recip`:
// RN(1 / s), or 0 when every element takes the division (s zero, or so small that its reciprocal is
// not finite).
template <int BITS>
__device__ __forceinline__ uint32_t encode_four(float4 x, float s, float recip) {
  constexpr float QMAX = BITS == 8 ? 127.0f : 7.0f;
  constexpr uint32_t MASK = BITS == 8 ? 0xFFu : 0xFu;    // two's-complement byte or nibble
  int c0, c1, c2, c3;
  bool h0, h1, h2, h3;
  c0 = encode_by_reciprocal(x.x, recip, QMAX, &h0);
  c1 = encode_by_reciprocal(x.y, recip, QMAX, &h1);
  c2 = encode_by_reciprocal(x.z, recip, QMAX, &h2);
  c3 = encode_by_reciprocal(x.w, recip, QMAX, &h3);
  if (recip == 0.0f || h0 || h1 || h2 || h3) {
    c0 = twa_encode_one(x.x, s, QMAX);
    c1 = twa_encode_one(x.y, s, QMAX);
    c2 = twa_encode_one(x.z, s, QMAX);
    c3 = twa_encode_one(x.w, s, QMAX);
  }
  return (static_cast<uint32_t>(c0) & MASK) | ((static_cast<uint32_t>(c1) & MASK) << BITS) |
         ((static_cast<uint32_t>(c2) & MASK) << (2 * BITS)) | ((static_cast<uint32_t>(c3) & MASK) << (3 * BITS));
}

// A warp produces one aligned 128-byte line of a column's codes per step -- 128 rows at 8 bits, 256
// at 4 -- including the padding up to the column stride, which is filled with the code 0.  A lane
// reads four consecutive rows (the warp 512 contiguous bytes per load) and stores one 32-bit word;
// the permutation of the 16-byte chunks stays inside the line, so every store covers the whole line.
// At 4 bits a lane encodes four rows of each half of the line and neighbouring lanes swap one half:
// even lanes complete words of the first half, odd lanes of the second.
template <int BITS>
__global__ void __launch_bounds__(BLOCK) encode_kernel(const float* __restrict__ P, long long D,
                                                       long long ld, const float* __restrict__ scales,
                                                       unsigned char* __restrict__ out,
                                                       long long out_stride) {
  constexpr int LINE_ROWS = 1024 / BITS;
  constexpr int UNROLL = 4;                           // lines a warp has in flight
  const int j = blockIdx.y;
  const float* col = P + j * ld;
  const float s = scales[j];
  const float recip = encode_reciprocal(s);
  unsigned char* dst = out + j * out_stride;
  const long long lines = out_stride / 128;
  const int lane = threadIdx.x & 31;
  const long long warp0 = (blockIdx.x * static_cast<long long>(BLOCK / 32) + (threadIdx.x >> 5)) * UNROLL;
  const long long step = static_cast<long long>(gridDim.x) * (BLOCK / 32) * UNROLL;
  // where this lane's word goes inside a line
  int byte;
  if (BITS == 8) byte = 4 * lane;
  else byte = (lane & 1) ? 64 + 2 * (lane - 1) : 2 * lane;
  for (long long l0 = warp0; l0 < lines; l0 += step) {
    // every load of the step first, then the arithmetic
    float4 xa[UNROLL], xb[BITS == 4 ? UNROLL : 1];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const long long r0 = (l0 + u) * LINE_ROWS;
      xa[u] = load_four(col, r0 + 4 * lane, D);
      if (BITS == 4) xb[u] = load_four(col, r0 + 128 + 4 * lane, D);
    }
    uint32_t w[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      if (BITS == 8) {
        w[u] = encode_four<8>(xa[u], s, recip);
      } else {
        const uint32_t ha = encode_four<4>(xa[u], s, recip);
        const uint32_t hb = encode_four<4>(xb[BITS == 4 ? u : 0], s, recip);
        const uint32_t got = __shfl_xor_sync(0xFFFFFFFFu, (lane & 1) ? ha : hb, 1);
        w[u] = (lane & 1) ? (got | (hb << 16)) : (ha | (got << 16));
      }
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      if (l0 + u < lines) {
        const long long q = (l0 + u) * 8 + (byte >> 4);                      // logical 16-byte chunk
        const long long slot = (q & ~31LL) | twa_chunk_slot(static_cast<int>(q & 31), j);
        *reinterpret_cast<uint32_t*>(dst + slot * 16 + (byte & 15)) = w[u];
      }
    }
  }
}

// Position of logical byte b of column j in the internal (chunk-permuted) order.
__device__ __forceinline__ long long internal_pos(long long b, int j) {
  const long long q = b >> 4;
  return (((q & ~31LL) | twa_chunk_slot(static_cast<int>(q & 31), j)) << 4) | (b & 15);
}

// internal (chunk-permuted, padded) -> canonical (tight); `mask` is XORed into every byte (0 today:
// both images hold two's-complement codes)
__global__ void __launch_bounds__(BLOCK) export_kernel(const unsigned char* __restrict__ in,
                                                       long long in_stride,
                                                       unsigned char* __restrict__ out,
                                                       long long row_bytes, unsigned char mask) {
  const int j = blockIdx.y;
  const unsigned char* src = in + j * in_stride;
  unsigned char* dst = out + j * row_bytes;
  for (long long b = blockIdx.x * static_cast<long long>(BLOCK) + threadIdx.x; b < row_bytes;
       b += static_cast<long long>(gridDim.x) * BLOCK)
    dst[b] = static_cast<unsigned char>(src[internal_pos(b, j)] ^ mask);
}

// canonical -> internal; bytes between the end of the column and the stride get the code 0
__global__ void __launch_bounds__(BLOCK) import_kernel(const unsigned char* __restrict__ in,
                                                       long long row_bytes,
                                                       unsigned char* __restrict__ out,
                                                       long long out_stride, unsigned char mask) {
  const int j = blockIdx.y;
  const unsigned char* src = in + j * row_bytes;
  unsigned char* dst = out + j * out_stride;
  for (long long b = blockIdx.x * static_cast<long long>(BLOCK) + threadIdx.x; b < out_stride;
       b += static_cast<long long>(gridDim.x) * BLOCK)
    dst[internal_pos(b, j)] = (b < row_bytes) ? static_cast<unsigned char>(src[b] ^ mask) : mask;
}

// Blocks of `kernel` (BLOCK threads, no dynamic shared memory) that fit on the device at once: a grid of
// that many blocks, or a divisor of it, runs as one wave with no tail.
template <typename K>
int resident_blocks(const twa_ctx* ctx, K kernel) {
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, BLOCK, 0) != cudaSuccess || per_sm < 1) per_sm = 1;
  return per_sm * ctx->sm_count;
}

int grid_for(const twa_ctx* ctx, long long items, int per_block, int blocks_per_sm) {
  long long g = (items + per_block - 1) / per_block;
  const long long cap = static_cast<long long>(ctx->sm_count) * blocks_per_sm;
  if (g > cap) g = cap;
  if (g > TWA_MAX_GRID) g = TWA_MAX_GRID;
  if (g < 1) g = 1;
  return static_cast<int>(g);
}

// Codes of every column of P32 into Pq->data with the scales already in Pq->scales.
int launch_encode(twa_ctx* ctx, const twa_basis* P32, int bits, const twa_basis* Pq) {
  const long long stride = twa_basis_col_stride(P32->D, bits);
  const long long steps = (stride / 128 + 3) / 4;                    // warp steps per column (4 lines each)
  const long long want = (steps + BLOCK / 32 - 1) / (BLOCK / 32);    // blocks that have work, per column
  const int fit = bits == 8 ? resident_blocks(ctx, encode_kernel<8>) : resident_blocks(ctx, encode_kernel<4>);
  long long per_col = fit / P32->n;
  if (per_col > want) per_col = want;
  if (per_col < 1) per_col = 1;
  const dim3 grid(static_cast<unsigned>(per_col), P32->n);
  const float* P = static_cast<const float*>(P32->data);
  unsigned char* out = static_cast<unsigned char*>(Pq->data);
  if (bits == 8)
    encode_kernel<8><<<grid, BLOCK, 0, ctx->stream>>>(P, P32->D, P32->col_stride / 4, Pq->scales, out, stride);
  else
    encode_kernel<4><<<grid, BLOCK, 0, ctx->stream>>>(P, P32->D, P32->col_stride / 4, Pq->scales, out, stride);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}

int launch_absmax(twa_ctx* ctx, const float* P, long long D, long long ld, int n, unsigned* absmax) {
  int total = grid_for(ctx, D, BLOCK * 16, 8);
  const int fit = resident_blocks(ctx, absmax_kernel);
  if (total > fit) total = fit;
  int per_col = total / n;
  if (per_col < 1) per_col = 1;
  absmax_kernel<<<dim3(per_col, n), BLOCK, 0, ctx->stream>>>(P, D, ld, absmax);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}

int launch_sumsq(twa_ctx* ctx, const float* v, long long D, void* ws, double* result) {
  char* w = static_cast<char*>(ws);
  const int grid = grid_for(ctx, D, BLOCK * 16, 4);
  sumsq_kernel<<<grid, BLOCK, 0, ctx->stream>>>(v, D, reinterpret_cast<double*>(w + TWA_WS_DPART), result,
                                                ctx->d_ticket);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}

}  // namespace

int twa_launch_scales(twa_ctx* ctx, const unsigned* absmax, int n, int bits, float* scales) {
  scales_kernel<<<1, 128, 0, ctx->stream>>>(absmax, n, bits == 8 ? 127.0f : 7.0f, scales, ctx->d_status);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}

extern "C" {

int64_t twa_basis_col_stride(int64_t D, int bits) {
  if (D < 1 || (bits != 32 && bits != 8 && bits != 4 && bits != 2 && bits != 1)) return 0;
  const int64_t row_bytes = (D * bits + 7) / 8;
  if (bits == 32) return (row_bytes + 127) / 128 * 128;
  return (row_bytes + 511) / 512 * 512;      // whole 512-byte segments: see twa_chunk_slot
}

size_t twa_basis_bytes(int64_t D, int n, int bits) {
  if (n < 1) return 0;
  return static_cast<size_t>(twa_basis_col_stride(D, bits)) * static_cast<size_t>(n);
}

size_t twa_workspace_bytes(int64_t, int, int) { return TWA_WS_BYTES; }

int twa_mean(twa_ctx* ctx, const float* W, int64_t D, int n, int64_t ldw, float* wbar_out) {
  if (!ctx || !W || !wbar_out || D < 1 || n < 1 || ldw < D) return TWA_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(W) & 15) || (ldw & 3) || (reinterpret_cast<uintptr_t>(wbar_out) & 15))
    return TWA_ERR_MISALIGNED;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  int grid = grid_for(ctx, D, BLOCK * 4, 8);
  const int fit = resident_blocks(ctx, mean_kernel);
  if (grid > fit) grid = fit;
  mean_kernel<<<grid, BLOCK, 0, ctx->stream>>>(W, D, n, ldw, wbar_out);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}

}  // extern "C"

namespace {

// twa_build_basis; with `absmax` (device, n words, zero on entry) the largest magnitude of every
// finished column is folded into it while the column is written for the last time.
int build_basis(twa_ctx* ctx, float* W, int64_t D, int n, int64_t ldw, float* wbar_out, twa_basis* P32_out, void* ws,
                size_t ws_bytes, unsigned* absmax) {
  if (!ctx || !W || !wbar_out || !P32_out) return TWA_ERR_INVALID_ARG;
  if (D < 1 || D > TWA_MAX_LAUNCH_ROWS || n < 1 || ldw < D) return TWA_ERR_INVALID_ARG;
  if (n > TWA_MAX_N) return TWA_ERR_UNSUPPORTED;
  if (!ws || ws_bytes < TWA_WS_BYTES) return TWA_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(W) & 15) || (ldw & 3) || (reinterpret_cast<uintptr_t>(ws) & 15) ||
      (reinterpret_cast<uintptr_t>(wbar_out) & 15))
    return TWA_ERR_MISALIGNED;
  int rc = twa_mean(ctx, W, D, n, ldw, wbar_out);
  if (rc) return rc;

  char* w = static_cast<char*>(ws);
  float* coef = reinterpret_cast<float*>(w + TWA_WS_COEF);
  double* norms = reinterpret_cast<double*>(w + TWA_WS_NORMS);          // [0]: after the sweep
  // squared norms of a panel's columns as given: the last doubles of the workspace's float region
  double* given = reinterpret_cast<double*>(w + TWA_WS_PARTIALS + sizeof(float) * TWA_MAX_GRID * TWA_MAX_N) - 8;
  const int egrid = grid_for(ctx, D, BLOCK * 16, 4);
  const int width = ctx->tune_build_panel == 1 ? 1 : 8;

  // One Gram-Schmidt sweep of column k against columns first .. k-1 (all coefficients from the same
  // vector), then its squared norm.
  auto sweep = [&](int first, int k) -> int {
    float* col = W + k * ldw;
    if (k > first) {
      twa_basis Q = {W + first * ldw, nullptr, D, 4 * ldw, k - first, 32};
      twa_project_epilogue epi = {coef, nullptr, 0.0f, 0.0f, k};
      int r = twa_launch_project(ctx, &Q, col, TWA_F32, epi, ws);         // c = Q^T v
      if (r) return r;
      r = twa_launch_lift(ctx, &Q, coef, -1.0f, col, col, false);         // v <- v - Q c
      if (r) return r;
    }
    return launch_sumsq(ctx, col, D, ws, norms);
  };

  if (width == 1) {
    // column by column: two sweeps against everything before, then normalise
    for (int j = 0; j < n; ++j) {
      float* col = W + j * ldw;
      rc = launch_sumsq(ctx, col, D, ws, given);                       // |a_j|^2
      if (rc) return rc;
      rc = sweep(0, j);
      if (rc) return rc;
      if (j > 0) {
        rc = sweep(0, j);
        if (rc) return rc;
      }
      normalise_kernel<<<egrid, BLOCK, 0, ctx->stream>>>(col, D, given, norms, j, ctx->d_status);
      TWA_CUDA_OK(ctx, cudaGetLastError());
    }
  } else {
    // Panels of up to 8 columns.  Twice: remove the earlier basis vectors from the whole panel in one
    // pass over them (projection of the panel, then update), then orthonormalise the panel's columns
    // among themselves (Gram form, or column sweeps and normalisations with TWA_TUNE_BUILD_PANEL = 2).  The first round makes the panel orthonormal up to the rounding its
    // cancellation amplifies; the second round, applied to unit vectors, removes that.
    for (int j0 = 0; j0 < n; j0 += width) {
      const int pb = n - j0 < width ? n - j0 : width;
      float* panel = W + j0 * ldw;
      if (ctx->tune_build_panel == 0) {
        // Gram form inside the panel: all coefficients of the panel's own Gram-Schmidt from its Gram
        // matrix, the new columns in one pass.  The squared norms of the columns as given come out of
        // the first projection, the Gram matrix out of the update (the first panel, which has neither,
        // takes its Gram matrix in a pass of its own and its norms from the diagonal); in the second
        // round the rank test compares against the columns' norms as this round found them (1, or 0
        // for a column already found dependent).
        for (int round = 0; round < 2; ++round) {
          if (j0 > 0) {
            rc = twa_launch_panel_project(ctx, W, D, ldw, j0, pb, ws, round == 0 ? given : nullptr);
            if (rc) return rc;
            rc = twa_launch_panel_lift(ctx, W, D, ldw, j0, pb, ws, given, round == 1);
          } else {
            rc = twa_launch_panel_gram(ctx, W, D, ldw, j0, pb, ws, given, true);
          }
          if (rc) return rc;
          rc = twa_launch_panel_apply(ctx, W, D, ldw, j0, pb, ws, round == 1 && absmax ? absmax + j0 : nullptr);
          if (rc) return rc;
        }
        continue;
      }
      for (int q = 0; q < pb; ++q) {
        rc = launch_sumsq(ctx, panel + q * ldw, D, ws, given + q);        // |a_j|^2 as given
        if (rc) return rc;
      }
      for (int round = 0; round < 2; ++round) {
        if (j0 > 0) {
          rc = twa_launch_panel_project(ctx, W, D, ldw, j0, pb, ws, nullptr);
          if (rc) return rc;
          rc = twa_launch_panel_lift(ctx, W, D, ldw, j0, pb, ws, nullptr, false);
          if (rc) return rc;
        }
        for (int q = 0; q < pb; ++q) {
          const int k = j0 + q;
          float* col = W + k * ldw;
          if (round == 1) {
            rc = launch_sumsq(ctx, col, D, ws, given + q);              // 1, or 0 for a column found dependent
            if (rc) return rc;
          }
          if (q > 0) {
            // one sweep against the panel's earlier columns, fused with the squared norm of the result
            double* dpart = reinterpret_cast<double*>(w + TWA_WS_DPART);
            double* dots_part = reinterpret_cast<double*>(w + TWA_WS_PARTIALS);   // [egrid][8], start of the float region
            inpanel_dots_kernel<<<egrid, BLOCK, 0, ctx->stream>>>(W + j0 * ldw, ldw, q, col, D, dots_part, coef,
                                                                  ctx->d_ticket, ctx->d_status, k);
            TWA_CUDA_OK(ctx, cudaGetLastError());
            inpanel_update_kernel<<<egrid, BLOCK, 0, ctx->stream>>>(W + j0 * ldw, ldw, q, col, D, coef, dpart, norms,
                                                                    ctx->d_ticket);
            TWA_CUDA_OK(ctx, cudaGetLastError());
          } else {
            rc = launch_sumsq(ctx, col, D, ws, norms);
            if (rc) return rc;
          }
          normalise_kernel<<<egrid, BLOCK, 0, ctx->stream>>>(col, D, given + q, norms, k, ctx->d_status);
          TWA_CUDA_OK(ctx, cudaGetLastError());
        }
      }
    }
  }
  // the schedules that finish a column with normalise_kernel take the maxima in a pass of their own
  if (absmax && ctx->tune_build_panel != 0) {
    rc = launch_absmax(ctx, W, D, ldw, n, absmax);
    if (rc) return rc;
  }
  P32_out->data = W;
  P32_out->scales = nullptr;
  P32_out->D = D;
  P32_out->col_stride = 4 * ldw;
  P32_out->n = n;
  P32_out->bits = 32;
  return TWA_OK;
}

int check_quantised_target(const twa_basis* Pq, int bits, const void* ws) {
  if (bits != 8 && bits != 4) return TWA_ERR_UNSUPPORTED;
  if (!Pq || !Pq->data || !Pq->scales) return TWA_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(Pq->data) & 15) || (reinterpret_cast<uintptr_t>(ws) & 15)) return TWA_ERR_MISALIGNED;
  return TWA_OK;
}

}  // namespace

extern "C" {

int twa_build_basis(twa_ctx* ctx, float* W, int64_t D, int n, int64_t ldw, float* wbar_out,
                    twa_basis* P32_out, void* ws, size_t ws_bytes) {
  return build_basis(ctx, W, D, n, ldw, wbar_out, P32_out, ws, ws_bytes, nullptr);
}

int twa_build_quantized(twa_ctx* ctx, float* W, int64_t D, int n, int64_t ldw, float* wbar_out,
                        twa_basis* P32_out, const int* bits, int widths, twa_basis* Pq, void* ws,
                        size_t ws_bytes) {
  if (!ctx || !bits || !Pq || widths < 1 || widths > 8) return TWA_ERR_INVALID_ARG;
  if (!ws || ws_bytes < TWA_WS_BYTES) return TWA_ERR_WORKSPACE;
  if (n < 1) return TWA_ERR_INVALID_ARG;
  if (n > TWA_MAX_N) return TWA_ERR_UNSUPPORTED;
  for (int k = 0; k < widths; ++k) {
    const int rc = check_quantised_target(&Pq[k], bits[k], ws);
    if (rc) return rc;
  }
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  unsigned* absmax = reinterpret_cast<unsigned*>(static_cast<char*>(ws) + TWA_WS_ABSMAX);
  TWA_CUDA_OK(ctx, cudaMemsetAsync(absmax, 0, sizeof(unsigned) * n, ctx->stream));
  int rc = build_basis(ctx, W, D, n, ldw, wbar_out, P32_out, ws, ws_bytes, absmax);
  if (rc) return rc;
  for (int k = 0; k < widths; ++k) {
    rc = twa_launch_scales(ctx, absmax, n, bits[k], Pq[k].scales);
    if (rc) return rc;
    rc = launch_encode(ctx, P32_out, bits[k], &Pq[k]);
    if (rc) return rc;
    Pq[k].D = D;
    Pq[k].col_stride = twa_basis_col_stride(D, bits[k]);
    Pq[k].n = n;
    Pq[k].bits = bits[k];
  }
  return TWA_OK;
}

int twa_quantize_basis(twa_ctx* ctx, const twa_basis* P32, int bits, twa_basis* Pq, void* ws,
                       size_t ws_bytes) {
  if (!ctx || !P32 || !Pq) return TWA_ERR_INVALID_ARG;
  if (bits != 8 && bits != 4) return TWA_ERR_UNSUPPORTED;
  if (!Pq->data || !Pq->scales) return TWA_ERR_INVALID_ARG;
  int rc = twa_check_basis(P32);
  if (rc) return rc;
  if (P32->bits != 32) return TWA_ERR_INVALID_ARG;
  if (!ws || ws_bytes < TWA_WS_BYTES) return TWA_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(Pq->data) & 15) || (reinterpret_cast<uintptr_t>(ws) & 15))
    return TWA_ERR_MISALIGNED;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  const long long D = P32->D;
  const int n = P32->n;
  const long long ld = P32->col_stride / 4;
  const float* P = static_cast<const float*>(P32->data);
  unsigned* absmax = reinterpret_cast<unsigned*>(static_cast<char*>(ws) + TWA_WS_ABSMAX);
  TWA_CUDA_OK(ctx, cudaMemsetAsync(absmax, 0, sizeof(unsigned) * n, ctx->stream));
  rc = launch_absmax(ctx, P, D, ld, n, absmax);
  if (rc) return rc;
  rc = twa_launch_scales(ctx, absmax, n, bits, Pq->scales);
  if (rc) return rc;
  rc = launch_encode(ctx, P32, bits, Pq);
  if (rc) return rc;
  const long long stride = twa_basis_col_stride(D, bits);
  Pq->D = D;
  Pq->col_stride = stride;
  Pq->n = n;
  Pq->bits = bits;
  return TWA_OK;
}

int twa_basis_export(twa_ctx* ctx, const twa_basis* Pq, void* codes_out, float* scales_out) {
  if (!ctx || !codes_out || !scales_out || !Pq) return TWA_ERR_INVALID_ARG;
  // the conversion kernels index bytes with 64-bit integers: up to TWA_MAX_ROWS rows
  twa_basis head = *Pq;
  if (Pq->D > TWA_MAX_LAUNCH_ROWS) head.D = TWA_MAX_LAUNCH_ROWS;
  int rc = twa_check_basis(&head);
  if (rc) return rc;
  if (Pq->D > TWA_MAX_ROWS || Pq->col_stride < (Pq->D * Pq->bits + 7) / 8) return TWA_ERR_INVALID_ARG;
  if (Pq->bits == 32) return TWA_ERR_UNSUPPORTED;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  const long long row_bytes = (Pq->D * Pq->bits + 7) / 8;
  int per = grid_for(ctx, row_bytes, BLOCK * 8, 8) / Pq->n;
  if (per < 1) per = 1;
  export_kernel<<<dim3(per, Pq->n), BLOCK, 0, ctx->stream>>>(
      static_cast<const unsigned char*>(Pq->data), Pq->col_stride,
      static_cast<unsigned char*>(codes_out), row_bytes, 0);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  TWA_CUDA_OK(ctx, cudaMemcpyAsync(scales_out, Pq->scales, sizeof(float) * Pq->n,
                                   cudaMemcpyDeviceToDevice, ctx->stream));
  return TWA_OK;
}

int twa_basis_import(twa_ctx* ctx, const void* codes, const float* scales, int64_t D, int n, int bits,
                     twa_basis* Pq) {
  if (!ctx || !codes || !scales || !Pq || !Pq->data || !Pq->scales) return TWA_ERR_INVALID_ARG;
  if (bits != 8 && bits != 4) return TWA_ERR_UNSUPPORTED;
  if (D < 1 || D > TWA_MAX_ROWS || n < 1) return TWA_ERR_INVALID_ARG;
  if (n > TWA_MAX_N) return TWA_ERR_UNSUPPORTED;
  if (reinterpret_cast<uintptr_t>(Pq->data) & 15) return TWA_ERR_MISALIGNED;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  const long long row_bytes = (D * bits + 7) / 8;
  const long long stride = twa_basis_col_stride(D, bits);
  int per = grid_for(ctx, stride, BLOCK * 8, 8) / n;
  if (per < 1) per = 1;
  import_kernel<<<dim3(per, n), BLOCK, 0, ctx->stream>>>(
      static_cast<const unsigned char*>(codes), row_bytes, static_cast<unsigned char*>(Pq->data),
      stride, 0);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  TWA_CUDA_OK(ctx, cudaMemcpyAsync(Pq->scales, scales, sizeof(float) * n, cudaMemcpyDeviceToDevice,
                                   ctx->stream));
  Pq->D = D;
  Pq->col_stride = stride;
  Pq->n = n;
  Pq->bits = bits;
  return TWA_OK;
}

}  // extern "C"
