// The paper's default construction (Sections 4.1, 4.5, 4.6; Algorithm 1): per layer l,
// e_i^l = (w_i^l - w_bar^l) / ||w_i^l - w_bar^l||, quantised with the uniform min-max scheme
// code = round((P - b^l) / a^l), a^l = (max - min) / (2^B - 1), b^l = min, one (a, b) pair per layer.
//
// Storage of the codes ("layered basis"): the same column-major, chunk-permuted bytes as the
// per-column format, but every layer starts on a 64-byte granule of the column, so that a warp's
// share of a tile always lies in one layer.  A table with one entry per granule maps it back to
// (layer, first flat row, number of valid rows).
#include <math.h>
#include <stdio.h>

#include <algorithm>
#include <vector>

#include "twa_common.cuh"

namespace {

constexpr int BLOCK = 256;
constexpr long long ITEM_ROWS = 8192;       // rows of one layer handled by one block

struct Item { int layer; long long r0, r1; };   // flat rows [r0, r1) of one layer

long long granule_rows(int bits) { return 64LL * 8 / bits; }
// Code width B of the quantiser (Section 4.6) -> width of the slot a code occupies in the stored
// columns, and the number of byte planes: 3-bit codes sit in 4-bit slots; 16-bit codes are two 8-bit
// planes (columns 0..n-1 hold the high bytes, n..2n-1 the low bytes).  0 = width not supported.
int slot_bits(int code_bits) {
  switch (code_bits) {
    case 1: return 1;
    case 2: return 2;
    case 3: case 4: return 4;
    case 8: case 16: return 8;
    default: return 0;
  }
}
int plane_count(int code_bits) { return code_bits == 16 ? 2 : 1; }
float top_code(int code_bits) { return static_cast<float>((1 << code_bits) - 1); }
constexpr size_t TABLE_SLACK = 8;                           // granule entries past the last column byte
constexpr int MAX_CTAS = 1024;                              // blocks of a step kernel
constexpr size_t CTA_TABLE_BYTES = (sizeof(int) * (MAX_CTAS + 1) + 255) / 256 * 256;

// host view of the layer partition
struct Partition {
  std::vector<long long> flat, internal;     // L+1 offsets each
  std::vector<Item> items;
  std::vector<int> first_item;               // L+1
  long long D_int;
};

int make_partition(const int64_t* offsets, int L, long long D, int bits, Partition* p) {
  if (!offsets || L < 1 || offsets[0] != 0 || offsets[L] != D) return TWA_ERR_INVALID_ARG;
  const long long gr = granule_rows(bits);
  p->flat.assign(offsets, offsets + L + 1);
  p->internal.resize(L + 1);
  p->first_item.resize(L + 1);
  p->items.clear();
  long long io = 0;
  for (int l = 0; l < L; ++l) {
    const long long len = offsets[l + 1] - offsets[l];
    if (len < 1) return TWA_ERR_INVALID_ARG;
    p->internal[l] = io;
    p->first_item[l] = static_cast<int>(p->items.size());
    for (long long r = offsets[l]; r < offsets[l + 1]; r += ITEM_ROWS)
      p->items.push_back({l, r, r + ITEM_ROWS < offsets[l + 1] ? r + ITEM_ROWS : offsets[l + 1]});
    io += (len + gr - 1) / gr * gr;
  }
  p->internal[L] = io;
  p->first_item[L] = static_cast<int>(p->items.size());
  p->D_int = io;
  return io <= TWA_MAX_LAUNCH_ROWS ? TWA_OK : TWA_ERR_UNSUPPORTED;
}

// ---- kernels ------------------------------------------------------------------------------
__device__ __forceinline__ double block_sum_d(double v, double* sh) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  double t = 0;
  if (threadIdx.x == 0)
    for (int w = 0; w < BLOCK / 32; ++w) t += sh[w];
  return t;
}

// Rows r .. r + 3 of p (r a multiple of 4); rows outside [lo, hi) read as zero.  One 16-byte load when p
// is 16-byte aligned and all four rows exist: a thread's loads then cover whole 32-byte sectors between
// them (with one float per load a warp touched 32 lines per instruction and the 4-bit pass ran at a
// third of the 8-bit one).
__device__ __forceinline__ float4 load_rows4(const float* __restrict__ p, long long r, long long lo, long long hi,
                                             bool aligned) {
  if (aligned && r >= lo && r + 3 < hi) return *reinterpret_cast<const float4*>(p + r);
  float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
  if (r >= lo && r < hi) x.x = p[r];
  if (r + 1 >= lo && r + 1 < hi) x.y = p[r + 1];
  if (r + 2 >= lo && r + 2 < hi) x.z = p[r + 2];
  if (r + 3 >= lo && r + 3 < hi) x.w = p[r + 3];
  return x;
}

// partial[item][i] = sum over the item's rows of (w - w_bar)^2
__global__ void __launch_bounds__(BLOCK) centred_sumsq_kernel(const float* __restrict__ W, long long ldw,
                                                              const float* __restrict__ wbar,
                                                              const Item* __restrict__ items, int n,
                                                              double* __restrict__ partial) {
  // blocks of one item and neighbouring columns run together, so the item's rows of the shared vectors
  // (w_bar) are fetched from memory once and found in the cache by the other columns
  const unsigned item_k = blockIdx.x / n;
  const int col_j = blockIdx.x % n;
  __shared__ double sh[BLOCK / 32];
  const Item it = items[item_k];
  const float* col = W + col_j * ldw;
  const bool aligned = ((reinterpret_cast<uintptr_t>(col) | reinterpret_cast<uintptr_t>(wbar)) & 15) == 0;
  double s = 0;
  for (long long g = (it.r0 & ~3LL) + 4 * threadIdx.x; g < it.r1; g += 4 * BLOCK) {
    // four rows a thread; rows outside the item read as zero on both sides and add nothing
    const float4 x = load_rows4(col, g, it.r0, it.r1, aligned), m = load_rows4(wbar, g, it.r0, it.r1, aligned);
    const double v0 = static_cast<double>(x.x) - static_cast<double>(m.x), v1 = static_cast<double>(x.y) - static_cast<double>(m.y);
    const double v2 = static_cast<double>(x.z) - static_cast<double>(m.z), v3 = static_cast<double>(x.w) - static_cast<double>(m.w);
    s += v0 * v0;
    s += v1 * v1;
    s += v2 * v2;
    s += v3 * v3;
  }
  const double t = block_sum_d(s, sh);
  if (threadIdx.x == 0) partial[static_cast<size_t>(item_k) * n + col_j] = t;
}

// inv[l][i] = 1 / sqrt(sum of the layer's partials in item order), 0 for a zero vector
__global__ void inv_norm_kernel(const double* __restrict__ partial, const int* __restrict__ first_item,
                                int L, int n, double* __restrict__ inv, int* status) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= L * n) return;
  const int l = idx / n, i = idx - l * n;
  double s = 0;
  for (int k = first_item[l]; k < first_item[l + 1]; ++k) s += partial[static_cast<size_t>(k) * n + i];
  if (!isfinite(s)) twa_set_status(status, TWA_ERR_NONFINITE, i);
  inv[idx] = (s > 0.0 && isfinite(s)) ? 1.0 / sqrt(s) : 0.0;
}

__global__ void __launch_bounds__(BLOCK) centre_scale_kernel(float* __restrict__ W, long long ldw,
                                                             const float* __restrict__ wbar,
                                                             const Item* __restrict__ items, int n,
                                                             const double* __restrict__ inv) {
  // blocks of one item and neighbouring columns run together, so the item's rows of the shared vectors
  // (w_bar) are fetched from memory once and found in the cache by the other columns
  const unsigned item_k = blockIdx.x / n;
  const int col_j = blockIdx.x % n;
  const Item it = items[item_k];
  float* col = W + col_j * ldw;
  const double f = inv[static_cast<size_t>(it.layer) * n + col_j];
  const bool aligned = ((reinterpret_cast<uintptr_t>(col) | reinterpret_cast<uintptr_t>(wbar)) & 15) == 0;
  for (long long g = (it.r0 & ~3LL) + 4 * threadIdx.x; g < it.r1; g += 4 * BLOCK) {
    const float4 x = load_rows4(col, g, it.r0, it.r1, aligned), m = load_rows4(wbar, g, it.r0, it.r1, aligned);
    float4 y;
    y.x = static_cast<float>((static_cast<double>(x.x) - static_cast<double>(m.x)) * f);
    y.y = static_cast<float>((static_cast<double>(x.y) - static_cast<double>(m.y)) * f);
    y.z = static_cast<float>((static_cast<double>(x.z) - static_cast<double>(m.z)) * f);
    y.w = static_cast<float>((static_cast<double>(x.w) - static_cast<double>(m.w)) * f);
    if (aligned && g >= it.r0 && g + 3 < it.r1) {
      *reinterpret_cast<float4*>(col + g) = y;
    } else {
      if (g >= it.r0 && g < it.r1) col[g] = y.x;
      if (g + 1 >= it.r0 && g + 1 < it.r1) col[g + 1] = y.y;
      if (g + 2 >= it.r0 && g + 2 < it.r1) col[g + 2] = y.z;
      if (g + 3 >= it.r0 && g + 3 < it.r1) col[g + 3] = y.w;
    }
  }
}

// partial min / max of one item over one column
__global__ void __launch_bounds__(BLOCK) minmax_kernel(const float* __restrict__ P, long long ld,
                                                       const Item* __restrict__ items, int n,
                                                       float* __restrict__ pmin, float* __restrict__ pmax) {
  // (column, item), the item running fastest: neighbouring blocks read neighbouring rows of one column
  const unsigned items_n = gridDim.x / n;
  const unsigned item_k = blockIdx.x % items_n;
  const int col_j = blockIdx.x / items_n;
  __shared__ float smin[BLOCK / 32], smax[BLOCK / 32];
  const Item it = items[item_k];
  const float* col = P + col_j * ld;
  float lo = INFINITY, hi = -INFINITY;
  bool bad = false;                              // fmin / fmax drop NaN: track non-finite input apart
  const bool aligned = (reinterpret_cast<uintptr_t>(col) & 15) == 0;
  for (long long g = (it.r0 & ~3LL) + 4 * threadIdx.x; g < it.r1; g += 4 * BLOCK) {
    const float4 x = load_rows4(col, g, it.r0, it.r1, aligned);
    const float v[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (g + i >= it.r0 && g + i < it.r1) {
        lo = fminf(lo, v[i]);
        hi = fmaxf(hi, v[i]);
        bad |= !isfinite(v[i]);
      }
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    lo = fminf(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, off));
    hi = fmaxf(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, off));
  }
  bad = __any_sync(0xFFFFFFFFu, bad);
  if ((threadIdx.x & 31) == 0) {
    smin[threadIdx.x >> 5] = bad ? NAN : lo;
    smax[threadIdx.x >> 5] = hi;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 0; w < BLOCK / 32; ++w) {
      bad |= isnan(smin[w]);
      lo = fminf(lo, smin[w]);
      hi = fmaxf(hi, smax[w]);
    }
    pmin[static_cast<size_t>(item_k) * n + col_j] = bad ? NAN : lo;
    pmax[static_cast<size_t>(item_k) * n + col_j] = hi;
  }
}

// a[l] = (max - min) / (2^B - 1), b[l] = min over the layer's items and all columns.  One block of 128
// threads per layer (min and max do not depend on the order).
__global__ void __launch_bounds__(128) factors_kernel(const float* __restrict__ pmin, const float* __restrict__ pmax,
                                                      const int* __restrict__ first_item, int L, int n, float levels,
                                                      float* __restrict__ a, float* __restrict__ b, int* status) {
  __shared__ float slo[4], shi[4];
  __shared__ int sbad[4];
  const int l = blockIdx.x;
  const size_t i0 = static_cast<size_t>(first_item[l]) * n, i1 = static_cast<size_t>(first_item[l + 1]) * n;
  float lo = INFINITY, hi = -INFINITY;
  bool bad = false;
  for (size_t i = i0 + threadIdx.x; i < i1; i += 128) {
    const float x = pmin[i], y = pmax[i];
    bad |= isnan(x) || isnan(y);
    lo = fminf(lo, x);
    hi = fmaxf(hi, y);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    lo = fminf(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, off));
    hi = fmaxf(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, off));
  }
  bad = __any_sync(0xFFFFFFFFu, bad);
  if ((threadIdx.x & 31) == 0) {
    slo[threadIdx.x >> 5] = lo;
    shi[threadIdx.x >> 5] = hi;
    sbad[threadIdx.x >> 5] = bad ? 1 : 0;
  }
  __syncthreads();
  if (threadIdx.x != 0) return;
  for (int w = 1; w < 4; ++w) {
    lo = fminf(lo, slo[w]);
    hi = fmaxf(hi, shi[w]);
    bad |= sbad[w] != 0;
  }
  if (bad) {
    twa_set_status(status, TWA_ERR_NONFINITE, l);
    a[l] = 0.0f;
    b[l] = 0.0f;
    return;
  }
  a[l] = __fdiv_rn(__fsub_rn(hi, lo), levels);
  b[l] = lo;
}

// The quantiser's code of an element: round((e - b) / a) on IEEE float32 operations, half to even,
// clamped to [0, top] (clamping first gives the same code: the bounds are integers; a NaN becomes 0
// either way).  The rounding is an addition of 2^23, whose low mantissa bits are then the code.
__device__ __forceinline__ uint32_t affine_code(float e, float bl, float al, float top) {
  const float q = fminf(fmaxf(__fdiv_rn(__fsub_rn(e, bl), al), 0.0f), top);
  return __float_as_uint(q + 8388608.0f) - 0x4B000000u;
}

// The same code without the division: with r = RN(1 / a) the product (e - b) r lies within
// (top + 1) 2^-23 of the IEEE quotient wherever the clamp does not decide, so both round to the same
// integer unless the product is within `near` = (top + 1) 2^-21 of a half-integer; then *hard is set and
// the caller repeats the group with affine_code.  The distance to the integer is exact in float32.
__device__ __forceinline__ uint32_t affine_code_by_reciprocal(float e, float bl, float r, float top, float near,
                                                             bool* hard) {
  const float q0 = fminf(fmaxf(__fsub_rn(e, bl) * r, 0.0f), top);
  const float y = q0 + 8388608.0f;
  *hard |= fabsf(q0 - (y - 8388608.0f)) >= 0.5f - near;
  return __float_as_uint(y) - 0x4B000000u;
}

// r = RN(1 / a) when the reciprocal path is valid for this layer and width, else 0: a normal scale, and a
// `near` band narrow enough to be met rarely (16-bit codes would meet it in every group).
__device__ __forceinline__ float affine_reciprocal(float al, float top) {
  return (al >= 0x1p-100f && top <= 255.0f) ? __frcp_rn(al) : 0.0f;
}

// Puts code u (k-th of a 16-byte chunk, slots of W bits) into the chunk's words.
template <int W>
__device__ __forceinline__ void put_code(uint32_t (&w)[4], int k, uint32_t u) {
  constexpr int PER_WORD = 32 / W;
  w[k / PER_WORD] |= u << (W * (k % PER_WORD));
}

// One thread writes one 16-byte chunk of one column: 128 / W rows of a layer (W = slot width), rows
// past the layer's end get the code 0.  PLANES == 2 (16-bit codes): the chunk of the high bytes goes
// to column j, that of the low bytes to column n + j.
template <int W, int PLANES>
__global__ void __launch_bounds__(BLOCK) affine_encode_kernel(const float* __restrict__ P, long long ld,
                                                              const long long* __restrict__ flat,
                                                              const long long* __restrict__ internal,
                                                              const float* __restrict__ a,
                                                              const float* __restrict__ b, float top, int n,
                                                              unsigned char* __restrict__ out,
                                                              long long out_stride) {
  constexpr int RPC = 128 / W;
  const int l = blockIdx.z, j = blockIdx.y;
  const long long len = flat[l + 1] - flat[l];
  const long long chunks = (internal[l + 1] - internal[l]) / RPC;
  const float al = a[l], bl = b[l];
  const float* col = P + j * ld + flat[l];
  uint4* dst = reinterpret_cast<uint4*>(out + j * out_stride);
  uint4* dst_lo = reinterpret_cast<uint4*>(out + (static_cast<long long>(n) + j) * out_stride);
  const float recip = PLANES == 2 ? 0.0f : affine_reciprocal(al, top);
  const float near = (top + 1.0f) * 0x1p-21f;
  const bool aligned = (reinterpret_cast<uintptr_t>(col) & 15) == 0;
  for (long long c = blockIdx.x * static_cast<long long>(BLOCK) + threadIdx.x; c < chunks;
       c += static_cast<long long>(gridDim.x) * BLOCK) {
    uint32_t w[4] = {0, 0, 0, 0}, wl[4] = {0, 0, 0, 0};
    bool hard = recip == 0.0f;
    if (!hard) {
#pragma unroll
      for (int k = 0; k < RPC; k += 4) {
        const long long r = c * RPC + k;
        const float4 x = load_rows4(col, r, 0, len, aligned);
        if (r < len) put_code<W>(w, k, affine_code_by_reciprocal(x.x, bl, recip, top, near, &hard));
        if (r + 1 < len) put_code<W>(w, k + 1, affine_code_by_reciprocal(x.y, bl, recip, top, near, &hard));
        if (r + 2 < len) put_code<W>(w, k + 2, affine_code_by_reciprocal(x.z, bl, recip, top, near, &hard));
        if (r + 3 < len) put_code<W>(w, k + 3, affine_code_by_reciprocal(x.w, bl, recip, top, near, &hard));
      }
    }
    if (hard) {
      w[0] = w[1] = w[2] = w[3] = 0u;
#pragma unroll
      for (int k = 0; k < RPC; ++k) {
        const long long r = c * RPC + k;
        const uint32_t u = (r < len && al != 0.0f) ? affine_code(col[r], bl, al, top) : 0u;
        if (PLANES == 2) {
          put_code<W>(w, k, u >> 8);
          put_code<W>(wl, k, u & 0xFFu);
        } else {
          put_code<W>(w, k, u);
        }
      }
    }
    const long long q = internal[l] / RPC + c;
    dst[(q & ~31LL) | twa_chunk_slot(static_cast<int>(q & 31), j)] = make_uint4(w[0], w[1], w[2], w[3]);
    if (PLANES == 2)
      dst_lo[(q & ~31LL) | twa_chunk_slot(static_cast<int>(q & 31), n + j)] = make_uint4(wl[0], wl[1], wl[2], wl[3]);
  }
}

// ---- row-chunked construction: the same arithmetic on rows [row0, row1) of the flat vector --------
// chunk[i * ld + (r - row0)] is candidate i at flat row r.  An item (at most 8192 rows of one layer)
// may straddle two chunks: its partial results are merged by the calls in stream order.
__global__ void __launch_bounds__(BLOCK) chunk_centred_sumsq_kernel(const float* __restrict__ chunk, long long ld,
                                                                    long long row0, long long row1,
                                                                    const float* __restrict__ wbar,
                                                                    const Item* __restrict__ items, int n,
                                                                    double* __restrict__ partial) {
  // blocks of one item and neighbouring columns run together, so the item's rows of the shared vectors
  // (w_bar) are fetched from memory once and found in the cache by the other columns
  const unsigned item_k = blockIdx.x / n;
  const int col_j = blockIdx.x % n;
  __shared__ double sh[BLOCK / 32];
  const Item it = items[item_k];
  const long long r0 = it.r0 > row0 ? it.r0 : row0, r1 = it.r1 < row1 ? it.r1 : row1;
  const float* col = chunk + col_j * ld - row0;
  const bool aligned = ((reinterpret_cast<uintptr_t>(col) | reinterpret_cast<uintptr_t>(wbar)) & 15) == 0;
  double s = 0;
  for (long long g = (r0 & ~3LL) + 4 * threadIdx.x; g < r1; g += 4 * BLOCK) {
    const float4 x = load_rows4(col, g, r0, r1, aligned), m = load_rows4(wbar, g, r0, r1, aligned);
    const double v0 = static_cast<double>(x.x) - static_cast<double>(m.x), v1 = static_cast<double>(x.y) - static_cast<double>(m.y);
    const double v2 = static_cast<double>(x.z) - static_cast<double>(m.z), v3 = static_cast<double>(x.w) - static_cast<double>(m.w);
    s += v0 * v0;
    s += v1 * v1;
    s += v2 * v2;
    s += v3 * v3;
  }
  const double t = block_sum_d(s, sh);
  if (threadIdx.x == 0) partial[static_cast<size_t>(item_k) * n + col_j] += t;
}

// e = (w - w_bar) / ||.|| for the chunk's rows (the expression of centre_scale_kernel), its min / max
// per item merged into pmin / pmax, and optionally the values themselves.
__global__ void __launch_bounds__(BLOCK) chunk_minmax_kernel(const float* __restrict__ chunk, long long ld,
                                                             long long row0, long long row1,
                                                             const float* __restrict__ wbar,
                                                             const Item* __restrict__ items, int n,
                                                             const double* __restrict__ inv, float* __restrict__ pmin,
                                                             float* __restrict__ pmax, float* __restrict__ q32,
                                                             long long ldq) {
  // blocks of one item and neighbouring columns run together, so the item's rows of the shared vectors
  // (w_bar) are fetched from memory once and found in the cache by the other columns
  const unsigned item_k = blockIdx.x / n;
  const int col_j = blockIdx.x % n;
  __shared__ float smin[BLOCK / 32], smax[BLOCK / 32];
  const Item it = items[item_k];
  const long long r0 = it.r0 > row0 ? it.r0 : row0, r1 = it.r1 < row1 ? it.r1 : row1;
  const float* col = chunk + col_j * ld - row0;
  const double f = inv[static_cast<size_t>(it.layer) * n + col_j];
  float lo = INFINITY, hi = -INFINITY;
  bool bad = false;
  const bool aligned = ((reinterpret_cast<uintptr_t>(col) | reinterpret_cast<uintptr_t>(wbar)) & 15) == 0;
  for (long long g = (r0 & ~3LL) + 4 * threadIdx.x; g < r1; g += 4 * BLOCK) {
    const float4 x = load_rows4(col, g, r0, r1, aligned), m = load_rows4(wbar, g, r0, r1, aligned);
    const float v[4] = {static_cast<float>((static_cast<double>(x.x) - static_cast<double>(m.x)) * f),
                        static_cast<float>((static_cast<double>(x.y) - static_cast<double>(m.y)) * f),
                        static_cast<float>((static_cast<double>(x.z) - static_cast<double>(m.z)) * f),
                        static_cast<float>((static_cast<double>(x.w) - static_cast<double>(m.w)) * f)};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (g + i >= r0 && g + i < r1) {
        if (q32) q32[col_j * ldq + (g + i - row0)] = v[i];
        lo = fminf(lo, v[i]);
        hi = fmaxf(hi, v[i]);
        bad |= !isfinite(v[i]);
      }
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    lo = fminf(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, off));
    hi = fmaxf(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, off));
  }
  bad = __any_sync(0xFFFFFFFFu, bad);
  if ((threadIdx.x & 31) == 0) {
    smin[threadIdx.x >> 5] = bad ? NAN : lo;
    smax[threadIdx.x >> 5] = hi;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 0; w < BLOCK / 32; ++w) {
      bad |= isnan(smin[w]);
      lo = fminf(lo, smin[w]);
      hi = fmaxf(hi, smax[w]);
    }
    const size_t at = static_cast<size_t>(item_k) * n + col_j;
    const float old_lo = pmin[at], old_hi = pmax[at];
    bad |= isnan(old_lo);
    pmin[at] = bad ? NAN : fminf(lo, old_lo);
    pmax[at] = fmaxf(hi, old_hi);
  }
}

__global__ void fill_kernel(float* p, size_t count, float v) {
  for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < count;
       i += static_cast<size_t>(gridDim.x) * blockDim.x)
    p[i] = v;
}

// Codes of the chunk's rows.  A 16-byte group of codes (16 or 32 rows counted from the layer's first
// row) may straddle two chunks: the storage starts as zeros and every call ORs its rows in.
template <int W, int PLANES>
__global__ void __launch_bounds__(BLOCK) chunk_affine_encode_kernel(const float* __restrict__ chunk, long long ld,
                                                                    long long row0, long long row1,
                                                                    const float* __restrict__ wbar,
                                                                    const double* __restrict__ inv, int n,
                                                                    const long long* __restrict__ flat,
                                                                    const long long* __restrict__ internal,
                                                                    const float* __restrict__ a,
                                                                    const float* __restrict__ b, float top,
                                                                    unsigned char* __restrict__ out,
                                                                    long long out_stride, int first_layer) {
  constexpr int RPC = 128 / W;
  const int l = first_layer + blockIdx.z, j = blockIdx.y;
  const long long lay0 = flat[l], lay1 = flat[l + 1];
  const long long f0 = (lay0 > row0 ? lay0 : row0) - lay0, f1 = (lay1 < row1 ? lay1 : row1) - lay0;   // rows of the layer
  if (f1 <= f0) return;
  const long long c0 = f0 / RPC, c1 = (f1 + RPC - 1) / RPC;
  const float al = a[l], bl = b[l];
  const double f = inv[static_cast<size_t>(l) * n + j];
  const float* col = chunk + j * ld - row0 + lay0;
  const float* wb = wbar + lay0;
  uint4* dst = reinterpret_cast<uint4*>(out + j * out_stride);
  uint4* dst_lo = reinterpret_cast<uint4*>(out + (static_cast<long long>(n) + j) * out_stride);
  const float recip = PLANES == 2 ? 0.0f : affine_reciprocal(al, top);
  const float near = (top + 1.0f) * 0x1p-21f;
  const bool aligned = ((reinterpret_cast<uintptr_t>(col) | reinterpret_cast<uintptr_t>(wb)) & 15) == 0;
  for (long long c = c0 + blockIdx.x * static_cast<long long>(BLOCK) + threadIdx.x; c < c1;
       c += static_cast<long long>(gridDim.x) * BLOCK) {
    uint32_t w[4] = {0, 0, 0, 0}, wl[4] = {0, 0, 0, 0};
    bool hard = recip == 0.0f;
    if (!hard) {
#pragma unroll
      for (int k = 0; k < RPC; k += 4) {
        const long long r = c * RPC + k;
        const float4 x = load_rows4(col, r, f0, f1, aligned), m = load_rows4(wb, r, f0, f1, aligned);
        const float e0 = static_cast<float>((static_cast<double>(x.x) - static_cast<double>(m.x)) * f);
        const float e1 = static_cast<float>((static_cast<double>(x.y) - static_cast<double>(m.y)) * f);
        const float e2 = static_cast<float>((static_cast<double>(x.z) - static_cast<double>(m.z)) * f);
        const float e3 = static_cast<float>((static_cast<double>(x.w) - static_cast<double>(m.w)) * f);
        if (r >= f0 && r < f1) put_code<W>(w, k, affine_code_by_reciprocal(e0, bl, recip, top, near, &hard));
        if (r + 1 >= f0 && r + 1 < f1) put_code<W>(w, k + 1, affine_code_by_reciprocal(e1, bl, recip, top, near, &hard));
        if (r + 2 >= f0 && r + 2 < f1) put_code<W>(w, k + 2, affine_code_by_reciprocal(e2, bl, recip, top, near, &hard));
        if (r + 3 >= f0 && r + 3 < f1) put_code<W>(w, k + 3, affine_code_by_reciprocal(e3, bl, recip, top, near, &hard));
      }
    }
    if (hard) {
      w[0] = w[1] = w[2] = w[3] = 0u;
#pragma unroll
      for (int k = 0; k < RPC; ++k) {
        const long long r = c * RPC + k;
        uint32_t u = 0;
        if (r >= f0 && r < f1 && al != 0.0f) {
          const float e = static_cast<float>((static_cast<double>(col[r]) - static_cast<double>(wb[r])) * f);
          u = affine_code(e, bl, al, top);
        }
        if (PLANES == 2) {
          put_code<W>(w, k, u >> 8);
          put_code<W>(wl, k, u & 0xFFu);
        } else {
          put_code<W>(w, k, u);
        }
      }
    }
    const long long q = internal[l] / RPC + c;
    uint4* at = dst + ((q & ~31LL) | twa_chunk_slot(static_cast<int>(q & 31), j));
    uint4 old = *at;
    old.x |= w[0]; old.y |= w[1]; old.z |= w[2]; old.w |= w[3];
    *at = old;
    if (PLANES == 2) {
      at = dst_lo + ((q & ~31LL) | twa_chunk_slot(static_cast<int>(q & 31), n + j));
      old = *at;
      old.x |= wl[0]; old.y |= wl[1]; old.z |= wl[2]; old.w |= wl[3];
      *at = old;
    }
  }
}

// fills the tail of every column (rows from the last layer's end to the column stride) with code 0
__global__ void tail_zero_kernel(unsigned char* out, long long out_stride, long long first_chunk,
                                 long long chunks) {
  const int j = blockIdx.y;
  uint4* dst = reinterpret_cast<uint4*>(out + j * out_stride);
  for (long long q = first_chunk + blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; q < chunks;
       q += static_cast<long long>(gridDim.x) * blockDim.x)
    dst[(q & ~31LL) | twa_chunk_slot(static_cast<int>(q & 31), j)] = make_uint4(0, 0, 0, 0);
}

// Canonical image for parity and checkpoints: unsigned codes in flat row order, one row of bytes per
// candidate; slots of W bits, row (8/W) k + s of a column in bits [s W, (s+1) W) of byte k.  PLANES == 2
// (16-bit codes): two bytes per row, low byte first, from the low-byte column n + j and the high-byte
// column j.
template <int W, int PLANES>
__global__ void __launch_bounds__(BLOCK) layered_export_kernel(const unsigned char* __restrict__ in,
                                                               long long in_stride,
                                                               const long long* __restrict__ flat,
                                                               const long long* __restrict__ internal, int L,
                                                               long long D, int n, unsigned char* __restrict__ out,
                                                               long long row_bytes) {
  constexpr int PER = 8 / W;
  const int j = blockIdx.y;
  unsigned char* dst = out + j * row_bytes;
  for (long long ob = blockIdx.x * static_cast<long long>(BLOCK) + threadIdx.x; ob < row_bytes;
       ob += static_cast<long long>(gridDim.x) * BLOCK) {
    // PLANES == 2: output byte ob is the low (ob even) or high (ob odd) byte of row ob / 2
    const int col = PLANES == 2 ? ((ob & 1) ? j : n + j) : j;
    const unsigned char* src = in + col * in_stride;
    unsigned v = 0;
#pragma unroll
    for (int h = 0; h < PER; ++h) {
      const long long r = PLANES == 2 ? (ob >> 1) : ob * PER + h;
      if (r >= D) break;
      int lo = 0, hi = L;                       // layer of flat row r: last l with flat[l] <= r
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (flat[mid] <= r) lo = mid; else hi = mid;
      }
      const long long ir = internal[lo] + (r - flat[lo]);
      const long long ib = ir * W / 8;
      const long long q = ib >> 4;
      const unsigned char byte = src[(((q & ~31LL) | twa_chunk_slot(static_cast<int>(q & 31), col)) << 4) | (ib & 15)];
      const unsigned code = (byte >> (W * (ir % PER))) & ((1u << W) - 1u);
      v |= code << (W * h);
    }
    dst[ob] = static_cast<unsigned char>(v);
  }
}

// device layout of the construction workspace
struct LwsLayout { size_t items, first_item, flat, internal, partial, pmin, pmax, inv, total; };
LwsLayout lws_layout(size_t n_items, int L, int n) {
  LwsLayout w;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = (o + bytes + 255) / 256 * 256; return at; };
  w.items = take(sizeof(Item) * n_items);
  w.first_item = take(sizeof(int) * (L + 1));
  w.flat = take(sizeof(long long) * (L + 1));
  w.internal = take(sizeof(long long) * (L + 1));
  w.partial = take(sizeof(double) * n_items * n);
  w.pmin = take(sizeof(float) * n_items * n);
  w.pmax = take(sizeof(float) * n_items * n);
  w.inv = take(sizeof(double) * static_cast<size_t>(L) * n);
  w.total = o;
  return w;
}

int upload_partition(twa_ctx* ctx, const Partition& p, int L, char* lws, const LwsLayout& w) {
  TWA_CUDA_OK(ctx, cudaMemcpyAsync(lws + w.items, p.items.data(), sizeof(Item) * p.items.size(),
                                   cudaMemcpyHostToDevice, ctx->stream));
  TWA_CUDA_OK(ctx, cudaMemcpyAsync(lws + w.first_item, p.first_item.data(), sizeof(int) * (L + 1),
                                   cudaMemcpyHostToDevice, ctx->stream));
  TWA_CUDA_OK(ctx, cudaMemcpyAsync(lws + w.flat, p.flat.data(), sizeof(long long) * (L + 1),
                                   cudaMemcpyHostToDevice, ctx->stream));
  TWA_CUDA_OK(ctx, cudaMemcpyAsync(lws + w.internal, p.internal.data(), sizeof(long long) * (L + 1),
                                   cudaMemcpyHostToDevice, ctx->stream));
  // the host vectors are pageable: the copies above have completed on return, but be explicit
  TWA_CUDA_OK(ctx, cudaStreamSynchronize(ctx->stream));
  return TWA_OK;
}

size_t count_items(const int64_t* offsets, int L) {
  size_t k = 0;
  for (int l = 0; l < L; ++l) k += static_cast<size_t>((offsets[l + 1] - offsets[l] + ITEM_ROWS - 1) / ITEM_ROWS);
  return k;
}

// Carves the caller's buffer of a layered basis (codes | a | b | granule table | flat offsets |
// internal offsets | block tables), builds and uploads the tables, and fills the descriptor.
// Entry k of the granule table: (layer, valid rows, first flat row, 0) of the 64-byte granule whose first
// internal row is k * gr; layer -1 behind the last layer.  A layer's internal rows are its flat rows
// rounded up to whole granules, so a granule lies in the last layer whose internal offset is not above
// its first row (empty layers share their offset with the layer after them and are passed over).
__global__ void __launch_bounds__(BLOCK) granule_table_kernel(const long long* __restrict__ flat,
                                                              const long long* __restrict__ internal, int L,
                                                              long long gr, size_t entries, int4* __restrict__ tab) {
  for (size_t k = blockIdx.x * static_cast<size_t>(BLOCK) + threadIdx.x; k < entries;
       k += static_cast<size_t>(gridDim.x) * BLOCK) {
    const long long row = static_cast<long long>(k) * gr;
    int4 e = make_int4(-1, 0, 0, 0);
    if (row < internal[L]) {
      int lo = 0, hi = L - 1;
      while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (internal[mid] <= row) lo = mid;
        else hi = mid - 1;
      }
      const long long len = flat[lo + 1] - flat[lo], k0 = row - internal[lo];
      if (k0 < len) {
        e.x = lo;
        e.y = static_cast<int>(len - k0 < gr ? len - k0 : gr);
        e.z = static_cast<int>(flat[lo] + k0);
      }
    }
    tab[k] = e;
  }
}

int prepare_layered_storage(twa_ctx* ctx, const Partition& p, long long D, int L, int n_cand, int code_bits,
                            void* mem, twa_layered_basis* out) {
  // carve the caller's buffer: codes | a | b | granule table | flat offsets | internal offsets
  char* m = static_cast<char*>(mem);
  const int bits = slot_bits(code_bits), planes = plane_count(code_bits);
  const int n = n_cand * planes;                       // stored columns
  const long long stride = twa_basis_col_stride(p.D_int, bits);
  const size_t codes_bytes = static_cast<size_t>(stride) * n;
  const size_t fl = (sizeof(float) * L + 255) / 256 * 256;
  const size_t n_gran = static_cast<size_t>(stride / 64);
  const size_t off_bytes = (sizeof(long long) * (L + 1) + 255) / 256 * 256;
  size_t o = (codes_bytes + 255) / 256 * 256;
  float* a = reinterpret_cast<float*>(m + o); o += fl;
  float* b = reinterpret_cast<float*>(m + o); o += fl;
  int* gran = reinterpret_cast<int*>(m + o); o += 16 * (n_gran + TABLE_SLACK);
  long long* d_flat = reinterpret_cast<long long*>(m + o); o += off_bytes;
  long long* d_int = reinterpret_cast<long long*>(m + o); o += off_bytes;
  int* d_cta_first = reinterpret_cast<int*>(m + o); o += CTA_TABLE_BYTES;
  int* d_cta_base = reinterpret_cast<int*>(m + o);

  // work split of the step kernels: contiguous tile ranges, and the layers each range meets
  // (slots below 4 bits: one segment per tile -- a tile of 1-bit codes already covers 4096 rows)
  const int kt = bits < 4 ? 1
                          : ((ctx->tune_tile_segments == 1 || ctx->tune_tile_segments == 2) ? ctx->tune_tile_segments
                                                                                           : (n <= 64 ? 2 : 1));
  const long long tile_rows = 512LL * 8 / bits * kt;
  const int tiles = static_cast<int>((p.D_int + tile_rows - 1) / tile_rows);
  int ctas = ctx->sm_count < tiles ? ctx->sm_count : tiles;
  if (ctas > MAX_CTAS) ctas = MAX_CTAS;
  const int tpc = (tiles + ctas - 1) / ctas;
  ctas = (tiles + tpc - 1) / tpc;
  std::vector<int> cta_first(ctas), cta_base(ctas + 1, 0);
  {
    int l = 0;
    for (int k = 0; k < ctas; ++k) {
      const long long r0 = static_cast<long long>(k) * tpc * tile_rows;       // < D_int
      long long r1 = r0 + tpc * tile_rows;
      if (r1 > p.D_int) r1 = p.D_int;
      while (p.internal[l + 1] <= r0) ++l;
      cta_first[k] = l;
      int last = l;
      while (p.internal[last + 1] < r1) ++last;
      cta_base[k + 1] = cta_base[k] + (last - l + 1);
    }
  }
  // granule table: layer, valid rows, first flat row of every 64-byte granule of a column, written on
  // the device from the two offset arrays (the table has a million entries at ViT-B/16 size: built on the
  // host and copied from pageable memory it cost more than the quantiser's kernels)
  {
    TWA_CUDA_OK(ctx, cudaMemcpyAsync(d_flat, p.flat.data(), sizeof(long long) * (L + 1),
                                     cudaMemcpyHostToDevice, ctx->stream));
    TWA_CUDA_OK(ctx, cudaMemcpyAsync(d_int, p.internal.data(), sizeof(long long) * (L + 1),
                                     cudaMemcpyHostToDevice, ctx->stream));
    TWA_CUDA_OK(ctx, cudaMemcpyAsync(d_cta_first, cta_first.data(), sizeof(int) * ctas, cudaMemcpyHostToDevice,
                                     ctx->stream));
    TWA_CUDA_OK(ctx, cudaMemcpyAsync(d_cta_base, cta_base.data(), sizeof(int) * (ctas + 1),
                                     cudaMemcpyHostToDevice, ctx->stream));
    // (with slack, so that the last tile of a two-segment tiling finds entries for all its granules)
    const size_t entries = n_gran + TABLE_SLACK;
    int tgrid = static_cast<int>((entries + BLOCK - 1) / BLOCK);
    if (tgrid > ctx->sm_count * 8) tgrid = ctx->sm_count * 8;
    granule_table_kernel<<<tgrid, BLOCK, 0, ctx->stream>>>(d_flat, d_int, L, granule_rows(bits), entries,
                                                          reinterpret_cast<int4*>(gran));
    TWA_CUDA_OK(ctx, cudaGetLastError());
    TWA_CUDA_OK(ctx, cudaStreamSynchronize(ctx->stream));       // the host arrays above end with this scope
  }

  unsigned char* codes = reinterpret_cast<unsigned char*>(m);
  out->codes = twa_basis{codes, nullptr, p.D_int, stride, n, bits};
  out->a = a;
  out->b = b;
  out->granules = gran;
  out->flat_offsets = reinterpret_cast<int64_t*>(d_flat);
  out->internal_offsets = reinterpret_cast<int64_t*>(d_int);
  out->D = D;
  out->L = L;
  out->code_bits = code_bits;
  out->planes = planes;
  out->cta_count = ctas;
  out->kt = kt;
  out->tiles = tiles;
  out->tiles_per_cta = tpc;
  out->total_runs = cta_base[ctas];
  out->cta_first_layer = d_cta_first;
  out->cta_run_base = d_cta_base;
  return TWA_OK;
}

}  // namespace

extern "C" {

size_t twa_layered_workspace_bytes(const int64_t* offsets_host, int L, int n) {
  if (!offsets_host || L < 1 || n < 1) return 0;
  return lws_layout(count_items(offsets_host, L), L, n).total;
}

int64_t twa_layered_rows(const int64_t* offsets_host, int L, int bits) {
  if (!offsets_host || L < 1 || slot_bits(bits) == 0) return 0;
  const long long gr = granule_rows(slot_bits(bits));
  long long io = 0;
  for (int l = 0; l < L; ++l) io += (offsets_host[l + 1] - offsets_host[l] + gr - 1) / gr * gr;
  return io;
}

size_t twa_layered_basis_bytes(const int64_t* offsets_host, int L, int n, int bits) {
  const int64_t rows = twa_layered_rows(offsets_host, L, bits);
  if (rows < 1 || n < 1) return 0;
  const int w = slot_bits(bits);
  const size_t codes = twa_basis_bytes(rows, n * plane_count(bits), w);
  const size_t granules = static_cast<size_t>(twa_basis_col_stride(rows, w) / 64);
  return codes + 256 + 2 * ((sizeof(float) * L + 255) / 256 * 256) + 16 * (granules + TABLE_SLACK) +
         (sizeof(long long) * (L + 1) + 255) / 256 * 256 * 2 + 2 * CTA_TABLE_BYTES;
}

int twa_build_centered(twa_ctx* ctx, float* W, int64_t D, int n, int64_t ldw, const int64_t* offsets_host,
                       int L, float* wbar_out, twa_basis* P32_out, void* lws, size_t lws_bytes) {
  if (!ctx || !W || !wbar_out || !P32_out || !offsets_host) return TWA_ERR_INVALID_ARG;
  if (D < 1 || D > TWA_MAX_LAUNCH_ROWS || n < 1 || ldw < D) return TWA_ERR_INVALID_ARG;
  if (n > TWA_MAX_N) return TWA_ERR_UNSUPPORTED;
  Partition p;
  int rc = make_partition(offsets_host, L, D, 8, &p);
  if (rc) return rc;
  const LwsLayout w = lws_layout(p.items.size(), L, n);
  if (!lws || lws_bytes < w.total) return TWA_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(W) & 15) || (ldw & 3) || (reinterpret_cast<uintptr_t>(lws) & 15))
    return TWA_ERR_MISALIGNED;
  rc = twa_mean(ctx, W, D, n, ldw, wbar_out);
  if (rc) return rc;
  char* ws = static_cast<char*>(lws);
  rc = upload_partition(ctx, p, L, ws, w);
  if (rc) return rc;
  const Item* items = reinterpret_cast<const Item*>(ws + w.items);
  const int* first_item = reinterpret_cast<const int*>(ws + w.first_item);
  double* partial = reinterpret_cast<double*>(ws + w.partial);
  double* inv = reinterpret_cast<double*>(ws + w.inv);
  const unsigned grid = static_cast<unsigned>(p.items.size() * n);      // (item, column), the column running fastest
  centred_sumsq_kernel<<<grid, BLOCK, 0, ctx->stream>>>(W, ldw, wbar_out, items, n, partial);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  inv_norm_kernel<<<(L * n + 255) / 256, 256, 0, ctx->stream>>>(partial, first_item, L, n, inv, ctx->d_status);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  centre_scale_kernel<<<grid, BLOCK, 0, ctx->stream>>>(W, ldw, wbar_out, items, n, inv);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  *P32_out = twa_basis{W, nullptr, D, 4 * ldw, n, 32};
  return TWA_OK;
}

int twa_quantize_affine(twa_ctx* ctx, const twa_basis* P32, const int64_t* offsets_host, int L, int bits,
                        void* mem, size_t mem_bytes, twa_layered_basis* out, void* lws, size_t lws_bytes) {
  if (!ctx || !P32 || !out || !offsets_host || !mem) return TWA_ERR_INVALID_ARG;
  const int wbits = slot_bits(bits), planes = plane_count(bits);
  if (wbits == 0) return TWA_ERR_UNSUPPORTED;
  int rc = twa_check_basis(P32);
  if (rc) return rc;
  if (P32->bits != 32) return TWA_ERR_INVALID_ARG;
  const long long D = P32->D;
  const int n = P32->n;
  if (n * planes > TWA_MAX_N) return TWA_ERR_UNSUPPORTED;
  Partition p;
  rc = make_partition(offsets_host, L, D, wbits, &p);
  if (rc) return rc;
  const LwsLayout w = lws_layout(p.items.size(), L, n);
  if (!lws || lws_bytes < w.total) return TWA_ERR_WORKSPACE;
  if (mem_bytes < twa_layered_basis_bytes(offsets_host, L, n, bits)) return TWA_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(mem) & 255) || (reinterpret_cast<uintptr_t>(lws) & 15)) return TWA_ERR_MISALIGNED;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  char* ws = static_cast<char*>(lws);
  rc = upload_partition(ctx, p, L, ws, w);
  if (rc) return rc;

  rc = prepare_layered_storage(ctx, p, D, L, n, bits, mem, out);
  if (rc) return rc;
  float* a = out->a;
  float* b = out->b;
  const long long stride = out->codes.col_stride;

  const Item* items = reinterpret_cast<const Item*>(ws + w.items);
  const int* first_item = reinterpret_cast<const int*>(ws + w.first_item);
  float* pmin = reinterpret_cast<float*>(ws + w.pmin);
  float* pmax = reinterpret_cast<float*>(ws + w.pmax);
  const float* P = static_cast<const float*>(P32->data);
  const long long ld = P32->col_stride / 4;
  const unsigned grid = static_cast<unsigned>(p.items.size() * n);      // (item, column), the column running fastest
  minmax_kernel<<<grid, BLOCK, 0, ctx->stream>>>(P, ld, items, n, pmin, pmax);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  const float top = top_code(bits);
  factors_kernel<<<L, 128, 0, ctx->stream>>>(pmin, pmax, first_item, L, n, top, a, b, ctx->d_status);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  long long max_len = 0;
  for (int l = 0; l < L; ++l) max_len = std::max(max_len, p.internal[l + 1] - p.internal[l]);
  const int rpc = 128 / wbits;
  long long gx = (max_len / rpc + BLOCK - 1) / BLOCK;
  if (gx > 64) gx = 64;
  if (gx < 1) gx = 1;
  if (L > 65535) return TWA_ERR_UNSUPPORTED;
  const dim3 egrid(static_cast<unsigned>(gx), static_cast<unsigned>(n), static_cast<unsigned>(L));
  unsigned char* codes = static_cast<unsigned char*>(out->codes.data);
  const long long* fl_d = reinterpret_cast<const long long*>(ws + w.flat);
  const long long* in_d = reinterpret_cast<const long long*>(ws + w.internal);
  if (planes == 2)
    affine_encode_kernel<8, 2><<<egrid, BLOCK, 0, ctx->stream>>>(P, ld, fl_d, in_d, a, b, top, n, codes, stride);
  else if (wbits == 8)
    affine_encode_kernel<8, 1><<<egrid, BLOCK, 0, ctx->stream>>>(P, ld, fl_d, in_d, a, b, top, n, codes, stride);
  else if (wbits == 4)
    affine_encode_kernel<4, 1><<<egrid, BLOCK, 0, ctx->stream>>>(P, ld, fl_d, in_d, a, b, top, n, codes, stride);
  else if (wbits == 2)
    affine_encode_kernel<2, 1><<<egrid, BLOCK, 0, ctx->stream>>>(P, ld, fl_d, in_d, a, b, top, n, codes, stride);
  else
    affine_encode_kernel<1, 1><<<egrid, BLOCK, 0, ctx->stream>>>(P, ld, fl_d, in_d, a, b, top, n, codes, stride);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  const long long total_chunks = stride / 16, first_tail = p.D_int / rpc;
  if (first_tail < total_chunks) {
    tail_zero_kernel<<<dim3(1, n * planes), 64, 0, ctx->stream>>>(codes, stride, first_tail, total_chunks);
    TWA_CUDA_OK(ctx, cudaGetLastError());
  }
  return TWA_OK;
}

int twa_layered_export(twa_ctx* ctx, const twa_layered_basis* lb, void* codes_out, float* a_out,
                       float* b_out) {
  if (!ctx || !lb || !codes_out || !a_out || !b_out) return TWA_ERR_INVALID_ARG;
  const int bits = lb->codes.bits, planes = lb->planes;
  if ((bits != 8 && bits != 4 && bits != 2 && bits != 1) || (planes != 1 && planes != 2)) return TWA_ERR_UNSUPPORTED;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  const int n = lb->codes.n / planes;
  const long long row_bytes = planes == 2 ? 2 * lb->D : (lb->D * bits + 7) / 8;
  long long gx = (row_bytes + BLOCK * 8 - 1) / (BLOCK * 8);
  if (gx > 1024) gx = 1024;
  const dim3 grid(static_cast<unsigned>(gx), static_cast<unsigned>(n));
  const unsigned char* in = static_cast<const unsigned char*>(lb->codes.data);
  const long long* fl = reinterpret_cast<const long long*>(lb->flat_offsets);
  const long long* il = reinterpret_cast<const long long*>(lb->internal_offsets);
  unsigned char* o = static_cast<unsigned char*>(codes_out);
  const long long st = lb->codes.col_stride;
  if (planes == 2) layered_export_kernel<8, 2><<<grid, BLOCK, 0, ctx->stream>>>(in, st, fl, il, lb->L, lb->D, n, o, row_bytes);
  else if (bits == 8) layered_export_kernel<8, 1><<<grid, BLOCK, 0, ctx->stream>>>(in, st, fl, il, lb->L, lb->D, n, o, row_bytes);
  else if (bits == 4) layered_export_kernel<4, 1><<<grid, BLOCK, 0, ctx->stream>>>(in, st, fl, il, lb->L, lb->D, n, o, row_bytes);
  else if (bits == 2) layered_export_kernel<2, 1><<<grid, BLOCK, 0, ctx->stream>>>(in, st, fl, il, lb->L, lb->D, n, o, row_bytes);
  else layered_export_kernel<1, 1><<<grid, BLOCK, 0, ctx->stream>>>(in, st, fl, il, lb->L, lb->D, n, o, row_bytes);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  TWA_CUDA_OK(ctx, cudaMemcpyAsync(a_out, lb->a, sizeof(float) * lb->L, cudaMemcpyDeviceToDevice, ctx->stream));
  TWA_CUDA_OK(ctx, cudaMemcpyAsync(b_out, lb->b, sizeof(float) * lb->L, cudaMemcpyDeviceToDevice, ctx->stream));
  return TWA_OK;
}

}  // extern "C"

// ------------------------------------------------------------------------------------------------
// Row-chunked form of twa_build_centered + twa_quantize_affine
// ------------------------------------------------------------------------------------------------
namespace {

// Items [k0, k1) and layers [l0, l1] that meet flat rows [row0, row1), and the number of items in all,
// from the layer offsets alone (make_partition's numbering: a layer's items follow one another,
// ITEM_ROWS rows each).  Returns false for offsets make_partition would reject.
bool chunk_range(const int64_t* offsets, int L, long long D, long long row0, long long row1, int* k0, int* k1,
                 int* l0, int* l1, size_t* n_items) {
  if (!offsets || L < 1 || offsets[0] != 0 || offsets[L] != D) return false;
  size_t first = 0;
  *l0 = *l1 = -1;
  for (int l = 0; l < L; ++l) {
    const long long a = offsets[l], b = offsets[l + 1];
    if (b <= a) return false;
    if (row0 >= a && row0 < b) {
      *l0 = l;
      *k0 = static_cast<int>(first + static_cast<size_t>((row0 - a) / ITEM_ROWS));
    }
    if (row1 - 1 >= a && row1 - 1 < b) {
      *l1 = l;
      *k1 = static_cast<int>(first + static_cast<size_t>((row1 - 1 - a) / ITEM_ROWS)) + 1;
    }
    first += static_cast<size_t>((b - a + ITEM_ROWS - 1) / ITEM_ROWS);
  }
  *n_items = first;
  return *l0 >= 0 && *l1 >= *l0;
}

}  // namespace

extern "C" {

int twa_layered_build_begin(twa_ctx* ctx, int64_t D, int n, const int64_t* offsets_host, int L, int bits, void* mem,
                            size_t mem_bytes, twa_layered_basis* out, void* lws, size_t lws_bytes) {
  if (!ctx || !out || !offsets_host || !mem) return TWA_ERR_INVALID_ARG;
  if (slot_bits(bits) == 0) return TWA_ERR_UNSUPPORTED;
  if (D < 1 || D > TWA_MAX_LAUNCH_ROWS || n < 1) return TWA_ERR_INVALID_ARG;
  if (n * plane_count(bits) > TWA_MAX_N || L > 65535) return TWA_ERR_UNSUPPORTED;
  Partition p;
  int rc = make_partition(offsets_host, L, D, slot_bits(bits), &p);
  if (rc) return rc;
  const LwsLayout w = lws_layout(p.items.size(), L, n);
  if (!lws || lws_bytes < w.total) return TWA_ERR_WORKSPACE;
  if (mem_bytes < twa_layered_basis_bytes(offsets_host, L, n, bits)) return TWA_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(mem) & 255) || (reinterpret_cast<uintptr_t>(lws) & 15)) return TWA_ERR_MISALIGNED;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  char* ws = static_cast<char*>(lws);
  rc = upload_partition(ctx, p, L, ws, w);
  if (rc) return rc;
  rc = prepare_layered_storage(ctx, p, D, L, n, bits, mem, out);
  if (rc) return rc;
  const size_t cells = p.items.size() * static_cast<size_t>(n);
  TWA_CUDA_OK(ctx, cudaMemsetAsync(ws + w.partial, 0, sizeof(double) * cells, ctx->stream));
  fill_kernel<<<64, 256, 0, ctx->stream>>>(reinterpret_cast<float*>(ws + w.pmin), cells, INFINITY);
  fill_kernel<<<64, 256, 0, ctx->stream>>>(reinterpret_cast<float*>(ws + w.pmax), cells, -INFINITY);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  TWA_CUDA_OK(ctx, cudaMemsetAsync(out->codes.data, 0, static_cast<size_t>(out->codes.col_stride) * out->codes.n,
                                   ctx->stream));
  return TWA_OK;
}

int twa_layered_build_feed(twa_ctx* ctx, const twa_layered_basis* lb, const int64_t* offsets_host, int pass,
                           const float* chunk, int64_t ld, int64_t row0, int64_t rows, float* wbar,
                           float* q32_out, int64_t ldq, void* lws, size_t lws_bytes) {
  if (!ctx || !lb || !offsets_host || !chunk || !wbar || pass < 0 || pass > 2) return TWA_ERR_INVALID_ARG;
  const long long D = lb->D;
  const int planes = lb->planes == 2 ? 2 : 1;
  const int n = lb->codes.n / planes, L = lb->L, bits = lb->codes.bits;
  if (rows < 1 || row0 < 0 || row0 + rows > D || ld < rows) return TWA_ERR_INVALID_ARG;
  if (q32_out && (pass != 1 || ldq < rows)) return TWA_ERR_INVALID_ARG;
  // the mean of the chunk is written with 16-byte stores at wbar + row0
  if ((reinterpret_cast<uintptr_t>(chunk) & 15) || (ld & 3) || (row0 & 3) || (reinterpret_cast<uintptr_t>(wbar) & 15))
    return TWA_ERR_MISALIGNED;
  const long long row1 = row0 + rows;
  int k0 = 0, k1 = 0, l0, l1, rc;
  size_t n_items;
  if (!chunk_range(offsets_host, L, D, row0, row1, &k0, &k1, &l0, &l1, &n_items) || k1 <= k0) return TWA_ERR_INVALID_ARG;
  const LwsLayout w = lws_layout(n_items, L, n);
  if (!lws || lws_bytes < w.total) return TWA_ERR_WORKSPACE;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  char* ws = static_cast<char*>(lws);
  const Item* items = reinterpret_cast<const Item*>(ws + w.items) + k0;
  const size_t cell0 = static_cast<size_t>(k0) * n;
  const unsigned grid = static_cast<unsigned>((k1 - k0) * n);            // (item, column), the column running fastest
  const double* inv = reinterpret_cast<const double*>(ws + w.inv);
  if (pass == 0) {
    rc = twa_mean(ctx, chunk, rows, n, ld, wbar + row0);
    if (rc) return rc;
    chunk_centred_sumsq_kernel<<<grid, BLOCK, 0, ctx->stream>>>(chunk, ld, row0, row1, wbar, items, n,
                                                                reinterpret_cast<double*>(ws + w.partial) + cell0);
  } else if (pass == 1) {
    chunk_minmax_kernel<<<grid, BLOCK, 0, ctx->stream>>>(chunk, ld, row0, row1, wbar, items, n, inv,
                                                         reinterpret_cast<float*>(ws + w.pmin) + cell0,
                                                         reinterpret_cast<float*>(ws + w.pmax) + cell0, q32_out, ldq);
  } else {
    const int rpc = 128 / bits;
    long long gx = (rows / rpc + 2 + BLOCK - 1) / BLOCK;
    if (gx > 64) gx = 64;
    const dim3 egrid(static_cast<unsigned>(gx), static_cast<unsigned>(n), static_cast<unsigned>(l1 - l0 + 1));
    const long long* fl_d = reinterpret_cast<const long long*>(ws + w.flat);
    const long long* in_d = reinterpret_cast<const long long*>(ws + w.internal);
    unsigned char* codes = static_cast<unsigned char*>(lb->codes.data);
    const float top = top_code(lb->code_bits);
    const long long st = lb->codes.col_stride;
#define TWA_CHUNK_ENCODE(W, PL) \
    chunk_affine_encode_kernel<W, PL><<<egrid, BLOCK, 0, ctx->stream>>>(chunk, ld, row0, row1, wbar, inv, n, fl_d, in_d, \
                                                                        lb->a, lb->b, top, codes, st, l0)
    if (planes == 2) TWA_CHUNK_ENCODE(8, 2);
    else if (bits == 8) TWA_CHUNK_ENCODE(8, 1);
    else if (bits == 4) TWA_CHUNK_ENCODE(4, 1);
    else if (bits == 2) TWA_CHUNK_ENCODE(2, 1);
    else TWA_CHUNK_ENCODE(1, 1);
#undef TWA_CHUNK_ENCODE
  }
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}

int twa_layered_build_end_pass(twa_ctx* ctx, const twa_layered_basis* lb, const int64_t* offsets_host, int pass,
                               void* lws, size_t lws_bytes) {
  if (!ctx || !lb || !offsets_host || pass < 0 || pass > 2) return TWA_ERR_INVALID_ARG;
  const int n = lb->codes.n / (lb->planes == 2 ? 2 : 1), L = lb->L;
  const LwsLayout w = lws_layout(count_items(offsets_host, L), L, n);
  if (!lws || lws_bytes < w.total) return TWA_ERR_WORKSPACE;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  char* ws = static_cast<char*>(lws);
  const int* first_item = reinterpret_cast<const int*>(ws + w.first_item);
  if (pass == 0) {
    inv_norm_kernel<<<(L * n + 255) / 256, 256, 0, ctx->stream>>>(reinterpret_cast<const double*>(ws + w.partial),
                                                                 first_item, L, n, reinterpret_cast<double*>(ws + w.inv),
                                                                 ctx->d_status);
  } else if (pass == 1) {
    factors_kernel<<<L, 128, 0, ctx->stream>>>(reinterpret_cast<const float*>(ws + w.pmin),
                                                             reinterpret_cast<const float*>(ws + w.pmax), first_item, L, n,
                                                             top_code(lb->code_bits), lb->a, lb->b, ctx->d_status);
  }
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}

}  // extern "C"
