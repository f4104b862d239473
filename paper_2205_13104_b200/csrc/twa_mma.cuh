// Device helpers shared by the tensor-pipe streaming kernels (twa_stream_mma.cu,
// twa_layered_step.cu): matrix loads, the integer MMA, the digit cut, and the producer loop.
#pragma once

#include "twa_common.cuh"

constexpr int MMA_WARPS = 16;
constexpr int MMA_THREADS = (MMA_WARPS + 1) * 32;
constexpr int DIGIT_SCRATCH = 256;             // bytes of digit scratch per warp
constexpr float RND = 12582912.0f;             // 2^23 + 2^22: x + RND rounds x to an integer (ties to even)

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}

// d += a (16 x 32, u8) * b (32 x 8, s8), int32 accumulation
__device__ __forceinline__ void mma_u8s8(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// d += a (16 x 32, s8) * b (32 x 8, s8), int32 accumulation
__device__ __forceinline__ void mma_s8(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// d = a (16 x 32, s8) * b (32 x 8, s8): the first product of a sum, no accumulator to clear
__device__ __forceinline__ void mma_s8_first(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "r"(0));
}

// d = a (16 x 32, u8) * b (32 x 8, s8): the first product of a sum, no accumulator to clear
__device__ __forceinline__ void mma_u8s8_first(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "r"(0));
}

// |v| < 2^22 -> float, exactly, without the conversion unit
__device__ __forceinline__ float small_int_to_float(int v) {
  return __int_as_float(0x4B400000 + v) - RND;
}

// Two neighbouring digit sums as one float: (128 * hi + lo) * w_lo, w_lo the weight of the lower digit.
// The integer has up to 27 bits; its conversion rounds once (2^-24 relative).
__device__ __forceinline__ float digit_pair_to_float(int hi, int lo, float w_lo) {
  return static_cast<float>(hi * 128 + lo) * w_lo;
}

// Four signed base-128 digits of t (|t| <= 64): t = d0 + d1/128 + d2/128^2 + d3/128^3 + eps,
// |eps| <= 2^-22, every digit in [-64, 64].  Returned packed, digit k in byte k.
__device__ __forceinline__ uint32_t cut_digits(float t) {
  const float m0 = t + RND;
  t = (t - (m0 - RND)) * 128.0f;
  const float m1 = t + RND;
  t = (t - (m1 - RND)) * 128.0f;
  const float m2 = t + RND;
  t = (t - (m2 - RND)) * 128.0f;
  const float m3 = t + RND;
  const uint32_t lo = __byte_perm(__float_as_uint(m0), __float_as_uint(m1), 0x0040);  // bytes m0.b0, m1.b0
  const uint32_t hi = __byte_perm(__float_as_uint(m2), __float_as_uint(m3), 0x0040);
  return __byte_perm(lo, hi, 0x5410);
}

// d += a (16 x 32, s8) * b (32 x 8, u8), int32 accumulation
__device__ __forceinline__ void mma_s8u8(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.s8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// d = a (16 x 32, s8) * b (32 x 8, u8): the first product of a sum, no accumulator to clear
__device__ __forceinline__ void mma_s8u8_first(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.s8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "r"(0));
}

// d += a (16 x 32, u8) * b (32 x 8, u8), int32 accumulation
__device__ __forceinline__ void mma_u8u8(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void ldmatrix_x2(uint32_t addr, uint32_t& r0, uint32_t& r1) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}

// ---- byte digits of the gradient (projection kernels) ---------------------------------------------
// A block of gradient values with largest magnitude below 2^(e-126) (e = its biased exponent) is
// turned into integers q = round(g * 2^sexp), |q| <= 2^22, by ONE fused multiply-add with the
// constant RND = 1.5 * 2^23: the float RND + q has the bit pattern 0x4B400000 + q, so its three low
// bytes are the base-256 digits of q + 2^22:
//     q = u0 + 256 u1 + 65536 (u2 - 64),   u0, u1 in [0, 255], u2 in [0, 128].
// The integer MMAs take the three bytes as unsigned operands next to a column of ones, whose dot
// product (the sum of the codes) removes the offset 64 of the top byte.  For float32 gradients a
// fourth byte carries the remainder: r = round((g * 2^sexp - q) * 254) in [-127, 127], stored as
// r + 128, again next to a column of ones.  Error of the cut: 2^-23 (three bytes) or 2^-31 (four)
// of the power of two above the block's largest magnitude.
constexpr int BYTE_DIGIT_ROWS = 8;              // rows of a digit matrix: u0, u1, u2, ones, r + 128, ones, 0, 0
constexpr int BYTE_DIGIT_STRIDE = 48;           // bytes between digit rows: 32 gradient rows + 16 of padding, so
                                                // that the eight 16-byte rows of a matrix load fall into
                                                // eight different groups of four banks
constexpr int BYTE_DIGIT_SET = BYTE_DIGIT_ROWS * BYTE_DIGIT_STRIDE;
constexpr int BYTE_DIGIT_SCRATCH = 2 * BYTE_DIGIT_SET;    // per warp: even and odd rows (4-bit codes)

struct ByteDigitScale {
  float up;        // 2^sexp
  float w0;        // 2^-sexp, the weight of u0
  bool live;       // false: every value of the block is below 2^-122 and contributes nothing
  bool bad;        // NaN or Inf among the values
};

// mb = largest |g| of the block as a bit pattern
__device__ __forceinline__ ByteDigitScale byte_digit_scale(unsigned mb) {
  const int ebits = static_cast<int>(mb >> 23);
  ByteDigitScale s;
  s.bad = ebits >= 255;
  s.live = ebits >= 5 && ebits < 255;
  int sexp = 148 - ebits;                                  // |g| 2^sexp < 2^22
  sexp = sexp > 126 ? 126 : sexp;
  s.up = __uint_as_float(static_cast<unsigned>(127 + sexp) << 23);
  s.w0 = __uint_as_float(static_cast<unsigned>(127 - sexp) << 23);
  return s;
}

// Fills the constant rows of a warp's digit matrices (ones in row 3, and in row 5 with four-byte
// digits; zeros elsewhere); rows 0-2 (and 4) are rewritten for every block of rows.
template <bool FOUR, int SETS = 2>
__device__ __forceinline__ void byte_digit_init(unsigned char* digw, int lane) {
  uint32_t* w = reinterpret_cast<uint32_t*>(digw);
#pragma unroll
  for (int i = 0; i < SETS * BYTE_DIGIT_SET / 128; ++i) {
    const int idx = lane + 32 * i;                         // word of the scratch
    const int row = (idx % (BYTE_DIGIT_SET / 4)) / (BYTE_DIGIT_STRIDE / 4);
    w[idx] = (row == 3 || (FOUR && row == 5)) ? 0x01010101u : 0u;
  }
}

// Writes the digits of the lane's value of gradient row `lane` into digit matrix `set`.
template <bool FOUR>
__device__ __forceinline__ void byte_digit_store(unsigned char* digw, int set, int lane, float g, float up) {
  const float y = fmaf(g, up, RND);
  const uint32_t b = __float_as_uint(y);
  unsigned char* d = digw + set * BYTE_DIGIT_SET + lane;
  d[0] = static_cast<unsigned char>(b);
  d[BYTE_DIGIT_STRIDE] = static_cast<unsigned char>(b >> 8);
  d[2 * BYTE_DIGIT_STRIDE] = static_cast<unsigned char>(b >> 16);
  if (FOUR) {
    const float rem = fmaf(g, up, -(y - RND));             // exact: g * up - q
    d[4 * BYTE_DIGIT_STRIDE] = static_cast<unsigned char>(__float_as_uint(fmaf(rem, 254.0f, RND + 128.0f)));
  }
}

// Address a lane hands to ldmatrix for the warp's digit matrices: matrix m = lane / 8 is the (m & 1)-th
// half (gradient rows 16 (m & 1) ...) of set m / 2, row lane % 8 is digit lane % 8.
__device__ __forceinline__ uint32_t byte_digit_ldmatrix_addr(const unsigned char* digw, int lane) {
  const int m = lane >> 3;
  return twa_smem_u32(digw + (m >> 1) * BYTE_DIGIT_SET + (lane & 7) * BYTE_DIGIT_STRIDE + (m & 1) * 16);
}

// Lane constants of the recombination: the accumulator columns of lane tig hold digits 2 tig, 2 tig + 1.
//   tig 0: u0 + 256 u1, weight w0;  tig 1: u2 - 64 ones, weight 65536 w0;
//   tig 2: (r + 128) - 128 ones, weight w0 / 254;  tig 3: nothing.
__device__ __forceinline__ int byte_digit_mult(int tig) { return tig == 0 ? 256 : (tig == 1 ? -64 : (tig == 2 ? -128 : 0)); }
__device__ __forceinline__ float byte_digit_weight(int tig, float w0) {
  return tig == 0 ? w0 : (tig == 1 ? w0 * 65536.0f : (tig == 2 ? w0 * (1.0f / 254.0f) : 0.0f));
}

// Producer loop: tile k of this block's sequence is t_first + k * t_step (k < t_count); with
// `reverse` the sequence is walked from its end; x_per_tile = elements of the codes' tensor map a tile
// advances along a column.  g_boxes 1-D boxes of 256 gradient elements follow the tile of P~ in a
// stage (project only).
__device__ __forceinline__ void producer_loop_mma(twa_smem_header* hdr, unsigned char* ring,
                                                  const CUtensorMap* map_p, const CUtensorMap* map_g,
                                                  int t_first, int t_step, int t_count, int stages,
                                                  unsigned stage_bytes, int x_per_tile, int g_boxes,
                                                  int g_elem_bytes, int tile_rows, unsigned g_off,
                                                  unsigned tx_bytes, bool reverse, int* status,
                                                  unsigned long long limit) {
  twa_prefetch_tensormap(map_p);
  if (g_boxes > 0) twa_prefetch_tensormap(map_g);
  volatile int* abort_flag = &hdr->abort_flag;
  int s = 0, issued = 0;
  unsigned phase = 0;
  bool ok = true;
  for (int k = 0; k < t_count; ++k) {
    if (issued >= stages) {
      if (!twa_mbar_wait(twa_smem_u32(&hdr->empty[s]), phase, abort_flag, limit)) {
        ok = false;
        break;
      }
    }
    const int tile = t_first + (reverse ? (t_count - 1 - k) : k) * t_step;
    const uint32_t fb = twa_smem_u32(&hdr->full[s]);
    const uint32_t dst = twa_smem_u32(ring + static_cast<size_t>(s) * stage_bytes);
    twa_mbar_expect_tx(fb, tx_bytes);
    twa_tma_load_2d(dst, map_p, tile * x_per_tile, 0, fb);
    for (int b = 0; b < g_boxes; ++b)
      twa_tma_load_1d(dst + g_off + b * 256 * g_elem_bytes, map_g, tile * tile_rows + b * 256, fb);
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

__device__ __forceinline__ void init_barriers(twa_smem_header* hdr, int stages) {
  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      twa_mbar_init(twa_smem_u32(&hdr->full[s]), 1);
      twa_mbar_init(twa_smem_u32(&hdr->empty[s]), MMA_WARPS);
    }
    hdr->abort_flag = 0;
    hdr->last_flag = 0;
    hdr->bad_flag = 0;
    hdr->amax_bits = 0;
    twa_fence_barrier_init();
  }
}

