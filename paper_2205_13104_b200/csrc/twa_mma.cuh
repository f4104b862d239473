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

// Producer loop: tile k of this block's sequence is t_first + k * t_step (k < t_count); with
// `reverse` the sequence is walked from its end.  g_boxes 1-D boxes of 256 gradient elements
// follow the tile of P~ in a stage (project only).
__device__ __forceinline__ void producer_loop_mma(twa_smem_header* hdr, unsigned char* ring,
                                                  const CUtensorMap* map_p, const CUtensorMap* map_g,
                                                  int t_first, int t_step, int t_count, int stages,
                                                  unsigned stage_bytes, int kt, int g_boxes,
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
    twa_tma_load_2d(dst, map_p, tile * TWA_TILE_COL_WORDS * kt, 0, fb);
    for (int b = 0; b < g_boxes; ++b)
      twa_tma_load_1d(dst + g_off + b * 256 * g_elem_bytes, map_g, tile * tile_rows + b * 256, fb);
    ++issued;
    if (++s == stages) {
      s = 0;
      if (issued > stages) phase ^= 1u;
    }
  }
  if (!ok) {
    twa_set_status(status, TWA_ERR_TIMEOUT, -1);
    const int live = issued < stages ? issued : stages;
    for (int q = 0; q < live; ++q) {      // let the copies already issued land
      const int last = ((issued - 1 - q) / stages) * stages + q;
      const unsigned par = static_cast<unsigned>(last / stages) & 1u;
      const unsigned long long t0 = twa_globaltimer();
      while (!twa_mbar_try_wait(twa_smem_u32(&hdr->full[q]), par)) {
        if (twa_globaltimer() - t0 > limit) break;
      }
    }
  }
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

