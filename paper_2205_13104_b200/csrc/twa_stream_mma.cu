// Projection and lift for 8- and 4-bit bases with the code x value products done as exact
// integer dot products on the tensor pipe (Section 4.2 / 4.3 of the paper; loop body of
// Algorithm 1; storage of Section 4.6).
//
// Why: the streams are HBM-bound only if the SM keeps up.  Turning every code into a float
// costs three issue slots per code (byte permute, subtract, FMA) plus the compiler's register
// traffic, which measured 5.7 instructions per code and 80 % issue utilisation at 60 % of DRAM
// throughput.  Here the codes go from shared memory to the tensor pipe as they are:
//
//   project:  g is cut, per 32 or 64 bytes of a column (32 to 128 rows), into four signed base-128
//             digits of a common power-of-two scale (block fixed point, 2^-29 of the block
//             maximum, finer than float32 relative to the block), and  sum_r code[r,j] * digit_k[r]  is one
//             integer MMA per 16 columns; the four digit sums are recombined in float32.
//   lift:     the n coefficients s_j * alpha_j are cut into digits once per kernel, and
//             sum_j code[r,j] * digit_k[j]  is an integer MMA per 16 rows and 32 columns.
//
// Integer sums are exact, so the results do not depend on the order of accumulation; the only
// roundings are the digit cut (absolute, 2^-29 of the block maximum), the float32 recombination
// and the float32 accumulation across tiles, which runs in a fixed order.
//
// Data movement is the same as in the float path (twa_stream.cu): persistent blocks, one
// producer lane issuing TMA copies into a ring of stages, full/empty mbarriers with bounded
// waits.  A tile is [n columns][512 bytes] in shared memory, one TMA box per stage; the 16-byte
// chunks of a column are stored permuted (twa_chunk_slot) so that ldmatrix reads of eight
// neighbouring columns hit eight different bank groups.
// Warp w of the 16 consumer warps owns bytes [32w, 32w+32) of every column of a tile; warps
// never wait for one another inside the tile loop.
#include <stdio.h>

#include "twa_mma.cuh"

namespace {

struct ProjectMmaArgs {
  long long D;
  int n, stages, tiles;
  int kt;                      // 512-byte segments of a column per tile (1 or 2)
  unsigned stage_bytes, g_off, tx_bytes, scratch_off;
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

struct LiftMmaArgs {
  long long D;
  int n, stages, tiles;
  int kt;                      // 512-byte segments of a column per tile (1 or 2)
  unsigned stage_bytes, tx_bytes, table_off;
  unsigned base_off;           // offset of the tile's rows of the base vector inside a stage (BTMA)
  const float* scales;
  const float* alpha;
  float alpha_mult;
  const float* base;
  float* out;
  int reverse;
  int* status;
  unsigned long long wait_limit_ns;
};

// =================================================================================================
// project
// =================================================================================================
// MT = number of 16-column groups, ceil(n / 16): a compile-time constant so that the MMA loops
// carry no guards and only the accumulators that exist are kept.
template <int BITS, bool GBF16, int MT, int KT>
__global__ void __launch_bounds__(MMA_THREADS, 1)
twa_project_mma_kernel(const __grid_constant__ CUtensorMap map_p,
                       const __grid_constant__ CUtensorMap map_g, const ProjectMmaArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  // stages start on 1024-byte boundaries (TMA destinations need 128)
  unsigned char* smem = smem_raw + ((1024u - (twa_smem_u32(smem_raw) & 1023u)) & 1023u);
  constexpr int SROWS = twa_tile_rows(BITS);           // rows behind one 512-byte segment: 512 or 1024
  constexpr int WROWS = SROWS / MMA_WARPS;             // rows behind 32 bytes: 32 or 64
  constexpr int GSZ = GBF16 ? 2 : 4;
  twa_smem_header* hdr = reinterpret_cast<twa_smem_header*>(smem);
  unsigned char* ring = smem + TWA_SMEM_HEADER;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gid = lane >> 2, tig = lane & 3;

  init_barriers(hdr, a.stages);
  if (threadIdx.x < TWA_MAX_N) hdr->c_part[threadIdx.x] = 0.0f;
  __syncthreads();

  float facc[MT][2];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) facc[mt][0] = facc[mt][1] = 0.0f;

  if (warp == MMA_WARPS) {
    if (lane == 0)
      producer_loop_mma(hdr, ring, &map_p, &map_g, blockIdx.x, gridDim.x,
                        (a.tiles - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) /
                            static_cast<int>(gridDim.x),
                        a.stages, a.stage_bytes, TWA_TILE_COL_BYTES / 8 * KT, SROWS * KT / 256, GSZ, SROWS * KT, a.g_off,
                        a.tx_bytes, false, a.status, a.wait_limit_ns);
  } else {
    unsigned char* digw = smem + a.scratch_off + warp * BYTE_DIGIT_SCRATCH;   // this warp's digit matrices
    constexpr bool FOUR = !GBF16;                       // float32 gradients carry a fourth byte digit
    byte_digit_init<FOUR>(digw, lane);
    __syncwarp();
    const uint32_t dig_addr = byte_digit_ldmatrix_addr(digw, lane);
    const int dmult = byte_digit_mult(tig);
    const int lm = lane >> 3, lr = lane & 7;            // ldmatrix: matrix and row this lane addresses
    const int jmax = a.n - 1;                           // last column that exists in shared memory
    constexpr int col_bytes = TWA_TILE_COL_BYTES * KT;
    // The warp owns bytes [32*KT*warp, 32*KT*(warp+1)) of every column: KT blocks of 32 bytes.
    // Offsets, inside a tile, of the 16-byte chunk this lane hands to ldmatrix for block u and
    // column group mt (they do not change from tile to tile).
    uint32_t aoff[KT][MT];
#pragma unroll
    for (int u = 0; u < KT; ++u)
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        int j = mt * 16 + lr + 8 * (lm & 1);
        j = j < jmax ? j : jmax;
        const int chunk = (warp * KT + u) * 2 + (lm >> 1);
        aoff[u][mt] = static_cast<uint32_t>(j * col_bytes + ((chunk >> 5) << 9) +
                                            (twa_chunk_slot(chunk & 31, j) << 4));
      }
    volatile int* abort_flag = &hdr->abort_flag;
    int s = 0;
    unsigned phase = 0;
    bool bad = false;
    for (int t = blockIdx.x; t < a.tiles; t += gridDim.x) {
      if (!twa_mbar_wait(twa_smem_u32(&hdr->full[s]), phase, abort_flag, a.wait_limit_ns)) {
        twa_set_status(a.status, TWA_ERR_TIMEOUT, -1);
        break;
      }
      const unsigned char* st = ring + static_cast<size_t>(s) * a.stage_bytes;
      const uint32_t tile_base = twa_smem_u32(st);
      // ---- the warp's rows of g: per block 1 (8-bit) or 2 (4-bit) per lane -------------------
      float g0[KT], g1[KT];
      unsigned mb = 0u;
#pragma unroll
      for (int u = 0; u < KT; ++u) {
        g1[u] = 0.0f;
        const int vw = warp * KT + u;                   // index of the 32-byte block in the column
        if (BITS == 8) {
          if (GBF16) g0[u] = __uint_as_float(static_cast<uint32_t>(
                         reinterpret_cast<const unsigned short*>(st + a.g_off)[vw * WROWS + lane]) << 16);
          else g0[u] = reinterpret_cast<const float*>(st + a.g_off)[vw * WROWS + lane];
        } else {
          if (GBF16) {
            const uint32_t pr = reinterpret_cast<const uint32_t*>(st + a.g_off)[vw * 32 + lane];
            g0[u] = twa_bf16_lo(pr);
            g1[u] = twa_bf16_hi(pr);
          } else {
            const float2 pr = reinterpret_cast<const float2*>(st + a.g_off)[vw * 32 + lane];
            g0[u] = pr.x;
            g1[u] = pr.y;
          }
          mb = max(mb, __float_as_uint(g1[u]) & 0x7FFFFFFFu);
        }
        mb = max(mb, __float_as_uint(g0[u]) & 0x7FFFFFFFu);
      }
      mb = __reduce_max_sync(0xFFFFFFFFu, mb);          // one digit scale for the warp's rows of the tile
      const ByteDigitScale ds = byte_digit_scale(mb);
      if (ds.bad) bad = true;                           // NaN or Inf in g
      if (ds.live) {
        // 4-bit codes enter the MMA times 16
        const float wl = byte_digit_weight(tig, BITS == 4 ? ds.w0 * 0.0625f : ds.w0);
        int c[MT][4];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) c[mt][0] = c[mt][1] = c[mt][2] = c[mt][3] = 0;
#pragma unroll
        for (int u = 0; u < KT; ++u) {
          byte_digit_store<FOUR>(digw, 0, lane, g0[u], ds.up);
          if (BITS == 4) byte_digit_store<FOUR>(digw, 1, lane, g1[u], ds.up);
          __syncwarp();
          uint32_t b0, b1, b2 = 0, b3 = 0;
          if (BITS == 8) {
            ldmatrix_x2(dig_addr, b0, b1);
          } else {
            uint32_t bb[4];
            ldmatrix_x4(dig_addr, bb);
            b0 = bb[0]; b1 = bb[1]; b2 = bb[2]; b3 = bb[3];   // second matrix pair: the odd rows
          }
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
            uint32_t r[4];
            ldmatrix_x4(tile_base + aoff[u][mt], r);
            if (BITS == 8) {
              mma_s8u8(c[mt], r, b0, b1);
            } else {
              uint32_t e[4], o[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                e[i] = (r[i] << 4) & 0xF0F0F0F0u;       // even rows: 16 * code
                o[i] = r[i] & 0xF0F0F0F0u;              // odd rows:  16 * code
              }
              mma_s8u8(c[mt], e, b0, b1);
              mma_s8u8(c[mt], o, b2, b3);
            }
          }
          __syncwarp();                                  // the digit matrices are rewritten by the next block
        }
        // digit sums -> float: |sum| < 2^31 always (at most 128 rows x 255 x 127 per digit, times 257)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          facc[mt][0] = fmaf(static_cast<float>(c[mt][0] + dmult * c[mt][1]), wl, facc[mt][0]);
          facc[mt][1] = fmaf(static_cast<float>(c[mt][2] + dmult * c[mt][3]), wl, facc[mt][1]);
        }
      }
      __syncwarp();
      if (lane == 0) twa_mbar_arrive(twa_smem_u32(&hdr->empty[s]));
      if (++s == a.stages) {
        s = 0;
        phase ^= 1u;
      }
    }
    if (bad) hdr->bad_flag = 1;
  }
  __syncthreads();                                       // every stage consumed; the ring is free

  // ---- column sums of the block: lanes -> warps -> block, in a fixed order ------------------
  float* part = reinterpret_cast<float*>(ring);         // [MMA_WARPS][TWA_MAX_N]
  if (warp < MMA_WARPS) {
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      float v0 = facc[mt][0], v1 = facc[mt][1];
      v0 += __shfl_xor_sync(0xFFFFFFFFu, v0, 1);
      v1 += __shfl_xor_sync(0xFFFFFFFFu, v1, 1);
      v0 += __shfl_xor_sync(0xFFFFFFFFu, v0, 2);
      v1 += __shfl_xor_sync(0xFFFFFFFFu, v1, 2);
      if (tig == 0) {
        part[warp * TWA_MAX_N + mt * 16 + gid] = v0;
        part[warp * TWA_MAX_N + mt * 16 + gid + 8] = v1;
      }
    }
  }
  __syncthreads();
  const int tid = threadIdx.x;
  if (tid < a.n) {
    float sum = 0.0f;
#pragma unroll
    for (int w = 0; w < MMA_WARPS; ++w) sum += part[w * TWA_MAX_N + tid];
    if (hdr->bad_flag) sum = __int_as_float(0x7FC00000);
    a.partials[static_cast<size_t>(blockIdx.x) * a.n + tid] = sum;
  }
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
      c = sum * static_cast<double>(a.scales[tid]);
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

// =================================================================================================
// lift
// =================================================================================================
// KS = number of 32-column steps, ceil(n / 32), a compile-time constant.
// VEC says how the rows of the base vector and of the output travel:
//   0  every lane loads its base rows and stores its results itself;
//   1  the tile's base rows ride the ring beside the codes (1-D boxes of 256 floats, zero past D),
//      so their latency is hidden by the depth of the ring and not by one tile of look-ahead;
//   2  as 1, and the results are written over the base rows in the stage and leave through one
//      bulk tensor store per warp and tile (clipped at D by the tensor map); the stage is handed
//      back one tile later, once that store has read it.
// 1 and 2 need 16-byte aligned vectors.
template <int BITS, int KS, int KT, int VEC>
__global__ void __launch_bounds__(MMA_THREADS, 1)
twa_lift_mma_kernel(const __grid_constant__ CUtensorMap map_p, const __grid_constant__ CUtensorMap map_b,
                    const __grid_constant__ CUtensorMap map_o, const LiftMmaArgs a) {
  constexpr bool BTMA = VEC >= 1, STMA = VEC == 2;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (twa_smem_u32(smem_raw) & 1023u)) & 1023u);
  constexpr int ROWS = twa_tile_rows(BITS);
  constexpr int LROWS = BITS == 8 ? 2 : 4;             // rows one lane finishes per chunk
  twa_smem_header* hdr = reinterpret_cast<twa_smem_header*>(smem);
  unsigned char* ring = smem + TWA_SMEM_HEADER;
  unsigned char* table = smem + a.table_off;           // digit k of coefficient j at table[k*128 + j]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gid = lane >> 2, tig = lane & 3;
  const int tid = threadIdx.x;

  init_barriers(hdr, a.stages);
  __syncthreads();

  // ---- digits of the coefficients a_j = s_j * alpha_j * mult, common scale over all j --------
  float coef = 0.0f;
  if (tid < TWA_MAX_N) {
    if (tid < a.n) coef = a.alpha[tid] * a.alpha_mult * a.scales[tid];
    atomicMax(&hdr->amax_bits, __float_as_uint(coef) & 0x7FFFFFFFu);
  }
  __syncthreads();
  const unsigned ebits = hdr->amax_bits >> 23;
  const bool bad = ebits >= 255u;                       // NaN or Inf among the coefficients
  const bool live = ebits >= 5u && !bad;                // all-zero (or vanishing) coefficients: w = base
  if (tid < TWA_MAX_N) {
    uint32_t d = 0;
    if (live) d = cut_digits(coef * __uint_as_float((259u - ebits) << 23));
#pragma unroll
    for (int k = 0; k < 4; ++k) table[k * TWA_MAX_N + tid] = static_cast<unsigned char>(d >> (8 * k));
  }
  __syncthreads();

  if (warp == MMA_WARPS) {
    if (lane == 0)
      producer_loop_mma(hdr, ring, &map_p, &map_b, blockIdx.x, gridDim.x,
                        (a.tiles - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) /
                            static_cast<int>(gridDim.x),
                        a.stages, a.stage_bytes, TWA_TILE_COL_BYTES / 8 * KT, BTMA ? ROWS * KT / 256 : 0, 4, ROWS * KT, a.base_off,
                        a.tx_bytes, a.reverse != 0, a.status, a.wait_limit_ns);
    return;
  }
  if (bad && tid == 0) twa_set_status(a.status, TWA_ERR_NONFINITE, -1);

  const float w0 = !live ? 0.0f : (ebits >= 6u ? __uint_as_float((ebits - 5u) << 23) : 5.877471754e-39f);
  const float w1 = w0 * 0.0078125f, w2 = w1 * 0.0078125f, w3 = w2 * 0.0078125f;
  float wb = tig == 0 ? w1 : (tig == 1 ? w3 : 0.0f);    // weight of the lower digit of this lane's pair
  if (BITS == 4) wb *= 0.0625f;                         // 4-bit codes enter the MMA times 16
  if (bad) wb = __int_as_float(0x7FC00000);             // NaN or Inf among the coefficients poisons every row

  // B fragments: k-slot 4*tig+i of a 32-column step holds column j0 + {2tig, 2tig+1, 8+2tig, 9+2tig}[i]
  // (and the same + 16 for the second register), the order the transposing loads deliver.
  uint32_t bfrag[KS][2];
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) {
    bfrag[ks][0] = bfrag[ks][1] = 0u;
    if (gid < 4) {
      const unsigned char* tk = table + gid * TWA_MAX_N + ks * 32 + 2 * tig;
      bfrag[ks][0] = static_cast<uint32_t>(*reinterpret_cast<const unsigned short*>(tk)) |
                     (static_cast<uint32_t>(*reinterpret_cast<const unsigned short*>(tk + 8)) << 16);
      bfrag[ks][1] = static_cast<uint32_t>(*reinterpret_cast<const unsigned short*>(tk + 16)) |
                     (static_cast<uint32_t>(*reinterpret_cast<const unsigned short*>(tk + 24)) << 16);
    }
  }

  const int lm = lane >> 3, lr = lane & 7;
  const int jmax = a.n - 1;
  constexpr int col_bytes = TWA_TILE_COL_BYTES * KT;
  // The warp owns bytes [32*KT*warp, 32*KT*(warp+1)) of every column: KT blocks of two 16-byte
  // chunks.  Lanes with tig < 2 finish chunk tig of a block: LROWS rows starting at LROWS * gid.
  // Offsets, inside a tile, of the chunk this lane hands to ldmatrix for block u, chunk ch and
  // 32-column step ks (they do not change from tile to tile).
  uint32_t loff[KT][2][KS];
#pragma unroll
  for (int u = 0; u < KT; ++u)
#pragma unroll
    for (int ch = 0; ch < 2; ++ch)
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        int j = ks * 32 + lm * 8 + lr;
        j = j < jmax ? j : jmax;
        const int chunk = (warp * KT + u) * 2 + ch;
        loff[u][ch][ks] = static_cast<uint32_t>(j * col_bytes + ((chunk >> 5) << 9) +
                                                (twa_chunk_slot(chunk & 31, j) << 4));
      }
  int lane_row[KT];
#pragma unroll
  for (int u = 0; u < KT; ++u)
    lane_row[u] = ((warp * KT + u) * 32 + 16 * tig) * (8 / BITS) + LROWS * gid;
  constexpr int tile_rows = ROWS * KT;
  const int D = static_cast<int>(a.D);                   // D < 2^31
  volatile int* abort_flag = &hdr->abort_flag;
  int s = 0;
  unsigned phase = 0;
  // the same tile sequence as the producer: this block's tiles, backwards when `reverse`
  const int t_count = (a.tiles - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) /
                      static_cast<int>(gridDim.x);
  for (int k = 0; k < t_count; ++k) {
    const int tile = static_cast<int>(blockIdx.x) + (a.reverse ? (t_count - 1 - k) : k) * static_cast<int>(gridDim.x);
    const int tile_row0 = tile * tile_rows;               // < D < 2^31
    const bool whole = tile_row0 <= D - tile_rows;        // no row of the tile lies past D
    float bv[KT][LROWS];
#pragma unroll
    for (int u = 0; u < KT; ++u) {
#pragma unroll
      for (int i = 0; i < LROWS; ++i) bv[u][i] = 0.0f;
      if (!BTMA && a.base && tig < 2) {
        const int row = tile_row0 + lane_row[u];
        if (whole || row <= D - LROWS) {
          if (LROWS == 2) {
            const float2 x = *reinterpret_cast<const float2*>(a.base + row);
            bv[u][0] = x.x; bv[u][1] = x.y;
          } else {
            const float4 x = *reinterpret_cast<const float4*>(a.base + row);
            bv[u][0] = x.x; bv[u][1] = x.y; bv[u][2] = x.z; bv[u][3] = x.w;
          }
        } else {
#pragma unroll
          for (int i = 0; i < LROWS; ++i)
            if (row + i < D) bv[u][i] = a.base[row + i];
        }
      }
    }
    if (!twa_mbar_wait(twa_smem_u32(&hdr->full[s]), phase, abort_flag, a.wait_limit_ns)) {
      twa_set_status(a.status, TWA_ERR_TIMEOUT, -1);
      break;
    }
    const uint32_t tile_base = twa_smem_u32(ring + static_cast<size_t>(s) * a.stage_bytes);
    if (BTMA && tig < 2) {
      const float* sb = reinterpret_cast<const float*>(ring + static_cast<size_t>(s) * a.stage_bytes + a.base_off);
#pragma unroll
      for (int u = 0; u < KT; ++u) {
        if (LROWS == 2) {
          const float2 x = *reinterpret_cast<const float2*>(sb + lane_row[u]);
          bv[u][0] = x.x; bv[u][1] = x.y;
        } else {
          const float4 x = *reinterpret_cast<const float4*>(sb + lane_row[u]);
          bv[u][0] = x.x; bv[u][1] = x.y; bv[u][2] = x.z; bv[u][3] = x.w;
        }
      }
    }
    float keep[KT][LROWS];
#pragma unroll
    for (int u = 0; u < KT; ++u) {
      float v[2][LROWS];                                // per 16-byte chunk of the block
#pragma unroll
      for (int ch = 0; ch < 2; ++ch) {
        int acc0[4];                                    // 8-bit: rows 2gid, 2gid+1; 4-bit: rows 4gid, 4gid+2
        int acc1[4];                                    // 4-bit only: rows 4gid+1, 4gid+3
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
          uint32_t r[4];
          ldmatrix_x4_trans(tile_base + loff[u][ch][ks], r);
          // the transposing load delivers byte pairs of two columns: regroup to four columns per register
          const uint32_t af[4] = {__byte_perm(r[0], r[1], 0x6420), __byte_perm(r[0], r[1], 0x7531),
                                  __byte_perm(r[2], r[3], 0x6420), __byte_perm(r[2], r[3], 0x7531)};
          if (BITS == 8) {
            if (ks == 0) mma_s8_first(acc0, af, bfrag[ks][0], bfrag[ks][1]);
            else mma_s8(acc0, af, bfrag[ks][0], bfrag[ks][1]);
          } else {
            uint32_t ae[4], ao[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              ae[i] = (af[i] << 4) & 0xF0F0F0F0u;       // even rows: 16 * code
              ao[i] = af[i] & 0xF0F0F0F0u;              // odd rows:  16 * code
            }
            if (ks == 0) {
              mma_s8_first(acc0, ae, bfrag[ks][0], bfrag[ks][1]);
              mma_s8_first(acc1, ao, bfrag[ks][0], bfrag[ks][1]);
            } else {
              mma_s8(acc0, ae, bfrag[ks][0], bfrag[ks][1]);
              mma_s8(acc1, ao, bfrag[ks][0], bfrag[ks][1]);
            }
          }
        }
        // digit sums -> float: lane tig = 0 holds the sums of digits 0 and 1 of its rows, tig = 1 those of
        // digits 2 and 3 (wb is the weight of the lower digit of the pair; 0 in lanes tig >= 2)
        if (BITS == 8) {
          v[ch][0] = digit_pair_to_float(acc0[0], acc0[1], wb);
          v[ch][1] = digit_pair_to_float(acc0[2], acc0[3], wb);
        } else {
          v[ch][0] = digit_pair_to_float(acc0[0], acc0[1], wb);
          v[ch][2] = digit_pair_to_float(acc0[2], acc0[3], wb);
          v[ch][1] = digit_pair_to_float(acc1[0], acc1[1], wb);
          v[ch][3] = digit_pair_to_float(acc1[2], acc1[3], wb);
        }
      }
      // The four digits of a row sit in lanes tig = 0 and 1 of its quad; lane tig = 0 finishes the rows of
      // chunk 0 and lane tig = 1 those of chunk 1: each hands the other the half it does not keep.
#pragma unroll
      for (int i = 0; i < LROWS; ++i) {
        const float mine = (tig & 1) ? v[1][i] : v[0][i];
        const float theirs = (tig & 1) ? v[0][i] : v[1][i];
        keep[u][i] = mine + __shfl_xor_sync(0xFFFFFFFFu, theirs, 1);
      }
    }
    if (STMA) {
      float* sb = reinterpret_cast<float*>(ring + static_cast<size_t>(s) * a.stage_bytes + a.base_off);
      if (tig < 2) {
#pragma unroll
        for (int u = 0; u < KT; ++u) {
          if (LROWS == 2) {
            *reinterpret_cast<float2*>(sb + lane_row[u]) =
                make_float2(bv[u][0] + keep[u][0], bv[u][1] + keep[u][1]);
          } else {
            *reinterpret_cast<float4*>(sb + lane_row[u]) =
                make_float4(bv[u][0] + keep[u][0], bv[u][1] + keep[u][1],
                            bv[u][2] + keep[u][2], bv[u][3] + keep[u][3]);
          }
        }
        twa_fence_proxy_async();                          // the lanes' writes, before the bulk store reads them
        // The bulk store clips in units of 16 bytes, so its tensor map ends at the last multiple of
        // four rows; the up to three rows after that are stored by the lanes that own them.
        if (!whole) {
#pragma unroll
          for (int u = 0; u < KT; ++u)
#pragma unroll
            for (int i = 0; i < LROWS; ++i) {
              const int row = tile_row0 + lane_row[u] + i;
              if (row >= (D & ~3) && row < D) a.out[row] = bv[u][i] + keep[u][i];
            }
        }
      }
      __syncwarp();
      if (lane == 0) {
        // the warp's rows of the tile are contiguous: [warp * KT * 32 * (8 / BITS), + KT * 32 * (8 / BITS))
        constexpr int wrows = KT * 32 * (8 / BITS);
        if (tile_row0 + warp * wrows < (D & ~3))          // no store starts past the end of the map
          twa_tma_store_1d(&map_o, tile_row0 + warp * wrows, twa_smem_u32(sb + warp * wrows));
        twa_bulk_commit();
        if (k > 0) {                                      // the previous tile's store has read its stage
          twa_bulk_wait_read<1>();
          twa_mbar_arrive(twa_smem_u32(&hdr->empty[s == 0 ? a.stages - 1 : s - 1]));
        }
      }
      if (++s == a.stages) {
        s = 0;
        phase ^= 1u;
      }
      continue;
    }
    __syncwarp();
    if (lane == 0) twa_mbar_arrive(twa_smem_u32(&hdr->empty[s]));
#pragma unroll
    for (int u = 0; u < KT; ++u) {
      if (tig < 2) {
        const int row = tile_row0 + lane_row[u];
        if (whole || row <= D - LROWS) {
          if (LROWS == 2) {
            *reinterpret_cast<float2*>(a.out + row) =
                make_float2(bv[u][0] + keep[u][0], bv[u][1] + keep[u][1]);
          } else {
            *reinterpret_cast<float4*>(a.out + row) =
                make_float4(bv[u][0] + keep[u][0], bv[u][1] + keep[u][1],
                            bv[u][2] + keep[u][2], bv[u][3] + keep[u][3]);
          }
        } else {
#pragma unroll
          for (int i = 0; i < LROWS; ++i)
            if (row + i < D) a.out[row + i] = bv[u][i] + keep[u][i];
        }
      }
    }
    if (++s == a.stages) {
      s = 0;
      phase ^= 1u;
    }
  }
  if (STMA && lane == 0) twa_bulk_wait_read<0>();         // shared memory must outlive the stores' reads
}

// =================================================================================================
// host side
// =================================================================================================
// Segments per tile column.  Taller tiles spread the per-tile work (digit scale, digit sums to float,
// barrier traffic) over more bytes, but fewer of them fit in the ring.  The rule below is the one the
// measurements on B200 agree with (1.3 B-sized n = 32, ResNet-50-sized n = 50, ViT-B/16-sized n = 100, both
// widths): the tallest tile of 4 (n <= 32 only), 2 or 1 segments of which at least `want` stages fit, with
// want = 2 for the 8-bit projection and the 4-bit lift, 3 for the 4-bit projection and the 8-bit lift.
//   n = 32: lift 7.99 -> 7.67 ms (8 bits, 4 segments) and 4.97 -> 4.66 ms (4 bits, 4 segments, two stages);
//           4-bit projection 3.55 ms with 2 segments against 3.79 ms with 4.
//   n = 100: 8-bit projection 1.29 -> 1.24 ms with 2 segments (two stages), 8-bit lift 1.38 ms with 1 against
//           1.39 ms with 2; 4-bit lift 0.754 -> 0.732 ms with 2, 4-bit projection 0.668 ms with 1 against 0.682.
// row_bytes = bytes per tile row that ride the ring beside the codes (g, or the base vector).
int choose_kt(const twa_ctx* ctx, int n, int bits, bool lift, int row_bytes, int fixed_smem) {
  const int t = ctx->tune_tile_segments;
  if (t == 1 || t == 2 || (t == 4 && n <= 32)) return t;
  const int want = (lift ? bits == 8 : bits == 4) ? 3 : 2;
  for (int kt = n <= 32 ? 4 : 2; kt > 1; kt >>= 1) {
    const int stage = (n * TWA_TILE_COL_BYTES * kt + twa_tile_rows(bits) * kt * row_bytes + 1023) / 1024 * 1024;
    if ((ctx->smem_optin - fixed_smem) / stage >= want) return kt;
  }
  return 1;
}

// The codes as a 2-D tensor of 8-byte elements {column bytes / 8, n}: a box dimension is limited to 256
// elements, and a tile of four 512-byte segments is 256 of these.
int encode_tile_map(twa_ctx* ctx, const twa_basis* P, int kt, CUtensorMap* map) {
  long long row_bytes = (P->D * P->bits + 7) / 8;
  // quantised columns are stored in whole, internally permuted 512-byte segments
  row_bytes = (row_bytes + 511) / 512 * 512;
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(row_bytes / 8), static_cast<cuuint64_t>(P->n)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(P->col_stride)};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(TWA_TILE_COL_BYTES / 8 * kt), static_cast<cuuint32_t>(P->n)};
  cuuint32_t es[2] = {1, 1};
  CUresult r = ctx->encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, P->data, dims, strides, box, es,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(ctx->last_error, sizeof(ctx->last_error), "cuTensorMapEncodeTiled(P) failed: %d",
             static_cast<int>(r));
    return TWA_ERR_CUDA;
  }
  return TWA_OK;
}

int encode_g_map(twa_ctx* ctx, const void* g, long long D, bool bf16, CUtensorMap* map) {
  cuuint64_t dims[1] = {static_cast<cuuint64_t>(D)};
  cuuint64_t strides[1] = {0};
  cuuint32_t box[1] = {256};
  cuuint32_t es[1] = {1};
  CUresult r = ctx->encode_tiled(
      map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 1,
      const_cast<void*>(g), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
      CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(ctx->last_error, sizeof(ctx->last_error), "cuTensorMapEncodeTiled(g) failed: %d",
             static_cast<int>(r));
    return TWA_ERR_CUDA;
  }
  return TWA_OK;
}

int round_up_i(int x, int m) { return (x + m - 1) / m * m; }

template <int BITS, bool GBF16, int MT>
int launch_project_mma_t(twa_ctx* ctx, const CUtensorMap& mp, const CUtensorMap& mg,
                         const ProjectMmaArgs& a, int grid, int smem) {
  // four segments per tile exist for n <= 32 only (MT <= 2)
  auto kern = (a.kt == 4 && MT <= 2) ? twa_project_mma_kernel<BITS, GBF16, MT, (MT <= 2 ? 4 : 1)>
              : a.kt == 2            ? twa_project_mma_kernel<BITS, GBF16, MT, 2>
                                     : twa_project_mma_kernel<BITS, GBF16, MT, 1>;
  static int smem_limit[3][64] = {{0}};   // per tile height and device
  int rc = twa_ensure_smem(ctx, reinterpret_cast<const void*>(kern), &smem_limit[a.kt >> 1][ctx->device & 63], smem);
  if (rc) return rc;
  kern<<<grid, MMA_THREADS, smem, ctx->stream>>>(mp, mg, a);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}

template <int BITS, bool GBF16>
int launch_project_mma_mt(twa_ctx* ctx, const CUtensorMap& mp, const CUtensorMap& mg,
                          const ProjectMmaArgs& a, int grid, int smem);

struct LiftMaps {
  CUtensorMap p, b, o;
};

template <int BITS, int KS, int VEC>
int launch_lift_mma_t(twa_ctx* ctx, const LiftMaps& m, const LiftMmaArgs& a, int grid, int smem) {
  auto kern = (a.kt == 4 && KS == 1) ? twa_lift_mma_kernel<BITS, KS, (KS == 1 ? 4 : 1), VEC>
              : a.kt == 2            ? twa_lift_mma_kernel<BITS, KS, 2, VEC>
                                     : twa_lift_mma_kernel<BITS, KS, 1, VEC>;
  static int smem_limit[3][64] = {{0}};   // per tile height and device
  int rc = twa_ensure_smem(ctx, reinterpret_cast<const void*>(kern), &smem_limit[a.kt >> 1][ctx->device & 63], smem);
  if (rc) return rc;
  kern<<<grid, MMA_THREADS, smem, ctx->stream>>>(m.p, m.b, m.o, a);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}

template <int BITS, bool GBF16>
int launch_project_mma_mt(twa_ctx* ctx, const CUtensorMap& mp, const CUtensorMap& mg,
                          const ProjectMmaArgs& a, int grid, int smem) {
  switch ((a.n + 15) >> 4) {
    case 1: return launch_project_mma_t<BITS, GBF16, 1>(ctx, mp, mg, a, grid, smem);
    case 2: return launch_project_mma_t<BITS, GBF16, 2>(ctx, mp, mg, a, grid, smem);
    case 3: return launch_project_mma_t<BITS, GBF16, 3>(ctx, mp, mg, a, grid, smem);
    case 4: return launch_project_mma_t<BITS, GBF16, 4>(ctx, mp, mg, a, grid, smem);
    case 5: return launch_project_mma_t<BITS, GBF16, 5>(ctx, mp, mg, a, grid, smem);
    case 6: return launch_project_mma_t<BITS, GBF16, 6>(ctx, mp, mg, a, grid, smem);
    case 7: return launch_project_mma_t<BITS, GBF16, 7>(ctx, mp, mg, a, grid, smem);
    default: return launch_project_mma_t<BITS, GBF16, 8>(ctx, mp, mg, a, grid, smem);
  }
}

template <int BITS, int VEC>
int launch_lift_mma_ks(twa_ctx* ctx, const LiftMaps& m, const LiftMmaArgs& a, int grid, int smem) {
  switch ((a.n + 31) >> 5) {
    case 1: return launch_lift_mma_t<BITS, 1, VEC>(ctx, m, a, grid, smem);
    case 2: return launch_lift_mma_t<BITS, 2, VEC>(ctx, m, a, grid, smem);
    case 3: return launch_lift_mma_t<BITS, 3, VEC>(ctx, m, a, grid, smem);
    default: return launch_lift_mma_t<BITS, 4, VEC>(ctx, m, a, grid, smem);
  }
}

template <int BITS>
int launch_lift_mma_vec(twa_ctx* ctx, const LiftMaps& m, const LiftMmaArgs& a, int grid, int smem, int vec) {
  switch (vec) {
    case 2: return launch_lift_mma_ks<BITS, 2>(ctx, m, a, grid, smem);
    case 1: return launch_lift_mma_ks<BITS, 1>(ctx, m, a, grid, smem);
    default: return launch_lift_mma_ks<BITS, 0>(ctx, m, a, grid, smem);
  }
}

// 1-D tensor map over a float vector of D elements with boxes of `box` elements
int encode_vector_map(twa_ctx* ctx, const float* v, long long D, int box, CUtensorMap* map) {
  cuuint64_t dims[1] = {static_cast<cuuint64_t>(D)};
  cuuint64_t strides[1] = {0};
  cuuint32_t bx[1] = {static_cast<cuuint32_t>(box)};
  cuuint32_t es[1] = {1};
  CUresult r = ctx->encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 1, const_cast<float*>(v), dims, strides, bx, es,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(ctx->last_error, sizeof(ctx->last_error), "cuTensorMapEncodeTiled(vector) failed: %d",
             static_cast<int>(r));
    return TWA_ERR_CUDA;
  }
  return TWA_OK;
}

}  // namespace

int twa_launch_project_mma(twa_ctx* ctx, const twa_basis* P, const void* g, twa_dtype g_dtype,
                           const twa_project_epilogue& epi, void* ws) {
  const bool bf16 = g_dtype == TWA_BF16;
  const int gsz = bf16 ? 2 : 4;
  const int fixed = TWA_SMEM_HEADER + MMA_WARPS * BYTE_DIGIT_SCRATCH + 1024;   // 1024: alignment slack
  const int kt = choose_kt(ctx, P->n, P->bits, false, gsz, fixed);
  const int rows = twa_tile_rows(P->bits) * kt;
  CUtensorMap mp, mg;
  int rc = encode_tile_map(ctx, P, kt, &mp);
  if (rc) return rc;
  rc = encode_g_map(ctx, g, P->D, bf16, &mg);
  if (rc) return rc;

  ProjectMmaArgs a;
  a.D = P->D;
  a.n = P->n;
  a.tiles = static_cast<int>((P->D + rows - 1) / rows);
  a.kt = kt;
  a.g_off = static_cast<unsigned>(P->n) * TWA_TILE_COL_BYTES * kt;
  a.tx_bytes = a.g_off + static_cast<unsigned>(rows * gsz);
  a.stage_bytes = static_cast<unsigned>(round_up_i(static_cast<int>(a.tx_bytes), 1024));
  int stages = (ctx->smem_optin - fixed) / static_cast<int>(a.stage_bytes);
  if (stages > TWA_MAX_STAGES) stages = TWA_MAX_STAGES;
  if (ctx->tune_stages >= 2 && ctx->tune_stages < stages) stages = ctx->tune_stages;
  if (stages < 2) return TWA_ERR_UNSUPPORTED;
  // the ring is reused for the block's [16][128] float partials after the tile loop
  while (stages * static_cast<int>(a.stage_bytes) < MMA_WARPS * TWA_MAX_N * 4) ++stages;
  a.stages = stages;
  a.scratch_off = TWA_SMEM_HEADER + static_cast<unsigned>(stages) * a.stage_bytes;
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
  const int smem = static_cast<int>(a.scratch_off) + MMA_WARPS * BYTE_DIGIT_SCRATCH + 1024;
  if (P->bits == 8)
    return bf16 ? launch_project_mma_mt<8, true>(ctx, mp, mg, a, grid, smem)
                : launch_project_mma_mt<8, false>(ctx, mp, mg, a, grid, smem);
  return bf16 ? launch_project_mma_mt<4, true>(ctx, mp, mg, a, grid, smem)
              : launch_project_mma_mt<4, false>(ctx, mp, mg, a, grid, smem);
}

int twa_launch_lift_mma(twa_ctx* ctx, const twa_basis* P, const float* alpha, float alpha_mult,
                        const float* base, float* out, bool reverse_tiles) {
  // How base and output travel (see the kernel): through the ring and bulk stores when tensor maps
  // can describe them (16-byte aligned starts) and the two vectors are a large share of the bytes
  // moved, 64 / (n * bits + 64).  Measured on B200: a third (n = 16 at 8 bits, n = 32 at 4 bits): base
  // through the ring 6.6 / 6.3 TB/s against 4.3 / 5.5 with the lanes' own loads, bulk stores in between;
  // a fifth (n = 32 at 8 bits): ring and bulk stores 6.7 against 6.45 (ring alone) and 6.3 (lanes);
  // a seventh and less (n >= 50 at 8 bits): the lanes' loads are hidden behind the wait for the codes
  // and the ring alone costs 3-4 %.
  const int nb = P->n * P->bits;
  int vec = ctx->tune_lift_base_path == 0 ? (nb <= 192 ? 1 : (nb <= 320 ? 2 : 0)) : ctx->tune_lift_base_path - 1;
  if (base == nullptr || ((reinterpret_cast<uintptr_t>(base) | reinterpret_cast<uintptr_t>(out)) & 15u) != 0) vec = 0;
  if (vec == 2 && P->D < 4) vec = 1;                      // nothing for a bulk store to write
  const int fixed = TWA_SMEM_HEADER + 4 * TWA_MAX_N + 1024;               // 1024: alignment slack
  const int kt = choose_kt(ctx, P->n, P->bits, true, vec >= 1 ? 4 : 0, fixed);
  const int rows = twa_tile_rows(P->bits) * kt;
  CUtensorMap mp;
  int rc = encode_tile_map(ctx, P, kt, &mp);
  if (rc) return rc;
  LiftMmaArgs a;
  a.D = P->D;
  a.n = P->n;
  a.tiles = static_cast<int>((P->D + rows - 1) / rows);
  a.kt = kt;
  const bool btma = vec >= 1;
  LiftMaps maps;
  maps.p = mp;
  maps.b = mp;
  maps.o = mp;
  if (btma) {
    rc = encode_vector_map(ctx, base, P->D, 256, &maps.b);
    if (rc) return rc;
  }
  if (vec == 2) {
    // rows [D & ~3, D) are stored by the lanes: a bulk store clips in units of 16 bytes
    rc = encode_vector_map(ctx, out, P->D & ~3ll, kt * 32 * (8 / P->bits), &maps.o);
    if (rc) return rc;
  }
  a.base_off = static_cast<unsigned>(P->n) * TWA_TILE_COL_BYTES * kt;
  a.tx_bytes = a.base_off + (btma ? static_cast<unsigned>(rows) * 4u : 0u);
  a.stage_bytes = static_cast<unsigned>(round_up_i(static_cast<int>(a.tx_bytes), 1024));
  int stages = (ctx->smem_optin - fixed) / static_cast<int>(a.stage_bytes);
  if (stages > TWA_MAX_STAGES) stages = TWA_MAX_STAGES;
  if (ctx->tune_stages >= 2 && ctx->tune_stages < stages) stages = ctx->tune_stages;
  if (stages < 2) return TWA_ERR_UNSUPPORTED;
  a.stages = stages;
  a.table_off = TWA_SMEM_HEADER + static_cast<unsigned>(stages) * a.stage_bytes;
  a.scales = P->scales;
  a.alpha = alpha;
  a.alpha_mult = alpha_mult;
  a.base = base;
  a.out = out;
  a.reverse = reverse_tiles ? 1 : 0;
  a.status = ctx->d_status;
  a.wait_limit_ns = ctx->wait_limit_ns;
  const int grid = ctx->sm_count < a.tiles ? ctx->sm_count : a.tiles;
  const int smem = static_cast<int>(a.table_off) + 4 * TWA_MAX_N + 1024;
  return P->bits == 8 ? launch_lift_mma_vec<8>(ctx, maps, a, grid, smem, vec)
                      : launch_lift_mma_vec<4>(ctx, maps, a, grid, smem, vec);
}
