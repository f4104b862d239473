// Projection of several gradients at once: C[b][j] = s_j * sum_r code[r,j] * G[b][r]
// (Section 4.2, the chain-rule equation, for every row of G), P~ read once per group of gradients.
//
// Same data path as the single-gradient kernel in twa_stream_mma.cu.  What the batch adds: the
// m16n8k32 integer MMA has eight result columns and one gradient's three byte digits and the
// column of ones that goes with them fill only four, so two gradients share every MMA (columns
// 0-3: the first, 4-7: the second; float32 gradients are cut to three bytes here too: 2^-23 of the
// largest magnitude of a warp's rows).  A tile of P~ in shared memory serves NP such pairs before
// its stage is released;
// the gradients of a group arrive as [NB][256] boxes of one 2-D tensor map over G (rows past the
// batch read as zero).
#include <stdio.h>

#include "twa_mma.cuh"
#include "twa_slabs.cuh"

namespace {

// Digit matrices of one pair of gradients: [8 digit rows][32 gradient rows]; with 4-bit codes one for
// the even and one for the odd rows.  A warp keeps one such set per pair of the group.
__host__ __device__ constexpr int pair_bytes(int bits) { return (bits == 8 ? 1 : 2) * BYTE_DIGIT_SET; }

// Digit matrix of a pair of gradients: rows u0, u1, u2, ones of the first, then of the second.
template <int BITS>
__device__ __forceinline__ void pair_digit_init(unsigned char* digw, int lane) {
  uint32_t* w = reinterpret_cast<uint32_t*>(digw);
#pragma unroll
  for (int i = 0; i < pair_bytes(BITS) / 128; ++i) {
    const int idx = lane + 32 * i;
    const int row = (idx % (BYTE_DIGIT_SET / 4)) / (BYTE_DIGIT_STRIDE / 4);
    w[idx] = (row & 3) == 3 ? 0x01010101u : 0u;
  }
}

// The three byte digits of gradient h's value for gradient row `lane` into digit matrix `set`.
__device__ __forceinline__ void pair_digit_store(unsigned char* digw, int set, int h, int lane, float g, float up) {
  const uint32_t b = __float_as_uint(fmaf(g, up, RND));
  unsigned char* d = digw + set * BYTE_DIGIT_SET + h * 4 * BYTE_DIGIT_STRIDE + lane;
  d[0] = static_cast<unsigned char>(b);
  d[BYTE_DIGIT_STRIDE] = static_cast<unsigned char>(b >> 8);
  d[2 * BYTE_DIGIT_STRIDE] = static_cast<unsigned char>(b >> 16);
}

// B fragments of a pair: result columns 0-3 = u0, u1, u2, ones of the pair's first gradient, 4-7 of its
// second; with 4-bit codes registers 2, 3 hold the odd rows' digits.
template <int BITS>
__device__ __forceinline__ void load_pair_fragments(uint32_t dig_addr, uint32_t (&bf)[4]) {
  if (BITS == 8) {
    ldmatrix_x2(dig_addr, bf[0], bf[1]);
  } else {
    ldmatrix_x4(dig_addr, bf);
  }
}

struct BatchArgs {
  long long D;
  int n, stages, tiles, b0, batch;
  unsigned stage_bytes, g_off, tx_bytes, scratch_off;
  unsigned pair_stride;         // bytes between the digit matrices of a warp's pairs; 0: one set, reused pair after pair
  const float* scales;
  float* partials;              // [grid][NB][n]
  unsigned* ticket;
  int* status;
  float* c_out;                 // [batch][n]
  int accumulate;               // 1: the results are added to c_out (a later row slab of the basis)
  unsigned long long wait_limit_ns;
};

// The block has no warp of its own for the copies (16 warps, four per scheduler, may use 128
// registers a thread; a 17th would cap every thread at 96, and this kernel's 2 x NP x MT float sums
// then leave too few to overlap the conversions).  Lane 0 of the last warp fills the ring: all stages
// before the loop, and stage s again right after its own warp has released it, once the other 15
// have too.  The warps run in step with the ring anyway, so that wait is short, and the other stages
// of the ring are in flight or have landed meanwhile.
template <int KT, int NB>
__device__ __forceinline__ void issue_tile(twa_smem_header* hdr, unsigned char* ring, const CUtensorMap* map_p,
                                           const CUtensorMap* map_g, const BatchArgs& a, int tile, int s, int tile_rows,
                                           int g_elem_bytes) {
  const uint32_t fb = twa_smem_u32(&hdr->full[s]);
  const uint32_t dst = twa_smem_u32(ring + static_cast<size_t>(s) * a.stage_bytes);
  twa_mbar_expect_tx(fb, a.tx_bytes);
  twa_tma_load_2d(dst, map_p, tile * TWA_TILE_COL_WORDS * KT, 0, fb);
  for (int q = 0; q < tile_rows / 256; ++q)
    twa_tma_load_2d(dst + a.g_off + q * NB * 256 * g_elem_bytes, map_g, tile * tile_rows + q * 256, a.b0, fb);
}

// NP pairs of gradients per launch (NB = 2 NP); MT, KT as in the single-gradient kernel.
constexpr int BATCH_THREADS = MMA_WARPS * 32;

template <int BITS, bool GBF16, int MT, int KT, int NP>
__global__ void __launch_bounds__(BATCH_THREADS, 1)
twa_project_batch_kernel(const __grid_constant__ CUtensorMap map_p, const __grid_constant__ CUtensorMap map_g,
                         const BatchArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (twa_smem_u32(smem_raw) & 1023u)) & 1023u);
  constexpr int NB = 2 * NP;
  constexpr int SROWS = twa_tile_rows(BITS);           // rows behind one 512-byte segment
  constexpr int GSZ = GBF16 ? 2 : 4;
  twa_smem_header* hdr = reinterpret_cast<twa_smem_header*>(smem);
  unsigned char* ring = smem + TWA_SMEM_HEADER;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gid = lane >> 2, tig = lane & 3;

  init_barriers(hdr, a.stages);
  __syncthreads();

  float facc[NP][MT][2];
#pragma unroll
  for (int p = 0; p < NP; ++p)
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) facc[p][mt][0] = facc[p][mt][1] = 0.0f;

  const bool filler = threadIdx.x == (MMA_WARPS - 1) * 32;
  const int my_tiles = blockIdx.x < a.tiles ? (a.tiles - 1 - static_cast<int>(blockIdx.x)) / static_cast<int>(gridDim.x) + 1 : 0;
  int issued = 0;
  if (filler) {
    twa_prefetch_tensormap(&map_p);
    twa_prefetch_tensormap(&map_g);
    for (; issued < my_tiles && issued < a.stages; ++issued)
      issue_tile<KT, NB>(hdr, ring, &map_p, &map_g, a, blockIdx.x + issued * gridDim.x, issued, SROWS * KT, GSZ);
  }
  {
    constexpr int PAIR_BYTES = pair_bytes(BITS);         // digit matrices of one pair of gradients
    // a set of digit matrices per pair where shared memory allows, else one set reused pair after pair
    const int sets = a.pair_stride ? NP : 1;
    unsigned char* digw = smem + a.scratch_off + warp * sets * PAIR_BYTES;
    for (int p = 0; p < sets; ++p) pair_digit_init<BITS>(digw + p * PAIR_BYTES, lane);
    __syncwarp();
    const uint32_t dig_addr = byte_digit_ldmatrix_addr(digw, lane);
    const int dmult = (tig & 1) ? -64 : 256;
    // weight of this lane's digit sums over the weight of u0; 4-bit codes enter the MMA times 16
    const float wfac = ((tig & 1) ? 65536.0f : 1.0f) * (BITS == 4 ? 0.0625f : 1.0f);
    const int lm = lane >> 3, lr = lane & 7;
    const int jmax = a.n - 1;
    constexpr int col_bytes = TWA_TILE_COL_BYTES * KT;
    uint32_t aoff[KT][MT];
#pragma unroll
    for (int u = 0; u < KT; ++u)
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        int j = mt * 16 + lr + 8 * (lm & 1);
        j = j < jmax ? j : jmax;
        const int chunk = (warp * KT + u) * 2 + (lm >> 1);
        aoff[u][mt] = static_cast<uint32_t>(j * col_bytes + ((chunk >> 5) << 9) + (twa_chunk_slot(chunk & 31, j) << 4));
      }
    // element offsets, inside one gradient's [256] slices of the stage, of this lane's rows for block u:
    // row r of the tile lives in box r / 256 at position r % 256
    int goff[KT];
#pragma unroll
    for (int u = 0; u < KT; ++u) {
      const int r = (warp * KT + u) * (SROWS / MMA_WARPS) + (BITS == 8 ? lane : 2 * lane);
      goff[u] = (r >> 8) * NB * 256 + (r & 255);
    }
    volatile int* abort_flag = &hdr->abort_flag;
    int s = 0;
    unsigned phase = 0;
    unsigned bad = 0u;                                   // lane b < NB: gradient b of the group is not finite
    for (int t = blockIdx.x; t < a.tiles; t += gridDim.x) {
      if (!twa_mbar_wait(twa_smem_u32(&hdr->full[s]), phase, abort_flag, a.wait_limit_ns)) {
        twa_set_status(a.status, TWA_ERR_TIMEOUT, -1);
        break;
      }
      const unsigned char* st = ring + static_cast<size_t>(s) * a.stage_bytes;
      const uint32_t tile_base = twa_smem_u32(st);
#pragma unroll
      for (int u = 0; u < KT; ++u) {
        // ---- digits of the warp's rows of every gradient of the group, one matrix per pair ------
        // The lane's row (4-bit codes: two rows) of every gradient and each gradient's largest magnitude;
        // lane b < NB then derives gradient b's digit scale once for the warp and the others fetch it.
        float g0[NB], g1[NB];
        unsigned mine = 0u;
#pragma unroll
        for (int b = 0; b < NB; ++b) {
          const int e = goff[u] + b * 256;
          g1[b] = 0.0f;
          if (GBF16) {
            const unsigned short* gs = reinterpret_cast<const unsigned short*>(st + a.g_off);
            g0[b] = __uint_as_float(static_cast<uint32_t>(gs[e]) << 16);
            if (BITS == 4) g1[b] = __uint_as_float(static_cast<uint32_t>(gs[e + 1]) << 16);
          } else {
            const float* gs = reinterpret_cast<const float*>(st + a.g_off);
            g0[b] = gs[e];
            if (BITS == 4) g1[b] = gs[e + 1];
          }
          unsigned mb = __float_as_uint(g0[b]) & 0x7FFFFFFFu;
          if (BITS == 4) mb = max(mb, __float_as_uint(g1[b]) & 0x7FFFFFFFu);
          mb = __reduce_max_sync(0xFFFFFFFFu, mb);
          if (b == 0 || lane == b) mine = mb;
        }
        const ByteDigitScale ds = byte_digit_scale(mine);
        if (ds.bad && lane < NB) bad = 1u;
        // a dead or non-finite gradient is cut with scale 0: its digits are those of zero
        const float up_mine = ds.live ? ds.up : 0.0f;
        const float w_mine = ds.live ? ds.w0 : 0.0f;
        float wl[NP];                                    // this lane's weight for pair p (0: nothing to add)
        uint32_t bf[NP][4];                              // B fragments of every pair
#pragma unroll
        for (int p = 0; p < NP; ++p) {
          const float up0 = __shfl_sync(0xFFFFFFFFu, up_mine, 2 * p), up1 = __shfl_sync(0xFFFFFFFFu, up_mine, 2 * p + 1);
          // lanes tig 0,1 finish the first gradient's digits (columns u0 u1 | u2 ones), tig 2,3 the second's
          wl[p] = __shfl_sync(0xFFFFFFFFu, w_mine, 2 * p + (tig >> 1)) * wfac;
          unsigned char* dp = digw + p * a.pair_stride;
          pair_digit_store(dp, 0, 0, lane, g0[2 * p], up0);
          pair_digit_store(dp, 0, 1, lane, g0[2 * p + 1], up1);
          if (BITS == 4) {
            pair_digit_store(dp, 1, 0, lane, g1[2 * p], up0);
            pair_digit_store(dp, 1, 1, lane, g1[2 * p + 1], up1);
          }
          if (a.pair_stride == 0) {
            __syncwarp();
            load_pair_fragments<BITS>(dig_addr, bf[p]);
            __syncwarp();                                // the digit matrices are rewritten by the next pair
          }
        }
        if (a.pair_stride != 0) {
          __syncwarp();
#pragma unroll
          for (int p = 0; p < NP; ++p) load_pair_fragments<BITS>(dig_addr + p * a.pair_stride, bf[p]);
          __syncwarp();                                  // rewritten for the next block of rows
        }
        // ---- every 16-column group of the tile is loaded (and unpacked) once for all pairs -------
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          uint32_t r[4], o[4];
          ldmatrix_x4(tile_base + aoff[u][mt], r);
          if (BITS == 4) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              o[i] = r[i] & 0xF0F0F0F0u;                  // odd rows:  16 * code
              r[i] = (r[i] << 4) & 0xF0F0F0F0u;           // even rows: 16 * code
            }
          }
#pragma unroll
          for (int p = 0; p < NP; ++p) {
            int c[4];
            mma_s8u8_first(c, r, bf[p][0], bf[p][1]);
            if (BITS == 4) mma_s8u8(c, o, bf[p][2], bf[p][3]);
            // digit sums -> float: |sum| < 2^31 (at most 64 rows x 255 x 127 per digit, times 257)
            facc[p][mt][0] = fmaf(static_cast<float>(c[0] + dmult * c[1]), wl[p], facc[p][mt][0]);
            facc[p][mt][1] = fmaf(static_cast<float>(c[2] + dmult * c[3]), wl[p], facc[p][mt][1]);
          }
        }
      }
      __syncwarp();
      if (lane == 0) twa_mbar_arrive(twa_smem_u32(&hdr->empty[s]));
      if (filler && issued < my_tiles) {
        // the stage just released takes this block's tile number `issued` once every warp is done with it
        if (twa_mbar_wait(twa_smem_u32(&hdr->empty[s]), phase, abort_flag, a.wait_limit_ns)) {
          issue_tile<KT, NB>(hdr, ring, &map_p, &map_g, a, blockIdx.x + issued * gridDim.x, s, SROWS * KT, GSZ);
          ++issued;
        } else {
          twa_set_status(a.status, TWA_ERR_TIMEOUT, -1);
        }
      }
      if (++s == a.stages) {
        s = 0;
        phase ^= 1u;
      }
    }
    if (bad) atomicOr(&hdr->bad_flag, 1 << lane);
    // every copy issued has landed before its issuer goes on, whatever the consumers did meanwhile
    if (filler && !twa_drain_ring(hdr, issued, a.stages, a.wait_limit_ns)) twa_set_status(a.status, TWA_ERR_TIMEOUT, -1);
  }
  __syncthreads();                                       // every stage consumed; the ring is free

  // ---- sums of the block: lanes -> warps -> block, in a fixed order --------------------------
  float* part = reinterpret_cast<float*>(ring);         // [MMA_WARPS][NB][TWA_MAX_N]
  {
#pragma unroll
    for (int p = 0; p < NP; ++p)
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        float v0 = facc[p][mt][0], v1 = facc[p][mt][1];
        v0 += __shfl_xor_sync(0xFFFFFFFFu, v0, 1);
        v1 += __shfl_xor_sync(0xFFFFFFFFu, v1, 1);
        if ((tig & 1) == 0) {                            // tig 0: first gradient of the pair, tig 2: second
          float* row = part + (warp * NB + 2 * p + (tig >> 1)) * TWA_MAX_N;
          row[mt * 16 + gid] = v0;
          row[mt * 16 + gid + 8] = v1;
        }
      }
  }
  __syncthreads();
  const int tid = threadIdx.x;
  const int outs = NB * a.n;
  for (int idx = tid; idx < outs; idx += blockDim.x) {
    const int b = idx / a.n, j = idx - b * a.n;
    float sum = 0.0f;
#pragma unroll
    for (int w = 0; w < MMA_WARPS; ++w) sum += part[(w * NB + b) * TWA_MAX_N + j];
    if ((hdr->bad_flag >> b) & 1) sum = __int_as_float(0x7FC00000);
    a.partials[static_cast<size_t>(blockIdx.x) * outs + idx] = sum;
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
    for (int idx = tid; idx < outs; idx += blockDim.x) {
      const int b = idx / a.n, j = idx - b * a.n;
      if (a.b0 + b >= a.batch) continue;
      double sum = 0.0;
      for (unsigned k = 0; k < gridDim.x; ++k)
        sum += static_cast<double>(__ldcg(&a.partials[static_cast<size_t>(k) * outs + idx]));
      float* out = a.c_out + static_cast<size_t>(a.b0 + b) * a.n + j;
      const double c = sum * static_cast<double>(a.scales[j]) + (a.accumulate ? static_cast<double>(*out) : 0.0);
      if (!isfinite(c)) twa_set_status(a.status, TWA_ERR_NONFINITE, a.b0 + b);
      *out = static_cast<float>(c);
    }
    if (tid == 0) *a.ticket = 0u;
  }
}

int encode_codes_map(twa_ctx* ctx, const twa_basis* P, int kt, CUtensorMap* map) {
  long long row_bytes = (P->D * P->bits + 7) / 8;
  row_bytes = (row_bytes + 511) / 512 * 512;             // whole, internally permuted 512-byte segments
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(row_bytes / 4), static_cast<cuuint64_t>(P->n)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(P->col_stride)};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(TWA_TILE_COL_WORDS * kt), static_cast<cuuint32_t>(P->n)};
  cuuint32_t es[2] = {1, 1};
  CUresult r = ctx->encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, P->data, dims, strides, box, es,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(ctx->last_error, sizeof(ctx->last_error), "cuTensorMapEncodeTiled(P~) failed: %d", static_cast<int>(r));
    return TWA_ERR_CUDA;
  }
  return TWA_OK;
}

int encode_batch_map(twa_ctx* ctx, const void* G, long long D, long long ldg, int batch, bool bf16, int nb,
                     CUtensorMap* map) {
  const int gsz = bf16 ? 2 : 4;
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(batch)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(ldg * gsz)};
  cuuint32_t box[2] = {256, static_cast<cuuint32_t>(nb)};
  cuuint32_t es[2] = {1, 1};
  CUresult r = ctx->encode_tiled(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                                 const_cast<void*>(G), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                 CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(ctx->last_error, sizeof(ctx->last_error), "cuTensorMapEncodeTiled(G) failed: %d", static_cast<int>(r));
    return TWA_ERR_CUDA;
  }
  return TWA_OK;
}

template <int BITS, bool GBF16, int MT, int KT, int NP>
int launch_one(twa_ctx* ctx, const CUtensorMap& mp, const CUtensorMap& mg, const BatchArgs& a, int grid, int smem) {
  auto kern = twa_project_batch_kernel<BITS, GBF16, MT, KT, NP>;
  static int smem_limit[64] = {0};
  int rc = twa_ensure_smem(ctx, reinterpret_cast<const void*>(kern), &smem_limit[ctx->device & 63], smem);
  if (rc) return rc;
  kern<<<grid, BATCH_THREADS, smem, ctx->stream>>>(mp, mg, a);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}

// Shapes of a pass: four pairs of gradients when at least three such stages fit in shared memory
// (with two 512-byte segments per tile column for n <= 64, one for wider bases), else two pairs
// and one segment.
template <int BITS, bool GBF16>
int launch_mt(twa_ctx* ctx, const CUtensorMap& mp, const CUtensorMap& mg, const BatchArgs& a, int kt, int nb, int grid,
              int smem) {
  const int mt = (a.n + 15) >> 4;
  if (nb == 8 && kt == 2) {
    switch (mt) {
      case 1: return launch_one<BITS, GBF16, 1, 2, 4>(ctx, mp, mg, a, grid, smem);
      case 2: return launch_one<BITS, GBF16, 2, 2, 4>(ctx, mp, mg, a, grid, smem);
      case 3: return launch_one<BITS, GBF16, 3, 2, 4>(ctx, mp, mg, a, grid, smem);
      default: return launch_one<BITS, GBF16, 4, 2, 4>(ctx, mp, mg, a, grid, smem);
    }
  }
  if (nb == 8) {
    switch (mt) {
      case 5: return launch_one<BITS, GBF16, 5, 1, 4>(ctx, mp, mg, a, grid, smem);
      case 6: return launch_one<BITS, GBF16, 6, 1, 4>(ctx, mp, mg, a, grid, smem);
      case 7: return launch_one<BITS, GBF16, 7, 1, 4>(ctx, mp, mg, a, grid, smem);
      default: return launch_one<BITS, GBF16, 8, 1, 4>(ctx, mp, mg, a, grid, smem);
    }
  }
  switch (mt) {
    case 1: return launch_one<BITS, GBF16, 1, 1, 2>(ctx, mp, mg, a, grid, smem);
    case 2: return launch_one<BITS, GBF16, 2, 1, 2>(ctx, mp, mg, a, grid, smem);
    case 3: return launch_one<BITS, GBF16, 3, 1, 2>(ctx, mp, mg, a, grid, smem);
    case 4: return launch_one<BITS, GBF16, 4, 1, 2>(ctx, mp, mg, a, grid, smem);
    case 5: return launch_one<BITS, GBF16, 5, 1, 2>(ctx, mp, mg, a, grid, smem);
    case 6: return launch_one<BITS, GBF16, 6, 1, 2>(ctx, mp, mg, a, grid, smem);
    case 7: return launch_one<BITS, GBF16, 7, 1, 2>(ctx, mp, mg, a, grid, smem);
    default: return launch_one<BITS, GBF16, 8, 1, 2>(ctx, mp, mg, a, grid, smem);
  }
}

int fixed_smem(int bits, int sets = 1) { return TWA_SMEM_HEADER + MMA_WARPS * sets * pair_bytes(bits) + 1024; }

unsigned stage_bytes_of(const twa_basis* P, int gsz, int kt, int nb) {
  const unsigned tx = static_cast<unsigned>(P->n) * TWA_TILE_COL_BYTES * kt + twa_tile_rows(P->bits) * kt * gsz * nb;
  return (tx + 1023) / 1024 * 1024;
}

// (segments per tile column, gradients per pass) for this basis, gradient type and device
void pass_shape(const twa_ctx* ctx, const twa_basis* P, int gsz, int* kt, int* nb) {
  const int kt8 = P->n <= 64 ? 2 : 1;
  const bool fits = (ctx->smem_optin - fixed_smem(P->bits)) / static_cast<int>(stage_bytes_of(P, gsz, kt8, 8)) >= 3;
  const bool partials_fit = static_cast<size_t>(ctx->sm_count) * 8 * P->n <= static_cast<size_t>(TWA_MAX_GRID) * TWA_MAX_N;
  if (fits && partials_fit) {
    *kt = kt8;
    *nb = 8;
  } else {
    *kt = 1;
    *nb = 4;
  }
}

}  // namespace

extern "C" int twa_project_batch_group(twa_ctx* ctx, const twa_basis* P, twa_dtype g_dtype) {
  if (!ctx || !P || P->bits == 32) return 1;
  int kt, nb;
  pass_shape(ctx, P, g_dtype == TWA_BF16 ? 2 : 4, &kt, &nb);
  return nb;
}

namespace {
int project_batch_rows(twa_ctx* ctx, const twa_basis* P, const void* G, long long ldg, int batch, twa_dtype g_dtype,
                       float* C_out, void* ws, int accumulate);
}

extern "C" int twa_project_batch(twa_ctx* ctx, const twa_basis* P, const void* G, int64_t ldg, int batch,
                                 twa_dtype g_dtype, float* C_out, void* ws, size_t ws_bytes) {
  if (!ctx || !P || !G || !C_out || batch < 1) return TWA_ERR_INVALID_ARG;
  if (g_dtype != TWA_F32 && g_dtype != TWA_BF16) return TWA_ERR_INVALID_ARG;
  int rc = check_basis_slabbed(ctx, P);
  if (rc) return rc;
  if (ldg < P->D) return TWA_ERR_INVALID_ARG;
  if (!ws || ws_bytes < TWA_WS_BYTES) return TWA_ERR_WORKSPACE;
  const bool bf16 = g_dtype == TWA_BF16;
  const int gsz = bf16 ? 2 : 4;
  if ((reinterpret_cast<uintptr_t>(G) & 15) || ((ldg * gsz) & 15)) return TWA_ERR_MISALIGNED;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  if (P->bits == 32) {
    // a float32 basis (the build's own format) has no integer path: one projection per gradient
    for (int b = 0; b < batch; ++b) {
      rc = twa_project(ctx, P, static_cast<const char*>(G) + static_cast<size_t>(b) * ldg * gsz, g_dtype,
                       C_out + static_cast<size_t>(b) * P->n, ws, ws_bytes);
      if (rc) return rc;
    }
    return TWA_OK;
  }
  // a basis of more rows than one launch takes: slab after slab, every slab after the first adding to C_out
  const SlabPlan plan = slab_plan(ctx, P->D);
  for (int k = 0; k < plan.count; ++k) {
    long long r0;
    const twa_basis v = slab_view(P, plan, k, &r0);
    rc = project_batch_rows(ctx, &v, static_cast<const char*>(G) + r0 * gsz, ldg, batch, g_dtype, C_out, ws, k > 0);
    if (rc) return rc;
  }
  return TWA_OK;
}

namespace {
int project_batch_rows(twa_ctx* ctx, const twa_basis* P, const void* G, long long ldg, int batch, twa_dtype g_dtype,
                       float* C_out, void* ws, int accumulate) {
  const bool bf16 = g_dtype == TWA_BF16;
  const int gsz = bf16 ? 2 : 4;
  int rc;
  int kt, nb;
  pass_shape(ctx, P, gsz, &kt, &nb);
  const int rows = twa_tile_rows(P->bits) * kt;
  CUtensorMap mp, mg;
  rc = encode_codes_map(ctx, P, kt, &mp);
  if (rc) return rc;
  rc = encode_batch_map(ctx, G, P->D, ldg, batch, bf16, nb, &mg);
  if (rc) return rc;
  BatchArgs a;
  a.D = P->D;
  a.n = P->n;
  a.tiles = static_cast<int>((P->D + rows - 1) / rows);
  a.batch = batch;
  a.g_off = static_cast<unsigned>(P->n) * TWA_TILE_COL_BYTES * kt;
  a.tx_bytes = a.g_off + static_cast<unsigned>(rows * gsz * nb);
  a.stage_bytes = (a.tx_bytes + 1023) / 1024 * 1024;
  int stages = (ctx->smem_optin - fixed_smem(P->bits)) / static_cast<int>(a.stage_bytes);
  // a set of digit matrices per pair if that costs no stage (or leaves three)
  int sets = 1;
  {
    const int with_sets = (ctx->smem_optin - fixed_smem(P->bits, nb / 2)) / static_cast<int>(a.stage_bytes);
    if (with_sets == stages || with_sets >= 3) {
      sets = nb / 2;
      stages = with_sets;
    }
  }
  a.pair_stride = sets > 1 ? static_cast<unsigned>(pair_bytes(P->bits)) : 0u;
  if (stages > TWA_MAX_STAGES) stages = TWA_MAX_STAGES;
  if (stages < 2) return TWA_ERR_UNSUPPORTED;
  // the ring is reused for the block's [16][NB][128] float sums after the tile loop
  if (static_cast<size_t>(stages) * a.stage_bytes < sizeof(float) * MMA_WARPS * nb * TWA_MAX_N) return TWA_ERR_UNSUPPORTED;
  a.stages = stages;
  a.scratch_off = TWA_SMEM_HEADER + static_cast<unsigned>(stages) * a.stage_bytes;
  a.scales = P->scales;
  a.partials = reinterpret_cast<float*>(static_cast<char*>(ws) + TWA_WS_PARTIALS);
  a.ticket = ctx->d_ticket;
  a.status = ctx->d_status;
  a.c_out = C_out;
  a.accumulate = accumulate;
  a.wait_limit_ns = ctx->wait_limit_ns;
  int grid = ctx->sm_count < a.tiles ? ctx->sm_count : a.tiles;
  while (static_cast<size_t>(grid) * nb * P->n > static_cast<size_t>(TWA_MAX_GRID) * TWA_MAX_N) --grid;
  const int smem = static_cast<int>(a.scratch_off) + MMA_WARPS * sets * pair_bytes(P->bits) + 1024;
  for (int b0 = 0; b0 < batch; b0 += nb) {
    a.b0 = b0;
    if (P->bits == 8)
      rc = bf16 ? launch_mt<8, true>(ctx, mp, mg, a, kt, nb, grid, smem) : launch_mt<8, false>(ctx, mp, mg, a, kt, nb, grid, smem);
    else
      rc = bf16 ? launch_mt<4, true>(ctx, mp, mg, a, kt, nb, grid, smem) : launch_mt<4, false>(ctx, mp, mg, a, kt, nb, grid, smem);
    if (rc) return rc;
  }
  return TWA_OK;
}
}  // namespace
