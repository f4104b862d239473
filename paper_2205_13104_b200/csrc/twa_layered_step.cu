// Subspace step for the paper's default construction (Algorithm 1 with its loop over the layers;
// Sections 4.2, 4.3, 4.5, 4.6): for every layer l
//     c^l = P~^l^T g^l,   beta^l <- (1 - eta*lambda) beta^l - eta c^l,   w^l = w_bar^l + P~^l beta^l,
// with P~^l = a^l * code + b^l, unsigned B-bit codes.
//
// Same data path as twa_stream_mma.cu (TMA tiles of the codes, integer MMAs against base-128
// digits of g and of the coefficients).  What the layers add:
//  * every block owns a contiguous range of tiles, so it meets few layers; a warp's share of a
//    tile (32*KT bytes of every column) lies inside one 64-byte granule, hence inside one layer,
//    and the granule table gives its layer, its first flat row and how many of its rows exist;
//  * g, w_bar and w are addressed by flat row (layers start anywhere, so bulk copies cannot be
//    aligned): four helper warps stage the tile's granule entries and its rows of g (or w_bar)
//    in the stage beside the codes, each helper several tiles ahead of the MMA warps, and
//    signal the stage's "full" barrier together with the bulk copy;
//  * projection sums are kept per (block, warp, layer) and combined in a fixed order by a small
//    second kernel, which also applies a^l, b^l * sum(g^l) and the coefficient update;
//  * the lift takes its digit fragments per layer from a table made by a third small kernel,
//    and adds the constant b^l * sum_i beta_i^l.
#include <stdio.h>

#include <vector>

#include "twa_mma.cuh"

namespace {

constexpr int ROW_FLOATS = 132;                 // one partial row: 128 column sums, sum of g, padding
constexpr int L_THREADS = (MMA_WARPS + 2) * 32; // MMA warps, the bulk-copy warp, the helper warp

struct LProjectArgs {
  int n, stages, tiles, tpc;
  long long D;
  unsigned stage_bytes, tx_bytes, scratch_off, aux_off, ering_off;
  const int4* gran;
  const void* g;
  const int* cta_first;
  const int* cta_base;
  float* partials;
  int* status;
  unsigned long long wait_limit_ns;
};

struct LLiftArgs {
  int n, stages, tiles, tpc;
  long long D;
  unsigned stage_bytes, tx_bytes, aux_off, ering_off;
  const int4* gran;
  const unsigned char* dig;      // [L][4][128] digit bytes of a^l * beta^l_i
  const int* ebits;              // [L] exponent field of the layer's largest |coefficient|
  const float* konst;            // [L] b^l * sum_i beta^l_i
  const float* base;
  float* out;
  int out_vector_ok;             // out is 16-byte aligned
  int* status;
  unsigned long long wait_limit_ns;
};

__device__ __forceinline__ void cp_async_4(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_16_zfill(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
// Untiled bulk copy global -> shared, completion counted in bytes on an mbarrier; both addresses
// 16-byte aligned, size a multiple of 16.
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, unsigned bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
// More bytes to expect on the barrier's current phase, without an arrival.
__device__ __forceinline__ void twa_mbar_expect_tx_only(uint32_t bar, unsigned bytes) {
  asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
// The barrier receives one arrival from this thread once all its copies issued so far have landed.
__device__ __forceinline__ void cp_async_arrive_noinc(uint32_t bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void init_barriers_layered(twa_smem_header* hdr, int stages) {
  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      twa_mbar_init(twa_smem_u32(&hdr->full[s]), 33);           // the bulk copy and the 32 helper lanes
      twa_mbar_init(twa_smem_u32(&hdr->empty[s]), MMA_WARPS);
    }
    hdr->abort_flag = 0;
    hdr->last_flag = 0;
    hdr->bad_flag = 0;
    twa_fence_barrier_init();
  }
}

// What a stage holds beside the codes: the tile's granule entries (16 bytes each), then one
// segment per granule with the granule's rows of the flat vector (g or w_bar).  A segment starts
// at the 4-byte word that holds the granule's first element, so a bfloat16 granule that starts at
// an odd flat row sits one element into its segment.
__host__ __device__ constexpr int granule_rows(int bits) { return 64 * 8 / bits; }
__host__ __device__ constexpr int segment_bytes(int bits) { return granule_rows(bits) * 4 + 16; }
__host__ __device__ constexpr int aux_bytes(int bits, int kt) { return 8 * kt * (16 + segment_bytes(bits)); }

// digit matrices of a projection warp: one per code slot of a byte (at least the two of the shared helpers)
__host__ __device__ constexpr int digit_sets(int bits) { return 8 / bits < 2 ? 2 : 8 / bits; }
__host__ __device__ constexpr int digit_scratch(int bits) { return digit_sets(bits) * BYTE_DIGIT_SET; }

constexpr int ENTRY_DEPTH = 16;                                  // tiles the helper reads entries ahead
constexpr int ENTRY_RING_BYTES = ENTRY_DEPTH * 16 * 16;          // up to 16 granules per tile

__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait_group() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// A tile whose first and last granule belong to the same layer, with the last one full, covers one
// contiguous run of flat rows (a layer's granules follow one another); when that run also starts
// on a 16-byte boundary of src the helper fetches it with a single bulk copy and the segments are
// packed (GR * ES bytes apart, no slack).  The helper and the MMA warps evaluate this same test on
// the tile's entries.  Without it a tile of 16 granules took 16 copies of 128 to 256 bytes.
template <int BITS, int KT, int ES>
__device__ __forceinline__ bool tile_is_packed(const int4* entries, const void* src) {
  constexpr int GR = granule_rows(BITS);
  const int4 e0 = entries[0], eN = entries[8 * KT - 1];
  return e0.x >= 0 && e0.x == eN.x && eN.y == GR &&
         ((reinterpret_cast<uintptr_t>(src) + static_cast<unsigned long long>(e0.z) * ES) & 15u) == 0;
}

// The helper warp: for every tile of the block's sequence, asynchronous copies of the granule
// entries and of the rows of `src` the tile's granules cover (flat rows have no alignment
// guarantee, which rules out bulk copies), straight into the tile's stage; each lane's copies report to the stage's "full"
// barrier.  The copies' addresses come from the entries, which the warp therefore fetches
// ENTRY_DEPTH tiles ahead into a ring of its own (`ering`), also asynchronously, so that it
// never waits for a load issued recently.  src may be NULL (only entries are staged).
template <int BITS, int KT, int ES>
__device__ __forceinline__ void helper_loop(twa_smem_header* hdr, unsigned char* ring, unsigned stage_bytes,
                                            unsigned aux_off, int stages, int t_first, int t_count,
                                            bool reverse, const int4* __restrict__ gran, const void* src,
                                            long long D, int4* ering, int lane, int* status,
                                            unsigned long long limit) {
  constexpr int GR = granule_rows(BITS);
  constexpr int GPT = 8 * KT;
  constexpr int SEG = segment_bytes(BITS);
  constexpr int QW = GR * ES / 16;                     // 16-byte pieces of a granule's rows
  constexpr int TQ = GPT * QW;                         // and of a tile's: a multiple of 32
  static_assert(TQ % 32 == 0, "pieces per tile");
  volatile int* abort_flag = &hdr->abort_flag;
  const char* sbytes = static_cast<const char*>(src);
  const long long total_bytes = D * ES;
  auto entries_of = [&](int k) {
    return gran + static_cast<size_t>(t_first + (reverse ? (t_count - 1 - k) : k)) * GPT + lane;
  };
  for (int j = 0; j < ENTRY_DEPTH; ++j) {              // one group per tile, also when it is empty
    if (lane < GPT && j < t_count) cp_async_16(twa_smem_u32(ering + j * GPT + lane), entries_of(j));
    cp_async_commit();
  }
  int s = 0, use = 0, slot = 0;
  for (int k = 0; k < t_count; ++k) {
    cp_async_wait_group<ENTRY_DEPTH - 1>();            // the group that brought tile k's entries
    __syncwarp();
    const int4* ep = ering + slot * GPT;
    if (use > 0 && !twa_mbar_wait(twa_smem_u32(&hdr->empty[s]), static_cast<unsigned>(use - 1) & 1u, abort_flag, limit)) {
      twa_set_status(status, TWA_ERR_TIMEOUT, -1);
      break;
    }
    const uint32_t aux = twa_smem_u32(ring + static_cast<size_t>(s) * stage_bytes + aux_off);
    if (lane < GPT) cp_async_16(aux + lane * 16, entries_of(k));
    if (src) {
      // Lane q looks after granule q.  A granule whose rows start on a 16-byte boundary of src and
      // fill a multiple of 16 bytes (every granule, when the layers' sizes are multiples of 8 rows)
      // goes as one bulk copy counted in bytes on the stage's barrier.
      const uint32_t fb = twa_smem_u32(&hdr->full[s]);
      bool settled = true;
      if (tile_is_packed<BITS, KT, ES>(ep, sbytes)) {
        // the whole tile lies in one layer: its rows are one aligned run of src, one bulk copy
        if (lane == 0) {
          twa_mbar_expect_tx_only(fb, GPT * GR * ES);
          bulk_copy_g2s(aux + GPT * 16, sbytes + static_cast<long long>(ep[0].z) * ES, GPT * GR * ES, fb);
        }
      } else if (lane < GPT) {
        const int4 e = ep[lane];
        if (e.x >= 0) {
          const char* from = sbytes + static_cast<long long>(e.z) * ES;
          const unsigned bytes = static_cast<unsigned>(e.y) * ES;
          if (((reinterpret_cast<uintptr_t>(from) | bytes) & 15) == 0) {
            twa_mbar_expect_tx_only(fb, bytes);
            bulk_copy_g2s(aux + GPT * 16 + lane * SEG, from, bytes, fb);
          } else {
            settled = false;
          }
        }
      }
      const unsigned todo = ~__ballot_sync(0xFFFFFFFFu, settled);
      if (todo) {
        // The other granules in 16-byte pieces, one per lane and pass: 16 bytes at a time where
        // the granule starts on a 16-byte boundary, else 4 bytes at a time.
#pragma unroll 1
        for (int i = 0; i < TQ / 32; ++i) {
          const int x = i * 32 + lane, q = x / QW, j = x % QW;
          if (!((todo >> q) & 1u)) continue;
          const int4 e = ep[q];
          const long long gbyte = static_cast<long long>(e.z) * ES;            // the granule's first row in src
          const uint32_t seg = aux + GPT * 16 + q * SEG;
          if (((reinterpret_cast<uintptr_t>(sbytes) + gbyte) & 15) == 0) {
            const int nbytes = e.y * ES - j * 16;                              // bytes of existing rows from here on
            if (nbytes > 0) cp_async_16_zfill(seg + j * 16, sbytes + gbyte + j * 16, nbytes < 16 ? nbytes : 16);
          } else {
            const long long byte0 = gbyte & ~3LL;                              // word holding the first row
            const int shift = ES == 2 ? (e.z & 1) : 0;
#pragma unroll
            for (int t = 0; t < (ES == 2 ? 5 : 4); ++t) {
              if (t == 4 && j != QW - 1) continue;                             // the one word past a shifted granule
              const int w = 4 * j + t;
              const int first = ES == 2 ? 2 * w - shift : w;                   // first row the word holds
              if (first < e.y) {
                const long long off = byte0 + 4LL * w;
                const long long rem = total_bytes - off;
                cp_async_4(seg + 4 * w, sbytes + off, rem >= 4 ? 4 : static_cast<int>(rem));
              }
            }
          }
        }
      }
    }
    cp_async_arrive_noinc(twa_smem_u32(&hdr->full[s]));
    __syncwarp();                                      // every lane has read the ring slot
    if (lane < GPT && k + ENTRY_DEPTH < t_count)
      cp_async_16(twa_smem_u32(ering + slot * GPT + lane), entries_of(k + ENTRY_DEPTH));
    cp_async_commit();
    if (++slot == ENTRY_DEPTH) slot = 0;
    if (++s == stages) {
      s = 0;
      ++use;
    }
  }
  cp_async_wait_group<0>();                            // nothing of this warp is in flight when it leaves
  if (*abort_flag) {                                   // a wait ran out: give the bulk copies issued so far time to land
    const unsigned long long t0 = twa_globaltimer();
    while (twa_globaltimer() - t0 < 200000ull) {
    }
  }
}

// ------------------------------------------------------------------------------------------------
template <int BITS, bool GBF16, int MT, int KT>
__global__ void __launch_bounds__(L_THREADS, 1)
layered_project_kernel(const __grid_constant__ CUtensorMap map_p, const LProjectArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (twa_smem_u32(smem_raw) & 1023u)) & 1023u);
  constexpr int RB = 32 * 8 / BITS;                    // rows behind 32 bytes of a column
  twa_smem_header* hdr = reinterpret_cast<twa_smem_header*>(smem);
  unsigned char* ring = smem + TWA_SMEM_HEADER;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gid = lane >> 2, tig = lane & 3;
  init_barriers_layered(hdr, a.stages);
  const int my_first = a.cta_first[blockIdx.x], my_base = a.cta_base[blockIdx.x];
  {
    // a warp writes a row of partial sums only for the layers it meets: the rest must read as zero
    float* mine = a.partials + static_cast<size_t>(my_base) * MMA_WARPS * ROW_FLOATS;
    const int count = (a.cta_base[blockIdx.x + 1] - my_base) * MMA_WARPS * ROW_FLOATS;
    for (int i = threadIdx.x; i < count; i += blockDim.x) mine[i] = 0.0f;
  }
  __syncthreads();
  const int t_first = blockIdx.x * a.tpc;
  const int t_count = (a.tiles - t_first) < a.tpc ? (a.tiles - t_first) : a.tpc;

  if (warp == MMA_WARPS) {
    if (lane == 0)
      producer_loop_mma(hdr, ring, &map_p, nullptr, t_first, 1, t_count, a.stages, a.stage_bytes, TWA_TILE_COL_BYTES / 8 * KT, 0, 0,
                        0, 0, a.tx_bytes, false, a.status, a.wait_limit_ns);
    return;
  }
  if (warp > MMA_WARPS) {
    helper_loop<BITS, KT, (GBF16 ? 2 : 4)>(hdr, ring, a.stage_bytes, a.aux_off, a.stages, t_first, t_count, false,
                                           a.gran, a.g, a.D, reinterpret_cast<int4*>(smem + a.ering_off), lane,
                                           a.status, a.wait_limit_ns);
    return;
  }
  constexpr int SUB = 8 / BITS;                        // codes per byte: one digit matrix each
  unsigned char* digw = smem + a.scratch_off + warp * digit_scratch(BITS);   // this warp's digit matrices
  constexpr bool FOUR = !GBF16;                        // float32 gradients carry a fourth byte digit
  byte_digit_init<FOUR, digit_sets(BITS)>(digw, lane);
  __syncwarp();
  const uint32_t dig_addr = byte_digit_ldmatrix_addr(digw, lane);
  const int dmult = byte_digit_mult(tig);
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
  const int gran_in_tile = (warp * 32 * KT) >> 6;      // the granule holding the warp's share of a column
  const int rig0 = ((warp * 32 * KT) & 63) * 8 / BITS; // first row of the share inside the granule
  constexpr int GES = GBF16 ? 2 : 4;
  const unsigned seg_off_loose = a.aux_off + 8 * KT * 16 + gran_in_tile * segment_bytes(BITS);
  const unsigned seg_off_packed = a.aux_off + 8 * KT * 16 + gran_in_tile * granule_rows(BITS) * GES;
  float facc[MT][2];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) facc[mt][0] = facc[mt][1] = 0.0f;
  float gsum = 0.0f;
  int cur_layer = -1;
  bool bad = false;
  auto flush = [&]() {
    float* row = a.partials + (static_cast<size_t>(my_base + cur_layer - my_first) * MMA_WARPS + warp) * ROW_FLOATS;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      float v0 = facc[mt][0], v1 = facc[mt][1];
      v0 += __shfl_xor_sync(0xFFFFFFFFu, v0, 1);
      v1 += __shfl_xor_sync(0xFFFFFFFFu, v1, 1);
      v0 += __shfl_xor_sync(0xFFFFFFFFu, v0, 2);
      v1 += __shfl_xor_sync(0xFFFFFFFFu, v1, 2);
      if (tig == 0) {
        row[mt * 16 + gid] = bad ? __int_as_float(0x7FC00000) : v0;
        row[mt * 16 + gid + 8] = bad ? __int_as_float(0x7FC00000) : v1;
      }
      facc[mt][0] = facc[mt][1] = 0.0f;
    }
    float gs = gsum;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) gs += __shfl_xor_sync(0xFFFFFFFFu, gs, off);
    if (lane == 0) row[128] = gs;
    gsum = 0.0f;
    bad = false;
  };

  volatile int* abort_flag = &hdr->abort_flag;
  int s = 0;
  unsigned phase = 0;
  for (int k = 0; k < t_count; ++k) {
    if (!twa_mbar_wait(twa_smem_u32(&hdr->full[s]), phase, abort_flag, a.wait_limit_ns)) {
      twa_set_status(a.status, TWA_ERR_TIMEOUT, -1);
      break;
    }
    const unsigned char* st = ring + static_cast<size_t>(s) * a.stage_bytes;
    const int4* entries = reinterpret_cast<const int4*>(st + a.aux_off);
    const int4 e = entries[gran_in_tile];
    const unsigned seg_off = tile_is_packed<BITS, KT, GES>(entries, a.g) ? seg_off_packed : seg_off_loose;
    // the granule's rows of g, staged by the helper; rows past the layer's end hold nothing.  Lane l
    // holds the SUB rows behind byte l of the warp's 32-byte block: row SUB * l + s meets code slot s.
    float gv[KT][SUB];
#pragma unroll
    for (int u = 0; u < KT; ++u) {
      const int r = rig0 + u * RB + SUB * lane;
#pragma unroll
      for (int q = 0; q < SUB; ++q) {
        float x;
        if (GBF16) {
          const unsigned short* gs = reinterpret_cast<const unsigned short*>(st + seg_off) + (e.z & 1);
          x = __uint_as_float(static_cast<uint32_t>(gs[r + q]) << 16);
        } else {
          x = reinterpret_cast<const float*>(st + seg_off)[r + q];
        }
        gv[u][q] = r + q < e.y ? x : 0.0f;
      }
    }
    if (e.x != cur_layer) {
      if (cur_layer >= 0) flush();
      cur_layer = e.x;
    }
    if (e.x >= 0) {
      const uint32_t tile_base = twa_smem_u32(st);
      unsigned mb = 0u;
#pragma unroll
      for (int u = 0; u < KT; ++u)
#pragma unroll
        for (int q = 0; q < SUB; ++q) {
          mb = max(mb, __float_as_uint(gv[u][q]) & 0x7FFFFFFFu);
          gsum += gv[u][q];
        }
      mb = __reduce_max_sync(0xFFFFFFFFu, mb);
      const ByteDigitScale ds = byte_digit_scale(mb);
      if (ds.bad) bad = true;
      if (ds.live) {
        // 4-bit codes enter the MMA times 16
        const float wl = byte_digit_weight(tig, BITS == 4 ? ds.w0 * 0.0625f : ds.w0);
        int c[MT][4];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) c[mt][0] = c[mt][1] = c[mt][2] = c[mt][3] = 0;
#pragma unroll
        for (int u = 0; u < KT; ++u) {
#pragma unroll
          for (int q = 0; q < SUB; ++q) byte_digit_store<FOUR>(digw, q, lane, gv[u][q], ds.up);
          __syncwarp();
          uint32_t bf[SUB < 2 ? 2 : SUB][2];             // B fragments: digit matrix q meets code slot q
          if (SUB == 1) {
            ldmatrix_x2(dig_addr, bf[0][0], bf[0][1]);
          } else {
#pragma unroll
            for (int q = 0; q < SUB / 2; ++q) {
              uint32_t bb[4];
              ldmatrix_x4(dig_addr + q * 2 * BYTE_DIGIT_SET, bb);
              bf[2 * q][0] = bb[0]; bf[2 * q][1] = bb[1]; bf[2 * q + 1][0] = bb[2]; bf[2 * q + 1][1] = bb[3];
            }
          }
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
            uint32_t r[4];
            ldmatrix_x4(tile_base + aoff[u][mt], r);
            if (BITS == 8) {
              mma_u8u8(c[mt], r, bf[0][0], bf[0][1]);
            } else if (BITS == 4) {
              uint32_t ev[4], od[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                ev[i] = (r[i] << 4) & 0xF0F0F0F0u;       // even rows: 16 * code, unsigned
                od[i] = r[i] & 0xF0F0F0F0u;              // odd rows
              }
              mma_u8u8(c[mt], ev, bf[0][0], bf[0][1]);
              mma_u8u8(c[mt], od, bf[1][0], bf[1][1]);
            } else {
              constexpr uint32_t MASK = 0x01010101u * ((1u << BITS) - 1u);
#pragma unroll
              for (int q = 0; q < SUB; ++q) {            // slot q of every byte: rows SUB * byte + q
                uint32_t x[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) x[i] = (r[i] >> (BITS * q)) & MASK;
                mma_u8u8(c[mt], x, bf[q][0], bf[q][1]);
              }
            }
          }
          __syncwarp();
        }
        // digit sums -> float: |sum| < 2^31 (at most 128 rows x 255 x 240 per digit, times 257)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          facc[mt][0] = fmaf(static_cast<float>(c[mt][0] + dmult * c[mt][1]), wl, facc[mt][0]);
          facc[mt][1] = fmaf(static_cast<float>(c[mt][2] + dmult * c[mt][3]), wl, facc[mt][1]);
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
  if (cur_layer >= 0) flush();
}

// Digits of the layer's coefficients on their common scale, one per stored column, and the constant
// b^l * sum_i beta^l_i.  One plane: column i carries a^l beta^l_i.  Two planes (16-bit codes, high
// bytes in columns 0..n-1, low bytes in n..2n-1): column i carries 256 a^l beta^l_i, column n + i
// carries a^l beta^l_i.  Called by the first 128 threads of a block; `amax` is shared and zero;
// beta_row holds the layer's n coefficients.
__device__ __forceinline__ void layer_coefficients(int l, int i, int n, int planes, float al, float bl,
                                                   const float* beta_row, unsigned* amax,
                                                   unsigned char* __restrict__ dig, int* __restrict__ ebits_out,
                                                   float* __restrict__ konst, int* status) {
  float coef = 0.0f;
  if (i < n) coef = beta_row[i] * al * (planes == 2 ? 256.0f : 1.0f);
  else if (planes == 2 && i < 2 * n) coef = beta_row[i - n] * al;
  atomicMax(amax, __float_as_uint(coef) & 0x7FFFFFFFu);
  asm volatile("bar.sync 1, 128;" ::: "memory");
  const unsigned ebits = *amax >> 23;
  const bool bad = ebits >= 255u, live = ebits >= 5u && !bad;
  uint32_t d = 0;
  if (live) d = cut_digits(coef * __uint_as_float((259u - ebits) << 23));
#pragma unroll
  for (int k = 0; k < 4; ++k) dig[static_cast<size_t>(l) * 512 + k * 128 + i] = static_cast<unsigned char>(d >> (8 * k));
  if (i == 0) {
    double sb = 0.0;
    for (int q = 0; q < n; ++q) sb += static_cast<double>(beta_row[q]);
    const double kk = static_cast<double>(bl) * sb;
    if (bad || !isfinite(kk)) twa_set_status(status, TWA_ERR_NONFINITE, l);
    konst[l] = static_cast<float>(kk);
    ebits_out[l] = bad ? -1 : (live ? static_cast<int>(ebits) : 0);
  }
}

constexpr int COMBINE_PARTS = 4;

// One block of 128 * COMBINE_PARTS threads per layer: fixed-order sum of the layer's partial rows,
// c = a S + b sum(g), the coefficient update, and (dig != NULL) the lift's coefficient digits.
// Part p sums a contiguous quarter of the blocks that met the layer; the parts are added in order.
__global__ void __launch_bounds__(128 * COMBINE_PARTS)
layered_combine_kernel(const float* __restrict__ partials, const int* __restrict__ cta_first,
                       const int* __restrict__ cta_base, int ctas, int n, int planes, const float* __restrict__ a,
                       const float* __restrict__ b, float* c_out, float* beta, float lr, float lambda,
                       const twa_adam_args adam, unsigned char* dig, int* ebits_out, float* konst, int* status) {
  __shared__ int range[2];
  __shared__ unsigned amax;
  __shared__ double part_s[COMBINE_PARTS][128], part_g[COMBINE_PARTS];
  __shared__ float beta_new[128];
  const int l = blockIdx.x, i = threadIdx.x & 127, p = threadIdx.x >> 7;
  if (threadIdx.x == 0) {
    range[0] = ctas;
    range[1] = -1;
    amax = 0u;
  }
  __syncthreads();
  for (int cta = threadIdx.x; cta < ctas; cta += blockDim.x) {        // which blocks met this layer
    const int f = cta_first[cta], cnt = cta_base[cta + 1] - cta_base[cta];
    if (l >= f && l < f + cnt) {
      atomicMin(&range[0], cta);
      atomicMax(&range[1], cta);
    }
  }
  __syncthreads();
  const int c0 = range[0], c1 = range[1] + 1;                          // contiguous: blocks own tile ranges in order
  const int per = (c1 - c0 + COMBINE_PARTS - 1) / COMBINE_PARTS;
  const int lo = c0 + p * per, hi = (lo + per) < c1 ? (lo + per) : c1;
  double S = 0.0, Sg = 0.0;
  for (int cta = lo; cta < hi; ++cta) {
    const float* rows = partials + static_cast<size_t>(cta_base[cta] + l - cta_first[cta]) * MMA_WARPS * ROW_FLOATS;
    float v[MMA_WARPS], vg[MMA_WARPS];
#pragma unroll
    for (int w = 0; w < MMA_WARPS; ++w) {
      v[w] = i < n * planes ? __ldcg(rows + w * ROW_FLOATS + i) : 0.0f;
      vg[w] = __ldcg(rows + w * ROW_FLOATS + 128);
    }
#pragma unroll
    for (int w = 0; w < MMA_WARPS; ++w) {
      S += static_cast<double>(v[w]);
      Sg += static_cast<double>(vg[w]);
    }
  }
  part_s[p][i] = S;
  if (i == 0) part_g[p] = Sg;
  __syncthreads();
  if (p != 0) return;
  S = 0.0;
  Sg = 0.0;
#pragma unroll
  for (int q = 0; q < COMBINE_PARTS; ++q) {
    S += part_s[q][i];
    Sg += part_g[q];
  }
  if (planes == 2) {                                                   // S of candidate i = 256 S_high + S_low
    part_s[0][i] = S;
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (i < n) S = 256.0 * S + part_s[0][n + i];
  }
  float bnew = 0.0f;
  if (i < n) {
    const double c = static_cast<double>(a[l]) * S + static_cast<double>(b[l]) * Sg;
    if (!isfinite(c)) twa_set_status(status, TWA_ERR_NONFINITE, l);
    if (c_out) c_out[static_cast<size_t>(l) * n + i] = static_cast<float>(c);
    if (beta) {
      // the coefficients are state that outlives the call: a coefficient whose c is not finite, and
      // every coefficient after a wait ran out in the projection, stays as it was
      const size_t at = static_cast<size_t>(l) * n + i;
      bnew = beta[at];
      if (isfinite(c) && __ldcg(status) != TWA_ERR_TIMEOUT) {
        bnew = twa_coefficient_update(bnew, c, lr, lambda, adam, at);
        beta[at] = bnew;
      }
    }
  }
  if (dig) {                                                           // only with beta: the step
    beta_new[i] = bnew;
    asm volatile("bar.sync 1, 128;" ::: "memory");
    layer_coefficients(l, i, n, planes, a[l], b[l], beta_new, &amax, dig, ebits_out, konst, status);
  }
}

// One block (128 threads) per layer: the lift's coefficient digits from given coefficients.
__global__ void layered_coef_kernel(const float* __restrict__ beta, int n, int planes, const float* __restrict__ a,
                                    const float* __restrict__ b, unsigned char* __restrict__ dig,
                                    int* __restrict__ ebits_out, float* __restrict__ konst, int* status) {
  __shared__ unsigned amax;
  __shared__ float row[128];
  const int l = blockIdx.x, i = threadIdx.x;
  if (i == 0) amax = 0u;
  row[i] = i < n ? beta[static_cast<size_t>(l) * n + i] : 0.0f;
  __syncthreads();
  layer_coefficients(l, i, n, planes, a[l], b[l], row, &amax, dig, ebits_out, konst, status);
}

// ------------------------------------------------------------------------------------------------
template <int BITS, int KS, int KT>
__global__ void __launch_bounds__(L_THREADS, 1)
layered_lift_kernel(const __grid_constant__ CUtensorMap map_p, const LLiftArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (twa_smem_u32(smem_raw) & 1023u)) & 1023u);
  constexpr int SUB = 8 / BITS;                        // codes per byte
  constexpr int LROWS = 2 * SUB;                       // rows a lane finishes per 16-byte chunk
  constexpr int SG = SUB > 4 ? 4 : SUB;                // code slots handled together (bounds the live registers)
  constexpr int NG = SUB / SG;
  constexpr int RB = 32 * 8 / BITS;
  twa_smem_header* hdr = reinterpret_cast<twa_smem_header*>(smem);
  unsigned char* ring = smem + TWA_SMEM_HEADER;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gid = lane >> 2, tig = lane & 3;
  init_barriers_layered(hdr, a.stages);
  __syncthreads();
  const int t_first = blockIdx.x * a.tpc;
  const int t_count = (a.tiles - t_first) < a.tpc ? (a.tiles - t_first) : a.tpc;
  if (warp == MMA_WARPS) {
    if (lane == 0)
      producer_loop_mma(hdr, ring, &map_p, nullptr, t_first, 1, t_count, a.stages, a.stage_bytes, TWA_TILE_COL_BYTES / 8 * KT, 0, 0,
                        0, 0, a.tx_bytes, true, a.status, a.wait_limit_ns);
    return;
  }
  if (warp > MMA_WARPS) {
    helper_loop<BITS, KT, 4>(hdr, ring, a.stage_bytes, a.aux_off, a.stages, t_first, t_count, true, a.gran, a.base,
                             a.D, reinterpret_cast<int4*>(smem + a.ering_off), lane, a.status, a.wait_limit_ns);
    return;
  }
  const int lm = lane >> 3, lr = lane & 7;
  const int jmax = a.n - 1;
  constexpr int col_bytes = TWA_TILE_COL_BYTES * KT;
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
        loff[u][ch][ks] = static_cast<uint32_t>(j * col_bytes + ((chunk >> 5) << 9) + (twa_chunk_slot(chunk & 31, j) << 4));
      }
  const int wb = warp * 32 * KT;
  const int gran_in_tile = wb >> 6;
  const int rig0 = (wb & 63) * 8 / BITS;
  const unsigned seg_off_loose = a.aux_off + 8 * KT * 16 + gran_in_tile * segment_bytes(BITS);
  const unsigned seg_off_packed = a.aux_off + 8 * KT * 16 + gran_in_tile * granule_rows(BITS) * 4;
  // rows (inside the granule) this lane finishes for block u: chunk tig, LROWS rows from LROWS * gid
  int rrow[KT];
#pragma unroll
  for (int u = 0; u < KT; ++u) rrow[u] = rig0 + u * RB + 16 * tig * (8 / BITS) + LROWS * gid;

  uint32_t bfrag[KS][2];
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) bfrag[ks][0] = bfrag[ks][1] = 0u;
  float wbw = 0.0f, kon = 0.0f;
  int cur_layer = -1;
  volatile int* abort_flag = &hdr->abort_flag;
  int s = 0;
  unsigned phase = 0;
  for (int k = 0; k < t_count; ++k) {                   // backwards, like the producer
    if (!twa_mbar_wait(twa_smem_u32(&hdr->full[s]), phase, abort_flag, a.wait_limit_ns)) {
      twa_set_status(a.status, TWA_ERR_TIMEOUT, -1);
      break;
    }
    const unsigned char* st = ring + static_cast<size_t>(s) * a.stage_bytes;
    const int4* entries = reinterpret_cast<const int4*>(st + a.aux_off);
    const int4 e = entries[gran_in_tile];
    const unsigned seg_off = (a.base && tile_is_packed<BITS, KT, 4>(entries, a.base)) ? seg_off_packed : seg_off_loose;
    const float* gs = reinterpret_cast<const float*>(st + seg_off);        // the granule's rows of base, staged
    // only lanes tig 0, 1 finish rows: the other two would read the same banks a chunk further on
    // (four-way conflicts on every such load)
    float bv[KT][LROWS];
#pragma unroll
    for (int u = 0; u < KT; ++u) {
      if (!a.base || tig >= 2) {
#pragma unroll
        for (int i = 0; i < LROWS; ++i) bv[u][i] = 0.0f;
      } else if (LROWS == 2) {
        const float2 x = *reinterpret_cast<const float2*>(gs + rrow[u]);
        bv[u][0] = x.x; bv[u][1] = x.y;
      } else {
#pragma unroll
        for (int v4 = 0; v4 < LROWS / 4; ++v4) {
          const float4 x = *reinterpret_cast<const float4*>(gs + rrow[u] + 4 * v4);
          bv[u][4 * v4] = x.x; bv[u][4 * v4 + 1] = x.y; bv[u][4 * v4 + 2] = x.z; bv[u][4 * v4 + 3] = x.w;
        }
      }
    }
    if (e.x != cur_layer && e.x >= 0) {                  // new layer: its digit fragments and factors
      cur_layer = e.x;
      const int eb = a.ebits[cur_layer];
      const float w0 = eb <= 0 ? 0.0f : (eb >= 6 ? __uint_as_float(static_cast<uint32_t>(eb - 5) << 23) : 5.877471754e-39f);
      const float w1 = w0 * 0.0078125f, w2 = w1 * 0.0078125f, w3 = w2 * 0.0078125f;
      wbw = tig == 0 ? w1 : (tig == 1 ? w3 : 0.0f);      // weight of the lower digit of this lane's pair
      if (BITS == 4) wbw *= 0.0625f;                     // 4-bit codes enter the MMA times 16
      kon = eb < 0 ? __int_as_float(0x7FC00000) : a.konst[cur_layer];
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        bfrag[ks][0] = bfrag[ks][1] = 0u;
        if (gid < 4) {
          const unsigned char* tk = a.dig + static_cast<size_t>(cur_layer) * 512 + gid * 128 + ks * 32 + 2 * tig;
          bfrag[ks][0] = static_cast<uint32_t>(*reinterpret_cast<const unsigned short*>(tk)) |
                         (static_cast<uint32_t>(*reinterpret_cast<const unsigned short*>(tk + 8)) << 16);
          bfrag[ks][1] = static_cast<uint32_t>(*reinterpret_cast<const unsigned short*>(tk + 16)) |
                         (static_cast<uint32_t>(*reinterpret_cast<const unsigned short*>(tk + 24)) << 16);
        }
      }
    }
    const uint32_t tile_base = twa_smem_u32(st);
    float keep[KT][LROWS];
#pragma unroll
    for (int u = 0; u < KT; ++u) {
#pragma unroll
      for (int i = 0; i < LROWS; ++i) keep[u][i] = 0.0f;
      if (e.x >= 0) {
#pragma unroll
        for (int grp = 0; grp < NG; ++grp) {              // code slots grp * SG .. grp * SG + SG - 1 of every byte
          float v[2][2 * SG];                             // per 16-byte chunk of the block
#pragma unroll
          for (int ch = 0; ch < 2; ++ch) {
            // acc[q]: (c0, c1) row SUB * (2 gid) + slot, (c2, c3) row SUB * (2 gid + 1) + slot
            int acc[SG][4];
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
              uint32_t r[4];
              ldmatrix_x4_trans(tile_base + loff[u][ch][ks], r);
              // the transposing load delivers byte pairs of two columns: regroup to four columns per register
              const uint32_t af[4] = {__byte_perm(r[0], r[1], 0x6420), __byte_perm(r[0], r[1], 0x7531),
                                      __byte_perm(r[2], r[3], 0x6420), __byte_perm(r[2], r[3], 0x7531)};
              if (BITS == 8) {
                if (ks == 0) mma_u8s8_first(acc[0], af, bfrag[ks][0], bfrag[ks][1]);
                else mma_u8s8(acc[0], af, bfrag[ks][0], bfrag[ks][1]);
              } else if (BITS == 4) {
                uint32_t ae[4], ao[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  ae[i] = (af[i] << 4) & 0xF0F0F0F0u;     // even rows: 16 * code, unsigned
                  ao[i] = af[i] & 0xF0F0F0F0u;            // odd rows
                }
                if (ks == 0) {
                  mma_u8s8_first(acc[0], ae, bfrag[ks][0], bfrag[ks][1]);
                  mma_u8s8_first(acc[SG - 1], ao, bfrag[ks][0], bfrag[ks][1]);
                } else {
                  mma_u8s8(acc[0], ae, bfrag[ks][0], bfrag[ks][1]);
                  mma_u8s8(acc[SG - 1], ao, bfrag[ks][0], bfrag[ks][1]);
                }
              } else {
                constexpr uint32_t MASK = 0x01010101u * ((1u << BITS) - 1u);
#pragma unroll
                for (int q = 0; q < SG; ++q) {
                  uint32_t x[4];
#pragma unroll
                  for (int i = 0; i < 4; ++i) x[i] = (af[i] >> (BITS * (grp * SG + q))) & MASK;
                  if (ks == 0) mma_u8s8_first(acc[q], x, bfrag[ks][0], bfrag[ks][1]);
                  else mma_u8s8(acc[q], x, bfrag[ks][0], bfrag[ks][1]);
                }
              }
            }
            // digit pairs (0,1) in lanes tig = 0, (2,3) in tig = 1
#pragma unroll
            for (int q = 0; q < SG; ++q) {
              v[ch][q] = digit_pair_to_float(acc[q][0], acc[q][1], wbw);
              v[ch][SG + q] = digit_pair_to_float(acc[q][2], acc[q][3], wbw);
            }
          }
          // lane tig = 0 finishes the rows of chunk 0, lane tig = 1 those of chunk 1: each hands the other
          // the digit-pair sums it does not keep
#pragma unroll
          for (int q = 0; q < 2 * SG; ++q) {
            const float mine = (tig & 1) ? v[1][q] : v[0][q];
            const float theirs = (tig & 1) ? v[0][q] : v[1][q];
            // row inside the lane's LROWS: SUB * (q / SG) + slot
            keep[u][SUB * (q / SG) + grp * SG + (q % SG)] = mine + __shfl_xor_sync(0xFFFFFFFFu, theirs, 1);
          }
        }
      }
    }
    __syncwarp();
    if (lane == 0) twa_mbar_arrive(twa_smem_u32(&hdr->empty[s]));
    if (e.x >= 0 && tig < 2) {
      constexpr int VW = LROWS < 4 ? LROWS : 4;            // floats per vector store
      const bool aligned = (e.z & (VW - 1)) == 0 && a.out_vector_ok;      // the lane's rows start on a vector boundary
#pragma unroll
      for (int u = 0; u < KT; ++u) {
        float* dst = a.out + static_cast<long long>(e.z) + rrow[u];
        float r[LROWS];
#pragma unroll
        for (int i = 0; i < LROWS; ++i) r[i] = bv[u][i] + keep[u][i] + kon;
        if (aligned && rrow[u] + LROWS <= e.y) {
          if (LROWS == 2) {
            *reinterpret_cast<float2*>(dst) = make_float2(r[0], r[1]);
          } else {
#pragma unroll
            for (int v4 = 0; v4 < LROWS / 4; ++v4)
              *reinterpret_cast<float4*>(dst + 4 * v4) = make_float4(r[4 * v4], r[4 * v4 + 1], r[4 * v4 + 2], r[4 * v4 + 3]);
          }
        } else {
#pragma unroll
          for (int i = 0; i < LROWS; ++i)
            if (rrow[u] + i < e.y) dst[i] = r[i];
        }
      }
    }
    if (++s == a.stages) {
      s = 0;
      phase ^= 1u;
    }
  }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
// The codes as a 2-D tensor of 8-byte elements {column bytes / 8, n} (a box dimension is limited to 256
// elements; a tile of four 512-byte segments is 256 of these).
int encode_codes_map(twa_ctx* ctx, const twa_basis* P, int kt, CUtensorMap* map) {
  long long row_bytes = (P->D * P->bits + 7) / 8;
  row_bytes = (row_bytes + 511) / 512 * 512;
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(row_bytes / 8), static_cast<cuuint64_t>(P->n)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(P->col_stride)};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(TWA_TILE_COL_BYTES / 8 * kt), static_cast<cuuint32_t>(P->n)};
  cuuint32_t es[2] = {1, 1};
  CUresult r = ctx->encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, P->data, dims, strides, box, es,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(ctx->last_error, sizeof(ctx->last_error), "cuTensorMapEncodeTiled(layered codes) failed: %d",
             static_cast<int>(r));
    return TWA_ERR_CUDA;
  }
  return TWA_OK;
}

struct StepLayout { size_t partials, dig, ebits, konst, total; };
StepLayout step_layout(const twa_layered_basis* lb) {
  StepLayout w;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = (o + bytes + 255) / 256 * 256; return at; };
  w.partials = take(sizeof(float) * static_cast<size_t>(lb->total_runs) * MMA_WARPS * ROW_FLOATS);
  w.dig = take(static_cast<size_t>(lb->L) * 512);
  w.ebits = take(sizeof(int) * lb->L);
  w.konst = take(sizeof(float) * lb->L);
  w.total = o;
  return w;
}

template <int BITS, bool GBF16, int MT>
int launch_lproject_t(twa_ctx* ctx, const CUtensorMap& mp, const LProjectArgs& a, int kt, int grid, int smem) {
  // slots below 4 bits are tiled with one segment only
  auto kern = (BITS >= 4 && kt == 2) ? layered_project_kernel<BITS, GBF16, MT, (BITS >= 4 ? 2 : 1)>
                                     : layered_project_kernel<BITS, GBF16, MT, 1>;
  static int smem_limit[2][64] = {{0}};
  int rc = twa_ensure_smem(ctx, reinterpret_cast<const void*>(kern), &smem_limit[kt - 1][ctx->device & 63], smem);
  if (rc) return rc;
  kern<<<grid, L_THREADS, smem, ctx->stream>>>(mp, a);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}

template <int BITS, bool GBF16>
int launch_lproject(twa_ctx* ctx, const CUtensorMap& mp, const LProjectArgs& a, int kt, int grid, int smem) {
  switch ((a.n + 15) >> 4) {
    case 1: return launch_lproject_t<BITS, GBF16, 1>(ctx, mp, a, kt, grid, smem);
    case 2: return launch_lproject_t<BITS, GBF16, 2>(ctx, mp, a, kt, grid, smem);
    case 3: return launch_lproject_t<BITS, GBF16, 3>(ctx, mp, a, kt, grid, smem);
    case 4: return launch_lproject_t<BITS, GBF16, 4>(ctx, mp, a, kt, grid, smem);
    case 5: return launch_lproject_t<BITS, GBF16, 5>(ctx, mp, a, kt, grid, smem);
    case 6: return launch_lproject_t<BITS, GBF16, 6>(ctx, mp, a, kt, grid, smem);
    case 7: return launch_lproject_t<BITS, GBF16, 7>(ctx, mp, a, kt, grid, smem);
    default: return launch_lproject_t<BITS, GBF16, 8>(ctx, mp, a, kt, grid, smem);
  }
}

template <int BITS, int KS>
int launch_llift_t(twa_ctx* ctx, const CUtensorMap& mp, const LLiftArgs& a, int kt, int grid, int smem) {
  // slots below 4 bits are tiled with one segment only
  auto kern = (BITS >= 4 && kt == 2) ? layered_lift_kernel<BITS, KS, (BITS >= 4 ? 2 : 1)> : layered_lift_kernel<BITS, KS, 1>;
  static int smem_limit[2][64] = {{0}};
  int rc = twa_ensure_smem(ctx, reinterpret_cast<const void*>(kern), &smem_limit[kt - 1][ctx->device & 63], smem);
  if (rc) return rc;
  kern<<<grid, L_THREADS, smem, ctx->stream>>>(mp, a);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}

template <int BITS>
int launch_llift(twa_ctx* ctx, const CUtensorMap& mp, const LLiftArgs& a, int kt, int grid, int smem) {
  switch ((a.n + 31) >> 5) {
    case 1: return launch_llift_t<BITS, 1>(ctx, mp, a, kt, grid, smem);
    case 2: return launch_llift_t<BITS, 2>(ctx, mp, a, kt, grid, smem);
    case 3: return launch_llift_t<BITS, 3>(ctx, mp, a, kt, grid, smem);
    default: return launch_llift_t<BITS, 4>(ctx, mp, a, kt, grid, smem);
  }
}

int stage_count(const twa_ctx* ctx, int fixed, int stage_bytes) {
  int s = (ctx->smem_optin - fixed) / stage_bytes;
  if (s > TWA_MAX_STAGES) s = TWA_MAX_STAGES;
  return s;
}

int do_project(twa_ctx* ctx, const twa_layered_basis* lb, const void* g, twa_dtype g_dtype, float* c_out,
               float* beta, float lr, float lambda, const twa_adam_args& adam, bool with_digits, char* sws) {
  const StepLayout w = step_layout(lb);
  const int n = lb->codes.n, kt = lb->kt;
  CUtensorMap mp;
  int rc = encode_codes_map(ctx, &lb->codes, kt, &mp);
  if (rc) return rc;
  LProjectArgs a;
  a.n = n;
  a.tiles = lb->tiles;
  a.tpc = lb->tiles_per_cta;
  a.D = lb->D;
  a.tx_bytes = static_cast<unsigned>(n) * TWA_TILE_COL_BYTES * kt;
  a.aux_off = a.tx_bytes;
  a.stage_bytes = (a.aux_off + aux_bytes(lb->codes.bits, kt) + 1023) / 1024 * 1024;
  a.stages = stage_count(ctx, TWA_SMEM_HEADER + MMA_WARPS * digit_scratch(lb->codes.bits) + ENTRY_RING_BYTES + 1024,
                         static_cast<int>(a.stage_bytes));
  if (a.stages < 2) return TWA_ERR_UNSUPPORTED;
  a.scratch_off = TWA_SMEM_HEADER + static_cast<unsigned>(a.stages) * a.stage_bytes;
  a.ering_off = a.scratch_off + MMA_WARPS * digit_scratch(lb->codes.bits);
  a.gran = reinterpret_cast<const int4*>(lb->granules);
  a.g = g;
  a.cta_first = lb->cta_first_layer;
  a.cta_base = lb->cta_run_base;
  a.partials = reinterpret_cast<float*>(sws + w.partials);
  a.status = ctx->d_status;
  a.wait_limit_ns = ctx->wait_limit_ns;
  const int smem = static_cast<int>(a.ering_off) + ENTRY_RING_BYTES + 1024;
  const bool bf16 = g_dtype == TWA_BF16;
  switch (lb->codes.bits) {
    case 8: rc = bf16 ? launch_lproject<8, true>(ctx, mp, a, kt, lb->cta_count, smem)
                      : launch_lproject<8, false>(ctx, mp, a, kt, lb->cta_count, smem); break;
    case 4: rc = bf16 ? launch_lproject<4, true>(ctx, mp, a, kt, lb->cta_count, smem)
                      : launch_lproject<4, false>(ctx, mp, a, kt, lb->cta_count, smem); break;
    case 2: rc = bf16 ? launch_lproject<2, true>(ctx, mp, a, kt, lb->cta_count, smem)
                      : launch_lproject<2, false>(ctx, mp, a, kt, lb->cta_count, smem); break;
    default: rc = bf16 ? launch_lproject<1, true>(ctx, mp, a, kt, lb->cta_count, smem)
                       : launch_lproject<1, false>(ctx, mp, a, kt, lb->cta_count, smem); break;
  }
  if (rc) return rc;
  const int planes = lb->planes == 2 ? 2 : 1;
  layered_combine_kernel<<<lb->L, 128 * COMBINE_PARTS, 0, ctx->stream>>>(
      a.partials, lb->cta_first_layer, lb->cta_run_base, lb->cta_count, n / planes, planes, lb->a, lb->b, c_out, beta, lr, lambda,
      adam, with_digits ? reinterpret_cast<unsigned char*>(sws + w.dig) : nullptr, reinterpret_cast<int*>(sws + w.ebits),
      reinterpret_cast<float*>(sws + w.konst), ctx->d_status);
  TWA_CUDA_OK(ctx, cudaGetLastError());
  return TWA_OK;
}

int do_lift(twa_ctx* ctx, const twa_layered_basis* lb, const float* beta, const float* base, float* out,
            bool digits_ready, char* sws) {
  const StepLayout w = step_layout(lb);
  const int n = lb->codes.n;
  // (One or two segments per tile, as fixed when the basis was quantised: a warp's share of a tile, 32 * KT bytes
  // of every column, must lie inside one 64-byte granule, i.e. inside one layer.)
  const int kt = lb->kt;
  const int tiles = lb->tiles, tpc = lb->tiles_per_cta;
  unsigned char* dig = reinterpret_cast<unsigned char*>(sws + w.dig);
  int* ebits = reinterpret_cast<int*>(sws + w.ebits);
  float* konst = reinterpret_cast<float*>(sws + w.konst);
  if (!digits_ready) {
    const int planes = lb->planes == 2 ? 2 : 1;
    layered_coef_kernel<<<lb->L, 128, 0, ctx->stream>>>(beta, n / planes, planes, lb->a, lb->b, dig, ebits, konst,
                                                        ctx->d_status);
    TWA_CUDA_OK(ctx, cudaGetLastError());
  }
  CUtensorMap mp;
  int rc = encode_codes_map(ctx, &lb->codes, kt, &mp);
  if (rc) return rc;
  LLiftArgs a;
  a.n = n;
  a.tiles = tiles;
  a.tpc = tpc;
  a.D = lb->D;
  a.tx_bytes = static_cast<unsigned>(n) * TWA_TILE_COL_BYTES * kt;
  a.aux_off = a.tx_bytes;
  a.stage_bytes = (a.aux_off + aux_bytes(lb->codes.bits, kt) + 1023) / 1024 * 1024;
  a.stages = stage_count(ctx, TWA_SMEM_HEADER + ENTRY_RING_BYTES + 1024, static_cast<int>(a.stage_bytes));
  if (a.stages < 2) return TWA_ERR_UNSUPPORTED;
  a.ering_off = TWA_SMEM_HEADER + static_cast<unsigned>(a.stages) * a.stage_bytes;
  a.gran = reinterpret_cast<const int4*>(lb->granules);
  a.dig = dig;
  a.ebits = ebits;
  a.konst = konst;
  a.base = base;
  a.out = out;
  a.out_vector_ok = (reinterpret_cast<uintptr_t>(out) & 15) == 0;
  a.status = ctx->d_status;
  a.wait_limit_ns = ctx->wait_limit_ns;
  const int smem = static_cast<int>(a.ering_off) + ENTRY_RING_BYTES + 1024;
  switch (lb->codes.bits) {
    case 8: return launch_llift<8>(ctx, mp, a, kt, lb->cta_count, smem);
    case 4: return launch_llift<4>(ctx, mp, a, kt, lb->cta_count, smem);
    case 2: return launch_llift<2>(ctx, mp, a, kt, lb->cta_count, smem);
    default: return launch_llift<1>(ctx, mp, a, kt, lb->cta_count, smem);
  }
}

int check_step_args(twa_ctx* ctx, const twa_layered_basis* lb, const void* sws, size_t sws_bytes) {
  if (!ctx || !lb || !lb->codes.data || !lb->a || !lb->b || !lb->granules || !lb->cta_first_layer ||
      !lb->cta_run_base)
    return TWA_ERR_INVALID_ARG;
  const int wb = lb->codes.bits;
  if (wb != 8 && wb != 4 && wb != 2 && wb != 1) return TWA_ERR_UNSUPPORTED;
  if (lb->codes.n < 1 || lb->codes.n > TWA_MAX_N || lb->L < 1 || lb->cta_count < 1 || (lb->kt != 1 && lb->kt != 2) ||
      (wb < 4 && lb->kt != 1) || (lb->planes == 2 && (lb->codes.n & 1)))
    return TWA_ERR_INVALID_ARG;
  if (!sws || sws_bytes < step_layout(lb).total) return TWA_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(sws) & 255) return TWA_ERR_MISALIGNED;
  return TWA_OK;
}

}  // namespace

extern "C" {

size_t twa_layered_step_workspace_bytes(const twa_layered_basis* lb) {
  if (!lb || lb->L < 1 || lb->total_runs < 1) return 0;
  return step_layout(lb).total;
}

int twa_layered_project(twa_ctx* ctx, const twa_layered_basis* lb, const void* g, twa_dtype g_dtype,
                        float* c_out, void* sws, size_t sws_bytes) {
  int rc = check_step_args(ctx, lb, sws, sws_bytes);
  if (rc) return rc;
  if (!g || !c_out || (g_dtype != TWA_F32 && g_dtype != TWA_BF16)) return TWA_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(g) & 3) return TWA_ERR_MISALIGNED;         // staged in 4-byte words
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  return do_project(ctx, lb, g, g_dtype, c_out, nullptr, 0.0f, 0.0f, twa_adam_args{}, false, static_cast<char*>(sws));
}

int twa_layered_lift(twa_ctx* ctx, const twa_layered_basis* lb, const float* beta, const float* base,
                     float* w_out, void* sws, size_t sws_bytes) {
  int rc = check_step_args(ctx, lb, sws, sws_bytes);
  if (rc) return rc;
  if (!beta || !w_out) return TWA_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(base) & 3) || (reinterpret_cast<uintptr_t>(w_out) & 3)) return TWA_ERR_MISALIGNED;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  return do_lift(ctx, lb, beta, base, w_out, false, static_cast<char*>(sws));
}

static int layered_step_impl(twa_ctx* ctx, const twa_layered_basis* lb, const void* g, twa_dtype g_dtype, float lr,
                             float lambda, const twa_adam_args& adam, float* beta, const float* wbar, float* w,
                             float* c_out, void* sws, size_t sws_bytes) {
  int rc = check_step_args(ctx, lb, sws, sws_bytes);
  if (rc) return rc;
  if (!g || !beta || !wbar || !w || (g_dtype != TWA_F32 && g_dtype != TWA_BF16)) return TWA_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(g) & 3) || (reinterpret_cast<uintptr_t>(wbar) & 3) ||
      (reinterpret_cast<uintptr_t>(w) & 3))
    return TWA_ERR_MISALIGNED;
  TWA_CUDA_OK(ctx, cudaSetDevice(ctx->device));
  rc = do_project(ctx, lb, g, g_dtype, c_out, beta, lr, lambda, adam, true, static_cast<char*>(sws));
  if (rc) return rc;
  return do_lift(ctx, lb, beta, wbar, w, true, static_cast<char*>(sws));
}

int twa_layered_step(twa_ctx* ctx, const twa_layered_basis* lb, const void* g, twa_dtype g_dtype, float lr,
                     float lambda, float* beta, const float* wbar, float* w, float* c_out, void* sws,
                     size_t sws_bytes) {
  return layered_step_impl(ctx, lb, g, g_dtype, lr, lambda, twa_adam_args{}, beta, wbar, w, c_out, sws, sws_bytes);
}

int twa_layered_step_adam(twa_ctx* ctx, const twa_layered_basis* lb, const void* g, twa_dtype g_dtype,
                          const twa_adam* opt, float* beta, float* m, float* v, const float* wbar, float* w,
                          float* c_out, void* sws, size_t sws_bytes) {
  twa_adam_args ad;
  int rc = twa_adam_device_args(opt, m, v, &ad);
  if (rc) return rc;
  return layered_step_impl(ctx, lb, g, g_dtype, opt->lr, opt->weight_decay, ad, beta, wbar, w, c_out, sws, sws_bytes);
}

}  // extern "C"
