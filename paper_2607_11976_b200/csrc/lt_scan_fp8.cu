// Alternative FP8 (e4m3) tensor-core scan kernel of the fused indexer top-k (sm_100a: TMA -> shared -> tcgen05.mma
// -> TMEM), selected with lt_tunables.path = LT_PATH_FUSED_ABS.  It is exact like the default kernel and, as
// measured, slower (three epilogue warps per scheduler instead of four); it is kept as the measured record of the
// only instruction selection that undercuts the default kernel's register-read bound.
//
// Eq. 1 of the paper, I[t, s] = k_scale[s] * sum_h w[t, h] * ReLU(x[t, h, s]) with x = q[t, h] . k[s], is
// evaluated here through the identity ReLU(x) = (x + |x|) / 2:
//
//     I[t, s] = k_scale[s] * ( sum_h (w[t, h] / 2) * |x[t, h, s]|  +  (1/2) * (sum_h w[t, h] q[t, h]) . k[s] ).
//
// The first sum costs ONE CUDA-core instruction per tensor-core accumulator (an FMA whose operand carries
// an absolute-value modifier) instead of two (max, then FMA): the paper's Sec. 3.2 "Filtering" observes that
// this CUDA-core finalisation is what the score's latency consists of.  The second term is linear in k[s],
// so the tensor core computes it as kLinTerms extra accumulator columns per query: a pre-pass
// (lin_terms_kernel) forms qlin[t] = sum_h w[t, h] q[t, h] in fp64 and splits it into kLinTerms e4m3
// vectors with power-of-two scales, qlin ~= sum_j scale[t][j] * c[t][j], residual <= 2^-20 of each element.
//
// One CTA keeps a block of 6 query rows resident in shared memory (two units of 3 queries: 192 head rows +
// 15 linear-term rows, padded to 208 operand rows each) and streams 128-key tiles of K past it.  Per key tile
// it issues two 128 x 208 x 128 UMMAs into two TMEM buffers; lanes index keys and columns index (query,
// head), so each epilogue thread owns one key and finishes the sums above as an in-thread chain of packed
// FMAs over TMEM columns.
//
//   kMode == kModeFilter  paper Sec. 3.2 "Filtering": gate the score against the row's threshold edge,
//                         ballot-compact the survivors of each warp into a staging list; a flush appends the
//                         list to the row's candidate buffer and counts its entries in the row's bin
//                         histogram; a spare warp re-derives the threshold bin from the histogram while the
//                         scan runs ("Threshold Refresh") and publishes it by plain store.
//   kMode == kModeDump    write every score (or -inf where masked) to a dense matrix: used for the sample
//                         phase, lt_indexer_scores, the unfused baseline and the exact fallback.
//
// Warp roles (480 threads): 0 TMA producer, 1 UMMA issuer (+ TMEM owner), 2 threshold refresh, 3..14
// epilogue.  Epilogue warp (lane quarter, g) finishes query g of unit 0 and then query g of unit 1 of every
// key tile for its 32 keys.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "lt_common.cuh"
#include "lt_host.h"
#include "lt_ptx.cuh"

namespace lt {

using namespace ptx;

namespace {

constexpr int kH = 64;
constexpr int kD = 128;
constexpr int kBlockQ = kRowsPerBlockFp8;   // query rows resident per CTA
constexpr int kUnitQ = 3;                   // query rows per UMMA
constexpr int kUnits = kBlockQ / kUnitQ;    // UMMAs per key tile = TMEM buffers
constexpr int kJ = kLinTerms;               // e4m3 terms of the linear part of one query
constexpr int kHeadRows = kUnitQ * kH;      // 192 operand rows (q[t][h]) of a unit
constexpr int kLinRows = 16;                // 15 linear-term rows of a unit + 1 unused
constexpr int kUmmaN = kHeadRows + kLinRows;  // 208
constexpr int kBufCols = 256;               // TMEM columns between the two accumulators
constexpr int kTmemCols = 512;
constexpr int kFirstEpiWarp = 3;
constexpr int kEpiWarps = 4 * kUnitQ;       // (lane quarter, query of the unit)
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kThreads = kFirstEpiWarp * 32 + kEpiThreads;
constexpr int kStageBytes = 128 * 128;      // one key tile: 128 rows x 128-byte swizzled rows
constexpr int kQTile = kUmmaN * 128;        // bytes of one unit's operand rows
constexpr int kQBytes = kUnits * kQTile;
constexpr int kStages = 9;                  // K-tile ring depth
constexpr int kSmemTiles = kQBytes + kStages * kStageBytes;
constexpr int kStageLen = 64;               // entries of one per-warp staging list
constexpr int kRowWBytes = kH * 4;          // bytes between the weights of consecutive rows of the block
constexpr int kRowLBytes = kLinScaleStride * 4;

static_assert(kBlockQ == kUnits * kUnitQ, "block = two units");
static_assert(kUnitQ * kJ <= kLinRows, "linear-term rows of a unit");
static_assert(kUmmaN % 16 == 0 && kUmmaN <= 256, "UMMA N");
static_assert(kQTile % 1024 == 0, "operand tiles stay 1024-byte aligned");

struct SmemTail {
  float w[kBlockQ * kH];                    // w / 2
  float lsc[kBlockQ * kLinScaleStride];     // scale of linear term j / 2
  float thr[8];
  float smin[8];
  float width[8];
  float inv_width[8];
  int vis[8];
  int dump_row[8];
  uint64_t bar_full[kStages];
  uint64_t bar_empty[kStages];
  uint64_t bar_q_full;
  uint64_t bar_q_empty;
  uint64_t bar_tmem_full[2];
  uint64_t bar_tmem_empty[2];
  uint32_t tmem_base;
  int abort_flag;     // [0] raised by a wait that ran out; every role unwinds on it
  int wait_limit_us;  // [1] bound of every wait (read by mbar_wait through the flag's address)
  int epi_abort;
  int done_seq;
  uint2 stage[kEpiWarps][kUnits][kStageLen];  // per warp and unit: (score bits, key index) of survivors
};

constexpr int smem_bytes() { return 1024 + kSmemTiles + static_cast<int>(sizeof(SmemTail)); }
static_assert(smem_bytes() <= 227 * 1024, "shared memory budget");

struct Item {
  int t0;        // first query row of the block
  int tile_lo;   // key tiles [tile_lo, tile_hi)
  int tile_hi;
  int slot;      // dump slot (fallback mode) or block number
};

// Work items are (key segment, query block) pairs, segment-major, so that CTAs running side by
// side stream the same part of K (L2 reuse) for different query blocks.
__device__ __forceinline__ bool resolve_item(const ScanParams& p, int n_blocks, int item, Item& it) {
  int seg = item / n_blocks;
  int qb = item - seg * n_blocks;
  int last_row;
  if (p.fb_list != nullptr) {
    it.t0 = p.fb_list[p.fb_round_base + qb] * kBlockQ;
    it.slot = qb;
    last_row = min(it.t0 + kBlockQ, p.T) - 1;
  } else {
    it.t0 = p.row_begin + qb * kBlockQ;
    it.slot = qb;
    last_row = min(it.t0 + kBlockQ, p.row_end) - 1;
  }
  int n_tiles = (p.n_keys + kTileKeys - 1) / kTileKeys;
  if (p.skip_masked_tiles) {
    int vis = visible_keys(last_row, p.n_keys, p.causal_offset);
    n_tiles = (vis + kTileKeys - 1) / kTileKeys;
  }
  it.tile_lo = seg * p.seg_tiles;
  it.tile_hi = min(it.tile_lo + p.seg_tiles, n_tiles);
  return it.tile_lo < it.tile_hi;
}

// Where the scale of view key s lives: at s * ks_stride, or with a paged key cache at the key's physical row.
template <bool kPaged>
__device__ __forceinline__ size_t scale_index(const ScanParams& p, int s) {
  if (kPaged) {
    long long phys = __ldg(p.page_table + (s / kPageKeys));
    if (!LT_IN_BOUNDS(phys >= 0 && phys < p.pool_pages, p.ctl)) phys = 0;  // a page-table entry outside the pool
    return static_cast<size_t>(phys) * kPageKeys + static_cast<size_t>(s % kPageKeys);
  }
  return static_cast<size_t>(s) * p.ks_stride;
}

// ---- the score of one key against one query ----------------------------------------------------
// 64 TMEM columns (per-head dots x_h) and kJ linear-term columns y_j ->
//     score = ks * ( sum_h wh[h] * |x_h| + sum_j ls[j] * y_j ),   wh = w / 2, ls = scale / 2.
// Head h lands in packed accumulator (h / 2) % 4, lane h % 2; finish() fixes the order of the final
// additions.  These functions produce every fp8 score the library ranks or dumps on the tensor-core
// path, so fused, dumped and fallback scores agree bit for bit.
struct Acc8 {
  uint64_t p[4];
};
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
// acc (+)= w * |x| for two heads at once.  The absolute value is taken in place on the two registers the
// TMEM load filled (they stay an aligned register pair); the assembler folds it into the FMA's operand.
template <bool kFirst>
__device__ __forceinline__ void abs_fma2(uint64_t& acc, uint64_t w, uint32_t& x0, uint32_t& x1) {
  asm("abs.f32 %0, %0;" : "+r"(x0));
  asm("abs.f32 %0, %0;" : "+r"(x1));
  if (kFirst) {
    asm("{\n.reg .b64 x;\nmov.b64 x, {%1, %2};\nmul.rn.f32x2 %0, %3, x;\n}\n" : "=l"(acc) : "r"(x0), "r"(x1), "l"(w));
  } else {
    asm("{\n.reg .b64 x;\nmov.b64 x, {%1, %2};\nfma.rn.f32x2 %0, %3, x, %0;\n}\n" : "+l"(acc) : "r"(x0), "r"(x1), "l"(w));
  }
}
// Eight heads starting at column J of a 32-column piece.  kOff: byte offset of the piece's weights
// from w_addr, folded into the load instructions as an immediate.
template <bool kFirst, int kOff, int J>
__device__ __forceinline__ void head_sum8(uint32_t (&v)[32], uint32_t w_addr, Acc8& acc) {
  uint64_t w01, w23, w45, w67;
  asm volatile("ld.shared.v2.b64 {%0, %1}, [%2+%3];" : "=l"(w01), "=l"(w23) : "r"(w_addr), "n"(kOff + J * 4));
  asm volatile("ld.shared.v2.b64 {%0, %1}, [%2+%3];" : "=l"(w45), "=l"(w67) : "r"(w_addr), "n"(kOff + J * 4 + 16));
  constexpr bool first = kFirst && J == 0;
  abs_fma2<first>(acc.p[0], w01, v[J + 0], v[J + 1]);
  abs_fma2<first>(acc.p[1], w23, v[J + 2], v[J + 3]);
  abs_fma2<first>(acc.p[2], w45, v[J + 4], v[J + 5]);
  abs_fma2<first>(acc.p[3], w67, v[J + 6], v[J + 7]);
}
template <bool kFirst, int kOff>
__device__ __forceinline__ void head_sum32(uint32_t (&v)[32], uint32_t w_addr, Acc8& acc) {
  head_sum8<kFirst, kOff, 0>(v, w_addr, acc);
  head_sum8<kFirst, kOff, 8>(v, w_addr, acc);
  head_sum8<kFirst, kOff, 16>(v, w_addr, acc);
  head_sum8<kFirst, kOff, 24>(v, w_addr, acc);
}
// sum_j ls[j] * y_j over the kJ linear-term columns (y holds 8 columns, the last 8 - kJ are not this query's)
template <int kOff>
__device__ __forceinline__ float lin_sum(const uint32_t (&y)[8], uint32_t l_addr) {
  float l0, l1, l2, l3, l4;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4+%5];" : "=f"(l0), "=f"(l1), "=f"(l2), "=f"(l3) : "r"(l_addr), "n"(kOff));
  asm volatile("ld.shared.f32 %0, [%1+%2];" : "=f"(l4) : "r"(l_addr), "n"(kOff + 16));
  static_assert(kJ == 5, "lin_sum is written for five terms");
  float s = l0 * __uint_as_float(y[0]);
  s = __fmaf_rn(l1, __uint_as_float(y[1]), s);
  s = __fmaf_rn(l2, __uint_as_float(y[2]), s);
  s = __fmaf_rn(l3, __uint_as_float(y[3]), s);
  s = __fmaf_rn(l4, __uint_as_float(y[4]), s);
  return s;
}
__device__ __forceinline__ float finish(const Acc8& acc, float lin, float ks) {
  uint64_t ab, cd, all;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(ab) : "l"(acc.p[0]), "l"(acc.p[1]));
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(cd) : "l"(acc.p[2]), "l"(acc.p[3]));
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(all) : "l"(ab), "l"(cd));
  float lo, hi;
  unpack2(all, lo, hi);
  return __fmaf_rn((lo + hi) + lin, ks, 0.f);  // the + 0 turns -0 into +0
}

// 32 lanes x 8 consecutive fp32 columns
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&v)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
               : "r"(taddr)
               : "memory");
}

// Flush one staging list: reserve room in the row's candidate buffer with a single atomic, copy the
// entries out with all lanes and count each of them in the row's histogram (fire-and-forget
// atomics).  Doing the bin arithmetic here, 32 entries at a time, keeps it out of the per-tile path;
// the refresh warp merely sees the counts a little later, which can only leave the gate looser.
// Entries beyond the capacity are dropped but still counted, and the tail counter runs past the
// capacity, which is how the final select learns that the row overflowed.
__device__ __forceinline__ void flush_stage(const uint2* list, int count, const ScanParams& p, int t, int lane, float smin,
                                            float width, float inv_width) {
  __syncwarp();
  uint32_t base = 0;
  if (lane == 0) base = atomicAdd(p.tail + t, static_cast<uint32_t>(count));
  base = __shfl_sync(0xffffffffu, base, 0);
  unsigned int* hist = p.hist + static_cast<size_t>(t) * kBins;
  uint2* cand = p.cand + static_cast<size_t>(t) * p.cap;
  for (int i = lane; i < count; i += 32) {
    const uint2 e = list[i];
    const uint32_t pos = base + i;
    if (pos < static_cast<uint32_t>(p.cap) && LT_IN_BOUNDS(t >= 0 && t < p.T && e.y < static_cast<uint32_t>(p.n_keys), p.ctl))
      cand[pos] = e;
    const int bin = bin_of(__uint_as_float(e.x), smin, width, inv_width);
    if (LT_IN_BOUNDS(bin >= 0 && bin < kBins && t >= 0 && t < p.T, p.ctl)) atomicAdd(hist + bin, 1u);
  }
  __syncwarp();
}

template <int kMode, bool kPaged>
__global__ void __launch_bounds__(kThreads, 1)
scan_fp8_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_l,
                const __grid_constant__ CUtensorMap tm_k, const ScanParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
  uint8_t* smem = smem_raw + pad;
  const uint32_t q_base = raw_addr + pad;
  const uint32_t k_base = q_base + kQBytes;
  SmemTail* st = reinterpret_cast<SmemTail*>(smem + kSmemTiles);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  // a fallback round with no flagged block left has nothing to do (uniform across the CTA)
  if (p.fb_list != nullptr && *p.fb_blocks <= p.fb_round_base) return;

  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) {
      mbar_init(smem_u32(&st->bar_full[i]), 1);
      mbar_init(smem_u32(&st->bar_empty[i]), 1);
    }
    mbar_init(smem_u32(&st->bar_q_full), 1);
    mbar_init(smem_u32(&st->bar_q_empty), 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&st->bar_tmem_full[i]), 1);
      mbar_init(smem_u32(&st->bar_tmem_empty[i]), kEpiWarps);
    }
    st->abort_flag = 0;
    st->wait_limit_us = static_cast<int>(p.wait_limit_us);
    st->epi_abort = 0;
    st->done_seq = 0;
    fence_mbar_init();
    prefetch_tensormap(&tm_q);
    prefetch_tensormap(&tm_l);
    prefetch_tensormap(&tm_k);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&st->tmem_base), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = st->tmem_base;
  volatile int* abort_flag = &st->abort_flag;

  // number of query blocks / items of this launch
  int n_blocks;
  if (p.fb_list != nullptr) {
    int avail = *p.fb_blocks - p.fb_round_base;
    n_blocks = avail < 0 ? 0 : (avail > p.fb_slots ? p.fb_slots : avail);
  } else {
    n_blocks = (p.row_end - p.row_begin + kBlockQ - 1) / kBlockQ;
  }
  const int n_tiles_all = (p.n_keys + kTileKeys - 1) / kTileKeys;
  const int n_seg = (n_tiles_all + p.seg_tiles - 1) / p.seg_tiles;
  const int n_items = n_blocks * n_seg;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      uint32_t n_done = 0;  // items issued so far (parity of the Q-block handshake)
      bool ok = true;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
        Item it;
        if (!resolve_item(p, n_blocks, item, it)) continue;
        // query block: wait until the UMMAs of the previous item no longer read it
        ok = mbar_wait<40>(smem_u32(&st->bar_q_empty), (n_done & 1) ^ 1, abort_flag);
        if (!ok) break;
        mbar_arrive_expect_tx(smem_u32(&st->bar_q_full), kQBytes);
        for (int u = 0; u < kUnits; ++u) {
          // 192 rows q[t][h] of the unit's three queries, then their 15 linear-term rows (+ 1 row nobody reads)
          tma_load_2d(q_base + u * kQTile, &tm_q, 0, (it.t0 + u * kUnitQ) * kH, smem_u32(&st->bar_q_full));
          tma_load_2d(q_base + u * kQTile + kHeadRows * 128, &tm_l, 0, (it.t0 + u * kUnitQ) * kJ, smem_u32(&st->bar_q_full));
        }
        ++n_done;
        for (int tile = it.tile_lo; tile < it.tile_hi; ++tile) {
          ok = mbar_wait<40>(smem_u32(&st->bar_empty[stage]), phase ^ 1, abort_flag);
          if (!ok) break;
          mbar_arrive_expect_tx(smem_u32(&st->bar_full[stage]), kStageBytes);
          if (!kPaged) {
            tma_load_2d(k_base + stage * kStageBytes, &tm_k, 0, tile * kTileKeys, smem_u32(&st->bar_full[stage]));
          } else {
            // paged key cache: a tile is two pages of 64 keys, each wherever the page table says (the map's
            // box is then 64 rows); pages past the end of the table are read from page 0 and masked later
            for (int pg = 0; pg < kTileKeys / kPageKeys; ++pg) {
              const int lp = tile * (kTileKeys / kPageKeys) + pg;
              int phys = lp < p.n_pages ? __ldg(p.page_table + lp) : 0;
              if (!LT_IN_BOUNDS(phys >= 0 && phys < p.pool_pages, p.ctl)) phys = 0;  // entry outside the pool
              tma_load_2d(k_base + stage * kStageBytes + pg * kPageKeys * 128, &tm_k, 0, phys * kPageKeys,
                          smem_u32(&st->bar_full[stage]));
            }
          }
          if (++stage == kStages) {
            stage = 0;
            phase ^= 1;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ UMMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(true, kUmmaN);
      int stage = 0;
      uint32_t phase = 0;
      uint32_t acc_phase = 0;  // flips once per key tile: each TMEM buffer is filled once per tile
      uint32_t n_done = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
        Item it;
        if (!resolve_item(p, n_blocks, item, it)) continue;
        ok = mbar_wait<40>(smem_u32(&st->bar_q_full), n_done & 1, abort_flag);
        if (!ok) break;
        ++n_done;
        for (int tile = it.tile_lo; tile < it.tile_hi && ok; ++tile) {
          ok = mbar_wait<40>(smem_u32(&st->bar_full[stage]), phase, abort_flag);
          if (!ok) break;
          for (int u = 0; u < kUnits; ++u) {
            ok = mbar_wait<40>(smem_u32(&st->bar_tmem_empty[u]), acc_phase ^ 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int kb = 0; kb < 4; ++kb) {
              uint64_t a = make_smem_desc_sw128(k_base + stage * kStageBytes) + (kb * 32 >> 4);
              uint64_t b = make_smem_desc_sw128(q_base + u * kQTile) + (kb * 32 >> 4);
              tc_mma<true>(tmem_base + u * kBufCols, a, b, idesc, kb > 0 ? 1u : 0u);
            }
            tc_commit(smem_u32(&st->bar_tmem_full[u]));
          }
          acc_phase ^= 1;
          tc_commit(smem_u32(&st->bar_empty[stage]));
          if (++stage == kStages) {
            stage = 0;
            phase ^= 1;
          }
        }
        tc_commit(smem_u32(&st->bar_q_empty));
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (+ refresh warp)
    const bool is_refresh = (warp == 2);
    const int n_sync = (kMode == kModeFilter) ? kEpiThreads + 32 : kEpiThreads;
    if (!(is_refresh && kMode != kModeFilter)) {
      const int e = threadIdx.x - kFirstEpiWarp * 32;  // epilogue thread number (valid for epilogue warps)
      const int ew = warp - kFirstEpiWarp;             // epilogue warp number
      const int quarter = warp & 3;                    // TMEM lane quarter this warp may read
      const int g = ew >> 2;                           // query g of each unit
      const int key_in_tile = quarter * 32 + lane;
      const uint32_t tlane = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
      const uint32_t tcol = tlane + static_cast<uint32_t>(g * kH);
      const uint32_t tlin = tlane + static_cast<uint32_t>(kHeadRows + g * kJ);
      const uint32_t w_addr = smem_u32(st->w) + g * kRowWBytes;
      const uint32_t l_addr = smem_u32(st->lsc) + g * kRowLBytes;
      uint32_t acc_phase = 0;
      int seq = 0;
      for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
        Item it;
        if (!resolve_item(p, n_blocks, item, it)) continue;
        ++seq;
        named_bar_sync(1, n_sync);  // A: everybody is done with the previous item's shared state
        if (!is_refresh) {
          for (int i = e; i < kBlockQ * kH; i += kEpiThreads) {
            int t = it.t0 + i / kH;
            st->w[i] = (t < p.T) ? 0.5f * p.w[static_cast<size_t>(t) * kH + (i % kH)] : 0.f;
          }
          if (e < kBlockQ * kLinScaleStride) {
            int t = it.t0 + e / kLinScaleStride;
            int j = e % kLinScaleStride;
            st->lsc[e] = (t < p.T && j < kJ) ? 0.5f * p.lin_scale[static_cast<size_t>(t) * kLinScaleStride + j] : 0.f;
          }
          if (e < kBlockQ) {
            int t = it.t0 + e;
            bool live = (p.fb_list != nullptr) ? (t < p.T) : (t < p.row_end);
            st->vis[e] = live ? visible_keys(t, p.n_keys, p.causal_offset) : 0;
            st->dump_row[e] = live ? ((p.fb_list != nullptr) ? it.slot * kBlockQ + e : t - p.row_begin) : -1;
            if (kMode == kModeFilter) {
              st->thr[e] = live ? __ldcg(p.thr + t) : INFINITY;
              st->smin[e] = live ? p.smin[t] : 0.f;
              st->width[e] = live ? p.width[t] : 0.f;
              st->inv_width[e] = (live && p.width[t] > 0.f) ? 1.f / p.width[t] : 0.f;
            }
          }
          if (e == 0) st->epi_abort = *abort_flag;
        }
        named_bar_sync(1, n_sync);  // B: shared state of this item is ready
        if (st->epi_abort) break;

        if (is_refresh) {
          // ---- paper Sec. 3.2 "Threshold Refresh": walk each row's histogram from the top bin
          // down until the cumulative count reaches k; publish the bin's lower edge by plain store.
          // The gate moves fast only while few keys have been seen, so the polling interval grows
          // geometrically (1 us -> 32 us): a stale edge merely admits a few more candidates, while a
          // busy polling warp would take issue slots from the epilogue warps of its scheduler.
          int cur_tb[kBlockQ];
#pragma unroll
          for (int r = 0; r < kBlockQ; ++r) cur_tb[r] = 0;
          unsigned int sleep_ns = 1000;
          while (true) {
#pragma unroll
            for (int r = 0; r < kBlockQ; ++r) {
              int t = it.t0 + r;
              if (t >= p.row_end) continue;
              const uint4* hp = reinterpret_cast<const uint4*>(p.hist + static_cast<size_t>(t) * kBins + lane * 8);
              uint4 h0 = __ldcg(hp), h1 = __ldcg(hp + 1);
              uint32_t c[8] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w};
              uint32_t mine = c[0] + c[1] + c[2] + c[3] + c[4] + c[5] + c[6] + c[7];
              // suffix sum over lanes: above = total count in bins owned by higher lanes
              uint32_t incl = mine;
#pragma unroll
              for (int d = 1; d < 32; d <<= 1) {
                uint32_t o = __shfl_down_sync(0xffffffffu, incl, d);
                if (lane + d < 32) incl += o;
              }
              uint32_t above = incl - mine;
              bool crosses = (above < static_cast<uint32_t>(p.topk)) && (incl >= static_cast<uint32_t>(p.topk));
              uint32_t who = __ballot_sync(0xffffffffu, crosses);
              if (who) {
                int src = __ffs(who) - 1;  // exactly one lane crosses
                int tb = 0;
                if (lane == src) {
                  uint32_t cum = above;
                  for (int j = 7; j >= 0; --j) {
                    cum += c[j];
                    if (cum >= static_cast<uint32_t>(p.topk)) {
                      tb = lane * 8 + j;
                      break;
                    }
                  }
                }
                tb = __shfl_sync(0xffffffffu, tb, src);
                if (tb > cur_tb[r]) {
                  cur_tb[r] = tb;
                  if (lane == 0) {
                    float edge = bin_edge(tb, st->smin[r], st->width[r]);
                    // never lower the gate this CTA already uses (the sample's edge may be higher)
                    if (edge > *reinterpret_cast<volatile float*>(&st->thr[r])) {
                      *reinterpret_cast<volatile float*>(&st->thr[r]) = edge;
                      __stcg(p.thr + t, edge);
                    }
                  }
                }
              }
            }
            // sleep in slices so that the end of the item is noticed quickly; lane 0 decides for the warp
            bool done = false;
            for (unsigned int slept = 0; slept < sleep_ns && !done; slept += 1000) {
              __nanosleep(1000);
              int d = 0;
              if (lane == 0) d = (*reinterpret_cast<volatile int*>(&st->done_seq) >= seq || *abort_flag) ? 1 : 0;
              done = __shfl_sync(0xffffffffu, d, 0) != 0;
            }
            if (done) break;
            if (sleep_ns < 32000) sleep_ns += sleep_ns >> 1;
          }
          continue;
        }

        // ---- epilogue proper: this warp finishes query g of both units for its 32 keys of every tile.
        // Every step with a long fixed latency is issued ahead of its use: the key scale of the
        // next tile and the row threshold are fetched before the arithmetic of the current one.
        int cnt[kUnits] = {0, 0};  // entries in this warp's staging lists (warp-uniform)
        const int vis_first = st->vis[0];
        const bool has_scale = p.k_scale != nullptr;
        bool ok = true;
        float ks_next = 1.f;
        {
          const int s0 = it.tile_lo * kTileKeys + key_in_tile;
          if (has_scale && s0 < p.n_keys) ks_next = __ldg(p.k_scale + scale_index<kPaged>(p, s0));
        }
        for (int tile = it.tile_lo; tile < it.tile_hi && ok; ++tile) {
          const int s = tile * kTileKeys + key_in_tile;
          const float ks = ks_next;
          {
            const int s1 = s + kTileKeys;
            if (has_scale && tile + 1 < it.tile_hi && s1 < p.n_keys)
              ks_next = __ldg(p.k_scale + scale_index<kPaged>(p, s1));
          }
          // keys of this tile that some row of the block may not see (diagonal or ragged last tile)
          const bool partial = (tile + 1) * kTileKeys > vis_first;
#pragma unroll
          for (int u = 0; u < kUnits; ++u) {
            const int r = u * kUnitQ + g;
            float thr = 0.f;
            if (kMode == kModeFilter) thr = *reinterpret_cast<volatile float*>(&st->thr[r]);
            ok = mbar_wait(smem_u32(&st->bar_tmem_full[u]), acc_phase, abort_flag);
            tc_fence_after();
            // the 64 + 8 columns of this query: all loads in flight, one wait.  The loads are issued even
            // after a failed wait (they then fetch values nobody uses): keeping them unconditional
            // keeps the destination registers free of copies.
            uint32_t va[32], vb[32], vl[8];
            tmem_ld32(tcol + u * kBufCols, va);
            tmem_ld32(tcol + u * kBufCols + 32, vb);
            tmem_ld8(tlin + u * kBufCols, vl);
            tmem_ld_wait();
            // this warp's columns of buffer u are in registers: hand the buffer back to the UMMA warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&st->bar_tmem_empty[u]));
            Acc8 acc;
            float lin;
            if (u == 0) {
              head_sum32<true, 0>(va, w_addr, acc);
              head_sum32<false, 128>(vb, w_addr, acc);
              lin = lin_sum<0>(vl, l_addr);
            } else {
              head_sum32<true, kUnitQ * kRowWBytes>(va, w_addr, acc);
              head_sum32<false, kUnitQ * kRowWBytes + 128>(vb, w_addr, acc);
              lin = lin_sum<kUnitQ * kRowLBytes>(vl, l_addr);
            }
            const float score = finish(acc, lin, ks);
            if (kMode == kModeDump) {
              const int dr = st->dump_row[r];
              if (dr >= 0 && s < p.n_keys &&
                  LT_IN_BOUNDS(s < p.dump_ld && dr < (p.fb_list != nullptr ? p.fb_slots * kBlockQ : p.row_end - p.row_begin), p.ctl))
                p.dump[static_cast<size_t>(dr) * p.dump_ld + s] = (s < st->vis[r]) ? score : -INFINITY;
            } else {
              // ---- paper Sec. 3.2 "Filtering": gate, ballot-compact into the warp's staging list,
              // count in the histogram; the list is flushed to the candidate buffer in batches
              bool pass = score >= thr;
              if (partial) pass = pass && (s < st->vis[r]);
              const uint32_t ballot = __ballot_sync(0xffffffffu, pass);
              if (ballot != 0) {
                const int t = it.t0 + r;
                const int n = __popc(ballot);
                uint2* list = st->stage[ew][u];
                if (cnt[u] + n > kStageLen) {
                  flush_stage(list, cnt[u], p, t, lane, st->smin[r], st->width[r], st->inv_width[r]);
                  cnt[u] = 0;
                }
                if (pass) list[cnt[u] + __popc(ballot & ((1u << lane) - 1u))] = make_uint2(__float_as_uint(score), static_cast<uint32_t>(s));
                cnt[u] += n;
              }
            }
            if (!ok) break;
          }
          acc_phase ^= 1;
        }
        if (kMode == kModeFilter) {
#pragma unroll
          for (int u = 0; u < kUnits; ++u)
            if (cnt[u] > 0) {
              const int r = u * kUnitQ + g;
              flush_stage(st->stage[ew][u], cnt[u], p, it.t0 + r, lane, st->smin[r], st->width[r], st->inv_width[r]);
            }
        }
        if (warp == kFirstEpiWarp && lane == 0) *reinterpret_cast<volatile int*>(&st->done_seq) = seq;
      }
    }
  }

  // ---------------------------------------------------------------------- teardown
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (st->abort_flag) {
    if (threadIdx.x == 0) atomicOr(&p.ctl->status, LT_STATUS_TIMEOUT);
    // give copies and UMMAs still in flight time to land before TMEM and shared memory go away
    uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---------------------------------------------------------------------------------------------
// pre-pass: the linear part of Eq. 1 as e4m3 operand rows
// ---------------------------------------------------------------------------------------------
// e4m3 (1-4-3, bias 7, no infinities): value of a storage code; the NaN codes do not occur (precondition).
__device__ __forceinline__ float e4m3_value(uint32_t c) {
  const uint32_t e = (c >> 3) & 15u, m = c & 7u;
  const float mag = e == 0 ? ldexpf(static_cast<float>(m), -9) : ldexpf(static_cast<float>(8u + m), static_cast<int>(e) - 10);
  return (c & 0x80u) ? -mag : mag;
}
// round to nearest even e4m3, saturating at +-448
__device__ __forceinline__ uint32_t e4m3_encode(float v) {
  uint16_t pair;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(pair) : "f"(0.f), "f"(v));
  return pair & 0xffu;
}

// One CTA of 128 threads per query row t; thread d owns coordinate d.
//   qlin[d] = sum_h w[t][h] * q[t][h][d]                       (fp64: products and sums are exact enough to
//                                                               make the split below the only approximation)
//   for j < kLinTerms:  scale_j = 2^e with max_d |r[d]| / scale_j in [128, 256);  c_j[d] = e4m3(r[d] / scale_j);
//                       r[d] -= scale_j * c_j[d]              (exact)
// Each term removes at least four bits of every coordinate's residual, so after five terms
// |r[d]| <= 2^-20 |qlin[d]| (or is below 2^-26 of the row's largest coordinate).
__global__ void __launch_bounds__(kD) lin_terms_kernel(const uint8_t* __restrict__ q, const float* __restrict__ w, int T,
                                                       uint8_t* __restrict__ lin_q, float* __restrict__ lin_scale) {
  const int t = blockIdx.x;
  const int d = threadIdx.x;
  __shared__ float sw[kH];
  __shared__ float red[4];
  if (d < kH) sw[d] = w[static_cast<size_t>(t) * kH + d];
  __syncthreads();
  double r = 0.0;
  const uint8_t* qt = q + static_cast<size_t>(t) * kH * kD;
#pragma unroll 8
  for (int h = 0; h < kH; ++h) r += static_cast<double>(sw[h]) * static_cast<double>(e4m3_value(qt[h * kD + d]));
  for (int j = 0; j < kJ; ++j) {
    float a = fabsf(static_cast<float>(r));
    // |r| rounded to fp32 only picks the scale; round up so that the maximum is never underestimated
    if (static_cast<double>(a) < fabs(r)) a = __uint_as_float(__float_as_uint(a) + 1u);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
    __syncthreads();
    if ((d & 31) == 0) red[d >> 5] = a;
    __syncthreads();
    const float mx = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
    float scale = 1.f;
    if (mx > 0.f) {
      int e;
      frexpf(mx, &e);            // mx = f * 2^e, f in [0.5, 1)
      e -= 8;                    // mx / 2^(e - 8) in [128, 256) ... keep a factor 1.75 below 448
      if (e < -120) e = -120;    // stay far from fp32 denormal scales
      scale = ldexpf(1.f, e);
    }
    const float c = static_cast<float>(r / static_cast<double>(scale));
    const uint32_t code = e4m3_encode(c);
    r -= static_cast<double>(scale) * static_cast<double>(e4m3_value(code));
    lin_q[(static_cast<size_t>(t) * kJ + j) * kD + d] = static_cast<uint8_t>(code);
    if (d == 0) lin_scale[static_cast<size_t>(t) * kLinScaleStride + j] = scale;
  }
  if (d >= kJ && d < kLinScaleStride) lin_scale[static_cast<size_t>(t) * kLinScaleStride + d] = 0.f;
}

// ---------------------------------------------------------------------------------------------
// host side: tensor maps and launch
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// 2-D map over a row-major [rows][128] byte matrix with a given row pitch; box = 128 bytes x box_rows,
// 128-byte swizzle, zero fill outside the matrix.
bool make_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t pitch_bytes, uint32_t box_rows) {
  EncodeTiledFn enc = get_encode_fn();
  if (enc == nullptr) return false;
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(kD), rows};
  cuuint64_t strides[1] = {pitch_bytes};
  cuuint32_t box[2] = {128, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

template <int kMode, bool kPaged>
cudaError_t launch_one(const CUtensorMap& tq, const CUtensorMap& tl, const CUtensorMap& tk, const ScanParams& p, int grid,
                       cudaStream_t stream) {
  constexpr int bytes = smem_bytes();
  cudaError_t e = cudaFuncSetAttribute(scan_fp8_kernel<kMode, kPaged>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) return e;
  scan_fp8_kernel<kMode, kPaged><<<grid, kThreads, bytes, stream>>>(tq, tl, tk, p);
  return cudaGetLastError();
}
// the paged variant is a separate instantiation so that the dense kernels carry none of its address arithmetic
template <int kMode>
cudaError_t launch(const CUtensorMap& tq, const CUtensorMap& tl, const CUtensorMap& tk, const ScanParams& p, int grid,
                   cudaStream_t stream) {
  return p.page_table != nullptr ? launch_one<kMode, true>(tq, tl, tk, p, grid, stream)
                                 : launch_one<kMode, false>(tq, tl, tk, p, grid, stream);
}

}  // namespace

cudaError_t launch_lin_terms(const void* q, const float* w, int T, void* lin_q, float* lin_scale, cudaStream_t stream) {
  lin_terms_kernel<<<T, kD, 0, stream>>>(static_cast<const uint8_t*>(q), w, T, static_cast<uint8_t*>(lin_q), lin_scale);
  return cudaGetLastError();
}

cudaError_t launch_scan_fp8(int mode, const void* q, int T, const void* k, long long n_keys_view, long long key_pitch_elems,
                            const ScanParams& params, int grid, cudaStream_t stream) {
  ScanParams p = params;
  if (p.wait_limit_us == 0) p.wait_limit_us = kDefaultWaitLimitUs;
  if (p.lin_q == nullptr || p.lin_scale == nullptr) return cudaErrorInvalidValue;
  CUtensorMap tq, tl, tk;
  if (!make_map(&tq, q, static_cast<uint64_t>(T) * kH, kD, kHeadRows)) return cudaErrorInvalidValue;
  if (!make_map(&tl, p.lin_q, static_cast<uint64_t>(T) * kJ, kD, kLinRows)) return cudaErrorInvalidValue;
  // dense keys: one 128-row box per tile; paged keys (k = the page pool, n_keys_view = its rows): 64-row boxes
  if (!make_map(&tk, k, static_cast<uint64_t>(n_keys_view), static_cast<uint64_t>(key_pitch_elems),
                p.page_table != nullptr ? kPageKeys : 128))
    return cudaErrorInvalidValue;
  return mode == kModeFilter ? launch<kModeFilter>(tq, tl, tk, p, grid, stream) : launch<kModeDump>(tq, tl, tk, p, grid, stream);
}

}  // namespace lt
