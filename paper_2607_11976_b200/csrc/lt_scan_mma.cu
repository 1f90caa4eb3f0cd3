// Tensor-core scan kernel of the fused indexer top-k (sm_100a: TMA -> shared -> tcgen05.mma -> TMEM).
//
// One CTA keeps a block of 8 query rows (8 x 64 heads = 512 operand rows of D = 128) resident in
// shared memory and streams 128-key tiles of K past it.  Per key tile it issues two 128 x 256 x 128
// UMMAs (unit u = queries 4u .. 4u+3) into the two 256-column halves of TMEM; lanes index keys and
// columns index (query, head), so each epilogue thread owns one key and finishes Eq. 1 of the paper
// (ReLU, head-weighted sum, key scale) as an in-thread chain of packed FMAs over TMEM columns.
//
//   kMode == kModeFilter  paper Sec. 3.2 "Filtering": gate the score against the row's threshold
//                         edge, ballot-compact the survivors of each warp into a staging list; a flush
//                         appends the list to the row's candidate buffer and counts its entries in the
//                         row's bin histogram; a spare warp re-derives the
//                         threshold bin from the histogram while the scan runs ("Threshold
//                         Refresh") and publishes it by plain store.
//   kMode == kModeDump    write every score (or -inf where masked) to a dense matrix: used for the
//                         sample phase, lt_indexer_scores, the unfused baseline and the exact fallback.
//
// Warp roles (608 threads): 0 TMA producer, 1 UMMA issuer (+ TMEM owner), 2 threshold refresh,
// 3..18 epilogue in four warpgroups.  Warpgroup g finishes query g of unit 0 (TMEM half 0) and then
// query g of unit 1 (half 1) of every key tile, so the UMMA warp refills one half while the other
// is drained.  A warp pulls its 64 columns of a half into registers with one wait, hands the half
// back at once and only then does the arithmetic; the four warps of a scheduler cover each
// other's barrier and TMEM latencies.  Survivors of the gate go to small
// per-warp staging lists in shared memory and are flushed to the row's candidate buffer in batches
// (one tail atomic per flush; paper Sec. 3.2 "Filtering").
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
constexpr int kBlockQ = 8;                  // query rows resident per CTA
constexpr int kUnitQ = 4;                   // query rows per UMMA (N = 4 * 64 = 256 columns)
constexpr int kUnits = kBlockQ / kUnitQ;    // UMMAs per key tile = TMEM halves
constexpr int kUmmaN = kUnitQ * kH;         // 256
constexpr int kTmemCols = 512;              // two accumulators of 256 fp32 columns
constexpr int kFirstEpiWarp = 3;
constexpr int kEpiWarps = 16;
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kThreads = kFirstEpiWarp * 32 + kEpiThreads;
constexpr int kSwizzleTile = 128 * 128;     // bytes: 128 rows x 128-byte swizzled rows
constexpr int kQTile = 256 * 128;           // bytes: 256 rows x 128-byte rows (one unit, one K-half)
constexpr int kStageLen = 64;               // entries of one per-warp staging list
constexpr int kUnitWBytes = kUnitQ * kH * 4;  // bytes between the weights of query g and query 4 + g

template <bool kFp8>
struct Cfg {
  static constexpr int kHalves = kFp8 ? 1 : 2;           // 128-byte row pieces along D
  static constexpr int kElemsPerRow128 = kFp8 ? 128 : 64;  // elements in a 128-byte row
  static constexpr int kStages = kFp8 ? 6 : 2;           // K-tile ring depth
  static constexpr int kKBlocks = kFp8 ? 4 : 8;          // UMMA K-steps per tile (K = 32 fp8 / 16 bf16 = 32 bytes)
  static constexpr int kQBytes = kUnits * kHalves * kQTile;
  static constexpr int kStageBytes = kHalves * kSwizzleTile;
  static constexpr int kSmemTiles = kQBytes + kStages * kStageBytes;
};

struct SmemTail {
  float w[kBlockQ * kH];
  float thr[kBlockQ];
  float smin[kBlockQ];
  float width[kBlockQ];
  float inv_width[kBlockQ];
  int vis[kBlockQ];
  int dump_row[kBlockQ];
  uint64_t bar_full[8];
  uint64_t bar_empty[8];
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

template <bool kFp8>
constexpr int smem_bytes() {
  return 1024 + Cfg<kFp8>::kSmemTiles + static_cast<int>(sizeof(SmemTail));
}

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

// ---- Eq. 1 for one key against one query ------------------------------------------------------
// 32 TMEM columns (per-head dots) -> ReLU -> weighted sum, accumulated into four packed fp32 pairs
// (eight independent chains).  Head h lands in pair (h / 2) % 4, lane h % 2; combine() fixes the
// order of the final additions.  These functions produce every score the library ranks or dumps
// on the tensor-core path, so fused, dumped and fallback scores agree bit for bit.
struct Acc8 {
  uint64_t p[4];
};
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
// acc (+)= w * ReLU(x) for two heads at once.  The ReLU is applied in place on the two registers
// the TMEM load filled, so that they stay an aligned register pair for the packed FMA.
//   kSat == false: ReLU(x) = max(x, 0)                                  (ALU pipe)
//   kSat == true : ReLU(x) = sat(x * 2^-25) * 2^25, the 2^25 being folded into the weight the
//                  caller stored for this head                          (FMA pipe)
// The saturating form needs |x| < 2^25 and no underflow of x * 2^-25; both hold for dot products of
// 128 e4m3 codes (|x| <= 448^2 * 128 < 2^25, non-zero |x| >= 2^-18).  Scaling by a power of two is
// exact, so w * 2^25 * (x * 2^-25) and w * x round to the same fp32 value: the two forms give
// bit-identical sums and are mixed only to spread the work over both pipes.
// kFirst: the accumulator starts at w * ReLU(x) (a multiply) instead of being zero-initialised.
template <bool kSat, bool kFirst>
__device__ __forceinline__ void relu_fma2(uint64_t& acc, uint64_t w, uint32_t& x0, uint32_t& x1) {
  // everything stays in the untyped 32-bit registers of the TMEM load (no typed copies)
  if (kSat) {
    asm("mul.sat.f32 %0, %0, 0f33000000;" : "+r"(x0));
    asm("mul.sat.f32 %0, %0, 0f33000000;" : "+r"(x1));
  } else {
    asm("max.f32 %0, %0, 0f00000000;" : "+r"(x0));
    asm("max.f32 %0, %0, 0f00000000;" : "+r"(x1));
  }
  if (kFirst) {
    asm("{\n.reg .b64 x;\nmov.b64 x, {%1, %2};\nmul.rn.f32x2 %0, %3, x;\n}\n" : "=l"(acc) : "r"(x0), "r"(x1), "l"(w));
  } else {
    asm("{\n.reg .b64 x;\nmov.b64 x, {%1, %2};\nfma.rn.f32x2 %0, %3, x, %0;\n}\n" : "+l"(acc) : "r"(x0), "r"(x1), "l"(w));
  }
}
// Weight stored in shared memory for head h: heads whose ReLU takes the saturating form carry 2^25.
template <bool kFp8>
__device__ __forceinline__ float stored_weight(float w, int h) {
  return (kFp8 && (h & 2)) ? w * 33554432.f : w;
}
// Eight heads starting at column J of a 32-column piece.  kOff: byte offset of the piece's weights
// from w_addr, folded into the load instructions as an immediate.
template <bool kFp8, bool kFirst, int kOff, int J>
__device__ __forceinline__ void head_sum8(uint32_t (&v)[32], uint32_t w_addr, Acc8& acc) {
  uint64_t w01, w23, w45, w67;
  asm volatile("ld.shared.v2.b64 {%0, %1}, [%2+%3];" : "=l"(w01), "=l"(w23) : "r"(w_addr), "n"(kOff + J * 4));
  asm volatile("ld.shared.v2.b64 {%0, %1}, [%2+%3];" : "=l"(w45), "=l"(w67) : "r"(w_addr), "n"(kOff + J * 4 + 16));
  constexpr bool first = kFirst && J == 0;
  relu_fma2<false, first>(acc.p[0], w01, v[J + 0], v[J + 1]);
  relu_fma2<kFp8, first>(acc.p[1], w23, v[J + 2], v[J + 3]);
  relu_fma2<false, first>(acc.p[2], w45, v[J + 4], v[J + 5]);
  relu_fma2<kFp8, first>(acc.p[3], w67, v[J + 6], v[J + 7]);
}
template <bool kFp8, bool kFirst, int kOff>
__device__ __forceinline__ void head_sum32(uint32_t (&v)[32], uint32_t w_addr, Acc8& acc) {
  head_sum8<kFp8, kFirst, kOff, 0>(v, w_addr, acc);
  head_sum8<kFp8, kFirst, kOff, 8>(v, w_addr, acc);
  head_sum8<kFp8, kFirst, kOff, 16>(v, w_addr, acc);
  head_sum8<kFp8, kFirst, kOff, 24>(v, w_addr, acc);
}
__device__ __forceinline__ float combine(const Acc8& acc, float ks) {
  uint64_t ab, cd, all;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(ab) : "l"(acc.p[0]), "l"(acc.p[1]));
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(cd) : "l"(acc.p[2]), "l"(acc.p[3]));
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(all) : "l"(ab), "l"(cd));
  float lo, hi;
  unpack2(all, lo, hi);
  return __fmaf_rn(lo + hi, ks, 0.f);  // the + 0 turns -0 into +0
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

// kU: units in use.  A chunk of at most kUnitQ rows (a decode step, a tail of a few tokens) has no row for the second
// unit: its launch issues, loads and finishes unit 0 only, which halves the tensor and the epilogue work per key tile.
template <bool kFp8, int kMode, bool kPaged, int kU = kUnits>
__global__ void __launch_bounds__(kThreads, 1)
scan_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k, const ScanParams p) {
  using C = Cfg<kFp8>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
  uint8_t* smem = smem_raw + pad;
  const uint32_t q_base = raw_addr + pad;
  const uint32_t k_base = q_base + C::kQBytes;
  SmemTail* st = reinterpret_cast<SmemTail*>(smem + C::kSmemTiles);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  // a fallback round with no flagged block left has nothing to do (uniform across the CTA)
  if (p.fb_list != nullptr && *p.fb_blocks <= p.fb_round_base) return;

  if (threadIdx.x == 0) {
    for (int i = 0; i < C::kStages; ++i) {
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
        mbar_arrive_expect_tx(smem_u32(&st->bar_q_full), kU * C::kHalves * kQTile);
        for (int u = 0; u < kU; ++u)
          for (int hf = 0; hf < C::kHalves; ++hf)
            tma_load_2d(q_base + (u * C::kHalves + hf) * kQTile, &tm_q, hf * C::kElemsPerRow128,
                        (it.t0 + u * kUnitQ) * kH, smem_u32(&st->bar_q_full));
        ++n_done;
        for (int tile = it.tile_lo; tile < it.tile_hi; ++tile) {
          ok = mbar_wait<40>(smem_u32(&st->bar_empty[stage]), phase ^ 1, abort_flag);
          if (!ok) break;
          // test hook (lt_tunables.debug_flags): CTA 0 never loads the first key tile of its first item, so
          // the UMMA warp's wait for it runs out and the whole CTA unwinds through the timeout path
          if ((p.debug_flags & LT_DEBUG_SKIP_ONE_KTILE) && blockIdx.x == 0 && n_done == 1 && tile == it.tile_lo) {
            ok = false;
            break;
          }
          mbar_arrive_expect_tx(smem_u32(&st->bar_full[stage]), C::kStageBytes);
          if (!kPaged) {
            for (int hf = 0; hf < C::kHalves; ++hf)
              tma_load_2d(k_base + stage * C::kStageBytes + hf * kSwizzleTile, &tm_k, hf * C::kElemsPerRow128,
                          tile * kTileKeys, smem_u32(&st->bar_full[stage]));
          } else {
            // paged key cache: a tile is two pages of 64 keys, each wherever the page table says (the map's
            // box is then 64 rows); pages past the end of the table are read from page 0 and masked later
            for (int pg = 0; pg < kTileKeys / kPageKeys; ++pg) {
              const int lp = tile * (kTileKeys / kPageKeys) + pg;
              int phys = lp < p.n_pages ? __ldg(p.page_table + lp) : 0;
              if (!LT_IN_BOUNDS(phys >= 0 && phys < p.pool_pages, p.ctl)) phys = 0;  // entry outside the pool
              for (int hf = 0; hf < C::kHalves; ++hf)
                tma_load_2d(k_base + stage * C::kStageBytes + hf * kSwizzleTile + pg * kPageKeys * 128, &tm_k,
                            hf * C::kElemsPerRow128, phys * kPageKeys, smem_u32(&st->bar_full[stage]));
            }
          }
          if (++stage == C::kStages) {
            stage = 0;
            phase ^= 1;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ UMMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(kFp8, kUmmaN);
      int stage = 0;
      uint32_t phase = 0;
      uint32_t acc_phase = 0;  // flips once per key tile: each TMEM half is filled once per tile
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
          for (int u = 0; u < kU; ++u) {
            ok = mbar_wait<40>(smem_u32(&st->bar_tmem_empty[u]), acc_phase ^ 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int kb = 0; kb < C::kKBlocks; ++kb) {
              const int hf = kFp8 ? 0 : (kb >> 2);
              const int step = kFp8 ? kb : (kb & 3);
              uint64_t a = make_smem_desc_sw128(k_base + stage * C::kStageBytes + hf * kSwizzleTile) + (step * 32 >> 4);
              uint64_t b = make_smem_desc_sw128(q_base + (u * C::kHalves + hf) * kQTile) + (step * 32 >> 4);
              tc_mma<kFp8>(tmem_base + u * kUmmaN, a, b, idesc, kb > 0 ? 1u : 0u);
            }
            tc_commit(smem_u32(&st->bar_tmem_full[u]));
          }
          acc_phase ^= 1;
          tc_commit(smem_u32(&st->bar_empty[stage]));
          if (++stage == C::kStages) {
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
      const int g = ew >> 2;                           // warpgroup 0..3: queries g (unit 0) and 4 + g (unit 1)
      const int key_in_tile = quarter * 32 + lane;
      const uint32_t tcol = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(g * kH);
      const uint32_t w_addr = smem_u32(st->w) + g * kH * 4;
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
            st->w[i] = (t < p.T) ? stored_weight<kFp8>(p.w[static_cast<size_t>(t) * kH + (i % kH)], i % kH) : 0.f;
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
            // sleep in slices so that the end of the item is noticed quickly; lane 0 reads the flags and the
            // whole warp follows its decision, so that no lane can leave while others still execute the
            // full-mask shuffles above
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

        // ---- epilogue proper: this warp finishes queries g and 4 + g for its 32 keys of every tile.
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
          for (int u = 0; u < kU; ++u) {
            const int r = u * kUnitQ + g;
            float thr = 0.f;
            if (kMode == kModeFilter) thr = *reinterpret_cast<volatile float*>(&st->thr[r]);
            ok = mbar_wait(smem_u32(&st->bar_tmem_full[u]), acc_phase, abort_flag);
            tc_fence_after();
            // the 64 columns of this query: both loads in flight, one wait.  The loads are issued even
            // after a failed wait (they then fetch values nobody uses): keeping them unconditional
            // keeps the 64 destination registers free of copies.
            uint32_t va[32], vb[32];
            tmem_ld32(tcol + u * kUmmaN, va);
            tmem_ld32(tcol + u * kUmmaN + 32, vb);
            tmem_ld_wait();
            // this warp's columns of half u are in registers: hand the half back to the UMMA warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&st->bar_tmem_empty[u]));
            Acc8 acc;
            if (u == 0) {
              head_sum32<kFp8, true, 0>(va, w_addr, acc);
              head_sum32<kFp8, false, 128>(vb, w_addr, acc);
            } else {
              head_sum32<kFp8, true, kUnitWBytes>(va, w_addr, acc);
              head_sum32<kFp8, false, kUnitWBytes + 128>(vb, w_addr, acc);
            }
            const float score = combine(acc, ks);
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
          for (int u = 0; u < kU; ++u)
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

// 2-D map over a row-major [rows][kD] matrix with a given row pitch; box = 128 bytes x box_rows,
// 128-byte swizzle, zero fill outside the matrix.
bool make_map(CUtensorMap* map, bool fp8, const void* base, uint64_t rows, uint64_t pitch_bytes, uint32_t box_rows) {
  EncodeTiledFn enc = get_encode_fn();
  if (enc == nullptr) return false;
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(kD), rows};
  cuuint64_t strides[1] = {pitch_bytes};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(fp8 ? 128 : 64), box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(map, fp8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base),
                   dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

template <bool kFp8, int kMode, bool kPaged, int kU>
cudaError_t launch_one(const CUtensorMap& tq, const CUtensorMap& tk, const ScanParams& p, int grid, cudaStream_t stream) {
  constexpr int bytes = smem_bytes<kFp8>();
  cudaError_t e = cudaFuncSetAttribute(scan_kernel<kFp8, kMode, kPaged, kU>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) return e;
  scan_kernel<kFp8, kMode, kPaged, kU><<<grid, kThreads, bytes, stream>>>(tq, tk, p);
  return cudaGetLastError();
}
// the paged variant is a separate instantiation so that the dense kernels carry none of its address arithmetic; the
// one-unit variant exists for the fused scan of a chunk of at most kUnitQ rows
template <bool kFp8, int kMode>
cudaError_t launch(const CUtensorMap& tq, const CUtensorMap& tk, const ScanParams& p, int grid, cudaStream_t stream) {
  if (kMode == kModeFilter && p.fb_list == nullptr && p.row_end - p.row_begin <= kUnitQ) {
    return p.page_table != nullptr ? launch_one<kFp8, kModeFilter, true, 1>(tq, tk, p, grid, stream)
                                   : launch_one<kFp8, kModeFilter, false, 1>(tq, tk, p, grid, stream);
  }
  return p.page_table != nullptr ? launch_one<kFp8, kMode, true, kUnits>(tq, tk, p, grid, stream)
                                 : launch_one<kFp8, kMode, false, kUnits>(tq, tk, p, grid, stream);
}

}  // namespace

namespace {
__global__ void wait_timeout_probe_kernel(unsigned int limit_us, int* result2) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag[2];  // flag, limit in microseconds
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag[0] = 0;
    abort_flag[1] = static_cast<int>(limit_us);
    fence_mbar_init();
  }
  __syncthreads();
  // phase 0 of `bar` never completes: the wait can only end by its time limit
  const bool ok = mbar_wait<40>(smem_u32(&bar), 0, abort_flag);
  __syncthreads();
  if (threadIdx.x == 0) {
    result2[0] = ok ? 1 : 0;
    result2[1] = abort_flag[0];
  }
}
}  // namespace

cudaError_t launch_wait_timeout_probe(unsigned int limit_us, int* result2, cudaStream_t stream) {
  wait_timeout_probe_kernel<<<1, 32, 0, stream>>>(limit_us, result2);
  return cudaGetLastError();
}

bool scan_mma_supported(int dtype, int H, int D) {
  return (dtype == LT_DTYPE_BF16 || dtype == LT_DTYPE_E4M3) && H == kH && D == kD;
}

cudaError_t launch_scan_mma(int dtype, int mode, const void* q, int T, const void* k, long long n_keys_view,
                            long long key_pitch_elems, const ScanParams& params, int grid, cudaStream_t stream) {
  ScanParams p = params;
  if (p.wait_limit_us == 0) p.wait_limit_us = kDefaultWaitLimitUs;
  if (mode != kModeFilter) p.debug_flags = 0;  // the test hooks act on the fused scan only
  const bool fp8 = (dtype == LT_DTYPE_E4M3);
  const size_t esz = fp8 ? 1 : 2;
  CUtensorMap tq, tk;
  if (!make_map(&tq, fp8, q, static_cast<uint64_t>(T) * kH, kD * esz, 256)) return cudaErrorInvalidValue;
  // dense keys: one 128-row box per tile; paged keys (k = the page pool, n_keys_view = its rows): 64-row boxes
  if (!make_map(&tk, fp8, k, static_cast<uint64_t>(n_keys_view), static_cast<uint64_t>(key_pitch_elems) * esz,
                p.page_table != nullptr ? kPageKeys : 128))
    return cudaErrorInvalidValue;
  if (fp8) {
    return mode == kModeFilter ? launch<true, kModeFilter>(tq, tk, p, grid, stream) : launch<true, kModeDump>(tq, tk, p, grid, stream);
  }
  return mode == kModeFilter ? launch<false, kModeFilter>(tq, tk, p, grid, stream) : launch<false, kModeDump>(tq, tk, p, grid, stream);
}

}  // namespace lt
