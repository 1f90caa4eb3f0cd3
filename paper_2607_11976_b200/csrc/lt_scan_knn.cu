// Tensor-core scan kernel of the k-NN (inner-product) variant (sm_100a: TMA -> shared -> tcgen05.mma -> TMEM).
//
// Paper Sec. 3.1 (Eq. 2 with f(q, x) = q . x) and Sec. 3.2 "Filtering", first case: "scores are produced
// directly by Tensor Cores", so the epilogue is a compare per score.  The corpus is streamed once per batch
// of 64 queries, which makes the kernel HBM-bound: D x 2 bytes per corpus vector against 64 x D MACs.
//
// One CTA keeps a block of 64 queries (64 x D bf16, D / 64 swizzled 8 KB slices) resident in shared memory
// and streams 128-vector tiles of the corpus past it, one 128-byte K-slice (128 vectors x 64 elements, 16 KB)
// per pipeline stage.  The D / 64 slices of a tile accumulate into one 128 x 64 fp32 accumulator in TMEM
// (lanes = corpus vectors, columns = queries); four accumulators rotate, so the UMMA warp runs up to three
// tiles ahead of the epilogue.
//
//   kMode == kModeFilter  gate every score against its query's threshold edge, ballot-compact the survivors
//                         of a warp straight into the query's candidate buffer (one tail atomic per ballot
//                         with a survivor: a few per tile) and count them in the query's bin histogram; a
//                         spare warp re-derives the threshold bins ("Threshold Refresh").
//   kMode == kModeDump    write every score to a dense matrix: sample phase, lt_knn_scores, exact fallback.
//
// Warp roles (352 threads): 0 TMA producer, 1 UMMA issuer (+ TMEM owner), 2 threshold refresh, 3..10 epilogue:
// two warps per TMEM lane quarter, the two sets of four taking alternate tiles.
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

constexpr int kQB = 64;                      // queries per block = UMMA N
constexpr int kSliceElems = 64;              // bf16 elements in a 128-byte row piece
constexpr int kQSliceBytes = kQB * 128;      // 8 KB: 64 query rows x 128 bytes
constexpr int kXSliceBytes = kTileKeys * 128;  // 16 KB: 128 corpus rows x 128 bytes
constexpr int kKnnStages = 6;                // 16 KB K-slices in flight per SM (a seventh, or L2 prefetches ahead, gained nothing)
constexpr int kKnnMaxSlices = 12;            // D <= 768
constexpr int kAccBufs = 4;                  // TMEM accumulators of 64 columns
constexpr int kKnnTmemCols = kAccBufs * kQB;  // 256
constexpr int kKnnFirstEpi = 3;
constexpr int kKnnEpiWarps = 8;
constexpr int kKnnThreads = (kKnnFirstEpi + kKnnEpiWarps) * 32;
constexpr int kKnnStageLen = 128;            // entries of one warp's staging list

struct KnnTail {
  float thr[kQB];
  float smin[kQB];
  float width[kQB];
  float inv_width[kQB];
  uint64_t bar_full[kKnnStages];
  uint64_t bar_empty[kKnnStages];
  uint64_t bar_q_full;
  uint64_t bar_q_empty;
  uint64_t bar_acc_full[kAccBufs];
  uint64_t bar_acc_empty[kAccBufs];
  uint32_t tmem_base;
  int abort_flag;     // [0] raised by a wait that ran out; every role unwinds on it
  int wait_limit_us;  // [1] bound of every wait (read by mbar_wait through the flag's address)
  int epi_abort;
  int done_seq;
  uint4 stage[kKnnEpiWarps][kKnnStageLen];  // per warp: (score bits, corpus index, query row, -) of survivors
};

constexpr int knn_smem_bytes(int n_slices) { return 1024 + n_slices * kQSliceBytes + kKnnStages * kXSliceBytes + static_cast<int>(sizeof(KnnTail)); }
static_assert(knn_smem_bytes(kKnnMaxSlices) <= 227 * 1024, "shared memory budget");

struct KnnItem {
  int qb;        // query block
  int tile_lo;   // corpus tiles [tile_lo, tile_hi)
  int tile_hi;
};

// Work items are (corpus segment, query block) pairs, segment-major.
__device__ __forceinline__ bool knn_item(const KnnScanParams& p, int qb_lo, int n_qb, int item, KnnItem& it) {
  const int seg = item / n_qb;
  it.qb = qb_lo + (item - seg * n_qb);
  const int n_tiles = (p.n_keys + kTileKeys - 1) / kTileKeys;
  it.tile_lo = seg * p.seg_tiles;
  it.tile_hi = min(it.tile_lo + p.seg_tiles, n_tiles);
  return it.tile_lo < it.tile_hi;
}

// Gate of 32 queries against one corpus vector per lane: bit q of the result = score[q] >= thr[q].
// The thresholds are read as eight 16-byte volatile loads (they move while the scan runs).
__device__ __forceinline__ uint32_t knn_gate32(const uint32_t (&v)[32], const float* thr, bool in_range) {
  uint32_t m = 0;
#pragma unroll
  for (int j = 0; j < 32; j += 4) {
    float t0, t1, t2, t3;
    asm volatile("ld.volatile.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(t0), "=f"(t1), "=f"(t2), "=f"(t3) : "r"(smem_u32(thr + j)));
    m |= (__uint_as_float(v[j + 0]) >= t0 ? 1u : 0u) << (j + 0);
    m |= (__uint_as_float(v[j + 1]) >= t1 ? 1u : 0u) << (j + 1);
    m |= (__uint_as_float(v[j + 2]) >= t2 ? 1u : 0u) << (j + 2);
    m |= (__uint_as_float(v[j + 3]) >= t3 ? 1u : 0u) << (j + 3);
  }
  return in_range ? m : 0u;
}

// Survivors go to one staging list per warp in shared memory, (score bits, corpus index, query row, -), for
// all 64 queries together: appending costs a ballot and a shared-memory store, nothing waits for global
// memory.  A list that may not hold the next ballot is flushed: every lane reserves a slot in its entry's
// candidate buffer with its own atomic (all of them in flight together: one round trip per 32 entries), stores
// the entry and counts it in the query's histogram.  Entries beyond the capacity are dropped but still counted
// (the tail then exceeds the capacity, which flags the row).  Paper Sec. 3.2 "Filtering": "a list in warp-local
// shared memory, flushed in batches".
__device__ __noinline__ void knn_flush(const uint4* list, int count, const KnnScanParams& p, int t0, const float* smin,
                                       const float* width, const float* inv_width) {
  const int lane = threadIdx.x & 31;
  __syncwarp();
  for (int i = lane; i < count; i += 32) {
    const uint4 e = list[i];
    const int t = static_cast<int>(e.z);
    const int r = t - t0;
    if (!LT_IN_BOUNDS(t >= 0 && t < p.T && r >= 0 && r < kQB && e.y < static_cast<uint32_t>(p.n_keys), p.ctl)) continue;
    const uint32_t pos = atomicAdd(p.tail + t, 1u);
    if (pos < static_cast<uint32_t>(p.cap)) p.cand[static_cast<size_t>(t) * p.cap + pos] = make_uint2(e.x, e.y);
    const int bin = bin_of(__uint_as_float(e.x), smin[r], width[r], inv_width[r]);
    if (LT_IN_BOUNDS(bin >= 0 && bin < kBins, p.ctl)) atomicAdd(p.hist + static_cast<size_t>(t) * kBins + bin, 1u);
  }
  __syncwarp();
}

// Appends the survivors of one tile.  mine: bit q set if this lane's vector survives query q; any: bit q set if
// some lane's does (a handful of bits per tile).  The loop runs over the set bits only and fetches the score of
// query q again from the tile's accumulator (one TMEM column), which keeps it a few dozen instructions long: a
// version unrolled over all 64 queries, taking the scores from the registers of the gate, ran out of the
// instruction cache.  Returns the new list length.
__device__ __forceinline__ int knn_stage(uint64_t any, uint64_t mine, uint32_t tacc, int s, int lane, uint4* list, int count,
                                         const KnnScanParams& p, int t0, const float* smin, const float* width,
                                         const float* inv_width) {
  while (any != 0ull) {
    const int q = __ffsll(static_cast<long long>(any)) - 1;
    any &= any - 1ull;
    const bool pass = (mine >> q) & 1ull;
    const uint32_t bal = __ballot_sync(0xffffffffu, pass);
    const uint32_t x = tmem_ld1(tacc + static_cast<uint32_t>(q));
    if (count + 32 > kKnnStageLen) {
      knn_flush(list, count, p, t0, smin, width, inv_width);
      count = 0;
    }
    tmem_ld_wait();
    // + 0 turns -0 into +0, so that the bit order of the scores is their value order
    if (pass) list[count + __popc(bal & ((1u << lane) - 1u))] =
        make_uint4(__float_as_uint(__fadd_rn(__uint_as_float(x), 0.f)), static_cast<uint32_t>(s), static_cast<uint32_t>(t0 + q), 0u);
    count += __popc(bal);
  }
  return count;
}

template <int kMode>
__global__ void __launch_bounds__(kKnnThreads, 1)
knn_scan_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_x, const KnnScanParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
  uint8_t* smem = smem_raw + pad;
  const int n_slices = p.D / kSliceElems;
  const uint32_t q_base = raw_addr + pad;
  const uint32_t x_base = q_base + n_slices * kQSliceBytes;
  KnnTail* st = reinterpret_cast<KnnTail*>(smem + n_slices * kQSliceBytes + kKnnStages * kXSliceBytes);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  // a fallback round has nothing to do unless some block of 8 rows in [row_begin, row_end) was flagged
  // (uniform across the grid)
  if (p.fb_flag != nullptr) {
    unsigned int any = 0u;
    for (int b = p.row_begin / kRowsPerBlock; b * kRowsPerBlock < p.row_end; ++b) any |= p.fb_flag[b];
    if (any == 0u) return;
  }

  if (threadIdx.x == 0) {
    for (int i = 0; i < kKnnStages; ++i) {
      mbar_init(smem_u32(&st->bar_full[i]), 1);
      mbar_init(smem_u32(&st->bar_empty[i]), 1);
    }
    mbar_init(smem_u32(&st->bar_q_full), 1);
    mbar_init(smem_u32(&st->bar_q_empty), 1);
    for (int i = 0; i < kAccBufs; ++i) {
      mbar_init(smem_u32(&st->bar_acc_full[i]), 1);
      mbar_init(smem_u32(&st->bar_acc_empty[i]), 4);  // the four quarter warps of the set that drains the tile
    }
    st->abort_flag = 0;
    st->wait_limit_us = static_cast<int>(p.wait_limit_us);
    st->epi_abort = 0;
    st->done_seq = 0;
    fence_mbar_init();
    prefetch_tensormap(&tm_q);
    prefetch_tensormap(&tm_x);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&st->tmem_base), kKnnTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = st->tmem_base;
  volatile int* abort_flag = &st->abort_flag;

  const int qb_lo = p.row_begin / kQB;
  const int n_qb = (p.row_end - 1) / kQB - qb_lo + 1;
  const int n_tiles_all = (p.n_keys + kTileKeys - 1) / kTileKeys;
  const int n_seg = (n_tiles_all + p.seg_tiles - 1) / p.seg_tiles;
  const int n_items = n_qb * n_seg;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0, cur_qb = -1;
      uint32_t phase = 0, n_done = 0;  // n_done: query blocks loaded so far (parity of the handshake)
      bool ok = true;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
        KnnItem it;
        if (!knn_item(p, qb_lo, n_qb, item, it)) continue;
        if (it.qb != cur_qb) {
          // a new query block: wait until the UMMAs of the previous one no longer read it
          ok = mbar_wait<40>(smem_u32(&st->bar_q_empty), (n_done & 1) ^ 1, abort_flag);
          if (!ok) break;
          mbar_arrive_expect_tx(smem_u32(&st->bar_q_full), n_slices * kQSliceBytes);
          for (int sl = 0; sl < n_slices; ++sl)
            tma_load_2d(q_base + sl * kQSliceBytes, &tm_q, sl * kSliceElems, it.qb * kQB, smem_u32(&st->bar_q_full));
          ++n_done;
          cur_qb = it.qb;
        }
        for (int tile = it.tile_lo; tile < it.tile_hi && ok; ++tile) {
          for (int sl = 0; sl < n_slices; ++sl) {
            ok = mbar_wait<40>(smem_u32(&st->bar_empty[stage]), phase ^ 1, abort_flag);
            if (!ok) break;
            mbar_arrive_expect_tx(smem_u32(&st->bar_full[stage]), kXSliceBytes);
            tma_load_2d(x_base + stage * kXSliceBytes, &tm_x, sl * kSliceElems, tile * kTileKeys, smem_u32(&st->bar_full[stage]));
            if (++stage == kKnnStages) {
              stage = 0;
              phase ^= 1;
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ UMMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(false, kQB);
      int stage = 0, cur_qb = -1;
      uint32_t phase = 0, n_done = 0, seq = 0;  // seq: tiles issued so far by this CTA
      bool ok = true;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
        KnnItem it;
        if (!knn_item(p, qb_lo, n_qb, item, it)) continue;
        if (it.qb != cur_qb) {
          if (cur_qb >= 0) tc_commit(smem_u32(&st->bar_q_empty));  // arrives once every UMMA issued so far is done
          ok = mbar_wait<40>(smem_u32(&st->bar_q_full), n_done & 1, abort_flag);
          if (!ok) break;
          ++n_done;
          cur_qb = it.qb;
        }
        for (int tile = it.tile_lo; tile < it.tile_hi && ok; ++tile, ++seq) {
          const uint32_t buf = seq & (kAccBufs - 1);
          ok = mbar_wait<40>(smem_u32(&st->bar_acc_empty[buf]), ((seq >> 2) & 1) ^ 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          for (int sl = 0; sl < n_slices; ++sl) {
            ok = mbar_wait<40>(smem_u32(&st->bar_full[stage]), phase, abort_flag);
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int step = 0; step < 4; ++step) {
              const uint64_t a = make_smem_desc_sw128(x_base + stage * kXSliceBytes) + (step * 32 >> 4);
              const uint64_t b = make_smem_desc_sw128(q_base + sl * kQSliceBytes) + (step * 32 >> 4);
              tc_mma<false>(tmem_base + buf * kQB, a, b, idesc, (sl > 0 || step > 0) ? 1u : 0u);
            }
            tc_commit(smem_u32(&st->bar_empty[stage]));
            if (++stage == kKnnStages) {
              stage = 0;
              phase ^= 1;
            }
          }
          if (!ok) break;
          tc_commit(smem_u32(&st->bar_acc_full[buf]));
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (+ refresh warp)
    const bool is_refresh = (warp == 2);
    constexpr int kEpiThreads = kKnnEpiWarps * 32;
    const int n_sync = (kMode == kModeFilter) ? kEpiThreads + 32 : kEpiThreads;
    if (!(is_refresh && kMode != kModeFilter)) {
      const int e = threadIdx.x - kKnnFirstEpi * 32;
      const int ew = warp - kKnnFirstEpi;
      const int quarter = warp & 3;
      const uint32_t set = static_cast<uint32_t>(ew >> 2);  // which of the two warp sets: takes tiles with seq % 2 == set
      const int key_in_tile = quarter * 32 + lane;
      const uint32_t tlane = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
      uint32_t seq = 0;  // tiles this CTA has gone through (same count as the UMMA warp's)
      // An "epoch" is a run of consecutive work items on the same query block: the per-query state in shared
      // memory is loaded, and the warps meet, only when the block changes (with one block of 64 queries: once).
      int item_seq = 0;  // epoch number
      int cur_qb = -1;
      int n_staged = 0;   // entries in this warp's staging list (warp-uniform)
      bool dead = false;  // a wait gave up: skip the remaining work, keep meeting the barriers
      for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
        KnnItem it;
        if (!knn_item(p, qb_lo, n_qb, item, it)) continue;
        const int t0 = it.qb * kQB;
        if (it.qb == cur_qb) {
          if (is_refresh) continue;  // the refresh warp served the whole epoch when it began
        } else {
        if (cur_qb >= 0 && !is_refresh) {
          // the previous epoch is over when both sets are through: tell the refresh warp
          if (kMode == kModeFilter && n_staged > 0) {
            knn_flush(st->stage[ew], n_staged, p, cur_qb * kQB, st->smin, st->width, st->inv_width);
            n_staged = 0;
          }
          named_bar_sync(2, kEpiThreads);
          if (warp == kKnnFirstEpi && lane == 0) *reinterpret_cast<volatile int*>(&st->done_seq) = item_seq;
        }
        ++item_seq;
        cur_qb = it.qb;
        named_bar_sync(1, n_sync);  // A: everybody is done with the previous epoch's shared state
        if (!is_refresh) {
          if (e < kQB && kMode == kModeFilter) {
            const int t = t0 + e;
            const bool live = t >= p.row_begin && t < p.row_end;
            st->thr[e] = live ? __ldcg(p.thr + t) : INFINITY;
            st->smin[e] = live ? p.smin[t] : 0.f;
            st->width[e] = live ? p.width[t] : 0.f;
            st->inv_width[e] = (live && p.width[t] > 0.f) ? 1.f / p.width[t] : 0.f;
          }
          if (e == 0) st->epi_abort = *abort_flag;
        }
        named_bar_sync(1, n_sync);  // B: shared state of this item is ready
        if (st->epi_abort) break;

        if (is_refresh) {
          // ---- paper Sec. 3.2 "Threshold Refresh": per query, walk the histogram from the top bin down until
          // the cumulative count reaches k and publish that bin's lower edge by plain store
          // A pass over 64 histograms takes tens of microseconds, a work item about as long: the end of the
          // item is checked before every row so that the epilogue warps never wait for this warp.
          unsigned int sleep_ns = 2000;
          bool done = false;
          while (!done) {
            for (int r = 0; r < kQB && !done; ++r) {
              const int t = t0 + r;
              // lane 0 reads the flags and the whole warp follows its decision, so that no lane can leave
              // while others still execute the full-mask shuffles below
              int d = 0;
              if (lane == 0) d = (*reinterpret_cast<volatile int*>(&st->done_seq) >= item_seq || *abort_flag) ? 1 : 0;
              done = __shfl_sync(0xffffffffu, d, 0) != 0;
              if (done || t < p.row_begin || t >= p.row_end) continue;
              const uint4* hp = reinterpret_cast<const uint4*>(p.hist + static_cast<size_t>(t) * kBins + lane * 8);
              const uint4 h0 = __ldcg(hp), h1 = __ldcg(hp + 1);
              const uint32_t c[8] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w};
              const uint32_t mine = c[0] + c[1] + c[2] + c[3] + c[4] + c[5] + c[6] + c[7];
              uint32_t incl = mine;
#pragma unroll
              for (int d = 1; d < 32; d <<= 1) {
                const uint32_t o = __shfl_down_sync(0xffffffffu, incl, d);
                if (lane + d < 32) incl += o;
              }
              const uint32_t above = incl - mine;
              const bool crosses = (above < static_cast<uint32_t>(p.topk)) && (incl >= static_cast<uint32_t>(p.topk));
              const uint32_t who = __ballot_sync(0xffffffffu, crosses);
              if (who) {
                const int src = __ffs(who) - 1;
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
                if (lane == 0 && tb > 0) {
                  const float edge = bin_edge(tb, st->smin[r], st->width[r]);
                  if (edge > *reinterpret_cast<volatile float*>(&st->thr[r])) {
                    *reinterpret_cast<volatile float*>(&st->thr[r]) = edge;
                    __stcg(p.thr + t, edge);
                  }
                }
              }
            }
            for (unsigned int slept = 0; slept < sleep_ns && !done; slept += 1000) {
              __nanosleep(1000);
              done = *reinterpret_cast<volatile int*>(&st->done_seq) >= item_seq || *abort_flag;
            }
            if (sleep_ns < 32000) sleep_ns += sleep_ns >> 1;
          }
          continue;
        }
        }  // epoch change

        // ---- epilogue proper: this warp drains the tiles of its set for its 32 corpus vectors
        bool ok = !dead;
        for (int tile = it.tile_lo; tile < it.tile_hi && ok; ++tile, ++seq) {
          if ((seq & 1u) != set) continue;
          const uint32_t buf = seq & (kAccBufs - 1);
          const int s = tile * kTileKeys + key_in_tile;
          ok = mbar_wait(smem_u32(&st->bar_acc_full[buf]), (seq >> 2) & 1, abort_flag);
          tc_fence_after();
          uint32_t va[32], vb[32];
          tmem_ld32(tlane + buf * kQB, va);
          tmem_ld32(tlane + buf * kQB + 32, vb);
          tmem_ld_wait();
          if (kMode == kModeDump) {
            // the dump needs nothing more from the accumulator: hand it back before the stores
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&st->bar_acc_empty[buf]));
          }
          if (!ok) {
            if (kMode == kModeFilter && lane == 0) mbar_arrive(smem_u32(&st->bar_acc_empty[buf]));
            break;
          }
          const bool in_range = s < p.n_keys;
          if (kMode == kModeDump) {
#pragma unroll
            for (int qq = 0; qq < kQB; ++qq) {
              // + 0 turns -0 into +0, so that the bit order of the scores is their value order
              const float score = __fadd_rn(__uint_as_float(qq < 32 ? va[qq & 31] : vb[qq & 31]), 0.f);
              const int t = t0 + qq;
              if (in_range && t >= p.row_begin && t < p.row_end && LT_IN_BOUNDS(s >= 0 && s < p.dump_ld, p.ctl))
                p.dump[static_cast<size_t>(t - p.row_begin) * p.dump_ld + s] = score;
            }
          } else {
            // ---- paper Sec. 3.2 "Filtering": a compare per score (rows outside the launch have thr = +inf;
            // -0 and +0 compare alike, so the raw accumulator is gated), then the few (query, warp) pairs
            // with a survivor are written out
            const uint32_t ma = knn_gate32(va, st->thr, in_range);
            const uint32_t mb = knn_gate32(vb, st->thr + 32, in_range);
            const uint32_t any_a = __reduce_or_sync(0xffffffffu, ma);
            const uint32_t any_b = __reduce_or_sync(0xffffffffu, mb);
            const uint64_t any = (static_cast<uint64_t>(any_b) << 32) | any_a;
            if (any != 0ull)
              n_staged = knn_stage(any, (static_cast<uint64_t>(mb) << 32) | ma, tlane + buf * kQB, s, lane, st->stage[ew], n_staged, p, t0,
                                   st->smin, st->width, st->inv_width);
            // the survivors' scores were fetched from the accumulator again: only now hand it back
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&st->bar_acc_empty[buf]));
          }
        }
        if (!ok) dead = true;
      }
      if (cur_qb >= 0 && !is_refresh) {
        if (kMode == kModeFilter && n_staged > 0) knn_flush(st->stage[ew], n_staged, p, cur_qb * kQB, st->smin, st->width, st->inv_width);
        named_bar_sync(2, kEpiThreads);
        if (warp == kKnnFirstEpi && lane == 0) *reinterpret_cast<volatile int*>(&st->done_seq) = item_seq;
      }
    }
  }

  // ---------------------------------------------------------------------- teardown
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (st->abort_flag) {
    if (threadIdx.x == 0) atomicOr(&p.ctl->status, LT_STATUS_TIMEOUT);
    uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kKnnTmemCols);
  }
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// host side: tensor maps and launch
// ---------------------------------------------------------------------------------------------
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn knn_encode_fn() {
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

// 2-D map over a row-major bf16 matrix [rows][d] with a given row pitch; box = 64 elements (128 bytes) x
// box_rows, 128-byte swizzle, zero fill outside the matrix.
bool knn_map(CUtensorMap* map, const void* base, uint64_t d, uint64_t rows, uint64_t pitch_bytes, uint32_t box_rows) {
  EncodeTiledFn enc = knn_encode_fn();
  if (enc == nullptr) return false;
  cuuint64_t dims[2] = {d, rows};
  cuuint64_t strides[1] = {pitch_bytes};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(kSliceElems), box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

template <int kMode>
cudaError_t knn_launch(const CUtensorMap& tq, const CUtensorMap& tx, const KnnScanParams& p, int grid, cudaStream_t stream) {
  const int bytes = knn_smem_bytes(p.D / kSliceElems);
  cudaError_t e = cudaFuncSetAttribute(knn_scan_kernel<kMode>, cudaFuncAttributeMaxDynamicSharedMemorySize, knn_smem_bytes(kKnnMaxSlices));
  if (e != cudaSuccess) return e;
  knn_scan_kernel<kMode><<<grid, kKnnThreads, bytes, stream>>>(tq, tx, p);
  return cudaGetLastError();
}

}  // namespace

bool scan_knn_supported(int D) { return D >= kSliceElems && D % kSliceElems == 0 && D <= kKnnMaxSlices * kSliceElems; }

cudaError_t launch_scan_knn(int mode, const void* q, int T, const void* x, long long n_keys_view, long long key_pitch_elems,
                            const KnnScanParams& params, int grid, cudaStream_t stream) {
  KnnScanParams p = params;
  if (p.wait_limit_us == 0) p.wait_limit_us = kDefaultWaitLimitUs;
  CUtensorMap tq, tx;
  if (!knn_map(&tq, q, static_cast<uint64_t>(p.D), static_cast<uint64_t>(T), static_cast<uint64_t>(p.D) * 2, kQB))
    return cudaErrorInvalidValue;
  if (!knn_map(&tx, x, static_cast<uint64_t>(p.D), static_cast<uint64_t>(n_keys_view), static_cast<uint64_t>(key_pitch_elems) * 2,
               kTileKeys))
    return cudaErrorInvalidValue;
  return mode == kModeFilter ? knn_launch<kModeFilter>(tq, tx, p, grid, stream) : knn_launch<kModeDump>(tq, tx, p, grid, stream);
}

}  // namespace lt
