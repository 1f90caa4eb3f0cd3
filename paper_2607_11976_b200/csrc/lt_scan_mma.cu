// Tensor-core scan kernel of the fused indexer top-k (sm_100a: TMA -> shared -> tcgen05.mma -> TMEM).
//
// One CTA keeps a block of 8 query rows (8 x 64 heads = 512 operand rows of D = 128) resident in
// shared memory and streams 128-key tiles of K past it.  Per key tile it issues two 128 x 256 x 128
// UMMAs (4 queries each) into a two-stage ring of TMEM accumulators; lanes index keys and columns
// index (query, head), so each epilogue thread owns one key and finishes Eq. 1 of the paper
// (ReLU, head-weighted sum, key scale) as an in-thread FFMA chain over TMEM columns.
//
//   kMode == kModeFilter  paper Sec. 3.2 "Filtering": gate the score against the row's threshold
//                         edge, ballot-compact the survivors of each warp into the row's candidate
//                         buffer (one tail atomic per ballot) and count them in the row's bin
//                         histogram; a spare warp re-derives the threshold bin from the histogram
//                         while the scan runs ("Threshold Refresh") and publishes it by plain store.
//   kMode == kModeDump    write every score (or -inf where masked) to a dense matrix: used for the
//                         sample phase, lt_indexer_scores, the unfused baseline and the exact fallback.
//
// Warp roles (384 threads): 0 TMA producer, 1 UMMA issuer (+ TMEM owner), 2 threshold refresh,
// 3 idle, 4..11 epilogue (two warpgroups; warpgroup g finishes queries 2g, 2g+1 of each unit).
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
constexpr int kUnits = kBlockQ / kUnitQ;    // UMMAs per key tile
constexpr int kUmmaN = kUnitQ * kH;         // 256
constexpr int kTmemCols = 512;              // two accumulator stages of 256 fp32 columns
constexpr int kEpiWarps = 8;
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kThreads = 128 + kEpiThreads;
constexpr int kSwizzleTile = 128 * 128;     // bytes: 128 rows x 128-byte swizzled rows
constexpr int kQTile = 256 * 128;           // bytes: 256 rows x 128-byte rows (one unit, one K-half)

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
  int vis[kBlockQ];
  int dump_row[kBlockQ];
  uint64_t bar_full[8];
  uint64_t bar_empty[8];
  uint64_t bar_q_full;
  uint64_t bar_q_empty;
  uint64_t bar_tmem_full[2];
  uint64_t bar_tmem_empty[2];
  uint32_t tmem_base;
  int abort_flag;
  int epi_abort;
  int done_seq;
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

// Eq. 1 for one key against one query: 64 TMEM columns (per-head dots) -> ReLU -> weighted sum.
// This one function produces every score the library ranks or dumps on the tensor-core path.
__device__ __forceinline__ void head_sum32(const uint32_t (&v)[32], const float* __restrict__ w, float& acc0, float& acc1) {
#pragma unroll
  for (int j = 0; j < 32; j += 4) {
    float4 ww = *reinterpret_cast<const float4*>(w + j);
    acc0 = __fmaf_rn(ww.x, fmaxf(__uint_as_float(v[j + 0]), 0.f), acc0);
    acc1 = __fmaf_rn(ww.y, fmaxf(__uint_as_float(v[j + 1]), 0.f), acc1);
    acc0 = __fmaf_rn(ww.z, fmaxf(__uint_as_float(v[j + 2]), 0.f), acc0);
    acc1 = __fmaf_rn(ww.w, fmaxf(__uint_as_float(v[j + 3]), 0.f), acc1);
  }
}

template <bool kFp8, int kMode>
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
        ok = mbar_wait(smem_u32(&st->bar_q_empty), (n_done & 1) ^ 1, abort_flag);
        if (!ok) break;
        mbar_arrive_expect_tx(smem_u32(&st->bar_q_full), C::kQBytes);
        for (int u = 0; u < kUnits; ++u)
          for (int hf = 0; hf < C::kHalves; ++hf)
            tma_load_2d(q_base + (u * C::kHalves + hf) * kQTile, &tm_q, hf * C::kElemsPerRow128,
                        (it.t0 + u * kUnitQ) * kH, smem_u32(&st->bar_q_full));
        ++n_done;
        for (int tile = it.tile_lo; tile < it.tile_hi; ++tile) {
          ok = mbar_wait(smem_u32(&st->bar_empty[stage]), phase ^ 1, abort_flag);
          if (!ok) break;
          mbar_arrive_expect_tx(smem_u32(&st->bar_full[stage]), C::kStageBytes);
          for (int hf = 0; hf < C::kHalves; ++hf)
            tma_load_2d(k_base + stage * C::kStageBytes + hf * kSwizzleTile, &tm_k, hf * C::kElemsPerRow128,
                        tile * kTileKeys, smem_u32(&st->bar_full[stage]));
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
      int acc = 0;
      uint32_t acc_phase = 0;
      uint32_t n_done = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
        Item it;
        if (!resolve_item(p, n_blocks, item, it)) continue;
        ok = mbar_wait(smem_u32(&st->bar_q_full), n_done & 1, abort_flag);
        if (!ok) break;
        ++n_done;
        for (int tile = it.tile_lo; tile < it.tile_hi && ok; ++tile) {
          ok = mbar_wait(smem_u32(&st->bar_full[stage]), phase, abort_flag);
          if (!ok) break;
          for (int u = 0; u < kUnits; ++u) {
            ok = mbar_wait(smem_u32(&st->bar_tmem_empty[acc]), acc_phase ^ 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int kb = 0; kb < C::kKBlocks; ++kb) {
              const int hf = kFp8 ? 0 : (kb >> 2);
              const int step = kFp8 ? kb : (kb & 3);
              uint64_t a = make_smem_desc_sw128(k_base + stage * C::kStageBytes + hf * kSwizzleTile) + (step * 32 >> 4);
              uint64_t b = make_smem_desc_sw128(q_base + (u * C::kHalves + hf) * kQTile) + (step * 32 >> 4);
              tc_mma<kFp8>(tmem_base + acc * kUmmaN, a, b, idesc, kb > 0 ? 1u : 0u);
            }
            tc_commit(smem_u32(&st->bar_tmem_full[acc]));
            acc ^= 1;
            if (acc == 0) acc_phase ^= 1;
          }
          tc_commit(smem_u32(&st->bar_empty[stage]));
          if (++stage == C::kStages) {
            stage = 0;
            phase ^= 1;
          }
        }
        tc_commit(smem_u32(&st->bar_q_empty));
      }
    }
  } else if (warp == 2 || warp >= 4) {
    // ------------------------------------------------------------------ epilogue (+ refresh warp)
    const bool is_refresh = (warp == 2);
    const int n_sync = (kMode == kModeFilter) ? kEpiThreads + 32 : kEpiThreads;
    if (!(is_refresh && kMode != kModeFilter)) {
      const int e = threadIdx.x - 128;        // epilogue thread number (valid for warp >= 4)
      const int quarter = warp & 3;           // TMEM lane quarter this warp may read
      const int g = (warp - 4) >> 2;          // warpgroup: queries 2g, 2g+1 of each unit
      const int key_in_tile = quarter * 32 + lane;
      int acc = 0;
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
            st->w[i] = (t < p.T) ? p.w[static_cast<size_t>(t) * kH + (i % kH)] : 0.f;
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
            }
          }
          if (e == 0) st->epi_abort = *abort_flag;
        }
        named_bar_sync(1, n_sync);  // B: shared state of this item is ready
        if (st->epi_abort) break;

        if (is_refresh) {
          // ---- paper Sec. 3.2 "Threshold Refresh": walk each row's histogram from the top bin
          // down until the cumulative count reaches k; publish the bin's lower edge by plain store.
          int cur_tb[kBlockQ];
#pragma unroll
          for (int r = 0; r < kBlockQ; ++r) cur_tb[r] = 0;
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
            if (*reinterpret_cast<volatile int*>(&st->done_seq) >= seq || *abort_flag) break;
            __nanosleep(400);
          }
          continue;
        }

        // ---- epilogue proper
        for (int tile = it.tile_lo; tile < it.tile_hi; ++tile) {
          const int s = tile * kTileKeys + key_in_tile;
          float ks = 1.f;
          if (p.k_scale != nullptr && s < p.n_keys) ks = __ldg(p.k_scale + static_cast<size_t>(s) * p.ks_stride);
          bool ok = true;
          for (int u = 0; u < kUnits; ++u) {
            ok = mbar_wait(smem_u32(&st->bar_tmem_full[acc]), acc_phase, abort_flag);
            if (!ok) break;
            tc_fence_after();
            float score[2];
#pragma unroll
            for (int qq = 0; qq < 2; ++qq) {
              const int r = u * kUnitQ + g * 2 + qq;
              const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                                     static_cast<uint32_t>(acc * kUmmaN + (g * 2 + qq) * kH);
              float acc0 = 0.f, acc1 = 0.f;
              uint32_t v[32];
              tmem_ld32(taddr, v);
              tmem_ld_wait();
              head_sum32(v, st->w + r * kH, acc0, acc1);
              tmem_ld32(taddr + 32, v);
              tmem_ld_wait();
              if (qq == 1) {
                // both queries' columns are in registers: hand the accumulator stage back
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&st->bar_tmem_empty[acc]));
              }
              head_sum32(v, st->w + r * kH + 32, acc0, acc1);
              score[qq] = (acc0 + acc1) * ks + 0.f;  // + 0 turns -0 into +0
            }
            acc ^= 1;
            if (acc == 0) acc_phase ^= 1;
#pragma unroll
            for (int qq = 0; qq < 2; ++qq) {
              const int r = u * kUnitQ + g * 2 + qq;
              const bool visible = s < st->vis[r];
              if (kMode == kModeDump) {
                int dr = st->dump_row[r];
                if (dr >= 0 && s < p.n_keys) p.dump[static_cast<size_t>(dr) * p.dump_ld + s] = visible ? score[qq] : -INFINITY;
              } else {
                // ---- paper Sec. 3.2 "Filtering": gate, ballot-compact, batched append, histogram
                const float thr = *reinterpret_cast<volatile float*>(&st->thr[r]);
                const bool pass = visible && (score[qq] >= thr);
                const uint32_t ballot = __ballot_sync(0xffffffffu, pass);
                if (ballot != 0) {
                  const int t = it.t0 + r;
                  uint32_t base = 0;
                  if (lane == 0) base = atomicAdd(p.tail + t, static_cast<uint32_t>(__popc(ballot)));
                  base = __shfl_sync(0xffffffffu, base, 0);
                  if (pass) {
                    uint32_t pos = base + __popc(ballot & ((1u << lane) - 1u));
                    if (pos < static_cast<uint32_t>(p.cap))
                      p.cand[static_cast<size_t>(t) * p.cap + pos] = make_uint2(__float_as_uint(score[qq]), static_cast<uint32_t>(s));
                    int b = bin_of(score[qq], st->smin[r], st->width[r]);
                    atomicAdd(p.hist + static_cast<size_t>(t) * kBins + b, 1u);
                  }
                }
              }
            }
          }
          if (!ok) break;
        }
        if (warp == 4 && lane == 0) *reinterpret_cast<volatile int*>(&st->done_seq) = seq;
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

template <bool kFp8, int kMode>
cudaError_t launch(const CUtensorMap& tq, const CUtensorMap& tk, const ScanParams& p, int grid, cudaStream_t stream) {
  constexpr int bytes = smem_bytes<kFp8>();
  cudaError_t e = cudaFuncSetAttribute(scan_kernel<kFp8, kMode>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e != cudaSuccess) return e;
  scan_kernel<kFp8, kMode><<<grid, kThreads, bytes, stream>>>(tq, tk, p);
  return cudaGetLastError();
}

}  // namespace

bool scan_mma_supported(int dtype, int H, int D) {
  return (dtype == LT_DTYPE_BF16 || dtype == LT_DTYPE_E4M3) && H == kH && D == kD;
}

cudaError_t launch_scan_mma(int dtype, int mode, const void* q, int T, const void* k, long long n_keys_view,
                            long long key_pitch_elems, const ScanParams& p, int grid, cudaStream_t stream) {
  const bool fp8 = (dtype == LT_DTYPE_E4M3);
  const size_t esz = fp8 ? 1 : 2;
  CUtensorMap tq, tk;
  if (!make_map(&tq, fp8, q, static_cast<uint64_t>(T) * kH, kD * esz, 256)) return cudaErrorInvalidValue;
  if (!make_map(&tk, fp8, k, static_cast<uint64_t>(n_keys_view), static_cast<uint64_t>(key_pitch_elems) * esz, 128))
    return cudaErrorInvalidValue;
  if (fp8) {
    return mode == kModeFilter ? launch<true, kModeFilter>(tq, tk, p, grid, stream) : launch<true, kModeDump>(tq, tk, p, grid, stream);
  }
  return mode == kModeFilter ? launch<false, kModeFilter>(tq, tk, p, grid, stream) : launch<false, kModeDump>(tq, tk, p, grid, stream);
}

}  // namespace lt
