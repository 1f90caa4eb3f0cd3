// Selection-side kernels of the indexer top-k: sample statistics, final select over the candidate
// buffers, full-row radix select (generic path, unfused baseline, exact fallback) and the generic
// SIMT scoring kernel.
#include <cuda_bf16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "lt_common.cuh"
#include "lt_host.h"

namespace lt {

namespace {

constexpr int kSelThreads = 1024;
constexpr int kSelBatch = 8;  // independent row loads in flight per thread of the full-row select
constexpr int kSelCap = 2 * LT_MAX_TOPK;  // 64-bit keys the final select can sort in shared memory

// ---------------------------------------------------------------------------------------------
// generic SIMT scoring: one CTA = one query row x 128 keys; thread = one key.
// ---------------------------------------------------------------------------------------------
template <int kDtype>
__device__ __forceinline__ float load_elem(const void* base, size_t i) {
  if (kDtype == LT_DTYPE_F32) return reinterpret_cast<const float*>(base)[i];
  if (kDtype == LT_DTYPE_BF16) return __uint_as_float(static_cast<uint32_t>(reinterpret_cast<const uint16_t*>(base)[i]) << 16);
  __half_raw hr = __nv_cvt_fp8_to_halfraw(reinterpret_cast<const uint8_t*>(base)[i], __NV_E4M3);
  return __half2float(__half(hr));
}

template <int kDtype>
__global__ void __launch_bounds__(128) simt_scores_kernel(const void* __restrict__ q, const float* __restrict__ w,
                                                          const void* __restrict__ k, const float* __restrict__ k_scale, int N,
                                                          int H, int D, int causal_offset, int row_begin, float* __restrict__ out,
                                                          long long ld) {
  extern __shared__ float sm[];
  float* qs = sm;                 // [H][D]
  float* ks = sm + H * D;         // [128][D + 1]
  const int t = row_begin + blockIdx.y;
  const int s0 = blockIdx.x * 128;
  for (int i = threadIdx.x; i < H * D; i += 128) qs[i] = load_elem<kDtype>(q, static_cast<size_t>(t) * H * D + i);
  for (int i = threadIdx.x; i < 128 * D; i += 128) {
    int r = i / D, d = i - r * D;
    int s = s0 + r;
    ks[r * (D + 1) + d] = (s < N) ? load_elem<kDtype>(k, static_cast<size_t>(s) * D + d) : 0.f;
  }
  __syncthreads();
  const int s = s0 + threadIdx.x;
  if (s >= N) return;
  const float* kr = ks + threadIdx.x * (D + 1);
  float total = 0.f;
  for (int h = 0; h < H; ++h) {
    const float* qh = qs + h * D;
    float dot = 0.f;
    for (int d = 0; d < D; ++d) dot = __fmaf_rn(qh[d], kr[d], dot);
    total = __fmaf_rn(w[static_cast<size_t>(t) * H + h], fmaxf(dot, 0.f), total);
  }
  if (k_scale != nullptr) total *= k_scale[s];
  total += 0.f;  // -0 -> +0
  const int vis = visible_keys(t, N, causal_offset);
  out[static_cast<size_t>(blockIdx.y) * ld + s] = (s < vis) ? total : -INFINITY;
}

// ---------------------------------------------------------------------------------------------
// sample statistics: one CTA per row.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) sample_stats_kernel(const float* __restrict__ sample, int n_sample, int rank,
                                                           float* __restrict__ smin_out, float* __restrict__ width_out,
                                                           float* __restrict__ thr_out) {
  __shared__ float red_min[8], red_max[8];
  __shared__ unsigned int hist[kBins];
  __shared__ float s_min, s_width;
  const int t = blockIdx.x;
  const float* row = sample + static_cast<size_t>(t) * n_sample;
  float mn = INFINITY, mx = -INFINITY;
  for (int i = threadIdx.x; i < n_sample; i += 256) {
    float v = row[i];
    mn = fminf(mn, v);
    mx = fmaxf(mx, v);
  }
  for (int d = 16; d > 0; d >>= 1) {
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, d));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
  }
  if ((threadIdx.x & 31) == 0) {
    red_min[threadIdx.x >> 5] = mn;
    red_max[threadIdx.x >> 5] = mx;
  }
  hist[threadIdx.x] = 0;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int i = 1; i < 8; ++i) {
      mn = fminf(mn, red_min[i]);
      mx = fmaxf(mx, red_max[i]);
    }
    if (n_sample <= 0) mn = mx = 0.f;
    s_min = mn;
    s_width = (mx - mn) / static_cast<float>(kBins);
  }
  __syncthreads();
  const float smin = s_min, width = s_width;
  for (int i = threadIdx.x; i < n_sample; i += 256) atomicAdd(&hist[bin_of(row[i], smin, width)], 1u);
  __syncthreads();
  if (threadIdx.x == 0) {
    // threshold bin = bin holding the rank-th largest sampled score; 0 (accept all) if the sample is smaller than that
    int tb = 0;
    unsigned int cum = 0;
    for (int b = kBins - 1; b >= 1; --b) {
      cum += hist[b];
      if (cum >= static_cast<unsigned int>(rank)) {
        tb = b;
        break;
      }
    }
    smin_out[t] = smin;
    width_out[t] = width;
    thr_out[t] = bin_edge(tb, smin, width);
  }
}

// ---------------------------------------------------------------------------------------------
// Stable LSD radix sort of src[0 .. n) by the high word of the keys (the score), descending, 8 bits per pass,
// between src and a second buffer alt of n keys; n <= kRadixSortMax, called by every thread of a CTA of
// kRadixThreads threads.  Warp w owns the contiguous slice [w, w + 1) * 32 * rounds of the input; within a warp
// `match.any` groups the lanes of equal digit, so a key's place is (keys of smaller digits) + (keys of its digit in
// lower warps) + (keys of its digit earlier in its own warp): the order of equal digits is kept, which is what
// makes least-significant-digit-first passes a sort.  A pass in which every key has the same digit (the leading
// bytes of a row's top scores mostly agree) moves nothing and is skipped.  The bitonic network this replaces costs
// ~3.3 k instructions per thread for 2048 keys, four of these passes ~0.7 k.
// Returns the buffer holding the result.  *sorted is false when two neighbours with equal scores ended in the
// wrong index order: the low words took no part, the caller then has to sort the full keys.
// ---------------------------------------------------------------------------------------------
constexpr int kRadixThreads = 512;
constexpr int kRadixSortMax = 4096;
__device__ __forceinline__ uint64_t* radix_sort_by_score_desc(uint64_t* src, uint64_t* alt, int n, bool* sorted) {
  constexpr int kWarps = kRadixThreads / 32;
  constexpr int kMaxRounds = kRadixSortMax / kRadixThreads;
  __shared__ unsigned int cnt[kWarps][256];
  __shared__ unsigned int base[256];
  __shared__ int s_skip, s_unsorted;
  __shared__ unsigned int s_and, s_or;  // bits every score word has / some score word has (known after pass 0)
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int rounds = (n + kRadixThreads - 1) / kRadixThreads;
  const int first = warp * 32 * rounds;
  if (tid == 0) {
    s_and = 0xffffffffu;
    s_or = 0u;
  }
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 32 + 8 * pass;
    // a byte that is the same in every score word (usually the leading one) needs no pass at all
    if (pass > 0 && (((s_and ^ s_or) >> (8 * pass)) & 255u) == 0u) continue;
    for (int i = tid; i < kWarps * 256; i += kRadixThreads) (&cnt[0][0])[i] = 0u;
    __syncthreads();
    uint64_t key[kMaxRounds];
    unsigned int loc[kMaxRounds];
    unsigned int all_bits = 0xffffffffu, any_bits = 0u;
#pragma unroll
    for (int r = 0; r < kMaxRounds; ++r) {
      if (r < rounds) {
        const int i = first + r * 32 + lane;
        const bool valid = i < n;
        key[r] = valid ? src[i] : 0ull;
        // digit 0 = largest byte, so that ascending places are descending scores; idle lanes get digits of their own
        const unsigned int d = valid ? 255u - (static_cast<unsigned int>(key[r] >> shift) & 255u) : 256u + lane;
        const unsigned int peers = __match_any_sync(0xffffffffu, d);
        const unsigned int rank = __popc(peers & ((1u << lane) - 1u));
        const unsigned int before = valid ? cnt[warp][d] : 0u;
        __syncwarp();
        if (valid && rank == 0) cnt[warp][d] = before + __popc(peers);
        __syncwarp();
        loc[r] = before + rank;
        if (valid) {
          all_bits &= static_cast<unsigned int>(key[r] >> 32);
          any_bits |= static_cast<unsigned int>(key[r] >> 32);
        }
      }
    }
    if (pass == 0) {
      all_bits = __reduce_and_sync(0xffffffffu, all_bits);
      any_bits = __reduce_or_sync(0xffffffffu, any_bits);
      if (lane == 0) {
        atomicAnd(&s_and, all_bits);
        atomicOr(&s_or, any_bits);
      }
    }
    __syncthreads();
    if (tid < 256) {
      unsigned int run = 0;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) {
        const unsigned int c = cnt[w][tid];
        cnt[w][tid] = run;
        run += c;
      }
      base[tid] = run;  // keys with this digit
    }
    __syncthreads();
    if (tid < 32) {
      unsigned int c[8], mine = 0;
      bool all_in_one = false;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        c[j] = base[lane * 8 + j];
        mine += c[j];
        all_in_one = all_in_one || c[j] == static_cast<unsigned int>(n);
      }
      unsigned int incl = mine;
#pragma unroll
      for (int dd = 1; dd < 32; dd <<= 1) {
        const unsigned int o = __shfl_up_sync(0xffffffffu, incl, dd);
        if (lane >= dd) incl += o;
      }
      unsigned int run = incl - mine;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        base[lane * 8 + j] = run;
        run += c[j];
      }
      const bool skip = __any_sync(0xffffffffu, all_in_one);
      if (lane == 0) s_skip = skip ? 1 : 0;
    }
    __syncthreads();
    if (s_skip) continue;  // uniform: nothing would move
#pragma unroll
    for (int r = 0; r < kMaxRounds; ++r) {
      if (r < rounds) {
        const int i = first + r * 32 + lane;
        if (i < n) {
          const unsigned int d = 255u - (static_cast<unsigned int>(key[r] >> shift) & 255u);
          alt[base[d] + cnt[warp][d] + loc[r]] = key[r];
        }
      }
    }
    __syncthreads();
    uint64_t* t = src;
    src = alt;
    alt = t;
  }
  if (tid == 0) s_unsorted = 0;
  __syncthreads();
  bool bad = false;
  for (int i = tid; i + 1 < n; i += kRadixThreads) {
    const uint64_t a = src[i], b = src[i + 1];
    bad = bad || ((a >> 32) == (b >> 32) && a < b);
  }
  if (bad) s_unsorted = 1;
  __syncthreads();
  *sorted = s_unsorted == 0;
  return src;
}

// ---------------------------------------------------------------------------------------------
// sort the first `count` keys of sel[] (shared) and write the row's outputs.  alt: an optional second buffer of
// kRadixSortMax keys; with it (and a CTA of kRadixThreads threads) rows of 512 .. kRadixSortMax keys are sorted
// by the radix passes above, and by the bitonic network only if equal scores were left in the wrong order.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void sort_and_write(uint64_t* sel, int count, int topk, int32_t* out_idx, float* out_score,
                                               int n_keys, Control* ctl, uint64_t* alt = nullptr) {
  bool sorted = false;
  if (alt != nullptr && count >= 512 && count <= kRadixSortMax) sel = radix_sort_by_score_desc(sel, alt, count, &sorted);
  if (!sorted) {
    const int n = next_pow2(count < 2 ? 2 : count);
    for (int i = count + threadIdx.x; i < n; i += blockDim.x) sel[i] = 0ull;
    __syncthreads();
    bitonic_sort_desc(sel, n, threadIdx.x, blockDim.x);
  }
  for (int j = threadIdx.x; j < topk; j += blockDim.x) {
    bool have = j < count;
    if (have && !LT_IN_BOUNDS(key_index(sel[j]) >= 0 && key_index(sel[j]) < n_keys, ctl)) have = false;  // never publish an index outside the keys
    out_idx[j] = have ? key_index(sel[j]) : -1;
    if (out_score != nullptr) out_score[j] = have ? key_score(sel[j]) : -INFINITY;
  }
}

// ---------------------------------------------------------------------------------------------
// Keeps the `keep` largest of the `count` distinct 64-bit keys in sel[0 .. count), compacted to sel[0 .. keep)
// in any order.  MSB radix select, 8 bits per pass, histogram in shared memory (hist: 256 counters, scratch: one
// counter); the digit of each pass is found by a warp suffix scan.  Called by every thread of the CTA.
// ---------------------------------------------------------------------------------------------
constexpr int kKeepPerThread = 8;  // keys a thread holds in registers per compaction slab
__device__ __forceinline__ void keep_top_keys(uint64_t* sel, int count, int keep, unsigned int* hist, unsigned int* scratch) {
  __shared__ uint64_t s_prefix64;
  __shared__ unsigned int s_need;
  __shared__ int s_settled;
  const int tid = threadIdx.x, lane = tid & 31, nthreads = blockDim.x;
  if (tid == 0) {
    s_prefix64 = 0;
    s_need = static_cast<unsigned int>(keep);
    s_settled = 0;
  }
  uint64_t mask = 0;
  for (int pass = 0; pass < 8; ++pass) {
    const int shift = 56 - 8 * pass;
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    const uint64_t prefix = s_prefix64;
    for (int i = tid; i < count; i += nthreads) {
      const uint64_t key = sel[i];
      if ((key & mask) == prefix) atomicAdd(&hist[static_cast<unsigned int>(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid < 32) {
      // suffix sums over the 256 digits, 8 per lane: the digit where the count from the top reaches `need`
      unsigned int c[8], mine = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        c[j] = hist[lane * 8 + j];
        mine += c[j];
      }
      unsigned int incl = mine;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const unsigned int o = __shfl_down_sync(0xffffffffu, incl, d);
        if (lane + d < 32) incl += o;
      }
      const unsigned int above = incl - mine, need = s_need;
      if (above < need && incl >= need) {  // exactly one lane
        unsigned int cum = above;
        for (int j = 7; j >= 0; --j) {
          if (cum + c[j] >= need) {
            s_prefix64 = prefix | (static_cast<uint64_t>(lane * 8 + j) << shift);
            s_need = need - cum;
            // every key with this prefix is wanted: the prefix padded with zeros already separates kept from
            // dropped keys, the remaining digits need no pass (the usual case once the score bytes are through)
            if (c[j] == need - cum) s_settled = 1;
            break;
          }
          cum += c[j];
        }
      }
    }
    mask |= 0xffull << shift;
    __syncthreads();
    if (s_settled) break;
  }
  const uint64_t kth = s_prefix64;  // the keep-th largest key, or a lower bound of it that no dropped key reaches
  // compaction in place, a slab of kKeepPerThread * nthreads keys at a time: every thread pulls its keys of
  // the slab into registers, then the kept ones are written from the front (never past what has been read)
  if (tid == 0) *scratch = 0;
  for (int slab = 0; slab < count; slab += kKeepPerThread * nthreads) {
    uint64_t mine[kKeepPerThread];
#pragma unroll
    for (int j = 0; j < kKeepPerThread; ++j) {
      const int i = slab + j * nthreads + tid;
      mine[j] = i < count ? sel[i] : 0ull;
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < kKeepPerThread; ++j) {
      const int i = slab + j * nthreads + tid;
      const bool take = i < count && mine[j] >= kth;
      const unsigned int ballot = __ballot_sync(0xffffffffu, take);
      if (ballot != 0) {
        unsigned int base = 0;
        if (lane == 0) base = atomicAdd(scratch, static_cast<unsigned int>(__popc(ballot)));
        base = __shfl_sync(0xffffffffu, base, 0);
        if (take) sel[base + __popc(ballot & ((1u << lane) - 1u))] = mine[j];
      }
    }
    __syncthreads();
  }
}

// ---------------------------------------------------------------------------------------------
// final select over one row's candidate buffer (paper Sec. 3.2 "Top-k Selection"): the final
// threshold bin is the highest bin whose cumulative count from the top reaches k; every candidate
// at or above its lower edge is pulled into shared memory (the bins above hold fewer than k of
// them), sorted by (score desc, index asc), and the first k are written out.
// ---------------------------------------------------------------------------------------------
constexpr int kFinalThreads = 512;
static_assert(kFinalThreads == kRadixThreads, "the radix sort is written for the final select's CTA size");

__global__ void __launch_bounds__(kFinalThreads) final_select_kernel(const FinalSelectParams p, int sel_cap) {
  extern __shared__ uint64_t sel[];  // sel_cap keys
  __shared__ unsigned int hist[kBins];
  __shared__ int s_tb;
  __shared__ unsigned int s_count;
  const int t = blockIdx.x;
  const int lane = threadIdx.x & 31;
  const unsigned int tail = p.tail[t];
  const int vis = visible_keys(t, p.N, p.causal_offset);
  const int kk = p.topk < vis ? p.topk : vis;
  bool redo = tail > static_cast<unsigned int>(p.cap);
  if (threadIdx.x == 0) {
    atomicMax(&p.ctl->max_survivors, static_cast<int>(tail > 0x7fffffffu ? 0x7fffffffu : tail));
    atomicAdd(&p.ctl->tot_survivors, static_cast<int>(tail > 0x000fffffu ? 0x000fffffu : tail));
    if (redo) atomicAdd(&p.ctl->overflow_rows, 1);
  }
  if (!redo) {
    // candidates are fetched eight rounds at a time so that the loads of a batch overlap; the first batch is
    // issued before the histogram work, which does not depend on it
    constexpr int kBatch = 8;
    const uint2* cand = p.cand + static_cast<size_t>(t) * p.cap;
    const unsigned int rounds = (tail + kFinalThreads - 1) / kFinalThreads;
    uint2 c[kBatch];
#pragma unroll
    for (int j = 0; j < kBatch; ++j) {
      const unsigned int i = j * kFinalThreads + threadIdx.x;
      c[j] = (i < tail) ? __ldcs(cand + i) : make_uint2(0xff800000u, 0u);  // -inf never passes a finite edge
    }
    if (threadIdx.x < kBins) hist[threadIdx.x] = p.hist[static_cast<size_t>(t) * kBins + threadIdx.x];
    if (threadIdx.x == 0) s_count = 0;
    __syncthreads();
    if (threadIdx.x < 32) {
      // suffix sums over the 256 bins, 8 bins per lane, exactly as the refresh warp of the scan does
      unsigned int c[8];
      unsigned int mine = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        c[j] = hist[lane * 8 + j];
        mine += c[j];
      }
      unsigned int incl = mine;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        unsigned int o = __shfl_down_sync(0xffffffffu, incl, d);
        if (lane + d < 32) incl += o;
      }
      const unsigned int above = incl - mine;
      const unsigned int need = static_cast<unsigned int>(kk);
      int tb = 0;
      if (above < need && incl >= need) {
        unsigned int cum = above;
        for (int j = 7; j >= 0; --j) {
          cum += c[j];
          if (cum >= need) {
            tb = lane * 8 + j;
            break;
          }
        }
      }
      // bin 0 is "everything else": a crossing inside lane 0 may legitimately report bin 0
      tb = __reduce_max_sync(0xffffffffu, tb);
      if (need == 0) tb = kBins - 1;
      if (lane == 0) s_tb = tb;
    }
    __syncthreads();
    const float smin = p.smin[t], width = p.width[t];
    const float edge = bin_edge(s_tb, smin, width);
    // every candidate at or above `from` goes to sel[] (one shared-memory atomic per warp); candidates beyond
    // sel_cap are counted but not stored
    auto gather = [&](float from, bool first_batch_loaded) {
      for (unsigned int r0 = 0; r0 < rounds; r0 += kBatch) {
        if (r0 > 0 || !first_batch_loaded) {
#pragma unroll
          for (int j = 0; j < kBatch; ++j) {
            const unsigned int i = (r0 + j) * kFinalThreads + threadIdx.x;
            c[j] = (i < tail) ? __ldcs(cand + i) : make_uint2(0xff800000u, 0u);
          }
        }
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
          const unsigned int i = (r0 + j) * kFinalThreads + threadIdx.x;
          const bool take = (i < tail) && (__uint_as_float(c[j].x) >= from);
          const unsigned int ballot = __ballot_sync(0xffffffffu, take);
          if (ballot != 0) {
            unsigned int base = 0;
            if (lane == 0) base = atomicAdd(&s_count, static_cast<unsigned int>(__popc(ballot)));
            base = __shfl_sync(0xffffffffu, base, 0);
            if (take) {
              const unsigned int pos = base + __popc(ballot & ((1u << lane) - 1u));
              if (pos < static_cast<unsigned int>(sel_cap)) sel[pos] = pack_key(__uint_as_float(c[j].x), static_cast<int>(c[j].y));
            }
          }
        }
      }
    };
    gather(edge, true);
    __syncthreads();
    unsigned int count = s_count;
    if (count > static_cast<unsigned int>(sel_cap) && s_tb >= 1 && s_tb < kBins - 1) {
      // The threshold bin alone holds more candidates than shared memory takes: equal-width bins over a range that
      // a few outliers stretch put most keys into a few bins (heavy-tailed scores).  Second level of the same
      // scheme inside that bin: kBins equal-width bins over [E(tb), E(tb + 1)), the bin in which the count from the
      // top reaches k, and a second gather from its lower edge.  Costs two more sweeps over the row's candidates
      // and spares the row the unfused fallback.
      const int tb = s_tb;
      const float lo = edge, hi = bin_edge(tb + 1, smin, width);
      const float w2 = (hi - lo) / static_cast<float>(kBins);
      if (w2 > 0.f) {
        __shared__ unsigned int fine[kBins];
        __shared__ unsigned int s_above;
        __shared__ float s_from;
        if (threadIdx.x < kBins) fine[threadIdx.x] = 0u;
        if (threadIdx.x < 32) {
          unsigned int above = 0;
          for (int b = tb + 1 + lane; b < kBins; b += 32) above += hist[b];
          above = __reduce_add_sync(0xffffffffu, above);
          if (lane == 0) {
            s_above = above;
            s_count = 0;
          }
        }
        __syncthreads();
        const float inv_w2 = 1.f / w2;
        for (unsigned int i = threadIdx.x; i < tail; i += kFinalThreads) {
          const float v = __uint_as_float(__ldg(&cand[i].x));
          if (v >= lo && v < hi) atomicAdd(&fine[bin_of(v, lo, w2, inv_w2)], 1u);
        }
        __syncthreads();
        if (threadIdx.x < 32) {
          // the fine bin in which the count from the top (bins above tb included) reaches kk
          unsigned int cf[8], mine = 0;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            cf[j] = fine[lane * 8 + j];
            mine += cf[j];
          }
          unsigned int incl = mine;
#pragma unroll
          for (int d = 1; d < 32; d <<= 1) {
            const unsigned int o = __shfl_down_sync(0xffffffffu, incl, d);
            if (lane + d < 32) incl += o;
          }
          const unsigned int need = static_cast<unsigned int>(kk) - s_above;  // >= 1: bins above tb hold fewer than kk
          const unsigned int above = incl - mine;
          int fb = 0;
          if (above < need && incl >= need) {
            unsigned int cum = above;
            for (int j = 7; j >= 0; --j) {
              cum += cf[j];
              if (cum >= need) {
                fb = lane * 8 + j;
                break;
              }
            }
          }
          fb = __reduce_max_sync(0xffffffffu, fb);
          // fine bin 0 starts at the coarse edge itself: nothing gained, the row is redone
          if (lane == 0) s_from = fb >= 1 ? fminf(bin_edge(fb, lo, w2), hi) : lo;
        }
        __syncthreads();
        if (s_from > lo) {
          gather(s_from, false);
          __syncthreads();
          count = s_count;
        }
      }
    }
    // count < kk cannot happen for an exact filter; treating it as "redo" keeps the result exact regardless
    if (count > static_cast<unsigned int>(sel_cap) || count < static_cast<unsigned int>(kk)) redo = true;
    if (!redo) {
      int n_keep = static_cast<int>(count);
      int32_t* out_idx = p.out_idx + static_cast<size_t>(t) * p.topk;
      float* out_score = p.out_score ? p.out_score + static_cast<size_t>(t) * p.topk : nullptr;
      // the upper half of sel[] is a second buffer for the radix sort whenever the keys fit the lower one
      uint64_t* alt = sel_cap >= 2 * kRadixSortMax ? sel + kRadixSortMax : nullptr;
      uint64_t* keys = sel;
      if (alt != nullptr && n_keep >= 512 && n_keep <= kRadixSortMax) {
        // The usual row: a few hundred candidates more than outputs (the threshold bin is included whole).  Sorting
        // all of them by score and writing the first kk is cheaper than selecting the kk-th key first.
        bool sorted;
        keys = radix_sort_by_score_desc(sel, alt, n_keep, &sorted);
        if (sorted) {
          for (int j = threadIdx.x; j < p.topk; j += kFinalThreads) {
            bool have = j < kk;
            if (have && !LT_IN_BOUNDS(key_index(keys[j]) >= 0 && key_index(keys[j]) < p.N, p.ctl)) have = false;
            out_idx[j] = have ? key_index(keys[j]) : -1;
            if (out_score != nullptr) out_score[j] = have ? key_score(keys[j]) : -INFINITY;
          }
          return;
        }
        alt = nullptr;  // equal scores in the wrong index order: the full-key path below, on wherever the keys are now
      }
      if (n_keep > kk && kk > 0) {
        // More candidates than outputs.  The packed keys are distinct (the index is part of them), so the kk-th
        // largest key is unique: find it by a radix select in shared memory and keep exactly the keys at or above it.
        keep_top_keys(keys, n_keep, kk, hist, &s_count);
        n_keep = kk;
      }
      sort_and_write(keys, n_keep, p.topk, out_idx, out_score, p.N, p.ctl, keys == sel ? alt : nullptr);
      return;
    }
  }
  if (threadIdx.x == 0) {
    p.row_flag[t] = 1;
    atomicOr(&p.ctl->status, LT_STATUS_FALLBACK);
    atomicAdd(&p.ctl->fb_rows, 1);
    if (atomicExch(p.block_flag + t / p.rows_per_block, 1u) == 0u) {
      int pos = atomicAdd(&p.ctl->fb_blocks, 1);
      p.fb_list[pos] = t / p.rows_per_block;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// full-row exact select: 4-pass MSB radix select for the k-th key, ordered collection of ties
// (lowest indices first), bitonic sort of the k winners.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSelThreads) select_rows_kernel(const SelectRowsParams p) {
  extern __shared__ uint64_t sel[];  // LT_MAX_TOPK keys
  __shared__ unsigned int hist[256];
  __shared__ unsigned int s_prefix, s_remaining, s_gt;
  __shared__ unsigned int warp_cnt[32];
  int t;
  if (p.fb_list != nullptr) {
    int j = p.fb_round_base + blockIdx.x / p.rows_per_block;
    if (j >= *p.fb_blocks) return;
    t = p.fb_list[j] * p.rows_per_block + blockIdx.x % p.rows_per_block;
    if (t >= p.T || !p.row_flag[t]) return;
  } else {
    t = p.row_begin + blockIdx.x;
    if (p.row_flag != nullptr && !p.row_flag[t]) return;  // only flagged rows are redone
  }
  const float* row = p.scores + static_cast<size_t>(blockIdx.x) * p.ld;
  const int vis = visible_keys(t, p.N, p.causal_offset);
  const int kk = p.topk < vis ? p.topk : vis;
  int32_t* out_idx = p.out_idx + static_cast<size_t>(t) * p.topk;
  float* out_score = p.out_score ? p.out_score + static_cast<size_t>(t) * p.topk : nullptr;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;

  if (vis <= p.topk) {
    // every visible key is selected
    for (int i = tid; i < vis; i += kSelThreads) sel[i] = pack_key(row[i], i);
    __syncthreads();
    sort_and_write(sel, vis, p.topk, out_idx, out_score, p.N, p.ctl);
    return;
  }

  if (tid == 0) {
    s_prefix = 0;
    s_remaining = static_cast<unsigned int>(kk);
  }
  unsigned int mask = 0;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    const unsigned int prefix = s_prefix;
    // Scores of one row share their leading bits, so consecutive candidates of a thread mostly want the
    // same counter: each thread run-length-encodes its digits and issues one atomic per run.
    unsigned int run_digit = 0x100u, run_len = 0;
    // (kSelBatch loads in flight per thread: one row is read by one SM, which is latency-bound otherwise)
    for (int base = 0; base < vis; base += kSelThreads * kSelBatch) {
      float v[kSelBatch];
#pragma unroll
      for (int j = 0; j < kSelBatch; ++j) {
        const int i = base + j * kSelThreads + tid;
        v[j] = i < vis ? row[i] : 0.f;
      }
#pragma unroll
      for (int j = 0; j < kSelBatch; ++j) {
        const int i = base + j * kSelThreads + tid;
        unsigned int digit = 0x100u;  // "not a candidate" (out of range or another prefix)
        if (i < vis) {
          const unsigned int key = score_to_key(__float_as_uint(v[j]));
          if ((key & mask) == prefix) digit = (key >> shift) & 255u;
        }
        if (digit < 0x100u) {
          if (digit == run_digit) {
            ++run_len;
          } else {
            if (run_len > 0) atomicAdd(&hist[run_digit], run_len);
            run_digit = digit;
            run_len = 1;
          }
        }
      }
    }
    if (run_len > 0) atomicAdd(&hist[run_digit], run_len);
    __syncthreads();
    if (tid == 0) {
      unsigned int remaining = s_remaining, cum = 0;
      int digit = 0;
      for (int d = 255; d >= 0; --d) {
        unsigned int c = hist[d];
        if (cum + c >= remaining) {
          digit = d;
          break;
        }
        cum += c;
      }
      s_remaining = remaining - cum;  // still needed among keys that share the longer prefix
      s_prefix = prefix | (static_cast<unsigned int>(digit) << shift);
    }
    mask |= 0xffu << shift;
    __syncthreads();
  }
  const unsigned int kth = s_prefix;                 // key of the k-th largest score
  const unsigned int need_eq = s_remaining;          // how many keys equal to it are selected
  const unsigned int n_gt = static_cast<unsigned int>(kk) - need_eq;
  if (tid == 0) s_gt = 0;
  // Collection.  Keys above the k-th go in any order (the sort follows).  Ties at the k-th value keep
  // the lowest indices, so they are ranked in index order: every warp owns one contiguous range of the
  // row, counts its ties, and after one prefix sum over the 32 warps writes them at their ranks.
  const int per_warp = (((vis + 31) / 32 + 31) / 32) * 32;  // range length: a multiple of 32 covering vis / 32
  const int lo = wid * per_warp;
  const int hi = min(vis, lo + per_warp);
  unsigned int my_eq = 0;
  for (int base = lo; base < hi; base += 32 * kSelBatch) {
    float v[kSelBatch];
#pragma unroll
    for (int j = 0; j < kSelBatch; ++j) {
      const int i = base + j * 32 + lane;
      v[j] = i < hi ? row[i] : 0.f;
    }
#pragma unroll
    for (int j = 0; j < kSelBatch; ++j) {
      const int i = base + j * 32 + lane;
      const bool eq = i < hi && score_to_key(__float_as_uint(v[j])) == kth;
      my_eq += __popc(__ballot_sync(0xffffffffu, eq));
    }
  }
  if (lane == 0) warp_cnt[wid] = my_eq;
  __syncthreads();
  unsigned int running = 0;
  for (int wq = 0; wq < wid; ++wq) running += warp_cnt[wq];
  for (int base0 = lo; base0 < hi; base0 += 32 * kSelBatch) {
   float v[kSelBatch];
#pragma unroll
   for (int j = 0; j < kSelBatch; ++j) {
     const int i = base0 + j * 32 + lane;
     v[j] = i < hi ? row[i] : 0.f;
   }
#pragma unroll
   for (int j = 0; j < kSelBatch; ++j) {
    const int i = base0 + j * 32 + lane;
    unsigned int key = 0;
    bool gt = false, eq = false;
    if (i < hi) {
      key = score_to_key(__float_as_uint(v[j]));
      gt = key > kth;
      eq = key == kth;
    }
    const uint64_t packed = (static_cast<uint64_t>(key) << 32) | (0xffffffffu - static_cast<unsigned int>(i));
    const unsigned int gt_ballot = __ballot_sync(0xffffffffu, gt);
    if (gt_ballot != 0) {
      unsigned int pos = 0;
      if (lane == 0) pos = atomicAdd(&s_gt, static_cast<unsigned int>(__popc(gt_ballot)));
      pos = __shfl_sync(0xffffffffu, pos, 0);
      if (gt) sel[pos + __popc(gt_ballot & ((1u << lane) - 1u))] = packed;
    }
    const unsigned int eq_ballot = __ballot_sync(0xffffffffu, eq);
    if (eq) {
      const unsigned int rank = running + __popc(eq_ballot & ((1u << lane) - 1u));
      if (rank < need_eq) sel[n_gt + rank] = packed;
    }
    running += __popc(eq_ballot);
   }
  }
  __syncthreads();
  sort_and_write(sel, kk, p.topk, out_idx, out_score, p.N, p.ctl);
}

}  // namespace

cudaError_t launch_simt_scores(int dtype, const void* q, const float* w, const void* k, const float* k_scale, int T, int N,
                               int H, int D, int causal_offset, int row_begin, int row_end, float* out, long long ld,
                               cudaStream_t stream) {
  (void)T;
  const int rows = row_end - row_begin;
  if (rows <= 0) return cudaSuccess;
  const size_t smem = (static_cast<size_t>(H) * D + 128 * (D + 1)) * sizeof(float);
  dim3 grid((N + 127) / 128, rows);
  cudaError_t e;
#define LT_SIMT_CASE(DT)                                                                                              \
  e = cudaFuncSetAttribute(simt_scores_kernel<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)); \
  if (e != cudaSuccess) return e;                                                                                       \
  simt_scores_kernel<DT><<<grid, 128, smem, stream>>>(q, w, k, k_scale, N, H, D, causal_offset, row_begin, out, ld);
  if (dtype == LT_DTYPE_F32) {
    LT_SIMT_CASE(LT_DTYPE_F32)
  } else if (dtype == LT_DTYPE_BF16) {
    LT_SIMT_CASE(LT_DTYPE_BF16)
  } else {
    LT_SIMT_CASE(LT_DTYPE_E4M3)
  }
#undef LT_SIMT_CASE
  return cudaGetLastError();
}

cudaError_t launch_sample_stats(const float* sample, int T, int n_sample, int rank, float* smin, float* width, float* thr,
                                cudaStream_t stream) {
  sample_stats_kernel<<<T, 256, 0, stream>>>(sample, n_sample, rank, smin, width, thr);
  return cudaGetLastError();
}

cudaError_t launch_final_select(const FinalSelectParams& p, cudaStream_t stream) {
  // room for every candidate at or above the final threshold edge: k plus the population of the threshold bin,
  // which for a small k over millions of keys can be several thousand (the select that follows cuts them to k)
  int sel_cap = next_pow2(2 * p.topk);
  if (sel_cap < 8192) sel_cap = 8192;
  if (sel_cap > kSelCap) sel_cap = kSelCap;
  const int smem = sel_cap * static_cast<int>(sizeof(uint64_t));
  cudaError_t e = cudaFuncSetAttribute(final_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  final_select_kernel<<<p.T, kFinalThreads, smem, stream>>>(p, sel_cap);
  return cudaGetLastError();
}

cudaError_t launch_select_rows(const SelectRowsParams& p, cudaStream_t stream) {
  const int smem = LT_MAX_TOPK * sizeof(uint64_t);
  cudaError_t e = cudaFuncSetAttribute(select_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  if (p.n_blocks <= 0) return cudaSuccess;
  select_rows_kernel<<<p.n_blocks, kSelThreads, smem, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace lt
