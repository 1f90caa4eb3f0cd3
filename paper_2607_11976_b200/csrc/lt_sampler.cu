// Previous-chunk sampler (paper Sec. 3.2 "Sampling"): count how often each key position occurs in a
// chunk's top-k result, rank the counts, and gather the keys of a caller-provided sample into a dense buffer that the
// scan kernel can score through an ordinary tensor map.  Integer / byte work only.
#include <cuda_runtime.h>
#include <stdint.h>

#include "lt_common.cuh"
#include "lt_host.h"

namespace lt {

namespace {

// counts[p] += 1 for every entry p of idx with 0 <= p < N (fire-and-forget atomics; 16-byte loads)
__global__ void __launch_bounds__(256) count_positions_kernel(const int32_t* __restrict__ idx, long long n, int N,
                                                              unsigned int* __restrict__ counts) {
  const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
  long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  const long long n4 = ((reinterpret_cast<uintptr_t>(idx) & 15u) == 0) ? n / 4 : 0;
  const int4* idx4 = reinterpret_cast<const int4*>(idx);
  for (long long j = i; j < n4; j += stride) {
    const int4 v = __ldg(idx4 + j);
    if (static_cast<unsigned int>(v.x) < static_cast<unsigned int>(N)) atomicAdd(counts + v.x, 1u);
    if (static_cast<unsigned int>(v.y) < static_cast<unsigned int>(N)) atomicAdd(counts + v.y, 1u);
    if (static_cast<unsigned int>(v.z) < static_cast<unsigned int>(N)) atomicAdd(counts + v.z, 1u);
    if (static_cast<unsigned int>(v.w) < static_cast<unsigned int>(N)) atomicAdd(counts + v.w, 1u);
  }
  for (long long j = n4 * 4 + i; j < n; j += stride) {
    const int v = __ldg(idx + j);
    if (static_cast<unsigned int>(v) < static_cast<unsigned int>(N)) atomicAdd(counts + v, 1u);
  }
}

// ---- ranking the counts: top n_out of the N distinct keys (count, position) ---------------------------------------
// A key packs the count above the complemented position, (count << pos_bits) | (2^pos_bits - 1 - position), so that
// larger keys mean (count descending, position ascending) and only count_bits + pos_bits bits carry information.
// A grid-wide MSB radix select, one launch per 8-bit digit of those bits: every CTA histograms the digit of the
// keys that still match the prefix found so far (per-thread run-length aggregation: neighbouring positions mostly
// share the digit), adds its 256 counters to the global histogram, and the last CTA to finish picks the digit in
// which the count from the top reaches the number of keys still wanted.  The keys are distinct (the position is
// part of them), so after the last digit the prefix IS the n_out-th largest key and no tie needs ranking.
struct RankState {
  unsigned int hist[256];
  unsigned long long prefix;
  unsigned int remaining;
  unsigned int done;
  unsigned int n_written;
  unsigned int pad[3];
};

constexpr int kRankBatch = 8;  // loads a thread keeps in flight (one CTA-wide load per batch entry)

__device__ __forceinline__ unsigned long long rank_key(unsigned int count, unsigned int pos, int pos_bits) {
  return (static_cast<unsigned long long>(count) << pos_bits) | ((1ull << pos_bits) - 1ull - pos);
}

__global__ void __launch_bounds__(256) rank_pass_kernel(const unsigned int* __restrict__ counts, int N, RankState* st, int shift,
                                                         int first_pass, int pos_bits, int want) {
  __shared__ unsigned int hist[256];
  __shared__ bool last;
  const unsigned long long mask = first_pass ? 0ull : (~0ull << (shift + 8));
  const unsigned long long prefix = st->prefix;
  hist[threadIdx.x] = 0;
  __syncthreads();
  unsigned int run_digit = 0x100u, run_len = 0;
  // each CTA walks one contiguous range of positions with coalesced loads, kRankBatch of them in flight per
  // thread (one load at a time is latency-bound: 16 dependent DRAM round trips per pass); a thread's consecutive
  // keys are 256 positions apart, which still share their leading digits (the count's high bytes)
  const int per_thread = (N + gridDim.x * blockDim.x - 1) / (gridDim.x * blockDim.x);
  const long long first = static_cast<long long>(blockIdx.x) * blockDim.x * per_thread + threadIdx.x;
  for (int j0 = 0; j0 < per_thread; j0 += kRankBatch) {
    unsigned int c[kRankBatch];
#pragma unroll
    for (int u = 0; u < kRankBatch; ++u) {
      const long long i = first + static_cast<long long>(j0 + u) * blockDim.x;
      c[u] = (j0 + u < per_thread && i < N) ? __ldg(counts + i) : 0u;
    }
#pragma unroll
    for (int u = 0; u < kRankBatch; ++u) {
      const long long i = first + static_cast<long long>(j0 + u) * blockDim.x;
      if (j0 + u >= per_thread || i >= N) continue;
      const unsigned long long key = rank_key(c[u], static_cast<unsigned int>(i), pos_bits);
      if ((key & mask) != prefix) continue;
      const unsigned int digit = static_cast<unsigned int>(key >> shift) & 255u;
      if (digit == run_digit) {
        ++run_len;
      } else {
        if (run_len > 0) atomicAdd(&hist[run_digit], run_len);
        run_digit = digit;
        run_len = 1;
      }
    }
  }
  if (run_len > 0) atomicAdd(&hist[run_digit], run_len);
  __syncthreads();
  if (hist[threadIdx.x] != 0) atomicAdd(&st->hist[threadIdx.x], hist[threadIdx.x]);
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) last = atomicAdd(&st->done, 1u) == gridDim.x - 1;
  __syncthreads();
  if (!last) return;
  __threadfence();
  // the complete histogram comes back with one load per thread (a single thread walking it in global memory
  // would pay 256 dependent L2 round trips)
  hist[threadIdx.x] = __ldcg(&st->hist[threadIdx.x]);
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned int remaining = first_pass ? static_cast<unsigned int>(want) : st->remaining;
    unsigned int cum = 0;
    int digit = 0;
    for (int d = 255; d >= 0; --d) {
      const unsigned int c = hist[d];
      if (cum + c >= remaining) {
        digit = d;
        break;
      }
      cum += c;
    }
    st->remaining = remaining - cum;
    st->prefix = prefix | (static_cast<unsigned long long>(digit) << shift);
    st->done = 0;
  }
  __syncthreads();
  st->hist[threadIdx.x] = 0;
}

// every key at or above the n_out-th largest goes to the list (any order; exactly n_out of them)
__global__ void __launch_bounds__(256) rank_collect_kernel(const unsigned int* __restrict__ counts, int N, RankState* st,
                                                            unsigned long long* __restrict__ keys, int n_out, int pos_bits) {
  const unsigned long long kth = st->prefix;
  const int lane = threadIdx.x & 31;
  const int per_thread = (N + gridDim.x * blockDim.x - 1) / (gridDim.x * blockDim.x);
  const long long first = static_cast<long long>(blockIdx.x) * blockDim.x * per_thread + threadIdx.x;
  for (int j0 = 0; j0 < per_thread; j0 += kRankBatch) {
    unsigned int c[kRankBatch];
#pragma unroll
    for (int u = 0; u < kRankBatch; ++u) {
      const long long i = first + static_cast<long long>(j0 + u) * blockDim.x;
      c[u] = (j0 + u < per_thread && i < N) ? __ldg(counts + i) : 0u;
    }
#pragma unroll
    for (int u = 0; u < kRankBatch; ++u) {
      const long long i = first + static_cast<long long>(j0 + u) * blockDim.x;
      unsigned long long key = 0;
      bool take = false;
      if (j0 + u < per_thread && i < N) {
        key = rank_key(c[u], static_cast<unsigned int>(i), pos_bits);
        take = key >= kth;
      }
      const unsigned int ballot = __ballot_sync(0xffffffffu, take);
      if (ballot != 0) {
        unsigned int base = 0;
        if (lane == 0) base = atomicAdd(&st->n_written, static_cast<unsigned int>(__popc(ballot)));
        base = __shfl_sync(0xffffffffu, base, 0);
        const unsigned int pos = base + __popc(ballot & ((1u << lane) - 1u));
        if (take && pos < static_cast<unsigned int>(n_out)) keys[pos] = key;
      }
    }
  }
}

// Order of the n_out winners (count descending, position ascending) by counting: the keys are distinct, so the
// number of larger keys IS a key's place in the output.  CTA (x, y) ranks 256 keys against slice y of the list
// held in shared memory; the slices' partial ranks meet in `rank` (zeroed by the caller).  n_out^2 comparisons
// spread over the whole GPU take a few microseconds where a one-CTA sort of the list took 80.
constexpr int kOrderSlice = 1024;

__global__ void __launch_bounds__(256) rank_count_larger_kernel(const unsigned long long* __restrict__ keys, int n_out,
                                                                 unsigned int* __restrict__ rank) {
  __shared__ unsigned long long slice[kOrderSlice];
  const int s0 = blockIdx.y * kOrderSlice;
  const int len = min(kOrderSlice, n_out - s0);
  for (int i = threadIdx.x; i < len; i += blockDim.x) slice[i] = keys[s0 + i];
  __syncthreads();
  const int me = blockIdx.x * blockDim.x + threadIdx.x;
  if (me >= n_out) return;
  const unsigned long long mine = keys[me];
  unsigned int larger = 0;
#pragma unroll 8
  for (int i = 0; i < len; ++i) larger += slice[i] > mine ? 1u : 0u;
  if (larger != 0) atomicAdd(rank + me, larger);
}

__global__ void __launch_bounds__(256) rank_write_kernel(const unsigned long long* __restrict__ keys, int n_out,
                                                          const unsigned int* __restrict__ rank, int pos_bits,
                                                          int32_t* __restrict__ out_pos, int32_t* __restrict__ out_count) {
  const int me = blockIdx.x * blockDim.x + threadIdx.x;
  if (me >= n_out) return;
  const unsigned long long key = keys[me];
  const unsigned int r = rank[me];
  if (r >= static_cast<unsigned int>(n_out)) return;  // cannot happen for distinct keys
  out_pos[r] = static_cast<int32_t>((1ull << pos_bits) - 1ull - (key & ((1ull << pos_bits) - 1ull)));
  if (out_count != nullptr) out_count[r] = static_cast<int32_t>(key >> pos_bits);
}

// out_k[j] = key row at position sample_idx[j] (or j * stride when no list is given), row_bytes bytes (a
// multiple of 16); out_scale[j] = its scale.  One 16-byte piece per thread; positions outside [0, N) are read as
// position 0.  With a paged key cache the position is translated to its physical row first.
__global__ void __launch_bounds__(256) gather_keys_kernel(const uint8_t* __restrict__ k, const float* __restrict__ k_scale,
                                                          const int32_t* __restrict__ sample_idx, long long stride,
                                                          int n_sample, int N, int row_bytes,
                                                          const int* __restrict__ page_table, long long pool_rows,
                                                          Control* ctl, uint8_t* __restrict__ out_k,
                                                          float* __restrict__ out_scale) {
  const int pieces = row_bytes >> 4;
  const long long g = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  const long long j = g / pieces;
  const int piece = static_cast<int>(g - j * pieces);
  if (j >= n_sample) return;
  long long s = sample_idx != nullptr ? static_cast<long long>(__ldg(sample_idx + j)) : j * stride;
  if (s < 0 || s >= N) s = 0;
  if (page_table != nullptr) {
    s = static_cast<long long>(__ldg(page_table + s / kPageKeys)) * kPageKeys + s % kPageKeys;
    if (!LT_IN_BOUNDS(s >= 0 && s < pool_rows, ctl)) s = 0;  // a page-table entry outside the pool
  }
  const uint4 v = __ldg(reinterpret_cast<const uint4*>(k + static_cast<size_t>(s) * row_bytes) + piece);
  reinterpret_cast<uint4*>(out_k + static_cast<size_t>(j) * row_bytes)[piece] = v;
  if (piece == 0 && k_scale != nullptr) out_scale[j] = __ldg(k_scale + s);
}

}  // namespace

cudaError_t launch_count_positions(const int32_t* idx, long long n, int N, unsigned int* counts, cudaStream_t stream) {
  if (n <= 0) return cudaSuccess;
  long long blocks = (n / 4 + 255) / 256;
  if (blocks < 1) blocks = 1;
  if (blocks > 148 * 16) blocks = 148 * 16;
  count_positions_kernel<<<static_cast<int>(blocks), 256, 0, stream>>>(idx, n, N, counts);
  return cudaGetLastError();
}

size_t rank_scratch_bytes(int n_out) { return 1280 + static_cast<size_t>(n_out) * 12; }

namespace {
int bits_for(unsigned long long max_value) {
  int b = 1;
  while (b < 64 && (max_value >> b) != 0ull) ++b;
  return b;
}
}  // namespace

// Ranks the N counts and writes the n_out most frequent positions; scratch: rank_scratch_bytes(n_out) bytes,
// 256-byte aligned.  max_count: an upper bound of any count (it fixes how many digits the select has to visit).
cudaError_t launch_rank_counts(const unsigned int* counts, int N, int n_out, unsigned long long max_count, void* scratch,
                               int32_t* out_pos, int32_t* out_count, cudaStream_t stream) {
  static_assert(sizeof(RankState) <= 1088, "state block");
  RankState* st = static_cast<RankState*>(scratch);
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(static_cast<uint8_t*>(scratch) + 1280);
  unsigned int* rank = reinterpret_cast<unsigned int*>(keys + n_out);
  cudaError_t e = cudaMemsetAsync(st, 0, sizeof(RankState), stream);
  if (e != cudaSuccess) return e;
  e = cudaMemsetAsync(rank, 0, static_cast<size_t>(n_out) * 4, stream);
  if (e != cudaSuccess) return e;
  if (max_count > 0xffffffffull) max_count = 0xffffffffull;
  const int pos_bits = bits_for(static_cast<unsigned long long>(N - 1));
  const int passes = (bits_for(max_count) + pos_bits + 7) / 8;
  int blocks = (N + 256 * kRankBatch - 1) / (256 * kRankBatch);
  if (blocks < 1) blocks = 1;
  if (blocks > 148 * 4) blocks = 148 * 4;
  for (int pass = 0; pass < passes; ++pass)
    rank_pass_kernel<<<blocks, 256, 0, stream>>>(counts, N, st, 8 * (passes - 1 - pass), pass == 0 ? 1 : 0, pos_bits, n_out);
  rank_collect_kernel<<<blocks, 256, 0, stream>>>(counts, N, st, keys, n_out, pos_bits);
  const int key_blocks = (n_out + 255) / 256;
  rank_count_larger_kernel<<<dim3(key_blocks, (n_out + kOrderSlice - 1) / kOrderSlice), 256, 0, stream>>>(keys, n_out, rank);
  rank_write_kernel<<<key_blocks, 256, 0, stream>>>(keys, n_out, rank, pos_bits, out_pos, out_count);
  return cudaGetLastError();
}

cudaError_t launch_gather_keys(const void* k, const float* k_scale, const int32_t* sample_idx, long long stride, int n_sample,
                               int N, int row_bytes, const int* page_table, long long pool_rows, Control* ctl, void* out_k,
                               float* out_scale, cudaStream_t stream) {
  const long long threads = static_cast<long long>(n_sample) * (row_bytes >> 4);
  gather_keys_kernel<<<static_cast<int>((threads + 255) / 256), 256, 0, stream>>>(
      static_cast<const uint8_t*>(k), k_scale, sample_idx, stride, n_sample, N, row_bytes, page_table, pool_rows, ctl,
      static_cast<uint8_t*>(out_k), out_scale);
  return cudaGetLastError();
}

}  // namespace lt
