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

// ---- ranking the counts: top n_out of the N distinct 64-bit keys (count << 32 | ~position) ---------------------
// A grid-wide MSB radix select, one launch per 8-bit digit: every CTA histograms the digit of the keys that
// still match the prefix found so far (per-thread run-length aggregation: neighbouring positions mostly share
// the digit), adds its 256 counters to the global histogram, and the last CTA to finish picks the digit in
// which the count from the top reaches the number of keys still wanted.  The keys are distinct (the position
// is part of them), so after eight digits the prefix IS the n_out-th largest key and no tie needs ranking.
struct RankState {
  unsigned int hist[256];
  unsigned long long prefix;
  unsigned int remaining;
  unsigned int done;
  unsigned int n_written;
  unsigned int pad[3];
};

__device__ __forceinline__ unsigned long long rank_key(unsigned int count, unsigned int pos) {
  return (static_cast<unsigned long long>(count) << 32) | (0xffffffffu - pos);
}

__global__ void __launch_bounds__(256) rank_pass_kernel(const unsigned int* __restrict__ counts, int N, RankState* st, int pass,
                                                         int want) {
  __shared__ unsigned int hist[256];
  __shared__ bool last;
  const int shift = 56 - 8 * pass;
  const unsigned long long mask = pass == 0 ? 0ull : (~0ull << (shift + 8));
  const unsigned long long prefix = st->prefix;
  hist[threadIdx.x] = 0;
  __syncthreads();
  unsigned int run_digit = 0x100u, run_len = 0;
  // each CTA walks one contiguous range of positions with coalesced loads; a thread's consecutive keys are
  // 256 positions apart, which still share their leading digits (the count's high bytes)
  const int per_thread = (N + gridDim.x * blockDim.x - 1) / (gridDim.x * blockDim.x);
  const long long first = static_cast<long long>(blockIdx.x) * blockDim.x * per_thread + threadIdx.x;
  for (int j = 0; j < per_thread; ++j) {
    const long long i = first + static_cast<long long>(j) * blockDim.x;
    if (i >= N) break;
    const unsigned long long key = rank_key(__ldg(counts + i), static_cast<unsigned int>(i));
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
    const unsigned int remaining = pass == 0 ? static_cast<unsigned int>(want) : st->remaining;
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
                                                            unsigned long long* __restrict__ keys, int n_out) {
  const unsigned long long kth = st->prefix;
  const int lane = threadIdx.x & 31;
  const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
  const long long n_round = (N + stride - 1) / stride * stride;
  for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < n_round; i += stride) {
    unsigned long long key = 0;
    bool take = false;
    if (i < N) {
      key = rank_key(__ldg(counts + i), static_cast<unsigned int>(i));
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

// one CTA: sort the n_out keys (descending = count descending, position ascending) and write the outputs
__global__ void __launch_bounds__(1024) rank_sort_kernel(const unsigned long long* __restrict__ keys, int n_out,
                                                          int32_t* __restrict__ out_pos, int32_t* __restrict__ out_count) {
  extern __shared__ uint64_t sel[];
  const int n = next_pow2(n_out < 2 ? 2 : n_out);
  for (int i = threadIdx.x; i < n; i += blockDim.x) sel[i] = i < n_out ? keys[i] : 0ull;
  __syncthreads();
  bitonic_sort_desc(sel, n, threadIdx.x, blockDim.x);
  for (int i = threadIdx.x; i < n_out; i += blockDim.x) {
    out_pos[i] = static_cast<int32_t>(0xffffffffu - static_cast<unsigned int>(sel[i]));
    if (out_count != nullptr) out_count[i] = static_cast<int32_t>(sel[i] >> 32);
  }
}

// out_k[j] = key row at position sample_idx[j] (or j * stride when no list is given), row_bytes bytes (a
// multiple of 16); out_scale[j] = its scale.  One 16-byte piece per thread; positions outside [0, N) are read as
// position 0.  With a paged key cache the position is translated to its physical row first.
__global__ void __launch_bounds__(256) gather_keys_kernel(const uint8_t* __restrict__ k, const float* __restrict__ k_scale,
                                                          const int32_t* __restrict__ sample_idx, long long stride,
                                                          int n_sample, int N, int row_bytes,
                                                          const int* __restrict__ page_table, uint8_t* __restrict__ out_k,
                                                          float* __restrict__ out_scale) {
  const int pieces = row_bytes >> 4;
  const long long g = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  const long long j = g / pieces;
  const int piece = static_cast<int>(g - j * pieces);
  if (j >= n_sample) return;
  long long s = sample_idx != nullptr ? static_cast<long long>(__ldg(sample_idx + j)) : j * stride;
  if (s < 0 || s >= N) s = 0;
  if (page_table != nullptr) s = static_cast<long long>(__ldg(page_table + s / kPageKeys)) * kPageKeys + s % kPageKeys;
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

size_t rank_scratch_bytes(int n_out) { return 1280 + static_cast<size_t>(n_out) * 8; }

// Ranks the N counts and writes the n_out most frequent positions; scratch: rank_scratch_bytes(n_out) bytes,
// 256-byte aligned.
cudaError_t launch_rank_counts(const unsigned int* counts, int N, int n_out, void* scratch, int32_t* out_pos, int32_t* out_count,
                               cudaStream_t stream) {
  static_assert(sizeof(RankState) <= 1088, "state block");
  RankState* st = static_cast<RankState*>(scratch);
  unsigned long long* keys = reinterpret_cast<unsigned long long*>(static_cast<uint8_t*>(scratch) + 1280);
  cudaError_t e = cudaMemsetAsync(st, 0, sizeof(RankState), stream);
  if (e != cudaSuccess) return e;
  int blocks = (N + 256 * 16 - 1) / (256 * 16);
  if (blocks < 1) blocks = 1;
  if (blocks > 148 * 4) blocks = 148 * 4;
  for (int pass = 0; pass < 8; ++pass) rank_pass_kernel<<<blocks, 256, 0, stream>>>(counts, N, st, pass, n_out);
  rank_collect_kernel<<<blocks, 256, 0, stream>>>(counts, N, st, keys, n_out);
  const int smem = next_pow2(n_out < 2 ? 2 : n_out) * 8;
  e = cudaFuncSetAttribute(rank_sort_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  rank_sort_kernel<<<1, 1024, smem, stream>>>(keys, n_out, out_pos, out_count);
  return cudaGetLastError();
}

cudaError_t launch_gather_keys(const void* k, const float* k_scale, const int32_t* sample_idx, long long stride, int n_sample,
                               int N, int row_bytes, const int* page_table, void* out_k, float* out_scale, cudaStream_t stream) {
  const long long threads = static_cast<long long>(n_sample) * (row_bytes >> 4);
  gather_keys_kernel<<<static_cast<int>((threads + 255) / 256), 256, 0, stream>>>(
      static_cast<const uint8_t*>(k), k_scale, sample_idx, stride, n_sample, N, row_bytes, page_table,
      static_cast<uint8_t*>(out_k), out_scale);
  return cudaGetLastError();
}

}  // namespace lt
