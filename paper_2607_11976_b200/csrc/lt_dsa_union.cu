// LiteDSA union list + membership masks (paper Sec. 3.3): one CTA per group of adjacent query rows
// marks the group's selected key positions in a bit-packed bitmap in shared memory (atomic OR, so a
// position selected by several rows is kept once), sweeps the bitmap into one ascending list shared by
// the group, and gives every row a bitmask over the list's slots.  Integer work only.
#include <cuda_runtime.h>
#include <stdint.h>

#include "lt_common.cuh"
#include "lt_host.h"

namespace lt {

namespace {

constexpr int kUnionThreads = 1024;
constexpr int kWindowWords = 49152;            // bitmap words per pass: 1,572,864 positions, 192 KB
constexpr int kWordsPerBlock = 8;              // one stored prefix per 8 words (256 positions)
constexpr int kWindowBlocks = kWindowWords / kWordsPerBlock;
constexpr int kUnionSmem = kWindowWords * 4 + kWindowBlocks * 4;

struct UnionParams {
  const int32_t* idx;   // [T][topk]
  int T, topk, N, group;
  int cap;              // group * topk: slots of one group's list
  int mask_words;       // ceil(cap / 32)
  int32_t* union_pos;   // [n_groups][cap], pre-filled with -1
  int32_t* union_len;   // [n_groups]
  uint32_t* mask;       // [T][mask_words], pre-zeroed
};

// exclusive prefix sum of one value per thread over the CTA; *total receives the sum
__device__ __forceinline__ unsigned int block_exclusive_scan(unsigned int v, unsigned int* warp_tot, unsigned int* total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  unsigned int incl = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const unsigned int o = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += o;
  }
  if (lane == 31) warp_tot[wid] = incl;
  __syncthreads();
  if (wid == 0) {
    const unsigned int t = warp_tot[lane];
    unsigned int ti = t;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const unsigned int o = __shfl_up_sync(0xffffffffu, ti, d);
      if (lane >= d) ti += o;
    }
    warp_tot[lane] = ti - t;  // exclusive prefix of the warp totals
    if (lane == 31) *total = ti;
  }
  __syncthreads();
  return warp_tot[wid] + incl - v;
}

__global__ void __launch_bounds__(kUnionThreads, 1) dsa_union_kernel(const UnionParams p) {
  extern __shared__ uint32_t smem_u[];
  uint32_t* bitmap = smem_u;                     // kWindowWords
  uint32_t* block_pref = smem_u + kWindowWords;  // kWindowBlocks: list slots before the block (within the window)
  __shared__ unsigned int warp_tot[32];
  __shared__ unsigned int s_total;
  const int tid = threadIdx.x;
  const int r0 = blockIdx.x * p.group;
  const int r1 = min(p.T, r0 + p.group);
  const long long n_entries = static_cast<long long>(r1 - r0) * p.topk;
  const int32_t* gidx = p.idx + static_cast<size_t>(r0) * p.topk;
  int32_t* out = p.union_pos + static_cast<size_t>(blockIdx.x) * p.cap;
  unsigned int list_len = 0;  // entries written by earlier windows (uniform across the CTA)

  for (long long wbase = 0; wbase < p.N; wbase += static_cast<long long>(kWindowWords) * 32) {
    const long long left = p.N - wbase;
    const int wn = static_cast<int>(left >= static_cast<long long>(kWindowWords) * 32 ? kWindowWords : (left + 31) / 32);
    const long long wend = wbase + static_cast<long long>(wn) * 32 < p.N ? wbase + static_cast<long long>(wn) * 32 : p.N;
    const int n_blocks = (wn + kWordsPerBlock - 1) / kWordsPerBlock;
    for (int i = tid; i < n_blocks * kWordsPerBlock; i += kUnionThreads) bitmap[i] = 0;
    __syncthreads();
    // 1. mark: the atomic OR deduplicates positions selected by several rows
    for (long long e = tid; e < n_entries; e += kUnionThreads) {
      const int pos = __ldg(gidx + e);
      if (pos >= wbase && pos < wend) atomicOr(&bitmap[(pos - wbase) >> 5], 1u << (pos & 31));
    }
    __syncthreads();
    // 2. slots before every 8-word block: each thread owns a run of consecutive blocks
    const int per_thread = (n_blocks + kUnionThreads - 1) / kUnionThreads;
    const int b0 = min(n_blocks, tid * per_thread), b1 = min(n_blocks, b0 + per_thread);
    unsigned int mine = 0;
    for (int b = b0; b < b1; ++b) {
#pragma unroll
      for (int j = 0; j < kWordsPerBlock; ++j) mine += __popc(bitmap[b * kWordsPerBlock + j]);
    }
    unsigned int run = block_exclusive_scan(mine, warp_tot, &s_total);
    // 3. sweep: the set bits of the thread's blocks, in ascending order, go to consecutive slots
    for (int b = b0; b < b1; ++b) {
      block_pref[b] = run;
#pragma unroll
      for (int j = 0; j < kWordsPerBlock; ++j) {
        const int w = b * kWordsPerBlock + j;
        uint32_t word = bitmap[w];
        while (word != 0) {
          const int bit = __ffs(word) - 1;
          word &= word - 1;
          out[list_len + run] = static_cast<int32_t>(wbase + static_cast<long long>(w) * 32 + bit);
          ++run;
        }
      }
    }
    __syncthreads();
    // 4. membership: slot of a position = slots before its block + set bits before it inside the block
    for (long long e = tid; e < n_entries; e += kUnionThreads) {
      const int pos = __ldg(gidx + e);
      if (pos >= wbase && pos < wend) {
        const int w = static_cast<int>((pos - wbase) >> 5);
        const int b = w / kWordsPerBlock;
        unsigned int slot = list_len + block_pref[b];
        for (int j = b * kWordsPerBlock; j < w; ++j) slot += __popc(bitmap[j]);
        slot += __popc(bitmap[w] & ((1u << (pos & 31)) - 1u));
        const int row = r0 + static_cast<int>(e / p.topk);
        atomicOr(p.mask + static_cast<size_t>(row) * p.mask_words + (slot >> 5), 1u << (slot & 31));
      }
    }
    list_len += s_total;
    __syncthreads();
  }
  if (tid == 0) p.union_len[blockIdx.x] = static_cast<int32_t>(list_len);
}

}  // namespace

cudaError_t launch_dsa_union(const int32_t* idx, int T, int topk, int N, int group, int32_t* union_pos, int32_t* union_len,
                             uint32_t* mask, cudaStream_t stream) {
  UnionParams p{};
  p.idx = idx;
  p.T = T;
  p.topk = topk;
  p.N = N;
  p.group = group;
  p.cap = group * topk;
  p.mask_words = (p.cap + 31) / 32;
  p.union_pos = union_pos;
  p.union_len = union_len;
  p.mask = mask;
  const int n_groups = (T + group - 1) / group;
  cudaError_t e = cudaMemsetAsync(union_pos, 0xff, static_cast<size_t>(n_groups) * p.cap * 4, stream);
  if (e != cudaSuccess) return e;
  e = cudaMemsetAsync(mask, 0, static_cast<size_t>(T) * p.mask_words * 4, stream);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(dsa_union_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kUnionSmem);
  if (e != cudaSuccess) return e;
  dsa_union_kernel<<<n_groups, kUnionThreads, kUnionSmem, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace lt
