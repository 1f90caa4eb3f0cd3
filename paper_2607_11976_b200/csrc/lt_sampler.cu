// Previous-chunk sampler (paper Sec. 3.2 "Sampling"): count how often each key position occurs in a
// chunk's top-k result, and gather the keys of a caller-provided sample into a dense buffer that the
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

// counts (u32) -> the same numbers as fp32, in place, so that the full-row select can rank them.
// Exact: a count is at most T * topk entries of one matrix, and the launcher rejects matrices with
// more than 2^24 entries per position bound (T <= 2^24).
__global__ void __launch_bounds__(256) counts_to_float_kernel(unsigned int* __restrict__ counts, int N) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < N) counts[i] = __float_as_uint(static_cast<float>(counts[i]));
}

__global__ void __launch_bounds__(256) float_to_counts_kernel(const float* __restrict__ f, int n, int32_t* __restrict__ out) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = static_cast<int32_t>(f[i]);
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

cudaError_t launch_counts_to_float(unsigned int* counts, int N, cudaStream_t stream) {
  counts_to_float_kernel<<<(N + 255) / 256, 256, 0, stream>>>(counts, N);
  return cudaGetLastError();
}

cudaError_t launch_float_to_counts(const float* f, int n, int32_t* out, cudaStream_t stream) {
  float_to_counts_kernel<<<(n + 255) / 256, 256, 0, stream>>>(f, n, out);
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
