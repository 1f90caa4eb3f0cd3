// Shared device helpers for the indexer top-k kernels (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/lt_indexer.h"

namespace lt {

constexpr int kBins = LT_BINS;
constexpr int kTileKeys = 128;  // keys per MMA tile (UMMA M)

// ---------------------------------------------------------------------------------------------
// workspace control block (device memory).  One per call.
// ---------------------------------------------------------------------------------------------
struct Control {
  int status;         // LT_STATUS_* bits
  int fb_rows;        // rows that took the fallback
  int max_survivors;  // largest tail[] of any row
  int tot_survivors;  // sum of tail[] (saturating)
  int overflow_rows;  // rows whose candidate buffer overflowed
  int fb_blocks;      // number of entries in the fallback block list
  int pad[2];
};

// ---------------------------------------------------------------------------------------------
// Index checks of the bounds-checking build (compiled with -DLT_DEBUG_BOUNDS; it stands in for a memory
// checker): LT_IN_BOUNDS(cond, ctl) is `cond`, and where it is false it records LT_STATUS_BOUNDS in the
// status word so that the caller can skip the access and carry on - nothing traps.  In the release build
// it is the constant true and costs nothing.
// ---------------------------------------------------------------------------------------------
#if defined(LT_DEBUG_BOUNDS)
__device__ __forceinline__ bool lt_in_bounds(bool cond, Control* ctl) {
  if (!cond && ctl != nullptr) atomicOr(&ctl->status, LT_STATUS_BOUNDS);
  return cond;
}
#define LT_IN_BOUNDS(cond, ctl) (::lt::lt_in_bounds((cond), (ctl)))
#else
#define LT_IN_BOUNDS(cond, ctl) (true)
#endif

// ---------------------------------------------------------------------------------------------
// total order on (score, index): larger key = better.  Scores are canonicalised (-0 -> +0)
// where they are produced, so bit order equals value order.
// ---------------------------------------------------------------------------------------------
__host__ __device__ __forceinline__ uint32_t score_to_key(uint32_t bits) {
  return (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
}
__host__ __device__ __forceinline__ uint32_t key_to_score_bits(uint32_t key) {
  return (key & 0x80000000u) ? (key & 0x7fffffffu) : ~key;
}
__device__ __forceinline__ uint64_t pack_key(float score, int idx) {
  return (static_cast<uint64_t>(score_to_key(__float_as_uint(score))) << 32) | (0xffffffffu - static_cast<uint32_t>(idx));
}
__device__ __forceinline__ int key_index(uint64_t key) { return static_cast<int>(0xffffffffu - static_cast<uint32_t>(key)); }
__device__ __forceinline__ float key_score(uint64_t key) {
  return __uint_as_float(key_to_score_bits(static_cast<uint32_t>(key >> 32)));
}

// ---------------------------------------------------------------------------------------------
// Equal-width bins over [s_min, s_max] (paper Sec. 3.2 "Sampling").  Bins are DEFINED by their
// lower edges E(b) = fma(b, width, s_min), b = 1..m-1, evaluated by this one function everywhere:
//   bin(s) = largest b in [1, m-1] with E(b) <= s, or 0 if s < E(1).
// Bin 0 therefore also holds everything below the sampled range, bin m-1 everything above it,
// and "s >= E(b)" is exactly "bin(s) >= b" for b >= 1, which makes the float gate and the
// integer histogram agree bit for bit.  Threshold bin 0 means "accept all".
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float bin_edge(int b, float smin, float width) {
  return b <= 0 ? -INFINITY : __fmaf_rn(static_cast<float>(b), width, smin);
}
// `inv_width` is only used for a first guess (1 / width, any rounding); the edge comparisons that
// follow decide, so the result does not depend on it.
__device__ __forceinline__ int bin_of(float s, float smin, float width, float inv_width) {
  if (!(s >= bin_edge(1, smin, width))) return 0;
  if (!(width > 0.f)) return kBins - 1;  // degenerate range: every edge equals s_min
  float g = (s - smin) * inv_width;
  int b = g >= static_cast<float>(kBins - 1) ? kBins - 1 : (g < 1.f ? 1 : static_cast<int>(g));
  while (b < kBins - 1 && s >= bin_edge(b + 1, smin, width)) ++b;
  while (b > 1 && s < bin_edge(b, smin, width)) --b;
  return b;
}
__device__ __forceinline__ int bin_of(float s, float smin, float width) {
  return bin_of(s, smin, width, width > 0.f ? 1.f / width : 0.f);
}

// ---------------------------------------------------------------------------------------------
// bitonic sort of n (power of two, >= 2) 64-bit keys in shared memory, descending.  Every thread
// handles whole compare-exchange pairs: pair t of a stage with distance j is (i, i | j) where i is t
// with a zero bit inserted at bit log2(j), so no thread idles on the upper element of a pair.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void bitonic_sort_desc(uint64_t* s, int n, int tid, int nthreads) {
  const int half = n >> 1;
  for (int k = 2; k <= n; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int t = tid; t < half; t += nthreads) {
        const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
        const int ixj = i | j;
        const uint64_t a = s[i], b = s[ixj];
        const bool desc = (i & k) == 0;
        if (desc ? (a < b) : (a > b)) {
          s[i] = b;
          s[ixj] = a;
        }
      }
      __syncthreads();
    }
  }
}

__host__ __device__ __forceinline__ int next_pow2(int v) {
  int p = 1;
  while (p < v) p <<= 1;
  return p;
}

// keys visible to row t
__host__ __device__ __forceinline__ int visible_keys(int t, int N, int causal_offset) {
  long long v = static_cast<long long>(causal_offset) + t + 1;
  return v < 0 ? 0 : (v > N ? N : static_cast<int>(v));
}

}  // namespace lt
