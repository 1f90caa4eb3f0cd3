// Measurement aid (no counterpart in the paper): a bare FP8 UMMA stream.  Every CTA keeps the tensor core of its SM
// busy with tcgen05.mma kind::f8f6f4 tiles of the scan's shape (keys x (queries x heads) x 32 bytes) on operands that
// stay in shared memory - no TMA, no epilogue, the accumulators are never read.  What this stream sustains is the
// ceiling of the tensor roofline the scan kernels are held against on the same board, at the clocks and the power the
// board grants it.  Two forms: one CTA per SM (cta_group::1, M 128 x N 256, the scan's form) and CTA pairs
// (cta_group::2, M 256 x N 256: each CTA holds its own 128 rows of A and half of B; the leader issues, follows the
// completions on its own barriers, and the peer waits for it at the closing cluster barrier).  Both do
// 2 x 128 x 256 x 128 x 2 flops per SM and iteration.
#include "lt_host.h"
#include "lt_ptx.cuh"

namespace lt {
namespace {
using namespace ptx;

constexpr int kStreamThreads = 128;
constexpr int kTileBytes = 128 * 128;  // 128 rows of 128 bytes, 128-byte swizzle atoms
constexpr int kStreamTmemCols = 512;

struct StreamTail {
  uint64_t bar[2];
  uint32_t tmem;
  int abort_flag;
  int wait_limit_us;  // directly behind abort_flag: mbar_wait reads it there
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n"
      "}\n" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// one arrival on the issuing CTA's barrier when the pair's UMMAs issued so far have completed
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

template <bool kPair>
__global__ void __launch_bounds__(kStreamThreads, 1) umma_stream_kernel(int iters, int* status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
  uint8_t* smem = smem_raw + pad;
  // A: one key tile.  B: two units of 256 rows (single CTA) or of this CTA's 128 rows (pair).
  constexpr int kBUnit = kPair ? kTileBytes : 2 * kTileBytes;
  const uint32_t a_addr = raw_addr + pad;
  const uint32_t b_addr = a_addr + kTileBytes;
  StreamTail* st = reinterpret_cast<StreamTail*>(smem + kTileBytes + 2 * kBUnit);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = kPair ? cluster_ctarank() : 0u;

  // operands: pseudo-random e4m3 codes, NaN codes (0x7f, 0xff) excluded
  uint32_t h = (blockIdx.x * 977u + threadIdx.x) * 2654435761u + 12345u;
  for (int i = threadIdx.x; i < (kTileBytes + 2 * kBUnit) / 4; i += kStreamThreads) {
    h = h * 1664525u + 1013904223u;
    reinterpret_cast<uint32_t*>(smem)[i] = ((h ^ (h >> 13)) & 0x7e7e7e7eu) | (h & 0x80808080u);
  }
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&st->bar[0]), 1);
    mbar_init(smem_u32(&st->bar[1]), 1);
    st->abort_flag = 0;
    st->wait_limit_us = static_cast<int>(kDefaultWaitLimitUs);
    fence_mbar_init();
  }
  fence_proxy_async();  // the generic-proxy writes above are read by the tensor core
  if (warp == 1) {
    if (kPair) {
      // one warp of each CTA of the pair, same shared-memory offset for the result
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&st->tmem)), "r"(kStreamTmemCols));
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::);
    } else {
      tmem_alloc(smem_u32(&st->tmem), kStreamTmemCols);
      tmem_relinquish();
    }
  }
  tc_fence_before();
  __syncthreads();
  if (kPair) cluster_sync_all();  // the peer's barriers and operands are in place before the leader's first UMMA
  tc_fence_after();
  const uint32_t tmem_base = st->tmem;
  volatile int* abort_flag = &st->abort_flag;

  if (warp == 0 && lane == 0) {
    // instruction descriptor: fp32 accumulators, e4m3 x e4m3, N = 256, M = 128 (256 over the pair)
    constexpr uint32_t idesc = (1u << 4) | (static_cast<uint32_t>(256 >> 3) << 17) | (static_cast<uint32_t>((kPair ? 256 : 128) >> 4) << 24);
    bool ok = true;
    // two iterations in flight: iteration it waits for the commit of iteration it - 2 on the same barrier.  Of a
    // pair only the leader issues and waits; its peer goes straight to the closing cluster barrier.
    if (!kPair || rank == 0) {
      for (int it = 0; it < iters + 2 && ok; ++it) {
        if (it >= 2) ok = mbar_wait<20>(smem_u32(&st->bar[it & 1]), ((it - 2) >> 1) & 1, abort_flag);
        if (!ok || it >= iters) continue;
        tc_fence_after();
#pragma unroll
        for (int u = 0; u < 2; ++u) {
#pragma unroll
          for (int kb = 0; kb < 4; ++kb) {
            const uint64_t a = make_smem_desc_sw128(a_addr) + (kb * 32 >> 4);
            const uint64_t b = make_smem_desc_sw128(b_addr + u * kBUnit) + (kb * 32 >> 4);
            if (kPair) tc_mma_pair(tmem_base + u * 256, a, b, idesc, kb > 0 ? 1u : 0u);
            else tc_mma<true>(tmem_base + u * 256, a, b, idesc, kb > 0 ? 1u : 0u);
          }
        }
        if (kPair) tc_commit_pair(smem_u32(&st->bar[it & 1]));
        else tc_commit(smem_u32(&st->bar[it & 1]));
      }
    }
    if (!ok) atomicOr(status, LT_STATUS_TIMEOUT);
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (kPair) cluster_sync_all();  // neither CTA frees tensor memory while the other may still be written
  if (warp == 1) {
    tc_fence_after();
    if (kPair) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kStreamTmemCols));
    else tmem_dealloc(tmem_base, kStreamTmemCols);
  }
}

template <bool kPair>
cudaError_t launch_stream(int iters, int* status, int grid, cudaStream_t stream) {
  const int smem = 1024 + kTileBytes + 2 * (kPair ? kTileBytes : 2 * kTileBytes) + 256;
  cudaError_t rc = cudaFuncSetAttribute(umma_stream_kernel<kPair>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (rc != cudaSuccess) return rc;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kStreamThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kPair ? 2 : 1;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, umma_stream_kernel<kPair>, iters, status);
}
}  // namespace

cudaError_t launch_umma_stream(bool pair, int iters, int* status, int grid, cudaStream_t stream) {
  return pair ? launch_stream<true>(iters, status, grid, stream) : launch_stream<false>(iters, status, grid, stream);
}

}  // namespace lt
