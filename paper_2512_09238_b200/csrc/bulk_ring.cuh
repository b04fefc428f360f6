// A shared-memory ring fed by 1-D bulk asynchronous copies (the TMA engine without a tensor
// map), for HBM-bound kernels that stream contiguous rows: one producer thread keeps
// kStages tiles in flight whatever the register budget of the consuming warps, and the
// consumers release a slot as soon as its data sits in their registers.
#pragma once
#include "ptx_sm100.cuh"

namespace tca {

__device__ __forceinline__ void bulk_copy_g2s(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(ptx::smem_u32(smem_dst)), "l"(gmem_src), "r"(bytes), "r"(ptx::smem_u32(bar))
               : "memory");
}

// Named barrier over the first `n_threads` threads of the CTA (the consumer warps).
__device__ __forceinline__ void consumer_sync(int n_threads) {
  asm volatile("bar.sync 1, %0;" ::"r"(n_threads) : "memory");
}

template <int kStages>
struct BulkRing {
  uint64_t full[kStages];
  uint64_t empty[kStages];

  __device__ __forceinline__ void init(uint32_t n_consumers) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(&full[s], 1);
      ptx::mbar_init(&empty[s], n_consumers);
    }
    ptx::fence_barrier_init();
  }
  // producer: wait until slot of tile n is free, then announce `bytes`
  __device__ __forceinline__ bool acquire(int n, uint32_t bytes, volatile int* abort_flag) {
    const int slot = n % kStages;
    if (n >= kStages && !ptx::mbar_wait(&empty[slot], uint32_t(n / kStages - 1) & 1u, abort_flag)) return false;
    ptx::mbar_arrive_expect_tx(&full[slot], bytes);
    return true;
  }
  // consumer: wait for tile n
  __device__ __forceinline__ bool wait_full(int n, volatile int* abort_flag) {
    return ptx::mbar_wait(&full[n % kStages], uint32_t(n / kStages) & 1u, abort_flag);
  }
  // consumer: this thread no longer needs tile n
  __device__ __forceinline__ void release(int n) { ptx::mbar_arrive(&empty[n % kStages]); }
};

}  // namespace tca
