// tca_selftest_wait_expiry: makes one bounded wait run out, on purpose and harmlessly.
//
// Every mbarrier wait in the tensor-core kernels gives up after a time limit and then leaves
// through one path: the waiter raises the CTA's abort flag, every other waiter of the CTA sees
// the flag at its next probe and returns, the CTA meets at a barrier, the status word of the
// workspace is set, copies in flight get time to land and TMEM is freed.  In production that
// path runs only when something is badly wrong, so this entry point runs it in miniature: one
// CTA with the same roles (a warp that owns TMEM, a waiter with the time limit, waiters that
// only see the abort flag) waits on a barrier that nothing ever arrives at.  Nothing traps and
// nothing waits without a limit; the kernel returns by itself after `limit_ns`.
#include "common.cuh"
#include "ptx_sm100.cuh"

namespace tca {
namespace {

__global__ void __launch_bounds__(128, 1)
wait_expiry_kernel(int* __restrict__ status, unsigned long long limit_ns, unsigned long long* __restrict__ waited_ns) {
  __shared__ uint64_t bars[2];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_word;
  volatile int* abort_flag = &abort_word;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    ptx::mbar_init(&bars[0], 1);   // nobody arrives at either barrier
    ptx::mbar_init(&bars[1], 1);
    ptx::fence_barrier_init();
    abort_word = 0;
  }
  if (warp == 0) {                 // hold TMEM while waiting, as the attention kernels do
    ptx::tmem_alloc(&tmem_slot, 32);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  const unsigned long long t0 = ptx::global_timer_ns();
  bool ok = true;
  if (warp == 1) {
    if (lane == 0) ok = ptx::mbar_wait(&bars[0], 0, abort_flag, limit_ns);            // runs out of time
  } else if (warp >= 2) {
    ok = ptx::mbar_wait(&bars[1], 0, abort_flag, 64ull * limit_ns + 1000000000ull);   // leaves on the flag
  }
  const unsigned long long t1 = ptx::global_timer_ns();
  if (warp == 1 && lane == 0 && waited_ns) *waited_ns = ok ? 0ull : t1 - t0;
  // ---- the teardown of the attention kernels
  ptx::tc_fence_before();
  __syncthreads();
  if (*abort_flag) ptx::abort_teardown(status, tid);
  if (warp == 0) ptx::tmem_dealloc(tmem_base, 32);
}

}  // namespace
}  // namespace tca

using namespace tca;

extern "C" int tca_selftest_wait_expiry(void* ws, uint64_t limit_ns, uint64_t* waited_ns_dev, void* stream) {
  TCA_CHECK_ARG(ws != nullptr && aligned(ws, 256));
  TCA_CHECK_ARG(limit_ns >= 1000 && limit_ns <= 100000000ull);   // 1 us .. 100 ms
  wait_expiry_kernel<<<1, 128, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<int*>(ws), static_cast<unsigned long long>(limit_ns),
      reinterpret_cast<unsigned long long*>(waited_ns_dev));
  return check_launch();
}
