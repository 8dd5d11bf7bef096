// A stand-alone check of the error path every tensor-core kernel shares: a bounded wait that runs out.
//
// One CTA, two warps, set up exactly like the pipeline kernels (mbarrier in shared memory, tensor memory
// allocated by warp 1, the same WaitCtx).  Warp 0 waits on a barrier that nothing ever arrives at and that no
// copy is bound to; after `ds.wait_ns` the wait gives up, raises the CTA's abort flag and records the timeout in
// the host-visible status word; the other lanes see the flag and leave; the CTA meets at its final barrier and
// warp 1 frees the tensor memory.  On the way the two warps pass a block-level barrier that carries the news of the
// timeout (named_barrier_or), as the kernels with such barriers in their loops do.  Nothing is in flight at any point, so giving up is safe by construction.
#pragma once
#include "tc_common.cuh"

namespace vdn {

__global__ void __launch_bounds__(64, 1) wait_expiry_selftest_kernel(tc::DevStatus ds, int* left_cleanly) {
  using namespace tc;
  __shared__ __align__(8) unsigned long long bar_storage;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag_storage;
  __shared__ int told_storage;
  volatile int* abort_flag = &abort_flag_storage;
  const uint32_t bar = smem_u32(&bar_storage);
  const WaitCtx wc(abort_flag, ds);
  const int warp = threadIdx.x >> 5;

  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_slot), 32);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = tmem_slot;

  bool ok = true;
  if (warp == 0) ok = mbar_wait(bar, 0, wc);      // never completes: lane 0's clock runs out, the others see the flag

  // Kernels whose threads also meet at block-level barriers inside their loops let a thread that gave up go to the
  // next such barrier and say so, so that nobody is left standing there: warp 1, which waited for nothing, must
  // learn of warp 0's timeout here.
  const bool any_gave_up = named_barrier_or(1, 64, !ok);
  if (threadIdx.x == 32) told_storage = any_gave_up ? 1 : 0;

  // ---- teardown, as in the pipeline kernels
  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 32);
  }
  // bit 0: the wait gave up and the CTA got here; bit 1: the warp that had not waited was told at the barrier
  if (threadIdx.x == 0 && left_cleanly) *left_cleanly = (ok ? 0 : 1) | (told_storage ? 2 : 0);
}

}  // namespace vdn
