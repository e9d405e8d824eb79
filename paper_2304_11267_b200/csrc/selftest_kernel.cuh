// Self-test of the kernels' failure path: what a tensor-core kernel of this library does when one of its bounded
// waits runs out.  One block goes through the same steps with the same primitives (tc_common.cuh) -- barriers
// initialised, tensor memory allocated, one thread waiting on a barrier that NOTHING ever arrives on, another on a
// second such barrier with the kernels' full budget -- except that the first wait's budget is a few thousand polls
// (well under a millisecond) instead of the kernels' 2^21.  The first waiter gives up: it raises the block's abort
// flag and records {code, block, site, tile} in the status block; the second waiter sees the flag at its next look
// and leaves; the block drains, releases its tensor memory and RETURNS NORMALLY.  Nothing traps, faults or spins
// without a limit, and the context stays usable.
#pragma once
#include "tc_common.cuh"

namespace sd_attn {

constexpr int SELFTEST_SITE = 99, SELFTEST_TILE = 7;
constexpr uint32_t SELFTEST_POLL_LIMIT = 1u << 12;

__global__ void __launch_bounds__(128) selftest_wait_timeout_kernel(int* status, int* survivors) {
    __shared__ __align__(8) uint64_t bar_never[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar_never[0]), 1);
        mbar_init(smem_u32(&bar_never[1]), 1);
        mbar_init_fence();
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_base_slot), 32);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    volatile int* abort_p = &abort_flag;
    bool ok = true;
    if (warp == 1 && lane == 0)   // gives up after SELFTEST_POLL_LIMIT polls
        ok = mbar_wait<SELFTEST_POLL_LIMIT>(smem_u32(&bar_never[0]), 0, abort_p, status, SELFTEST_SITE, SELFTEST_TILE);
    if (warp == 2 && lane == 0)   // the kernels' own budget: released by the abort flag long before it runs out
        ok = mbar_wait(smem_u32(&bar_never[1]), 0, abort_p, status, SELFTEST_SITE + 1, 0);
    // teardown as in the kernels: every thread arrives, copies in flight (none here) get a bounded chance to land,
    // tensor memory is released
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0 && abort_flag) mbar_drain(smem_u32(&bar_never[0]), 1);   // (parity 1: the phase before the first, complete)
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem_base_slot, 32);
    }
    if (survivors && !ok) atomicAdd(survivors, 1);   // both waiters returned false
}

}  // namespace sd_attn
