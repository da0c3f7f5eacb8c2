// A one-CTA kernel that makes a bounded wait run out, for the test of the time-out path.
//
// Every mbarrier wait inside the attention kernels is bounded (mbar_wait): on expiry the waiting role raises the CTA's
// abort flag, all roles leave their loops, the CTA takes its normal teardown and the launch reports VPP_DEV_TIMEOUT in
// *status.  In a correct launch no wait ever expires, so that path would never run in a test.  This kernel runs the same
// primitive with a short limit on a barrier that nothing will ever arrive at -- no copy, no MMA and no tensor memory
// are involved, so nothing can fault or hang -- and then does what the kernels' teardown does.
#pragma once
#include "ptx.cuh"

namespace vpp {

__global__ void __launch_bounds__(64, 1) bounded_wait_test_kernel(int32_t* status, long long limit_cycles) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int s_abort;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        fence_mbar_init();
        s_abort = 0;
    }
    __syncthreads();
    // warp 0 waits for an arrival that never comes; warp 1 waits on the same barrier and must be released by the abort
    // flag its neighbour raises (or by its own limit), like the other roles of a CTA whose producer gave up
    const bool ok = mbar_wait_for(b, 0, &s_abort, 900 + (threadIdx.x >> 5), limit_cycles);
    __syncthreads();
    if (threadIdx.x == 0) {
        // teardown as in the attention kernels: a raised abort flag becomes the launch's device status
        if (s_abort != 0) atomicCAS(status, 0, 3 /* VPP_DEV_TIMEOUT */);
        else if (ok) atomicCAS(status, 0, -1);   // (cannot happen: nothing arrives on the barrier)
    }
}

}  // namespace vpp
