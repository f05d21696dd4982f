// Self-test of the bounded-wait path that every compute kernel of the library shares.
//
// One CTA with the same skeleton as the compute kernels: mbarriers in shared memory, a TMEM allocation, roles that wait
// on barriers, and the common teardown.  Nothing ever arrives on the two barriers, so both waits run out by
// construction - after LIMIT_NS instead of the compute kernels' two seconds - and the kernel leaves through the path a
// pipeline fault would take: the role that gives up sets the CTA's abort flag, the other role sees the flag (or its own
// limit) and stops waiting, every warp reaches the teardown, TMEM is freed, and the device status word is set.
// No fault, trap or unbounded loop is involved; the context stays usable.
#pragma once
#include "ptx.cuh"

namespace attn {

template <unsigned long long LIMIT_NS>
__global__ void __launch_bounds__(96) wait_timeout_selftest_kernel(int* status)
{
    using namespace ptx;
    __shared__ __align__(8) uint64_t bars[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        mbar_init(smem_u32(&bars[0]), 1);
        mbar_init(smem_u32(&bars[1]), 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 2) { tmem_alloc(smem_u32(&tmem_base_s), 32); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 0) {                     // a single-thread role (like a producer or an MMA issuer)
        if (lane == 0) mbar_wait<LIMIT_NS>(smem_u32(&bars[0]), 0, &abort_flag);
        __syncwarp();
    } else if (warp == 1) {              // a whole-warp role (like the softmax or compute warps)
        const bool ok = mbar_wait<LIMIT_NS>(smem_u32(&bars[1]), 0, &abort_flag);
        (void)__all_sync(0xffffffffu, ok);
    }
    // teardown, as in the compute kernels
    if (abort_flag) {
        for (int t = 0; t < 64; ++t) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 2) tmem_dealloc(tmem_base_s, 32);
    if (tid == 0 && abort_flag) atomicExch(status, 1);
}

}  // namespace attn
