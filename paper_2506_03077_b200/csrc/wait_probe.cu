// Test kernel for the bounded waits of the tensor-core kernels.
//
// Every mbarrier wait of the library goes through mbar_wait (sm100.cuh), which gives up after a time limit,
// raises the CTA's abort flag and the library's fault flag, and lets the kernel wind down: other roles see the
// abort flag and leave their loops, copies in flight get time to land, tensor memory is freed, the kernel
// returns, and the host reads STREAMBP_E_DEVICE_TIMEOUT.  None of that can be exercised with a real product
// or attention launch without breaking one on purpose.  This kernel runs the same wait, with the limit as a
// parameter (a millisecond instead of two seconds), on a barrier that nothing ever arrives at, and then winds
// down the same way; the GPU is never hung and the context stays usable.
#include "sm100.cuh"

namespace sbp {
namespace {

__global__ void __launch_bounds__(64, 1) wait_probe_kernel(unsigned long long limit_ns) {
    pdl_enter();
    __shared__ __align__(8) unsigned long long bar_storage;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_storage;
    const uint32_t bar = smem_u32(&bar_storage);
    volatile int *abort_flag = &abort_storage;
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_slot), 32);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    // warp 0 waits with the short limit and is the one that gives up; warp 1 waits with the ordinary limit and
    // must leave because it sees the abort flag, as the roles of a real kernel do
    const bool ok = warp == 0 ? mbar_wait_warp(bar, 0, abort_flag, limit_ns) : mbar_wait_warp(bar, 0, abort_flag);
    (void)ok;
    __syncwarp();
    if (*abort_flag) {   // the drain real kernels give their copies in flight
        const unsigned long long t0 = global_timer();
        while (global_timer() - t0 < 200000ull) { }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, 32);
    }
}

}  // namespace

int wait_probe_launch(unsigned long long limit_ns, cudaStream_t st) {
    SBP_LAUNCH(wait_probe_kernel, 1, 64, 0, st, limit_ns);
    return STREAMBP_OK;
}

int wait_probe_take_fault() { return take_fault_local(); }

}  // namespace sbp
