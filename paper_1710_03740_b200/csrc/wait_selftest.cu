// Self-test of the bounded device-side wait that every pipeline kernel of this library relies on
// (tc_ptx.cuh, mbar_wait): one CTA initialises an mbarrier that nothing ever arrives on and waits
// for it with a short limit.  The wait must give up, the kernel must record why in the status word
// and return normally, leaving the CUDA context usable.  This is how the time-out path
// (kernel -> status word -> MPT_ERR_TIMEOUT -> poisoned mpt_ctx) is exercised without a hang.
#include "mpt_common.cuh"
#include "tc_ptx.cuh"

namespace mpt {

__global__ void __launch_bounds__(32) k_wait_selftest(unsigned long long limit_ns, uint32_t *status)
{
    __shared__ __align__(8) uint64_t bar;
    __shared__ uint32_t abort_word;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    if (threadIdx.x == 0) {
        const bool arrived = mbar_wait(smem_u32(&bar), 0u, &abort_word, limit_ns);
        if (!arrived && status) atomicCAS(status, 0u, (uint32_t)KERR_WAIT_SELFTEST | 0x20u | ((uint32_t)blockIdx.x << 8));
    }
}

cudaError_t launch_wait_selftest(unsigned limit_us, uint32_t *status, cudaStream_t st)
{
    k_wait_selftest<<<1, 32, 0, st>>>((unsigned long long)limit_us * 1000ull, status);
    return cudaGetLastError();
}

}  // namespace mpt
