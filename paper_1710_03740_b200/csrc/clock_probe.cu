// SM clock probe: a one-warp kernel that measures the clock its SM is running at, by counting SM
// cycles (%clock64) over a window of wall time (%globaltimer).  Enqueued between two kernels of a
// stream it tells at which clock the neighbouring kernels ran - what a power-capped GPU does
// between a tensor-core product and the streaming pass that follows it cannot be seen at the
// 100 ms period of nvidia-smi.
#include "mpt_common.cuh"
#include "tc_ptx.cuh"

namespace mpt {

__global__ void __launch_bounds__(32) k_clock_probe(unsigned long long window_ns, float *mhz_out)
{
    if (threadIdx.x != 0) return;
    const unsigned long long t0 = global_ns();
    const long long c0 = clock64();
    unsigned long long t1 = t0;
    // bounded by construction: the global timer advances on its own
    while (t1 - t0 < window_ns) t1 = global_ns();
    const long long c1 = clock64();
    *mhz_out = (float)((double)(c1 - c0) * 1000.0 / (double)(t1 - t0));
}

cudaError_t launch_clock_probe(unsigned window_us, float *mhz_out, cudaStream_t st)
{
    k_clock_probe<<<1, 32, 0, st>>>((unsigned long long)window_us * 1000ull, mhz_out);
    return cudaGetLastError();
}

}  // namespace mpt
