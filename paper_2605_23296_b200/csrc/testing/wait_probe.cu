// Test-only probe, built into its own shared library (never into libcompact_attn): one CTA waits,
// with the library's bounded wait, on an mbarrier that nothing ever arrives at.  The wait must run
// out, record its code in the status word it was given, and the kernel must return.  This is the
// only way the give-up path of the kernels' waits is ever executed: in the product every barrier
// is arrived at.
#include <cuda_runtime.h>

#include <cstdint>

#include "cpa_device.cuh"

namespace {

__global__ void wait_probe_kernel(int32_t* status, uint32_t limit, int32_t* trace) {
    __shared__ __align__(8) uint64_t bar_mem;
    const uint32_t bar = (uint32_t)__cvta_generic_to_shared(&bar_mem);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    __syncthreads();
    bool dead = false;
    const bool done = mbar_wait(bar, 0u, dead, status, limit);   // phase 0 never completes
    // a second wait after the first gave up must return at once
    const bool again = mbar_wait(bar, 0u, dead, status, 0xFFFFFFFFu);
    if (threadIdx.x == 0) {
        trace[0] = done ? 1 : 0;
        trace[1] = dead ? 1 : 0;
        trace[2] = again ? 1 : 0;
        trace[3] = 1;   // the kernel reached its end
    }
}

}  // namespace

// d_status: device int32 the wait reports to (a plan's status word = the first int32 of its index
// buffer); d_trace: device int32[4] = (wait completed, dead flag, second wait completed, reached end);
// limit: tries before the wait gives up.  Returns 0 or the cudaError_t of the launch.
extern "C" __attribute__((visibility("default"))) int cpa_test_wait_probe(int32_t* d_status, int32_t* d_trace,
                                                                            uint32_t limit, void* stream) {
    if (!d_status || !d_trace || limit > (1u << 16)) return -1;
    wait_probe_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(d_status, limit, d_trace);
    return (int)cudaGetLastError();
}
