// Self-test hooks of the library: exported, but not part of the public header.  They exist so that the
// bounded-wait primitive, which no healthy run ever exercises to its end, can be driven to its give-up on
// purpose without hanging or faulting anything.
#include "common.cuh"
#include "launch.h"

namespace griffin {

// Two warps.  Thread 0 initialises a barrier on which nobody will ever arrive and waits on it through the
// library's wait_or_abort with the given limit; the wait must run out, raise the workspace's status word
// and return false, after which the second warp (which waits on the same barrier and can only leave
// through the CTA's abort flag, as the consumers of the real kernels do) leaves too.
// out[0] = 1 if the wait returned false, out[1] = the cycles it took.
__global__ void __launch_bounds__(64) wait_gives_up_kernel(void *ws, long long limit_cycles, long long *out) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const long long t0 = clock64();
        const bool got = wait_or_abort(&bar, 0, &abort_flag, ws, 99, limit_cycles);
        out[0] = got ? 0 : 1;
        out[1] = clock64() - t0;
    } else if (threadIdx.x >= 32) {
        // waiters that only ever leave through the abort flag (bounded by the library's own limit)
        wait_or_abort(&bar, 0, &abort_flag, nullptr, 98);
    }
}

}  // namespace griffin

extern "C" griffin_status griffin_selftest_wait_gives_up(void *workspace, long long limit_cycles, long long *out /*device, 2*/,
                                                         void *stream) {
    if (workspace == nullptr || out == nullptr) return GRIFFIN_ERR_INVALID_ARG;
    if (limit_cycles < 1 || limit_cycles > 100000000ll) return GRIFFIN_ERR_INVALID_ARG;  // at most ~50 ms
    griffin::wait_gives_up_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(workspace, limit_cycles, out);
    griffin::count_launches(1);
    return cudaGetLastError() == cudaSuccess ? GRIFFIN_OK : GRIFFIN_ERR_CUDA;
}
