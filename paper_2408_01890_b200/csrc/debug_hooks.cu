// Test hook: exercises the bounded device-side wait of the tensor-core kernels without any of their machinery.
#include "common.cuh"
#include "tc_common.cuh"

namespace lisa {
namespace {

// One warp; lane 0 waits on an mbarrier that expects one arrival and never gets it.  The wait gives up by itself after
// `limit_cycles`, the CTA records it in the status word exactly as the real kernels do, and returns.
__global__ void wait_timeout_kernel(long long limit_cycles, int* status) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        tc::mbar_init(&bar, 1);
        tc::fence_barrier_init();
    }
    __syncthreads();
    bool ok = true;
    if (threadIdx.x == 0) ok = tc::mbar_wait(&bar, 0, &abort_flag, limit_cycles);
    __syncthreads();
    if (threadIdx.x == 0 && (!ok || abort_flag)) atomicAdd(status + 1, 1);
}

}  // namespace
}  // namespace lisa

extern "C" lisa_status_t lisa_debug_wait_timeout(int64_t limit_cycles, lisa_stream_t stream) {
    if (limit_cycles < 1 || limit_cycles > 100000000) return LISA_ERR_INVALID_ARG;   // at most ~50 ms of waiting
    int* status = lisa::status_words();
    if (!status) return LISA_ERR_CUDA;
    lisa::wait_timeout_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>((long long)limit_cycles, status);
    lisa::count_launches(1);
    return cudaGetLastError() == cudaSuccess ? LISA_OK : LISA_ERR_CUDA;
}
