// Diagnostic entry point: shows, without touching any gradient data, that a bounded device-side wait of this
// library ends by itself and reports DETOX_ERR_TIMEOUT when nothing ever completes the barrier it waits on.
#include "common.cuh"
#include "mbarrier.cuh"

namespace detox {
namespace {

// One CTA, one warp.  Lane 0 waits on an mbarrier that expects one arrival which never comes; the other lanes
// wait on the same barrier and leave as soon as lane 0 has raised the abort flag (or their own limit passes).
__global__ void bounded_wait_selftest_kernel(int* __restrict__ status, long long limit) {
    __shared__ uint64_t bar;
    __shared__ int abort_word;
    volatile int* abort_flag = &abort_word;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_word = 0;
        mbar_fence_init();
    }
    __syncwarp();
    const bool ok = mbar_wait(&bar, 0u, abort_flag, status, limit);
    // ok can only be false here; a true would mean that the wait returned without the phase having completed
    if (ok) atomicExch(status, -1);
}

}  // namespace
}  // namespace detox

extern "C" detox_status detox_selftest_bounded_wait(int32_t* status, int64_t limit_cycles, void* stream) {
    if (!status || limit_cycles < 1 || limit_cycles > 2000000000LL) return DETOX_ERR_BAD_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(status, 0, sizeof(int32_t), s) != cudaSuccess) return DETOX_ERR_CUDA;
    detox::bounded_wait_selftest_kernel<<<1, 32, 0, s>>>(status, (long long)limit_cycles);
    return detox::launch_status();
}
