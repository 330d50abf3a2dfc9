// Harmless exercise of the bounded-wait path: a wait that runs out and returns, on a barrier of its own.
#include "tc_common.cuh"

namespace {

// One warp.  An mbarrier that expects one arrival is set up in shared memory and nobody ever arrives on it; lane 0
// waits on it through the same tc::mbar_wait the pipelines use, with the caller's cycle limit.  No TMA, no tensor
// memory, no cluster and no second CTA are involved, so nothing is in flight when the wait gives up: the kernel
// records the outcome the way the pipelines do (OR a code into the error word) and returns.
__global__ void bounded_wait_selftest_kernel(uint32_t* err, long long limit_cycles, long long* waited_cycles) {
    __shared__ __align__(8) uint64_t bar;
    if (threadIdx.x == 0) {
        tc::mbar_init(&bar, 1);
        tc::fence_barrier_init();
    }
    __syncwarp();
    if (threadIdx.x == 0) {
        const long long t0 = clock64();
        const bool done = tc::mbar_wait(&bar, 0, limit_cycles);
        if (waited_cycles) *waited_cycles = clock64() - t0;
        if (!done) atomicOr(err, FREE_DEV_ERR_FULL_WAIT);
    }
}

}  // namespace

extern "C" int free_device_error_code(uint32_t word) { return word ? FREE_ERR_DEVICE_TIMEOUT : FREE_OK; }

extern "C" int free_selftest_bounded_wait(uint32_t* device_error, int64_t limit_cycles, int64_t* waited_cycles, void* stream) {
    if (!device_error) return FREE_ERR_ARG;
    if (limit_cycles < 1 || limit_cycles > 100000000) return FREE_ERR_SHAPE;      // at most ~50 ms of spinning
    if ((reinterpret_cast<uintptr_t>(device_error) & 3u) || (reinterpret_cast<uintptr_t>(waited_cycles) & 7u)) return FREE_ERR_ALIGN;
    bounded_wait_selftest_kernel<<<1, 32, 0, reinterpret_cast<cudaStream_t>(stream)>>>(device_error, (long long)limit_cycles,
                                                                                      reinterpret_cast<long long*>(waited_cycles));
    return free_check_launch();
}
