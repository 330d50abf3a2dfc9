// Shared host/device helpers of the free_b200 library.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include "../../include/free_b200.h"

#define FREE_CUDA_TRY(expr)                                   \
    do {                                                      \
        cudaError_t _e = (expr);                              \
        if (_e != cudaSuccess) { (void)cudaGetLastError(); return FREE_ERR_CUDA; } \
    } while (0)

#define FREE_TRY(expr)                                        \
    do { int _r = (expr); if (_r != FREE_OK) return _r; } while (0)

static inline bool free_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static inline int free_check_launch() {
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? FREE_OK : FREE_ERR_CUDA;
}

static inline size_t free_round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// ---- programmatic dependent launch ---------------------------------------------------------------------------
// The kernels of a pass form a chain on one stream, and at small batches the gaps between them (launch latency, the
// set-up of barriers, tensor memory and descriptors, the tail of the last wave) are a large part of a step.  A kernel
// launched with free_launch(overlap = true, ...) may be brought onto the SMs while its predecessor in the stream is still
// running: it does its set-up, then calls free_grid_dep_wait(), which returns once the predecessor has completed and its
// writes are visible, and then lets its own successor come up early in turn (free_grid_dep_launch()).  Both calls do
// nothing in a kernel that was launched the ordinary way.  Nothing before free_grid_dep_wait() may read or write
// global memory that another kernel of the stream touches.
#ifdef __CUDACC__
__device__ __forceinline__ void free_grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void free_grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

bool free_launch_overlap_enabled();      // process-wide switch (free_set_launch_overlap), on by default
// The early launch pays where kernels are short.  On long kernels it measured 1% SLOWER (one round of 196 608 token rows:
// 961 against 971 TFLOP/s on one pod, the GPU at its power cap either way), so it is used up to this many token rows.
static inline bool free_overlap_for_rows(long long rows) { return free_launch_overlap_enabled() && rows <= 16384; }

template <typename... KArgs, typename... Args>
static inline int free_launch(bool overlap, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return FREE_ERR_CUDA; }
    return FREE_OK;
}
#endif

__device__ __forceinline__ float free_gelu_tanh(float a) {
    // 0.5 a (1 + tanh(sqrt(2/pi) (a + 0.044715 a^3)))
    const float k0 = 0.7978845608028654f, k1 = 0.044715f;
    float t = tanhf(k0 * (a + k1 * a * a * a));
    return 0.5f * a * (1.0f + t);
}

__device__ __forceinline__ float free_silu(float a) { return a / (1.0f + expf(-a)); }

__device__ __forceinline__ float free_warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double free_warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
