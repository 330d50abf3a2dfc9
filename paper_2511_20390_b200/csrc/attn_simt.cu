// Multi-head self-attention on CUDA cores for the fp32 mode: softmax(q k^T / sqrt(d_h)) v over all
// tokens of a sequence (non-causal).  One warp per query row; scores of the whole row are kept in shared
// memory (two passes: scores + max, then exp / sum / weighted sum of v), so the result is the plain
// definition with fp32 rounding only.  Operands are token-major: qkv [n_seq, n_tok, 3, heads, d_head].
#include "internal.h"

namespace {

constexpr int kRowsPerCta = 8;
constexpr int kMaxDh = 128;

template <typename T> __device__ __forceinline__ float ld(const T* p);
template <> __device__ __forceinline__ float ld<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ld<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void st(T* p, float v);
template <> __device__ __forceinline__ void st<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void st<__nv_bfloat16>(__nv_bfloat16* p, float v) { *p = __float2bfloat16(v); }

template <typename T>
__global__ void __launch_bounds__(kRowsPerCta * 32) attention_simt_kernel(int n_tok, int heads, int dh, const T* qkv, T* out) {
    extern __shared__ float smem[];                  // [rows][n_tok] scores, then [rows][kMaxDh] query
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int seq = blockIdx.z, head = blockIdx.y;
    const int row = blockIdx.x * kRowsPerCta + warp;
    float* sc = smem + (size_t)warp * n_tok;
    float* qs = smem + (size_t)kRowsPerCta * n_tok + warp * kMaxDh;
    if (row >= n_tok) return;
    const int D = heads * dh;
    const long long tok_stride = 3LL * D;
    const T* base = qkv + (long long)seq * n_tok * tok_stride;
    const T* q = base + (long long)row * tok_stride + head * dh;
    for (int c = lane; c < dh; c += 32) qs[c] = ld(q + c);
    __syncwarp();
    const float scale = rsqrtf((float)dh);
    float mx = -INFINITY;
    for (int j = lane; j < n_tok; j += 32) {
        const T* k = base + (long long)j * tok_stride + D + head * dh;
        float acc = 0.f;
        for (int c = 0; c < dh; ++c) acc = fmaf(qs[c], ld(k + c), acc);
        acc *= scale;
        sc[j] = acc;
        mx = fmaxf(mx, acc);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float sum = 0.f;
    for (int j = lane; j < n_tok; j += 32) { float p = expf(sc[j] - mx); sc[j] = p; sum += p; }
    sum = free_warp_sum(sum);
    __syncwarp();
    const float inv = 1.f / sum;
    for (int c = lane; c < dh; c += 32) {
        float acc = 0.f;
        for (int j = 0; j < n_tok; ++j) {
            const T* v = base + (long long)j * tok_stride + 2 * D + head * dh;
            acc = fmaf(sc[j], ld(v + c), acc);
        }
        st(out + ((long long)seq * n_tok + row) * D + head * dh + c, acc * inv);
    }
}

}  // namespace

int attention_simt(int dtype, int n_seq, int n_tok, int heads, int d_head, const void* qkv, void* out, cudaStream_t s) {
    if (n_seq < 1 || n_tok < 1 || heads < 1 || d_head < 1 || !qkv || !out) return FREE_ERR_ARG;
    if (d_head > kMaxDh) return FREE_ERR_UNSUPPORTED;
    size_t smem = ((size_t)kRowsPerCta * n_tok + kRowsPerCta * kMaxDh) * sizeof(float);
    if (smem > 200 * 1024) return FREE_ERR_UNSUPPORTED;
    dim3 grid((n_tok + kRowsPerCta - 1) / kRowsPerCta, heads, n_seq);
    if (dtype == FREE_FP32) {
        FREE_CUDA_TRY(cudaFuncSetAttribute(attention_simt_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attention_simt_kernel<float><<<grid, kRowsPerCta * 32, smem, s>>>(n_tok, heads, d_head, (const float*)qkv, (float*)out);
    } else {
        FREE_CUDA_TRY(cudaFuncSetAttribute(attention_simt_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attention_simt_kernel<__nv_bfloat16><<<grid, kRowsPerCta * 32, smem, s>>>(n_tok, heads, d_head, (const __nv_bfloat16*)qkv, (__nv_bfloat16*)out);
    }
    return free_check_launch();
}
