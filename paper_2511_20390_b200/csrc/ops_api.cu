// Public single-operation entry points (the same kernels the passes launch), used to check each
// kernel against the CPU oracle on its own.
#include "internal.h"
#include <mutex>

namespace {

// token-major qkv [n_seq, n_tok, 3, heads, d_head] -> head-major q, k [n_seq, heads, n_tok, d_pad] (zero padded)
// and v^T [n_seq, heads, d_pad, n_tok]: the operand layout of the tensor-core attention kernel.
__global__ void repack_qkv_kernel(int n_seq, int n_tok, int heads, int dh, int dp, const __nv_bfloat16* qkv,
                                  __nv_bfloat16* q, __nv_bfloat16* k, __nv_bfloat16* vt) {
    const long long total = (long long)n_seq * heads * n_tok * dp;
    const __nv_bfloat16 zero = __float2bfloat16(0.f);
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(i % dp);
        const int t = (int)((i / dp) % n_tok);
        const int h = (int)((i / ((long long)dp * n_tok)) % heads);
        const int s = (int)(i / ((long long)dp * n_tok * heads));
        const long long src = (((long long)s * n_tok + t) * 3) * heads * dh + (long long)h * dh + c;
        const bool in = c < dh;
        q[i] = in ? qkv[src] : zero;
        k[i] = in ? qkv[src + (long long)heads * dh] : zero;
        vt[(((long long)s * heads + h) * dp + c) * n_tok + t] = in ? qkv[src + 2LL * heads * dh] : zero;
    }
}

// v of token-major qkv [n_seq, n_tok, 3, heads, d_head] -> v^T [n_seq, heads, d_pad, n_tok] (zero padded)
__global__ void repack_vt_kernel(int n_seq, int n_tok, int heads, int dh, int dp, const __nv_bfloat16* qkv, __nv_bfloat16* vt) {
    const long long total = (long long)n_seq * heads * dp * n_tok;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int t = (int)(i % n_tok);
        const int c = (int)((i / n_tok) % dp);
        const int h = (int)((i / ((long long)n_tok * dp)) % heads);
        const int s = (int)(i / ((long long)n_tok * dp * heads));
        vt[i] = c < dh ? qkv[(((long long)s * n_tok + t) * 3 + 2) * heads * dh + (long long)h * dh + c] : __float2bfloat16(0.f);
    }
}

}  // namespace

extern "C" size_t free_op_linear_workspace_bytes(void) { return 256; }

extern "C" int free_op_linear(int dtype, int epilogue, int out_dtype, int M, int N, int K,
                              const void* A, const void* W, const float* bias, void* out,
                              float* resid, const float* gate, int64_t gate_stride, int rows_per_seq,
                              void* ws, size_t ws_bytes, void* stream) {
    if (dtype != FREE_FP32 && dtype != FREE_BF16) return FREE_ERR_ARG;
    if (out_dtype != FREE_FP32 && out_dtype != FREE_BF16) return FREE_ERR_ARG;
    if (epilogue < FREE_EPI_BIAS || epilogue > FREE_EPI_GATE_RESIDUAL) return FREE_ERR_ARG;
    if (M < 1 || N < 1 || K < 1) return FREE_ERR_SHAPE;
    if (!A || !W) return FREE_ERR_ARG;
    if (!free_aligned16(A) || !free_aligned16(W) || !free_aligned16(out) || !free_aligned16(resid)) return FREE_ERR_ALIGN;
    if (!ws || ws_bytes < 256) return FREE_ERR_WORKSPACE;
    LinearArgs a;
    a.M = M; a.N = N; a.K = K; a.A = A; a.W = W; a.bias = bias; a.epi = epilogue; a.out_dtype = out_dtype; a.out = out;
    a.resid = resid; a.gate = gate; a.gate_stride = gate_stride; a.rows_per_seq = rows_per_seq > 0 ? rows_per_seq : 1;
    a.err = reinterpret_cast<uint32_t*>(ws);
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (dtype == FREE_FP32) return linear_fp32(a, s);
    if (!linear_bf16_supported(N, K)) return FREE_ERR_UNSUPPORTED;
    return linear_bf16(a, s);
}

extern "C" size_t free_op_attention_workspace_bytes(int dtype, int n_seq, int n_tok, int heads, int d_head) {
    if (dtype != FREE_BF16 || !attention_tc_supported(n_tok, d_head)) return 256;
    return 256 + 3 * free_round_up((size_t)n_seq * heads * n_tok * attention_tc_dpad(d_head) * 2, 256);
}

extern "C" int free_op_attention(int dtype, int n_seq, int n_tok, int heads, int d_head,
                                 const void* qkv, void* out, void* ws, size_t ws_bytes, void* stream) {
    if (dtype != FREE_FP32 && dtype != FREE_BF16) return FREE_ERR_ARG;
    if (n_seq < 1 || n_tok < 1 || heads < 1 || d_head < 1) return FREE_ERR_SHAPE;
    if (!qkv || !out) return FREE_ERR_ARG;
    if (!free_aligned16(qkv) || !free_aligned16(out) || !free_aligned16(ws)) return FREE_ERR_ALIGN;
    if (!ws || ws_bytes < free_op_attention_workspace_bytes(dtype, n_seq, n_tok, heads, d_head)) return FREE_ERR_WORKSPACE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (dtype == FREE_FP32 || !attention_tc_supported(n_tok, d_head))
        return attention_simt(dtype, n_seq, n_tok, heads, d_head, qkv, out, s);
    if (attention_tc2_supported(n_tok, d_head)) {
        // the two-tile kernel reads q and k from the caller's matrix as it is; only v^T is prepared
        const int dp2 = attention_tc2_dpad(d_head);
        __nv_bfloat16* vt2 = (__nv_bfloat16*)((char*)ws + 256);
        const long long tot = (long long)n_seq * heads * n_tok * dp2;
        const unsigned g2 = (unsigned)((tot + 255) / 256 > 148 * 16 ? 148 * 16 : (tot + 255) / 256);
        repack_vt_kernel<<<g2, 256, 0, s>>>(n_seq, n_tok, heads, d_head, dp2, (const __nv_bfloat16*)qkv, vt2);
        FREE_TRY(free_check_launch());
        const int D = heads * d_head;
        return attention_tc2(n_seq, n_tok, heads, d_head, qkv, 3LL * D, 3 * D, 0, D, vt2, out, reinterpret_cast<uint32_t*>(ws), s);
    }
    const int dp = attention_tc_dpad(d_head);
    const size_t per = free_round_up((size_t)n_seq * heads * n_tok * dp * 2, 256);
    char* base = (char*)ws + 256;
    __nv_bfloat16 *q = (__nv_bfloat16*)base, *k = (__nv_bfloat16*)(base + per), *vt = (__nv_bfloat16*)(base + 2 * per);
    const long long total = (long long)n_seq * heads * n_tok * dp;
    const unsigned grid = (unsigned)((total + 255) / 256 > 148 * 16 ? 148 * 16 : (total + 255) / 256);
    repack_qkv_kernel<<<grid, 256, 0, s>>>(n_seq, n_tok, heads, d_head, dp, (const __nv_bfloat16*)qkv, q, k, vt);
    FREE_TRY(free_check_launch());
    return attention_tc(n_seq, n_tok, heads, d_head, dp, q, k, vt, out, reinterpret_cast<uint32_t*>(ws), s);
}

// ------------------------------------------------------------------------------------------------
// Attention without any allocation, for callers that cannot provide a workspace.
//
// Some callers may not allocate device memory at all: code running while a CUDA graph is being captured or
// replayed with a frozen memory plan, plugins of inference servers whose memory pool is owned by the host
// application, and real-time loops that forbid cudaMalloc / cudaFree because those calls synchronise the
// device.  For them the scratch of the tensor-core attention (the head-major copies of q, k and v^T) lives in
// this file-scope device array.  Every GPU that loads the library holds these 12 MiB until the process exits.
// ------------------------------------------------------------------------------------------------
#define FREE_STATIC_ATTN_BYTES (3ull * FREE_STATIC_ATTN_MAX_ELEMS * 2ull)
static __device__ __align__(256) unsigned char g_attn_scratch[FREE_STATIC_ATTN_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
unsigned char* g_scratch_ptr[kMaxDevices] = {};   // device address of g_attn_scratch on each device, once resolved

// In host code `g_attn_scratch` names a host-side shadow of the symbol, not device memory: the device address
// has to be asked for, once per device, with that device current.
int scratch_for_current_device(unsigned char** out) {
    int dev = 0;
    FREE_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return FREE_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        FREE_CUDA_TRY(cudaGetSymbolAddress(&p, g_attn_scratch));
        if (!p) return FREE_ERR_CUDA;
        g_scratch_ptr[dev] = static_cast<unsigned char*>(p);
    }
    *out = g_scratch_ptr[dev];
    return FREE_OK;
}
}  // namespace

extern "C" int free_op_attention_static(int n_seq, int n_tok, int heads, int d_head, const void* qkv, void* out,
                                        uint32_t* device_error, void* stream) {
    if (n_seq < 1 || n_tok < 1 || heads < 1 || d_head < 1) return FREE_ERR_SHAPE;
    if (!qkv || !out || !device_error) return FREE_ERR_ARG;
    if (!free_aligned16(qkv) || !free_aligned16(out) || (reinterpret_cast<uintptr_t>(device_error) & 3u)) return FREE_ERR_ALIGN;
    if (!attention_tc_supported(n_tok, d_head)) return FREE_ERR_UNSUPPORTED;
    const int dp = attention_tc_dpad(d_head);
    const unsigned long long elems = (unsigned long long)n_seq * heads * n_tok * dp;
    if (elems > FREE_STATIC_ATTN_MAX_ELEMS) return FREE_ERR_WORKSPACE;      // beyond the built-in scratch
    unsigned char* base = nullptr;
    FREE_TRY(scratch_for_current_device(&base));
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    // the scratch keeps the previous call's contents: the repack below overwrites every element this call reads
    // (padding included); only the caller's error word has to start at zero
    FREE_CUDA_TRY(cudaMemsetAsync(device_error, 0, 4, s));
    const size_t per = (size_t)FREE_STATIC_ATTN_MAX_ELEMS * 2;
    __nv_bfloat16 *q = (__nv_bfloat16*)base, *k = (__nv_bfloat16*)(base + per), *vt = (__nv_bfloat16*)(base + 2 * per);
    const unsigned grid = (unsigned)((elems + 255) / 256 > 148 * 16 ? 148 * 16 : (elems + 255) / 256);
    repack_qkv_kernel<<<grid, 256, 0, s>>>(n_seq, n_tok, heads, d_head, dp, (const __nv_bfloat16*)qkv, q, k, vt);
    FREE_TRY(free_check_launch());
    return attention_tc(n_seq, n_tok, heads, d_head, dp, q, k, vt, out, device_error, s);
}
