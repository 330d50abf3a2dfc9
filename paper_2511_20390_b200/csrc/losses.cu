// Drafter training objectives (Sec. 3.2) as one fused reduction: noise MSE (Eq. mse), cosine feature loss (Eq. cos),
// Smooth-L1 on feature residuals (Eqs. smooth, huber) and their weighted sum (Eq. free_loss), forward values only.
//
// Bandwidth-bound: both feature tensors and both noise tensors are read once.  One warp per token row keeps the row's
// dot product, the two squared norms and its Smooth-L1 sum in fp32 lanes (a row is D <= a few thousand values), folds
// them into fp64 per warp, and the CTA then walks its share of the noise elements.  Per-CTA partial sums go to the
// workspace; a second, single-CTA launch adds them in a fixed order, so the result does not depend on scheduling.
#include "internal.h"

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

struct LossArgs {
    long long rows; int D;                 // feature rows (sequences * tokens), width
    long long n_eps;                       // noise elements over the whole batch
    const void *f_pred, *f_ref;
    const float *e_pred, *e_ref;
    float beta, eps_cos;
    double* partial;                       // [grid][3]: sum of cosine terms, Smooth-L1 sum, squared noise error
};

template <typename T> __device__ __forceinline__ void load8(const T* p, float (&v)[8]);
template <> __device__ __forceinline__ void load8<float>(const float* p, float (&v)[8]) {
    const float4 a = __ldcs(reinterpret_cast<const float4*>(p)), b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
template <> __device__ __forceinline__ void load8<__nv_bfloat16>(const __nv_bfloat16* p, float (&v)[8]) {
    const uint4 u = __ldcs(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) { v[2 * i] = __uint_as_float(w[i] << 16); v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u); }
}

// phi_beta(u) with the two constants 0.5 / beta and 0.5 * beta formed once per thread
__device__ __forceinline__ float huber(float u, float beta, float half_inv_beta, float half_beta) {
    const float a = fabsf(u);
    return a < beta ? a * a * half_inv_beta : a - half_beta;
}

template <typename T>
__global__ void __launch_bounds__(kThreads) loss_partial_kernel(LossArgs a) {
    __shared__ double red[kWarps][3];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const T* fp = reinterpret_cast<const T*>(a.f_pred);
    const T* fr = reinterpret_cast<const T*>(a.f_ref);
    double cos_sum = 0.0, hub_sum = 0.0, sq_sum = 0.0;
    const bool vec = (a.D % 8) == 0;
    const float hib = 0.5f / a.beta, hb = 0.5f * a.beta;
    for (long long row = (long long)blockIdx.x * kWarps + warp; row < a.rows; row += (long long)gridDim.x * kWarps) {
        const T* p = fp + row * a.D;
        const T* r = fr + row * a.D;
        float dot = 0.f, np2 = 0.f, nr2 = 0.f, hub = 0.f;
        if (vec) {
#pragma unroll 2
            for (int c = lane * 8; c < a.D; c += 256) {
                float x[8], y[8];
                load8<T>(p + c, x); load8<T>(r + c, y);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    dot = fmaf(x[i], y[i], dot); np2 = fmaf(x[i], x[i], np2); nr2 = fmaf(y[i], y[i], nr2);
                    hub += huber(x[i] - y[i], a.beta, hib, hb);
                }
            }
        } else {
            for (int c = lane; c < a.D; c += 32) {
                const float x = (float)p[c], y = (float)r[c];
                dot = fmaf(x, y, dot); np2 = fmaf(x, x, np2); nr2 = fmaf(y, y, nr2);
                hub += huber(x - y, a.beta, hib, hb);
            }
        }
        dot = free_warp_sum(dot); np2 = free_warp_sum(np2); nr2 = free_warp_sum(nr2); hub = free_warp_sum(hub);
        if (lane == 0) {
            const double den = sqrt((double)np2) * sqrt((double)nr2) + (double)a.eps_cos;
            cos_sum += 1.0 - (double)dot / den;
            hub_sum += (double)hub;
        }
    }
    // noise elements: the grid's threads stride over float4s, the tail goes to thread 0 of CTA 0
    {
        const long long n4 = ((reinterpret_cast<uintptr_t>(a.e_pred) | reinterpret_cast<uintptr_t>(a.e_ref)) & 15u) == 0 ? a.n_eps / 4 : 0;
        float sq = 0.f;
        int run = 0;
        for (long long i = (long long)blockIdx.x * kThreads + threadIdx.x; i < n4; i += (long long)gridDim.x * kThreads) {
            const float4 x = __ldcs(reinterpret_cast<const float4*>(a.e_pred) + i), y = __ldcs(reinterpret_cast<const float4*>(a.e_ref) + i);
            const float d0 = x.x - y.x, d1 = x.y - y.y, d2 = x.z - y.z, d3 = x.w - y.w;
            sq = fmaf(d0, d0, sq); sq = fmaf(d1, d1, sq); sq = fmaf(d2, d2, sq); sq = fmaf(d3, d3, sq);
            if (++run == 64) { sq_sum += (double)sq; sq = 0.f; run = 0; }       // short fp32 runs, fp64 beyond
        }
        sq_sum += (double)sq;
        if (blockIdx.x == 0 && threadIdx.x == 0)
            for (long long i = n4 * 4; i < a.n_eps; ++i) { const double d = (double)a.e_pred[i] - (double)a.e_ref[i]; sq_sum += d * d; }
        sq_sum = free_warp_sum(sq_sum);
    }
    if (lane == 0) { red[warp][0] = cos_sum; red[warp][1] = hub_sum; red[warp][2] = sq_sum; }
    __syncthreads();
    if (threadIdx.x < 3) {
        double s = 0.0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) s += red[w][threadIdx.x];
        a.partial[(long long)blockIdx.x * 3 + threadIdx.x] = s;
    }
}

__global__ void __launch_bounds__(32) loss_final_kernel(int n_part, const double* partial, long long rows, int D, long long n_eps,
                                                        float lambda_f, float lambda_s, double* out) {
    const int lane = threadIdx.x;
    if (lane < 3) {
        double s = 0.0;
        for (int i = 0; i < n_part; ++i) s += partial[(long long)i * 3 + lane];
        const double denom = lane == 0 ? (double)rows : (lane == 1 ? (double)rows * D : (double)n_eps);
        out[lane == 2 ? 0 : lane + 1] = s / denom;             // out = (L_noise, L_feat, L_smooth, L_total)
    }
    __syncwarp();
    if (lane == 0) out[3] = out[0] + (double)lambda_f * out[1] + (double)lambda_s * out[2];
}

}  // namespace

extern "C" size_t free_drafter_loss_workspace_bytes(void) { return (size_t)148 * 8 * 3 * sizeof(double); }

extern "C" int free_drafter_loss(int dtype, int n_seq, int n_tok, int D, int64_t d_eps,
                                 const float* eps_pred, const float* eps_ref, const void* f_pred, const void* f_ref,
                                 float lambda_f, float lambda_s, float beta, float eps_cos,
                                 double* out, void* ws, size_t ws_bytes, void* stream) {
    if (!eps_pred || !eps_ref || !f_pred || !f_ref || !out) return FREE_ERR_ARG;
    if (dtype != FREE_FP32 && dtype != FREE_BF16) return FREE_ERR_ARG;
    if (n_seq < 1 || n_tok < 1 || D < 1 || d_eps < 1 || !(beta > 0.f) || eps_cos < 0.f) return FREE_ERR_SHAPE;
    if (!ws || ws_bytes < free_drafter_loss_workspace_bytes()) return FREE_ERR_WORKSPACE;
    if (!free_aligned16(f_pred) || !free_aligned16(f_ref) || !free_aligned16(ws) || (reinterpret_cast<uintptr_t>(out) & 7u)) return FREE_ERR_ALIGN;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const long long rows = (long long)n_seq * n_tok;
    long long want = (rows + kWarps - 1) / kWarps;
    const long long by_eps = ((long long)n_seq * d_eps / 4 + kThreads - 1) / kThreads;
    if (by_eps > want) want = by_eps;
    const int grid = (int)(want > 148 * 8 ? 148 * 8 : (want < 1 ? 1 : want));
    LossArgs a{rows, D, (long long)n_seq * d_eps, f_pred, f_ref, eps_pred, eps_ref, beta, eps_cos, reinterpret_cast<double*>(ws)};
    if (dtype == FREE_FP32) loss_partial_kernel<float><<<grid, kThreads, 0, s>>>(a);
    else loss_partial_kernel<__nv_bfloat16><<<grid, kThreads, 0, s>>>(a);
    FREE_TRY(free_check_launch());
    loss_final_kernel<<<1, 32, 0, s>>>(grid, a.partial, rows, D, a.n_eps, lambda_f, lambda_s, out);
    return free_check_launch();
}
