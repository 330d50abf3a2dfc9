// Verification straight from the noise predictions of the packed target pass: classifier-free guidance, the
// reverse-transition means m_k = coef_x x_k - coef_eps eps_k (Eq. ddpm_update), Algorithm 2 (reflection maximal
// coupling) with the first-rejection break of Algorithm 1 and the relaxed acceptance of Eq. acc_relax, in one kernel.
// The means never exist in memory: compared with "tail kernel, then spec_verify" the [B,K,d] mean tensor is neither
// written nor read, and the packed states x_k are the drafts themselves (x_1..x_{K-1} = x_hat_0..x_hat_{K-2}), so
// each draft row is fetched from HBM once and found in L2 when it is needed in its second role.
//
// Bandwidth-bound: every operand is streamed with 16-byte coalesced loads.  One thread-block cluster owns one sample.
// Per draft each thread accumulates s1 = |d|^2 and s2 = d.r in fp64 (d = m_hat - m, r = x_hat - m_hat, m formed in
// fp64 registers); warp shuffles, shared memory and distributed shared memory reduce them in a fixed order, and every
// CTA derives the same decisions.  Optional early exit: drafts are examined in chunks and the rows after the chunk
// that holds the first rejection are never read.
#include "internal.h"
#include <cooperative_groups.h>
#include <math.h>

namespace cg = cooperative_groups;

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

struct FusedArgs {
    int B, K, G, chunk;
    long long d;
    float cfg;
    const float* eps;
    const float* x_first; long long x_first_stride;
    const float *mh, *xh, *coef_x, *coef_eps, *sigma2, *lambda, *u;
    const int32_t* n_valid;
    float* x_out; int32_t* n_accept; float* logratio; float* dist2; float* means_out;
};

struct Row {                      // operands of draft k of this sample
    const float *ec, *eu, *x, *mh, *xh;
    float* means;                 // or nullptr
    double cx, ce, w;
};

template <bool G2>
__device__ __forceinline__ double mean_of(const Row& r, float ec, float eu, float x) {
    double e = (double)ec;
    if (G2) e = fma(r.w, e - (double)eu, (double)eu);          // eps_u + w (eps_c - eps_u)
    return fma(r.cx, (double)x, -r.ce * e);
}

template <bool G2>
__device__ __forceinline__ float accumulate(const Row& r, double& s1, double& s2, float ec, float eu, float x, float mh, float xh) {
    const double m = mean_of<G2>(r, ec, eu, x);
    const double dm = (double)mh - m, rr = (double)xh - (double)mh;
    s1 = fma(dm, dm, s1);
    s2 = fma(dm, rr, s2);
    return (float)m;
}

template <bool G2>
__device__ __forceinline__ void accumulate4(const Row& r, long long i, double& s1, double& s2, const float4& ec, const float4& eu,
                                            const float4& x, const float4& mh, const float4& xh) {
    float4 m;
    m.x = accumulate<G2>(r, s1, s2, ec.x, eu.x, x.x, mh.x, xh.x);
    m.y = accumulate<G2>(r, s1, s2, ec.y, eu.y, x.y, mh.y, xh.y);
    m.z = accumulate<G2>(r, s1, s2, ec.z, eu.z, x.z, mh.z, xh.z);
    m.w = accumulate<G2>(r, s1, s2, ec.w, eu.w, x.w, mh.w, xh.w);
    if (r.means) reinterpret_cast<float4*>(r.means)[i] = m;
}

template <int CLUSTER, bool VEC4, bool G2>
__global__ void __launch_bounds__(kThreads, 4) spec_verify_fused_kernel(FusedArgs a) {
    __shared__ double warp_part[FREE_MAX_K][kWarps][2];
    __shared__ double cta_part[FREE_MAX_K][2];
    __shared__ double tot[FREE_MAX_K][2];
    __shared__ double ell_s[FREE_MAX_K];
    __shared__ int ok_s[FREE_MAX_K];

    const int rank = (CLUSTER > 1) ? (int)cg::this_cluster().block_rank() : 0;
    const int b = blockIdx.x / CLUSTER;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = a.K;
    int nv = a.n_valid ? a.n_valid[b] : K;
    nv = nv < 0 ? 0 : (nv > K ? K : nv);
    const long long d = a.d;
    const int stride = CLUSTER * kThreads;
    const int first = rank * kThreads + tid;

    auto row = [&](int k) -> Row {
        const size_t bk = (size_t)b * K + k;
        Row r;
        r.ec = a.eps + bk * a.G * d;
        r.eu = G2 ? r.ec + d : r.ec;
        r.x = k == 0 ? a.x_first + (size_t)b * a.x_first_stride : a.xh + (bk - 1) * d;
        r.mh = a.mh + bk * d;
        r.xh = a.xh + bk * d;
        r.means = a.means_out ? a.means_out + bk * d : nullptr;
        r.cx = (double)a.coef_x[bk];
        r.ce = (double)a.coef_eps[bk];
        r.w = (double)a.cfg;
        return r;
    };

    // ---------------- phase A, chunk by chunk: partial sums, decisions, stop after the first rejection
    const int chunk = a.chunk > 0 ? a.chunk : (K > 0 ? K : 1);
    int examined = 0, jrej = -1, err = 0;
    for (int k0 = 0; k0 < nv; k0 += chunk) {
        const int k1 = k0 + chunk < nv ? k0 + chunk : nv;
        for (int k = k0; k < k1; ++k) {
            const Row r = row(k);
            double s1 = 0.0, s2 = 0.0;
            if (VEC4) {
                const float4* pc = reinterpret_cast<const float4*>(r.ec);
                const float4* pu = reinterpret_cast<const float4*>(r.eu);
                const float4* px = reinterpret_cast<const float4*>(r.x);
                const float4* ph = reinterpret_cast<const float4*>(r.mh);
                const float4* pd = reinterpret_cast<const float4*>(r.xh);
                const long long n4 = d >> 2;
                long long i = first;
                for (; i + stride < n4; i += 2LL * stride) {          // two 16-byte loads per stream in flight per thread
                    const float4 c0 = __ldg(pc + i), u0 = G2 ? __ldg(pu + i) : c0, x0 = __ldg(px + i), h0 = __ldg(ph + i), d0 = __ldg(pd + i);
                    const float4 c1 = __ldg(pc + i + stride), u1 = G2 ? __ldg(pu + i + stride) : c1, x1 = __ldg(px + i + stride),
                                 h1 = __ldg(ph + i + stride), d1 = __ldg(pd + i + stride);
                    accumulate4<G2>(r, i, s1, s2, c0, u0, x0, h0, d0);
                    accumulate4<G2>(r, i + stride, s1, s2, c1, u1, x1, h1, d1);
                }
                for (; i < n4; i += stride) {
                    const float4 c0 = __ldg(pc + i), u0 = G2 ? __ldg(pu + i) : c0, x0 = __ldg(px + i), h0 = __ldg(ph + i), d0 = __ldg(pd + i);
                    accumulate4<G2>(r, i, s1, s2, c0, u0, x0, h0, d0);
                }
            } else {
                for (long long i = first; i < d; i += stride) {
                    const float m = accumulate<G2>(r, s1, s2, __ldg(r.ec + i), __ldg(r.eu + i), __ldg(r.x + i), __ldg(r.mh + i), __ldg(r.xh + i));
                    if (r.means) r.means[i] = m;
                }
            }
            s1 = free_warp_sum(s1);
            s2 = free_warp_sum(s2);
            if (lane == 0) { warp_part[k][warp][0] = s1; warp_part[k][warp][1] = s2; }
        }
        __syncthreads();
        if (tid < k1 - k0) {
            const int k = k0 + tid;
            double s1 = 0.0, s2 = 0.0;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) { s1 += warp_part[k][w][0]; s2 += warp_part[k][w][1]; }
            cta_part[k][0] = s1; cta_part[k][1] = s2;
        }
        if (CLUSTER > 1) cg::this_cluster().sync(); else __syncthreads();
        if (tid < k1 - k0) {                              // every CTA derives the same values in the same order
            const int k = k0 + tid;
            double s1 = 0.0, s2 = 0.0;
            if (CLUSTER > 1) {
                cg::cluster_group cl = cg::this_cluster();
                for (int r = 0; r < CLUSTER; ++r) {
                    const double* rp = cl.map_shared_rank(&cta_part[0][0], r);
                    s1 += rp[2 * k]; s2 += rp[2 * k + 1];
                }
            } else { s1 = cta_part[k][0]; s2 = cta_part[k][1]; }
            const size_t bk = (size_t)b * K + k;
            const double sg = (double)a.sigma2[bk];
            const double lam = a.lambda ? (double)a.lambda[bk] : 1.0;
            const double uu = (double)a.u[bk];
            const bool bad = !(sg > 0.0) || isinf(sg);
            const double ell = bad ? nan("") : -lam * (s2 + 0.5 * s1) / sg;
            const double log_u = uu <= 0.0 ? -INFINITY : log(uu);
            ell_s[k] = ell;
            ok_s[k] = bad ? -1 : (log_u <= fmin(0.0, ell) ? 1 : 0);
            tot[k][0] = s1; tot[k][1] = s2;
        }
        __syncthreads();
        for (int k = k0; k < k1; ++k) {                   // the same scan in every thread of every CTA
            if (ok_s[k] < 0) err = 1;
            else if (ok_s[k] == 0 && jrej < 0) jrej = k;
        }
        examined = k1;
        if (err || jrej >= 0) break;
    }
    // no CTA may leave while a peer can still read its shared memory
    if (CLUSTER > 1) cg::this_cluster().sync();

    const int j = jrej >= 0 ? jrej : nv;
    if (rank == 0) {
        if (tid == 0) a.n_accept[b] = err ? FREE_ERR_SIGMA : j;
        if (a.logratio && tid < K) a.logratio[(size_t)b * K + tid] = tid < examined ? (float)ell_s[tid] : nanf("");
        if (a.dist2 && tid < K) a.dist2[(size_t)b * K + tid] = tid < examined ? (float)tot[tid][0] : nanf("");
    }
    if (err || nv == 0) return;

    // ---------------- phase B: this CTA's slice of the finalised state
    float* out = a.x_out + (size_t)b * d;
    if (j == nv) {                                        // every draft accepted: the last draft is the state
        const float* src = a.xh + ((size_t)b * K + nv - 1) * d;
        if (VEC4) {
            for (long long i = first; i < (d >> 2); i += stride) reinterpret_cast<float4*>(out)[i] = __ldg(reinterpret_cast<const float4*>(src) + i);
        } else {
            for (long long i = first; i < d; i += stride) out[i] = __ldg(src + i);
        }
        return;
    }
    const double s1 = tot[j][0], s2 = tot[j][1];
    const double coef = s1 > 0.0 ? 2.0 * s2 / s1 : 0.0;   // 2 (e.r) / |d| folded with e = d / |d|
    const bool ident = !(s1 > 0.0);
    const Row r = row(j);
    auto refl = [&](float ec, float eu, float x, float mh, float xh) -> float {
        if (ident) return xh;
        const double m = mean_of<G2>(r, ec, eu, x);
        const double dm = (double)mh - m, rr = (double)xh - (double)mh;
        return (float)(m + rr - coef * dm);
    };
    if (VEC4) {
        const float4* pc = reinterpret_cast<const float4*>(r.ec);
        const float4* pu = reinterpret_cast<const float4*>(r.eu);
        const float4* px = reinterpret_cast<const float4*>(r.x);
        const float4* ph = reinterpret_cast<const float4*>(r.mh);
        const float4* pd = reinterpret_cast<const float4*>(r.xh);
        for (long long i = first; i < (d >> 2); i += stride) {
            const float4 c0 = __ldg(pc + i), u0 = G2 ? __ldg(pu + i) : c0, x0 = __ldg(px + i), h0 = __ldg(ph + i), d0 = __ldg(pd + i);
            float4 o;
            o.x = refl(c0.x, u0.x, x0.x, h0.x, d0.x); o.y = refl(c0.y, u0.y, x0.y, h0.y, d0.y);
            o.z = refl(c0.z, u0.z, x0.z, h0.z, d0.z); o.w = refl(c0.w, u0.w, x0.w, h0.w, d0.w);
            reinterpret_cast<float4*>(out)[i] = o;
        }
    } else {
        for (long long i = first; i < d; i += stride)
            out[i] = refl(__ldg(r.ec + i), __ldg(r.eu + i), __ldg(r.x + i), __ldg(r.mh + i), __ldg(r.xh + i));
    }
}

template <int CLUSTER, bool VEC4, bool G2>
int launch(const FusedArgs& a, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(a.B * CLUSTER), 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CLUSTER; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    FREE_CUDA_TRY(cudaLaunchKernelEx(&cfg, spec_verify_fused_kernel<CLUSTER, VEC4, G2>, a));
    return FREE_OK;
}

template <int CLUSTER, bool VEC4>
int launch_g(const FusedArgs& a, cudaStream_t s) {
    return a.G == 2 ? launch<CLUSTER, VEC4, true>(a, s) : launch<CLUSTER, VEC4, false>(a, s);
}

}  // namespace

int spec_verify_fused_launch(int B, int K, long long d, int G, float cfg_scale,
                             const float* eps, const float* x_first, long long x_first_stride,
                             const float* m_draft, const float* x_draft, const float* coef_x, const float* coef_eps,
                             const float* sigma2, const float* lambda, const float* u, const int32_t* n_valid, int chunk,
                             float* x_out, int32_t* n_accept, float* logratio_out, float* dist2_out, float* means_out, cudaStream_t s) {
    if (B < 0 || !eps || !x_first || !m_draft || !x_draft || !coef_x || !coef_eps || !sigma2 || !u || !x_out || !n_accept)
        return FREE_ERR_ARG;
    if (G != 1 && G != 2) return FREE_ERR_ARG;
    if (K < 1 || K > FREE_MAX_K || d < 1 || chunk < 0 || x_first_stride < d) return FREE_ERR_SHAPE;
    if (B == 0) return FREE_OK;
    if ((long long)B * 8 > 2147483647LL) return FREE_ERR_SHAPE;
    if (!free_aligned16(eps) || !free_aligned16(x_first) || !free_aligned16(m_draft) || !free_aligned16(x_draft) ||
        !free_aligned16(x_out) || !free_aligned16(means_out))
        return FREE_ERR_ALIGN;
    FusedArgs a{B, K, G, chunk, d, cfg_scale, eps, x_first, x_first_stride, m_draft, x_draft, coef_x, coef_eps,
                sigma2, lambda, u, n_valid, x_out, n_accept, logratio_out, dist2_out, means_out};
    const bool vec = (d % 4) == 0 && (x_first_stride % 4) == 0;      // every row stays 16-byte aligned only then
    if (!vec) return d >= 4096 ? launch_g<4, false>(a, s) : launch_g<1, false>(a, s);
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) { (void)cudaGetLastError(); sms = 148; }
    const long long resident = 4LL * sms;                 // 256-thread CTAs of this kernel that fit on the GPU at once
    int width = d >= 8192 ? 8 : (d >= 4096 ? 4 : (d >= 2048 ? 2 : 1));
    while (width > 2 && (long long)B * width > resident) width >>= 1;
    switch (width) {
        case 8: return launch_g<8, true>(a, s);
        case 4: return launch_g<4, true>(a, s);
        case 2: return launch_g<2, true>(a, s);
        default: return launch_g<1, true>(a, s);
    }
}

extern "C" int spec_verify_fused(int B, int K, int64_t d, int G, float cfg_scale,
                                 const float* eps, const float* x_first, const float* m_draft, const float* x_draft,
                                 const float* coef_x, const float* coef_eps, const float* sigma2, const float* lambda,
                                 const float* u, const int32_t* n_valid, int chunk,
                                 float* x_out, int32_t* n_accept, float* logratio_out, float* dist2_out, float* means_out, void* stream) {
    return spec_verify_fused_launch(B, K, (long long)d, G, cfg_scale, eps, x_first, (long long)d, m_draft, x_draft, coef_x, coef_eps,
                                    sigma2, lambda, u, n_valid, chunk, x_out, n_accept, logratio_out, dist2_out, means_out,
                                    reinterpret_cast<cudaStream_t>(stream));
}
