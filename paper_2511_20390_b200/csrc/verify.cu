// Fused verifier: Algorithm 2 (reflection maximal coupling) over K drafts per sample with the
// first-rejection break of Algorithm 1 and the relaxed acceptance of Eq. acc_relax.
//
// Bandwidth-bound: every operand is read once from HBM with 16-byte coalesced loads.  One thread-block
// cluster owns one sample.  Phase A: each CTA of the cluster streams its slice of every draft's
// (m, m_hat, x_hat) rows and accumulates s1 = |d|^2, s2 = d.r in fp64 (d = m_hat - m, r = x_hat - m_hat);
// warp shuffles reduce within a warp, shared memory within the CTA, distributed shared memory across
// the cluster, always in a fixed order so that results do not depend on scheduling.  Every CTA then
// derives the K log-ratios and the first rejection j itself.  Phase B: each CTA writes its slice of
// x_out, re-reading row j (just touched, so served from L2).
#include "common.cuh"
#include <cooperative_groups.h>
#include <math.h>

namespace cg = cooperative_groups;

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

struct VerifyArgs {
    int B, K;
    long long d;
    const float *m, *mh, *xh, *sigma2, *lambda, *u;
    const int32_t* n_valid;
    float* x_out;
    int32_t* n_accept;
    float* logratio;
};

__device__ __forceinline__ void accumulate(double& s1, double& s2, float m, float mh, float xh) {
    double dm = (double)mh - (double)m;
    double r = (double)xh - (double)mh;
    s1 = fma(dm, dm, s1);
    s2 = fma(dm, r, s2);
}

template <int CLUSTER, bool VEC4>
__global__ void __launch_bounds__(kThreads) spec_verify_kernel(VerifyArgs a) {
    __shared__ double warp_part[FREE_MAX_K][kWarps][2];
    __shared__ double cta_part[FREE_MAX_K][2];
    __shared__ double ell_s[FREE_MAX_K];
    __shared__ int ok_s[FREE_MAX_K];
    __shared__ int decision[2];   // [0] = n_accept or error code, [1] = 1 if sigma error

    const int rank = (CLUSTER > 1) ? (int)cg::this_cluster().block_rank() : 0;
    const int b = blockIdx.x / CLUSTER;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = a.K;
    int nv = a.n_valid ? a.n_valid[b] : K;
    nv = nv < 0 ? 0 : (nv > K ? K : nv);
    const long long d = a.d;
    const size_t row0 = (size_t)b * K * d;
    const int stride = CLUSTER * kThreads;
    const int first = rank * kThreads + tid;

    // ---------------- phase A: partial sums of every present draft
    for (int k = 0; k < nv; ++k) {
        double s1 = 0.0, s2 = 0.0;
        const size_t off = row0 + (size_t)k * d;
        if (VEC4) {
            const float4* pm = reinterpret_cast<const float4*>(a.m + off);
            const float4* ph = reinterpret_cast<const float4*>(a.mh + off);
            const float4* px = reinterpret_cast<const float4*>(a.xh + off);
            const long long n4 = d >> 2;
            long long i = first;
            for (; i + 3LL * stride < n4; i += 4LL * stride) {   // four independent 16-byte loads per stream in flight
                float4 m0 = __ldg(pm + i), h0 = __ldg(ph + i), x0 = __ldg(px + i);
                float4 m1 = __ldg(pm + i + stride), h1 = __ldg(ph + i + stride), x1 = __ldg(px + i + stride);
                float4 m2 = __ldg(pm + i + 2 * stride), h2 = __ldg(ph + i + 2 * stride), x2 = __ldg(px + i + 2 * stride);
                float4 m3 = __ldg(pm + i + 3 * stride), h3 = __ldg(ph + i + 3 * stride), x3 = __ldg(px + i + 3 * stride);
                accumulate(s1, s2, m0.x, h0.x, x0.x); accumulate(s1, s2, m0.y, h0.y, x0.y);
                accumulate(s1, s2, m0.z, h0.z, x0.z); accumulate(s1, s2, m0.w, h0.w, x0.w);
                accumulate(s1, s2, m1.x, h1.x, x1.x); accumulate(s1, s2, m1.y, h1.y, x1.y);
                accumulate(s1, s2, m1.z, h1.z, x1.z); accumulate(s1, s2, m1.w, h1.w, x1.w);
                accumulate(s1, s2, m2.x, h2.x, x2.x); accumulate(s1, s2, m2.y, h2.y, x2.y);
                accumulate(s1, s2, m2.z, h2.z, x2.z); accumulate(s1, s2, m2.w, h2.w, x2.w);
                accumulate(s1, s2, m3.x, h3.x, x3.x); accumulate(s1, s2, m3.y, h3.y, x3.y);
                accumulate(s1, s2, m3.z, h3.z, x3.z); accumulate(s1, s2, m3.w, h3.w, x3.w);
            }
            for (; i + stride < n4; i += 2 * stride) {     // two independent 16-byte loads per stream in flight
                float4 m0 = __ldg(pm + i), h0 = __ldg(ph + i), x0 = __ldg(px + i);
                float4 m1 = __ldg(pm + i + stride), h1 = __ldg(ph + i + stride), x1 = __ldg(px + i + stride);
                accumulate(s1, s2, m0.x, h0.x, x0.x); accumulate(s1, s2, m0.y, h0.y, x0.y);
                accumulate(s1, s2, m0.z, h0.z, x0.z); accumulate(s1, s2, m0.w, h0.w, x0.w);
                accumulate(s1, s2, m1.x, h1.x, x1.x); accumulate(s1, s2, m1.y, h1.y, x1.y);
                accumulate(s1, s2, m1.z, h1.z, x1.z); accumulate(s1, s2, m1.w, h1.w, x1.w);
            }
            for (; i < n4; i += stride) {
                float4 m0 = __ldg(pm + i), h0 = __ldg(ph + i), x0 = __ldg(px + i);
                accumulate(s1, s2, m0.x, h0.x, x0.x); accumulate(s1, s2, m0.y, h0.y, x0.y);
                accumulate(s1, s2, m0.z, h0.z, x0.z); accumulate(s1, s2, m0.w, h0.w, x0.w);
            }
        } else {
            for (long long i = first; i < d; i += stride)
                accumulate(s1, s2, __ldg(a.m + off + i), __ldg(a.mh + off + i), __ldg(a.xh + off + i));
        }
        s1 = free_warp_sum(s1);
        s2 = free_warp_sum(s2);
        if (lane == 0) { warp_part[k][warp][0] = s1; warp_part[k][warp][1] = s2; }
    }
    __syncthreads();
    if (tid < nv) {
        double s1 = 0.0, s2 = 0.0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) { s1 += warp_part[tid][w][0]; s2 += warp_part[tid][w][1]; }
        cta_part[tid][0] = s1; cta_part[tid][1] = s2;
    }
    if (CLUSTER > 1) cg::this_cluster().sync(); else __syncthreads();

    // ---------------- decisions (every CTA computes the same values)
    if (tid < nv) {
        double s1 = 0.0, s2 = 0.0;
        if (CLUSTER > 1) {
            cg::cluster_group cl = cg::this_cluster();
            for (int r = 0; r < CLUSTER; ++r) {
                const double* rp = cl.map_shared_rank(&cta_part[0][0], r);
                s1 += rp[2 * tid]; s2 += rp[2 * tid + 1];
            }
        } else { s1 = cta_part[tid][0]; s2 = cta_part[tid][1]; }
        const size_t bk = (size_t)b * K + tid;
        const double sg = (double)a.sigma2[bk];
        const double lam = a.lambda ? (double)a.lambda[bk] : 1.0;
        const double uu = (double)a.u[bk];
        const bool bad = !(sg > 0.0) || isinf(sg);
        const double ell = bad ? nan("") : -lam * (s2 + 0.5 * s1) / sg;
        const double log_u = uu <= 0.0 ? -INFINITY : log(uu);
        ell_s[tid] = ell;
        ok_s[tid] = bad ? -1 : (log_u <= fmin(0.0, ell) ? 1 : 0);
        // totals for the reflection, reused in phase B through shared memory
        warp_part[tid][0][0] = s1; warp_part[tid][0][1] = s2;
    }
    // no CTA may leave (or overwrite cta_part) while a peer still reads its shared memory
    if (CLUSTER > 1) cg::this_cluster().sync(); else __syncthreads();
    if (tid == 0) {
        int j = 0, err = 0;
        for (int k = 0; k < nv; ++k) if (ok_s[k] < 0) err = 1;
        while (!err && j < nv && ok_s[j] == 1) ++j;
        decision[0] = err ? FREE_ERR_SIGMA : j;
        decision[1] = err;
    }
    __syncthreads();
    const int j = decision[0];
    if (rank == 0) {
        if (tid == 0) a.n_accept[b] = j;
        if (a.logratio && tid < K) a.logratio[(size_t)b * K + tid] = tid < nv ? (float)ell_s[tid] : nanf("");
    }
    if (decision[1] || nv == 0) return;

    // ---------------- phase B: this CTA's slice of the finalised state
    float* out = a.x_out + (size_t)b * d;
    if (j == nv) {                      // every draft accepted: the last draft is the state
        const size_t off = row0 + (size_t)(nv - 1) * d;
        if (VEC4) {
            const float4* px = reinterpret_cast<const float4*>(a.xh + off);
            float4* po = reinterpret_cast<float4*>(out);
            for (long long i = first; i < (d >> 2); i += stride) po[i] = __ldg(px + i);
        } else {
            for (long long i = first; i < d; i += stride) out[i] = __ldg(a.xh + off + i);
        }
        return;
    }
    const double s1 = warp_part[j][0][0], s2 = warp_part[j][0][1];
    const double coef = s1 > 0.0 ? 2.0 * s2 / s1 : 0.0;       // 2 (e.r) / |d| folded with e = d / |d|
    const bool ident = !(s1 > 0.0);
    const size_t off = row0 + (size_t)j * d;
    auto refl = [&](float m, float mh, float xh) -> float {
        if (ident) return xh;
        double dm = (double)mh - (double)m, r = (double)xh - (double)mh;
        return (float)((double)m + r - coef * dm);
    };
    if (VEC4) {
        const float4* pm = reinterpret_cast<const float4*>(a.m + off);
        const float4* ph = reinterpret_cast<const float4*>(a.mh + off);
        const float4* px = reinterpret_cast<const float4*>(a.xh + off);
        float4* po = reinterpret_cast<float4*>(out);
        for (long long i = first; i < (d >> 2); i += stride) {
            float4 m0 = __ldg(pm + i), h0 = __ldg(ph + i), x0 = __ldg(px + i), o;
            o.x = refl(m0.x, h0.x, x0.x); o.y = refl(m0.y, h0.y, x0.y);
            o.z = refl(m0.z, h0.z, x0.z); o.w = refl(m0.w, h0.w, x0.w);
            po[i] = o;
        }
    } else {
        for (long long i = first; i < d; i += stride)
            out[i] = refl(__ldg(a.m + off + i), __ldg(a.mh + off + i), __ldg(a.xh + off + i));
    }
}

template <int CLUSTER, bool VEC4>
int launch(const VerifyArgs& a, cudaStream_t stream) {
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
    FREE_CUDA_TRY(cudaLaunchKernelEx(&cfg, spec_verify_kernel<CLUSTER, VEC4>, a));
    return FREE_OK;
}

}  // namespace

extern "C" int spec_verify(int B, int K, int64_t d,
                           const float* m_target, const float* m_draft, const float* x_draft,
                           const float* sigma2, const float* lambda, const float* u, const int32_t* n_valid,
                           float* x_out, int32_t* n_accept, float* logratio_out, void* stream) {
    if (B < 0 || !m_target || !m_draft || !x_draft || !sigma2 || !u || !x_out || !n_accept) return FREE_ERR_ARG;
    if (K < 1 || K > FREE_MAX_K || d < 1) return FREE_ERR_SHAPE;
    if (B == 0) return FREE_OK;
    if ((long long)B * 8 > 2147483647LL) return FREE_ERR_SHAPE;
    if (!free_aligned16(m_target) || !free_aligned16(m_draft) || !free_aligned16(x_draft) || !free_aligned16(x_out))
        return FREE_ERR_ALIGN;
    VerifyArgs a{B, K, (long long)d, m_target, m_draft, x_draft, sigma2, lambda, u, n_valid, x_out, n_accept, logratio_out};
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const bool vec = (d % 4) == 0;     // rows stay 16-byte aligned only then
    // cluster width: enough CTAs per sample that one float4 per thread and draft remains, but not more clusters than
    // fit on the GPU at once when the batch is large: one full wave of narrower clusters streams better than several
    // waves with a ragged last one (measured at d = 16384, K = 16, B = 256: 5.8 TB/s with pairs, 5.6 TB/s with eight)
    if (!vec) return d >= 4096 ? launch<4, false>(a, s) : launch<1, false>(a, s);
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) { (void)cudaGetLastError(); sms = 148; }
    const long long resident = 4LL * sms;                 // 256-thread CTAs of this kernel per GPU
    int width = d >= 8192 ? 8 : (d >= 4096 ? 4 : (d >= 2048 ? 2 : 1));
    while (width > 2 && (long long)B * width > resident) width >>= 1;
    switch (width) {
        case 8: return launch<8, true>(a, s);
        case 4: return launch<4, true>(a, s);
        case 2: return launch<2, true>(a, s);
        default: return launch<1, true>(a, s);
    }
}
