// Verification straight from the head output of the packed target pass: classifier-free guidance, the reverse-transition
// means m_k = coef_x x_k - coef_eps eps_k (Eq. ddpm_update), Algorithm 2 (reflection maximal coupling) with the
// first-rejection break of Algorithm 1 and the relaxed acceptance of Eq. acc_relax, in one kernel.  The means never
// exist in memory: compared with "tail kernel, then spec_verify" the [B,K,d] mean tensor is neither written nor read,
// and the packed states x_k are the drafts themselves (x_1..x_{K-1} = x_hat_0..x_hat_{K-2}), read once from HBM.
//
// Bandwidth-bound.  One thread-block cluster owns one sample.  A work item is one run of P consecutive floats of a
// patch row: contiguous both in the head output (per-token vector ordered channel, row-in-patch, column-in-patch)
// and in the image.  The two offsets of every item of a CTA's slice are computed once into shared memory (they do
// not depend on the draft); the streaming loop then only loads and accumulates s1 = |d|^2, s2 = d.r in fp64
// (d = m_hat - m, r = x_hat - m_hat).  Reductions: warp shuffle -> shared memory -> distributed shared memory, in a
// fixed order.  Optional early exit: drafts are examined in chunks and the rows after the chunk that holds the first
// rejection are never read.
#include "internal.h"
#include <cooperative_groups.h>
#include <math.h>

namespace cg = cooperative_groups;

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kTabBytesMax = 40 * 1024;

struct FusedArgs {
    int B, K, G, C, H, W, p, c_out, chunk;
    float cfg;
    const float* head;
    const float* x_first; long long x_first_stride;
    const float *mh, *xh, *coef_x, *coef_eps, *sigma2, *lambda, *u;
    const int32_t* n_valid;
    float* x_out; int32_t* n_accept; float* logratio; float* means_out;
};

__device__ __forceinline__ void ldp(const float* p, float (&v)[1]) { v[0] = __ldg(p); }
__device__ __forceinline__ void ldp(const float* p, float (&v)[2]) { const float2 t = __ldg(reinterpret_cast<const float2*>(p)); v[0] = t.x; v[1] = t.y; }
__device__ __forceinline__ void ldp(const float* p, float (&v)[4]) { const float4 t = __ldg(reinterpret_cast<const float4*>(p)); v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; }
__device__ __forceinline__ void stp(float* p, const float (&v)[1]) { p[0] = v[0]; }
__device__ __forceinline__ void stp(float* p, const float (&v)[2]) { *reinterpret_cast<float2*>(p) = make_float2(v[0], v[1]); }
__device__ __forceinline__ void stp(float* p, const float (&v)[4]) { *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]); }

// The operands of one item of draft k.
template <int P>
struct Item { float ec[P], eu[P], x[P], mh[P], xh[P]; };

struct Row {                      // base pointers and coefficients of draft k of this sample
    const float *hc, *hu, *x, *mh, *xh;
    double cx, ce;
};

template <int P, bool G2>
__device__ __forceinline__ void load_item(const Row& r, int2 o, Item<P>& it) {
    ldp(r.hc + o.x, it.ec);
    if (G2) ldp(r.hu + o.x, it.eu);
    ldp(r.x + o.y, it.x);
    ldp(r.mh + o.y, it.mh);
    ldp(r.xh + o.y, it.xh);
}

template <bool G2>
__device__ __forceinline__ double mean_of(const Row& r, double w, float ec, float eu, float x) {
    double e = (double)ec;
    if (G2) e = fma(w, e - (double)eu, (double)eu);
    return fma(r.cx, (double)x, -r.ce * e);
}

template <int CLUSTER, int P, bool TAB>
__global__ void __launch_bounds__(kThreads, 3) spec_verify_fused_kernel(FusedArgs a) {
    extern __shared__ int2 tab[];
    __shared__ double warp_part[FREE_MAX_K][kWarps][2];
    __shared__ double cta_part[FREE_MAX_K][2];
    __shared__ double tot[FREE_MAX_K][2];
    __shared__ double ell_s[FREE_MAX_K];
    __shared__ int ok_s[FREE_MAX_K];

    const int rank = (CLUSTER > 1) ? (int)cg::this_cluster().block_rank() : 0;
    const int b = blockIdx.x / CLUSTER;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K = a.K, p = a.p, pv = p / P;
    int nv = a.n_valid ? a.n_valid[b] : K;
    nv = nv < 0 ? 0 : (nv > K ? K : nv);
    const int gw = a.W / p, n_tok = (a.H / p) * gw, od = a.c_out * p * p;
    const int d = a.C * a.H * a.W;
    const int per_tok = a.C * p * pv;                    // items per token: (channel, row-in-patch, run within the row)
    const int n_items = n_tok * per_tok;                 // = d / P
    const int ipc = (n_items + CLUSTER - 1) / CLUSTER;   // items of one CTA: a contiguous range
    const int i0 = rank * ipc;
    const int n_loc = n_items - i0 < ipc ? (n_items - i0 > 0 ? n_items - i0 : 0) : ipc;

    auto offsets = [&](int li) -> int2 {                 // (offset in the head output of one stream, offset in the image)
        const int i = i0 + li;
        const int tok = i / per_tok, rem = i - tok * per_tok;
        const int c = rem / (p * pv), rem2 = rem - c * (p * pv);
        const int pr = rem2 / pv, run = rem2 - pr * pv;
        const int trow = tok / gw, tcol = tok - trow * gw;
        return make_int2(tok * od + (c * p + pr) * p + run * P, (c * a.H + trow * p + pr) * a.W + tcol * p + run * P);
    };
    if (TAB) {
        for (int li = tid; li < n_loc; li += kThreads) tab[li] = offsets(li);
        __syncthreads();
    }
    auto off = [&](int li) -> int2 { return TAB ? tab[li] : offsets(li); };

    const size_t stream_sz = (size_t)n_tok * od;
    const double wg = (double)a.cfg;
    auto row = [&](int k) -> Row {
        const size_t bk = (size_t)b * K + k;
        Row r;
        r.hc = a.head + bk * a.G * stream_sz;
        r.hu = r.hc + (a.G == 2 ? stream_sz : 0);
        r.x = k == 0 ? a.x_first + (size_t)b * a.x_first_stride : a.xh + (bk - 1) * d;
        r.mh = a.mh + bk * d;
        r.xh = a.xh + bk * d;
        r.cx = (double)a.coef_x[bk];
        r.ce = (double)a.coef_eps[bk];
        return r;
    };

    auto accumulate_row = [&](auto g2, int k) {
        constexpr bool G2 = decltype(g2)::value;
        const Row r = row(k);
        double s1 = 0.0, s2 = 0.0;
        auto acc = [&](const Item<P>& it, int2 o) {
#pragma unroll
            for (int e = 0; e < P; ++e) {
                const double m = mean_of<G2>(r, wg, it.ec[e], it.eu[e], it.x[e]);
                const double dm = (double)it.mh[e] - m, rr = (double)it.xh[e] - (double)it.mh[e];
                s1 = fma(dm, dm, s1);
                s2 = fma(dm, rr, s2);
            }
            if (a.means_out) {
                float mv[P];
#pragma unroll
                for (int e = 0; e < P; ++e) mv[e] = (float)mean_of<G2>(r, wg, it.ec[e], it.eu[e], it.x[e]);
                stp(a.means_out + ((size_t)b * K + k) * d + o.y, mv);
            }
        };
        int li = tid;
        if (P < 4) {
            for (; li + 3 * kThreads < n_loc; li += 4 * kThreads) {      // 160 bytes (P = 2) of loads in flight per thread
                Item<P> t0, t1, t2, t3;
                const int2 o0 = off(li), o1 = off(li + kThreads), o2 = off(li + 2 * kThreads), o3 = off(li + 3 * kThreads);
                load_item<P, G2>(r, o0, t0); load_item<P, G2>(r, o1, t1); load_item<P, G2>(r, o2, t2); load_item<P, G2>(r, o3, t3);
                acc(t0, o0); acc(t1, o1); acc(t2, o2); acc(t3, o3);
            }
        }
        for (; li + kThreads < n_loc; li += 2 * kThreads) {
            Item<P> t0, t1;
            const int2 o0 = off(li), o1 = off(li + kThreads);
            load_item<P, G2>(r, o0, t0); load_item<P, G2>(r, o1, t1);
            acc(t0, o0); acc(t1, o1);
        }
        for (; li < n_loc; li += kThreads) {
            Item<P> t0;
            const int2 o0 = off(li);
            load_item<P, G2>(r, o0, t0);
            acc(t0, o0);
        }
        s1 = free_warp_sum(s1);
        s2 = free_warp_sum(s2);
        if (lane == 0) { warp_part[k][warp][0] = s1; warp_part[k][warp][1] = s2; }
    };

    // ---------------- phase A, chunk by chunk: partial sums, decisions, stop after the first rejection
    const int chunk = a.chunk > 0 ? a.chunk : (K > 0 ? K : 1);
    int examined = 0, jrej = -1, err = 0;
    for (int k0 = 0; k0 < nv; k0 += chunk) {
        const int k1 = k0 + chunk < nv ? k0 + chunk : nv;
        for (int k = k0; k < k1; ++k) {
            if (a.G == 2) accumulate_row(std::true_type{}, k); else accumulate_row(std::false_type{}, k);
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
        for (int k = k0; k < k1; ++k) {
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
    }
    if (err || nv == 0) return;

    // ---------------- phase B: this CTA's slice of the finalised state
    float* out = a.x_out + (size_t)b * d;
    if (j == nv) {                                        // every draft accepted: the last draft is the state
        const float* src = a.xh + ((size_t)b * K + nv - 1) * d;
        for (int li = tid; li < n_loc; li += kThreads) {
            const int2 o = off(li);
            float v[P];
            ldp(src + o.y, v);
            stp(out + o.y, v);
        }
        return;
    }
    const double s1 = tot[j][0], s2 = tot[j][1];
    const double coef = s1 > 0.0 ? 2.0 * s2 / s1 : 0.0;   // 2 (e.r) / |d| folded with e = d / |d|
    const bool ident = !(s1 > 0.0);
    const Row r = row(j);
    auto reflect_items = [&](auto g2) {
        constexpr bool G2 = decltype(g2)::value;
        for (int li = tid; li < n_loc; li += kThreads) {
            const int2 o = off(li);
            Item<P> it;
            load_item<P, G2>(r, o, it);
            float v[P];
#pragma unroll
            for (int e = 0; e < P; ++e) {
                const double m = mean_of<G2>(r, wg, it.ec[e], it.eu[e], it.x[e]);
                const double dm = (double)it.mh[e] - m, rr = (double)it.xh[e] - (double)it.mh[e];
                v[e] = ident ? it.xh[e] : (float)(m + rr - coef * dm);
            }
            stp(out + o.y, v);
        }
    };
    if (a.G == 2) reflect_items(std::true_type{}); else reflect_items(std::false_type{});
}

template <int CLUSTER, int P, bool TAB>
int launch(const FusedArgs& a, size_t tab_bytes, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(a.B * CLUSTER), 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = TAB ? tab_bytes : 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CLUSTER; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    FREE_CUDA_TRY(cudaLaunchKernelEx(&cfg, spec_verify_fused_kernel<CLUSTER, P, TAB>, a));
    return FREE_OK;
}

template <int CLUSTER, int P>
int launch_tab(const FusedArgs& a, cudaStream_t s) {
    const long long n_items = (long long)a.C * a.H * a.W / P;
    const size_t tab_bytes = (size_t)((n_items + CLUSTER - 1) / CLUSTER) * sizeof(int2);
    return tab_bytes <= (size_t)kTabBytesMax ? launch<CLUSTER, P, true>(a, tab_bytes, s) : launch<CLUSTER, P, false>(a, 0, s);
}

template <int P>
int launch_width(const FusedArgs& a, int width, cudaStream_t s) {
    switch (width) {
        case 8: return launch_tab<8, P>(a, s);
        case 4: return launch_tab<4, P>(a, s);
        case 2: return launch_tab<2, P>(a, s);
        default: return launch_tab<1, P>(a, s);
    }
}

}  // namespace

int spec_verify_fused_launch(int B, int K, int C, int H, int W, int patch, int c_out, int G, float cfg_scale,
                             const float* head_out, const float* x_first, long long x_first_stride,
                             const float* m_draft, const float* x_draft, const float* coef_x, const float* coef_eps,
                             const float* sigma2, const float* lambda, const float* u, const int32_t* n_valid, int chunk,
                             float* x_out, int32_t* n_accept, float* logratio_out, float* means_out, cudaStream_t s) {
    if (B < 0 || !head_out || !x_first || !m_draft || !x_draft || !coef_x || !coef_eps || !sigma2 || !u || !x_out || !n_accept)
        return FREE_ERR_ARG;
    if (G != 1 && G != 2) return FREE_ERR_ARG;
    if (K < 1 || K > FREE_MAX_K || chunk < 0) return FREE_ERR_SHAPE;
    if (C < 1 || c_out < C || patch < 1 || H < patch || W < patch || H % patch || W % patch) return FREE_ERR_SHAPE;
    const long long d = (long long)C * H * W, stream_sz = (long long)(H / patch) * (W / patch) * c_out * patch * patch;
    if (d > (1LL << 30) || stream_sz > (1LL << 30) || x_first_stride < d) return FREE_ERR_SHAPE;
    if (B == 0) return FREE_OK;
    if ((long long)B * 8 > 2147483647LL) return FREE_ERR_SHAPE;
    if (!free_aligned16(head_out) || !free_aligned16(x_first) || !free_aligned16(m_draft) || !free_aligned16(x_draft) ||
        !free_aligned16(x_out) || !free_aligned16(means_out))
        return FREE_ERR_ALIGN;
    FusedArgs a{B, K, G, C, H, W, patch, c_out, chunk, cfg_scale, head_out, x_first, x_first_stride, m_draft, x_draft,
                coef_x, coef_eps, sigma2, lambda, u, n_valid, x_out, n_accept, logratio_out, means_out};
    // run width: as wide as the patch row, the image row stride and the sample stride allow with 16-byte-aligned bases
    int P = patch % 4 == 0 ? 4 : (patch % 2 == 0 ? 2 : 1);
    while (P > 1 && (d % P || stream_sz % P || x_first_stride % P)) P >>= 1;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) { (void)cudaGetLastError(); sms = 148; }
    const long long resident = 3LL * sms;                 // 256-thread CTAs of this kernel that fit on the GPU at once
    int width = d >= 8192 ? 8 : (d >= 4096 ? 4 : (d >= 2048 ? 2 : 1));
    while (width > 2 && (long long)B * width > resident) width >>= 1;
    switch (P) {
        case 4: return launch_width<4>(a, width, s);
        case 2: return launch_width<2>(a, width, s);
        default: return launch_width<1>(a, width, s);
    }
}

extern "C" int spec_verify_fused(int B, int K, int C, int H, int W, int patch, int c_out, int G, float cfg_scale,
                                 const float* head_out, const float* x_first, const float* m_draft, const float* x_draft,
                                 const float* coef_x, const float* coef_eps, const float* sigma2, const float* lambda,
                                 const float* u, const int32_t* n_valid, int chunk,
                                 float* x_out, int32_t* n_accept, float* logratio_out, float* means_out, void* stream) {
    return spec_verify_fused_launch(B, K, C, H, W, patch, c_out, G, cfg_scale, head_out, x_first, (long long)C * H * W,
                                    m_draft, x_draft, coef_x, coef_eps, sigma2, lambda, u, n_valid, chunk,
                                    x_out, n_accept, logratio_out, means_out, reinterpret_cast<cudaStream_t>(stream));
}
