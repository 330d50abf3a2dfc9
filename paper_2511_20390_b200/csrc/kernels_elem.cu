// Bandwidth-bound row and elementwise kernels of the DiT pass: conditioning features, patch embedding,
// LayerNorm + adaLN modulation, feature conversion, and the tail that turns the head's output into the
// guided noise prediction and the reverse-transition mean (Eq. ddpm_update).
#include "internal.h"
#include <math.h>

namespace {

template <typename T> __device__ __forceinline__ void store_act(T* p, float v);
template <> __device__ __forceinline__ void store_act<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void store_act<__nv_bfloat16>(__nv_bfloat16* p, float v) { *p = __float2bfloat16(v); }

// ---------------------------------------------------------------------------------------------
// Sinusoidal timestep features [cos(tau w_i), sin(tau w_i)], w_i = 10000^(-i/half), and the label of
// every sequence (the unconditional stream of a guided state uses the null class).
template <typename T>
__global__ void cond_setup_kernel(int n_states, int G, int freq_dim, int n_classes, int N_sched,
                                  const int32_t* t_idx, const int32_t* labels, const float* t_embed_value,
                                  T* temb, int32_t* lab_seq) {
    const int q = blockIdx.x;                 // sequence
    const int st = q / G, g = q % G;
    int t = t_idx[st];
    t = t < 0 ? 0 : (t >= N_sched ? N_sched - 1 : t);
    const double tau = (double)t_embed_value[t];
    const int half = freq_dim / 2;
    for (int i = threadIdx.x; i < half; i += blockDim.x) {
        const double w = exp(-log(10000.0) * (double)i / (double)half);
        store_act(temb + (size_t)q * freq_dim + i, (float)cos(tau * w));
        store_act(temb + (size_t)q * freq_dim + half + i, (float)sin(tau * w));
    }
    if (threadIdx.x == 0) {
        int y = labels[st];
        y = y < 0 ? 0 : (y > n_classes ? n_classes : y);
        lab_seq[q] = g == 0 ? y : n_classes;
    }
}

// ---------------------------------------------------------------------------------------------
// Patch embedding: token (i, j) of a state gathers its C*p*p patch (order: channel, row, column),
// out = pe_w . patch + pe_b + pos[token], written once per guidance stream.  Thread t of a CTA owns output
// channels t, t + 256, ... and keeps their weight rows in registers (PD = C p p values each); the CTA walks
// over (state, token) pairs, so weights are read once per CTA and every store is a coalesced row segment.
template <typename T, int PD, int CPT>
__global__ void __launch_bounds__(256) patch_embed_kernel(int n_items, int G, int C, int H, int W, int p, int D,
                                                          const float* __restrict__ x_in, long long x_stride,
                                                          const float* __restrict__ pe_w, const float* __restrict__ pe_b,
                                                          const float* __restrict__ pos, T* __restrict__ out) {
    __shared__ float patch[2][PD];
    const int gw = W / p, n_tok = (H / p) * gw;
    float w[CPT][PD], b[CPT];
#pragma unroll
    for (int j = 0; j < CPT; ++j) {
        const int o = threadIdx.x + j * 256;
        b[j] = o < D ? pe_b[o] : 0.f;
#pragma unroll
        for (int e = 0; e < PD; ++e) w[j][e] = o < D ? pe_w[(long long)o * PD + e] : 0.f;
    }
    auto gather = [&](int item, float* dst) {
        if (threadIdx.x < PD && item < n_items) {
            const int st = item / n_tok, tok = item % n_tok, ti = tok / gw, tj = tok % gw;
            const int e = threadIdx.x, c = e / (p * p), r = (e / p) % p, cc = e % p;
            dst[e] = x_in[(long long)st * x_stride + ((long long)c * H + ti * p + r) * W + tj * p + cc];
        }
    };
    int item = blockIdx.x, buf = 0;
    gather(item, patch[0]);
    __syncthreads();
    for (; item < n_items; item += gridDim.x, buf ^= 1) {
        gather(item + gridDim.x, patch[buf ^ 1]);                 // next item's patch while this one is used
        const int st = item / n_tok, tok = item % n_tok;
#pragma unroll
        for (int j = 0; j < CPT; ++j) {
            const int o = threadIdx.x + j * 256;
            if (o < D) {
                float acc = 0.f;
#pragma unroll
                for (int e = 0; e < PD; ++e) acc = fmaf(w[j][e], patch[buf][e], acc);
                acc += b[j] + __ldg(pos + (long long)tok * D + o);
                for (int g = 0; g < G; ++g)
                    store_act(out + ((long long)(st * G + g) * n_tok + tok) * D + o, acc);
            }
        }
        __syncthreads();
    }
}

// Wide models (D a multiple of 128, 16-value patches): the transposed weight matrix [16][D] sits in shared memory, a warp
// takes four consecutive tokens at a time and a lane the same 4-column groups of all of them, so that every 16-byte
// weight read feeds 16 multiply-adds and every store is a full row segment.  Bound by the output's HBM bandwidth.
template <typename T, int VPL>
__global__ void __launch_bounds__(256, 2) patch_embed_wide_kernel(int n_items, int G, int C, int H, int W, int p, int D,
                                                                  const float* __restrict__ x_in, long long x_stride,
                                                                  const float* __restrict__ pe_w, const float* __restrict__ pe_b,
                                                                  const float* __restrict__ pos, T* __restrict__ out) {
    constexpr int PD = 16, TOKW = 4;
    extern __shared__ float4 pe_smem[];
    float* wt = reinterpret_cast<float*>(pe_smem);                    // [PD][D]
    float* patches = wt + (size_t)PD * D;                             // [warps][TOKW][PD]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wpc = blockDim.x >> 5;
    for (int i = threadIdx.x; i < PD * D; i += blockDim.x) { const int o = i / PD, e = i % PD; wt[(size_t)e * D + o] = pe_w[i]; }
    __syncthreads();
    float* mine = patches + warp * TOKW * PD;
    const int gw = W / p, n_tok = (H / p) * gw;
    const int n_groups = n_items / TOKW;                              // the host checks n_tok % TOKW == 0
    const int warps = gridDim.x * wpc;
    auto gather2 = [&](int group, float& a, float& b) {               // this lane's two of the group's 64 patch values
        const int e = lane & 15;
        const int c = e / (p * p), r = (e / p) % p, cc = e % p;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int item = group * TOKW + (lane >> 4) + 2 * h;
            const int st = item / n_tok, tok = item % n_tok, ti = tok / gw, tj = tok % gw;
            const float v = x_in[(long long)st * x_stride + ((long long)c * H + ti * p + r) * W + tj * p + cc];
            if (h == 0) a = v; else b = v;
        }
    };
    int group = blockIdx.x * wpc + warp;
    float na = 0.f, nb = 0.f;
    if (group < n_groups) gather2(group, na, nb);
    for (; group < n_groups; group += warps) {
        __syncwarp();
        mine[(lane >> 4) * PD + (lane & 15)] = na;
        mine[((lane >> 4) + 2) * PD + (lane & 15)] = nb;
        __syncwarp();
        if (group + warps < n_groups) gather2(group + warps, na, nb);  // the next group's values while this one is computed
        float pt[TOKW][PD];
#pragma unroll
        for (int t = 0; t < TOKW; ++t)
#pragma unroll
            for (int e4 = 0; e4 < PD / 4; ++e4) {
                const float4 v = reinterpret_cast<const float4*>(mine + t * PD)[e4];
                pt[t][4 * e4] = v.x; pt[t][4 * e4 + 1] = v.y; pt[t][4 * e4 + 2] = v.z; pt[t][4 * e4 + 3] = v.w;
            }
        const int item0 = group * TOKW, st = item0 / n_tok, tok0 = item0 % n_tok;   // four tokens of one state
#pragma unroll 1
        for (int i = 0; i < VPL; ++i) {
            const int c0 = (i * 32 + lane) * 4;
            const float4 bias = __ldg(reinterpret_cast<const float4*>(pe_b + c0));
            float4 acc[TOKW];
#pragma unroll
            for (int t = 0; t < TOKW; ++t) {
                const float4 ps = __ldg(reinterpret_cast<const float4*>(pos + (long long)(tok0 + t) * D + c0));
                acc[t] = make_float4(bias.x + ps.x, bias.y + ps.y, bias.z + ps.z, bias.w + ps.w);
            }
#pragma unroll
            for (int e = 0; e < PD; ++e) {
                const float4 w4 = *reinterpret_cast<const float4*>(wt + (size_t)e * D + c0);
#pragma unroll
                for (int t = 0; t < TOKW; ++t) {
                    acc[t].x = fmaf(w4.x, pt[t][e], acc[t].x); acc[t].y = fmaf(w4.y, pt[t][e], acc[t].y);
                    acc[t].z = fmaf(w4.z, pt[t][e], acc[t].z); acc[t].w = fmaf(w4.w, pt[t][e], acc[t].w);
                }
            }
#pragma unroll
            for (int t = 0; t < TOKW; ++t)
                for (int g = 0; g < G; ++g) {
                    T* dst = out + ((long long)(st * G + g) * n_tok + tok0 + t) * D + c0;
                    if (sizeof(T) == 4) {
                        *reinterpret_cast<float4*>(dst) = acc[t];
                    } else {
                        __nv_bfloat162 lo = __floats2bfloat162_rn(acc[t].x, acc[t].y), hi = __floats2bfloat162_rn(acc[t].z, acc[t].w);
                        uint2 pk;
                        pk.x = *reinterpret_cast<uint32_t*>(&lo);
                        pk.y = *reinterpret_cast<uint32_t*>(&hi);
                        *reinterpret_cast<uint2*>(dst) = pk;
                    }
                }
        }
    }
}

// Any patch size / width: one CTA per (state, token), weights read from global memory.
template <typename T>
__global__ void __launch_bounds__(128) patch_embed_generic_kernel(int G, int C, int H, int W, int p, int D,
                                                                  const float* x_in, long long x_stride, const float* pe_w,
                                                                  const float* pe_b, const float* pos, T* out) {
    extern __shared__ float patch_dyn[];
    const int gw = W / p, n_tok = (H / p) * gw, pd = C * p * p;
    const int st = blockIdx.x / n_tok, tok = blockIdx.x % n_tok;
    const int ti = tok / gw, tj = tok % gw;
    const float* x = x_in + (long long)st * x_stride;
    for (int e = threadIdx.x; e < pd; e += blockDim.x) {
        int c = e / (p * p), r = (e / p) % p, cc = e % p;
        patch_dyn[e] = x[((long long)c * H + ti * p + r) * W + tj * p + cc];
    }
    __syncthreads();
    for (int o = threadIdx.x; o < D; o += blockDim.x) {
        const float* w = pe_w + (long long)o * pd;
        float acc = 0.f;
        for (int e = 0; e < pd; ++e) acc = fmaf(w[e], patch_dyn[e], acc);
        acc += pe_b[o] + pos[(long long)tok * D + o];
        for (int g = 0; g < G; ++g)
            store_act(out + ((long long)(st * G + g) * n_tok + tok) * D + o, acc);
    }
}

// ---------------------------------------------------------------------------------------------
// LayerNorm (no affine, eps 1e-6, biased variance, two-pass statistics) + y = ln (1 + scale) + shift.
// One warp per row.  VPL > 0: the row (D = 128 * VPL) lives in registers as VPL float4 per lane; warps stride
// over the rows and issue the loads of their next row before reducing the current one, so that each warp always
// has a full row of 16-byte loads in flight (the kernel is a pure stream: read 4 D, write 2 D or 4 D bytes per row).
// SPLIT (bf16 only): y is written as two bf16 planes, hi = bf16(y) at y[0 .. M D) and lo = bf16(y - hi) at
// y[M D .. 2 M D), so that a tensor-core product can recover fp32-level accuracy from hi and lo terms.
template <typename T, int VPL, bool SPLIT = false>
__global__ void __launch_bounds__(VPL >= 9 ? 384 : 256, VPL >= 9 ? 1 : 2)
ln_modulate_kernel(int M, int D, int rows_per_seq, const float* __restrict__ x, const float* __restrict__ shift,
                   const float* __restrict__ scale, long long mod_stride, T* __restrict__ y) {
    free_grid_dep_wait();                  // x is the previous kernel's output
    free_grid_dep_launch();
    const int lane = threadIdx.x % 32;
    const int warps = gridDim.x * (blockDim.x / 32);
    const int gwarp = blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
    int row = gwarp;
    const float invD = 1.f / (float)D;
    if (VPL > 0) {
        // A warp takes a contiguous run of rows, so that the modulation of its sequence stays in registers (re-read from
        // L1 for every row it cost 13% of this kernel's time); the next row's loads are in flight while this one is reduced.
        const int rpw = (M + warps - 1) / warps;
        row = gwarp * rpw;
        const int row_end = row + rpw < M ? row + rpw : M;
        float4 v[VPL > 0 ? VPL : 1], nx[VPL > 0 ? VPL : 1], msc[VPL > 0 ? VPL : 1], msh[VPL > 0 ? VPL : 1];
        int cur_seq = -1;
        if (row < row_end) {
#pragma unroll
            for (int i = 0; i < VPL; ++i) nx[i] = __ldcs(reinterpret_cast<const float4*>(x + (long long)row * D) + i * 32 + lane);
        }
        for (; row < row_end; ++row) {
#pragma unroll
            for (int i = 0; i < VPL; ++i) v[i] = nx[i];
            if (row + 1 < row_end) {
#pragma unroll
                for (int i = 0; i < VPL; ++i) nx[i] = __ldcs(reinterpret_cast<const float4*>(x + (long long)(row + 1) * D) + i * 32 + lane);
            }
            const int seq = row / rows_per_seq;
            if (seq != cur_seq) {                               // warp-uniform: once per sequence
                const long long mo = (long long)seq * mod_stride;
#pragma unroll
                for (int i = 0; i < VPL; ++i) {
                    const int c0 = (i * 32 + lane) * 4;
                    msh[i] = __ldg(reinterpret_cast<const float4*>(shift + mo + c0));
                    const float4 sc = __ldg(reinterpret_cast<const float4*>(scale + mo + c0));
                    msc[i] = make_float4(1.f + sc.x, 1.f + sc.y, 1.f + sc.z, 1.f + sc.w);
                }
                cur_seq = seq;
            }
            float s = 0.f;
#pragma unroll
            for (int i = 0; i < VPL; ++i) s += (v[i].x + v[i].y) + (v[i].z + v[i].w);
            const float mu = free_warp_sum(s) * invD;
            float q = 0.f;
#pragma unroll
            for (int i = 0; i < VPL; ++i) {
                float a = v[i].x - mu, b = v[i].y - mu, c = v[i].z - mu, d = v[i].w - mu;
                q += (a * a + b * b) + (c * c + d * d);
            }
            const float rstd = rsqrtf(free_warp_sum(q) * invD + 1e-6f);
#pragma unroll
            for (int i = 0; i < VPL; ++i) {
                float o0 = (v[i].x - mu) * rstd * msc[i].x + msh[i].x;
                float o1 = (v[i].y - mu) * rstd * msc[i].y + msh[i].y;
                float o2 = (v[i].z - mu) * rstd * msc[i].z + msh[i].z;
                float o3 = (v[i].w - mu) * rstd * msc[i].w + msh[i].w;
                if (sizeof(T) == 4) {
                    reinterpret_cast<float4*>(y + (long long)row * D)[i * 32 + lane] = make_float4(o0, o1, o2, o3);
                } else {
                    __nv_bfloat162 lo = __floats2bfloat162_rn(o0, o1), hi = __floats2bfloat162_rn(o2, o3);
                    uint2 pk;
                    pk.x = *reinterpret_cast<uint32_t*>(&lo);
                    pk.y = *reinterpret_cast<uint32_t*>(&hi);
                    reinterpret_cast<uint2*>(y + (long long)row * D)[i * 32 + lane] = pk;
                    if (SPLIT) {                                    // residual plane: what bf16 rounding lost
                        const float2 f01 = __bfloat1622float2(lo), f23 = __bfloat1622float2(hi);
                        __nv_bfloat162 r01 = __floats2bfloat162_rn(o0 - f01.x, o1 - f01.y), r23 = __floats2bfloat162_rn(o2 - f23.x, o3 - f23.y);
                        pk.x = *reinterpret_cast<uint32_t*>(&r01);
                        pk.y = *reinterpret_cast<uint32_t*>(&r23);
                        reinterpret_cast<uint2*>(y + (long long)M * D + (long long)row * D)[i * 32 + lane] = pk;
                    }
                }
            }
        }
    } else {
        for (; row < M; row += warps) {
            const float* xr = x + (long long)row * D;
            const long long mo = (long long)(row / rows_per_seq) * mod_stride;
            float s = 0.f;
            for (int c = lane; c < D; c += 32) s += xr[c];
            const float mu = free_warp_sum(s) * invD;
            float q = 0.f;
            for (int c = lane; c < D; c += 32) { float a = xr[c] - mu; q += a * a; }
            const float rstd = rsqrtf(free_warp_sum(q) * invD + 1e-6f);
            for (int c = lane; c < D; c += 32) {
                const float o = (xr[c] - mu) * rstd * (1.f + scale[mo + c]) + shift[mo + c];
                store_act(y + (long long)row * D + c, o);
                if (SPLIT) store_act(y + (long long)M * D + (long long)row * D + c, o - (float)y[(long long)row * D + c]);
            }
        }
    }
}

// Head matrix and bias with their rows regrouped from the model's (row-in-patch, column-in-patch, channel) order to
// (channel, row-in-patch, column-in-patch), so that the C noise channels of a token are one contiguous run of the head's
// output.  SPLIT: two bf16 planes (hi, lo) for the three-GEMM product; else an fp32 copy.
template <bool SPLIT>
__global__ void head_weights_kernel(int p, int c_out, int D, const float* __restrict__ w, const float* __restrict__ b,
                                    void* __restrict__ out0, __nv_bfloat16* __restrict__ lo, float* __restrict__ b_out) {
    const long long n = (long long)p * p * c_out * D;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        const int row = (int)(i / D), col = (int)(i % D);
        const int ch = row / (p * p), pix = row % (p * p);
        const int src = pix * c_out + ch;
        const float v = w[(long long)src * D + col];
        if (SPLIT) {
            const __nv_bfloat16 h = __float2bfloat16(v);
            reinterpret_cast<__nv_bfloat16*>(out0)[i] = h;
            lo[i] = __float2bfloat16(v - __bfloat162float(h));
        } else {
            reinterpret_cast<float*>(out0)[i] = v;
        }
        if (col == 0) b_out[row] = b ? b[src] : 0.f;
    }
}

template <typename T>
__global__ void convert_kernel(long long n, const float* __restrict__ x, T* __restrict__ y) {
    const long long n4 = n / 4, stride = (long long)gridDim.x * blockDim.x, i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y)) & 15u) == 0) {
        for (long long i = i0; i < n4; i += stride) {
            const float4 v = __ldcs(reinterpret_cast<const float4*>(x) + i);
            if (sizeof(T) == 4) {
                reinterpret_cast<float4*>(y)[i] = v;
            } else {
                __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
                uint2 pk;
                pk.x = *reinterpret_cast<uint32_t*>(&lo);
                pk.y = *reinterpret_cast<uint32_t*>(&hi);
                reinterpret_cast<uint2*>(y)[i] = pk;
            }
        }
        for (long long i = n4 * 4 + i0; i < n; i += stride) store_act(y + i, x[i]);
    } else {
        for (long long i = i0; i < n; i += stride) store_act(y + i, x[i]);
    }
}

// ---------------------------------------------------------------------------------------------
// Tail of the pass.  For latent element (state, c, y, x): the head's token (y/p, x/p) holds the value at
// vector position ((y%p) p + x%p) c_out + c; the first C channels are the noise prediction.  Guidance:
// eps = eps_u + w (eps_c - eps_u).  mean = coef_x[t] x - coef_eps[t] eps.  Optionally draws the next
// state sample = mean + sqrt(sigma2[t]) noise (drafter step / target step of the sampling loop).
struct TailArgs {
    int n_states, G, d, N_sched;
    float cfg_scale;
    const float* head_out; const float* x_in; long long x_stride;
    const int32_t* t_idx; const float *coef_x, *coef_eps, *sigma2;
    float* mean_out; long long mean_stride;
    float* eps_out; long long eps_stride;
    const float* noise; long long noise_stride;
    float* sample_out; long long sample_stride;
    float* sample_out2; long long sample2_stride; const int32_t* sample2_mask;
};

// Guidance, the reverse-transition mean (Eq. ddpm_update) and optionally the sample, elementwise over the images the
// head wrote: head_out [n_states, G, d].
__global__ void __launch_bounds__(256) head_to_mean_kernel(TailArgs a) {
    const int d = a.d;
    const long long total = (long long)a.n_states * d;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int st = (int)(i / d), e = (int)(i % d);
        float eps = a.head_out[(long long)st * a.G * d + e];
        if (a.G == 2) {
            const float eu = a.head_out[((long long)st * a.G + 1) * d + e];
            eps = eu + a.cfg_scale * (eps - eu);
        }
        int t = a.t_idx[st];
        t = t < 0 ? 0 : (t >= a.N_sched ? a.N_sched - 1 : t);
        const float xv = a.x_in[(long long)st * a.x_stride + e];
        const float mean = a.coef_x[t] * xv - a.coef_eps[t] * eps;
        if (a.mean_out) a.mean_out[(long long)st * a.mean_stride + e] = mean;
        if (a.eps_out) a.eps_out[(long long)st * a.eps_stride + e] = eps;
        if (a.noise) {
            const float smp = mean + sqrtf(fmaxf(a.sigma2[t], 0.f)) * a.noise[(long long)st * a.noise_stride + e];
            if (a.sample_out) a.sample_out[(long long)st * a.sample_stride + e] = smp;
            if (a.sample_out2 && (!a.sample2_mask || a.sample2_mask[st])) a.sample_out2[(long long)st * a.sample2_stride + e] = smp;
        }
    }
}

}  // namespace

int cond_setup(int dtype, int n_states, int G, int freq_dim, int n_classes, int N_sched,
               const int32_t* t_idx, const int32_t* labels, const float* t_embed_value,
               void* temb, int32_t* lab_seq, cudaStream_t s) {
    const int S = n_states * G;
    if (dtype == FREE_FP32)
        cond_setup_kernel<float><<<S, 128, 0, s>>>(n_states, G, freq_dim, n_classes, N_sched, t_idx, labels, t_embed_value, (float*)temb, lab_seq);
    else
        cond_setup_kernel<__nv_bfloat16><<<S, 128, 0, s>>>(n_states, G, freq_dim, n_classes, N_sched, t_idx, labels, t_embed_value, (__nv_bfloat16*)temb, lab_seq);
    return free_check_launch();
}

template <typename T>
static int patch_embed_launch(int n_states, int G, int C, int H, int W, int p, int D, const float* x_in, long long x_stride,
                              const float* pe_w, const float* pe_b, const float* pos, T* out, cudaStream_t s) {
    const int n_tok = (H / p) * (W / p), pd = C * p * p;
    const int n_items = n_states * n_tok;
    if (pd == 16 && D % 128 == 0 && D / 128 <= 9 && n_tok % 4 == 0 && free_aligned16(pe_b) && free_aligned16(pos) && free_aligned16(out)) {
        const int vpl = D / 128, wpc = 8;
        const size_t smem = (size_t)16 * D * 4 + (size_t)wpc * 4 * 16 * 4;
        const int n_groups = n_items / 4;
        const unsigned need = (unsigned)((n_groups + wpc - 1) / wpc), cap = 148u * 2u;
        const unsigned grid = need < cap ? need : cap;
        cudaError_t attr = cudaSuccess;
#define FREE_PE_WIDE(V) do { static cudaError_t once = cudaFuncSetAttribute(patch_embed_wide_kernel<T, V>, cudaFuncAttributeMaxDynamicSharedMemorySize, 16 * 128 * V * 4 + 8 * 4 * 16 * 4); attr = once; \
            if (attr == cudaSuccess) patch_embed_wide_kernel<T, V><<<grid, 256, smem, s>>>(n_items, G, C, H, W, p, D, x_in, x_stride, pe_w, pe_b, pos, out); } while (0)
        switch (vpl) {
            case 3: FREE_PE_WIDE(3); break;
            case 9: FREE_PE_WIDE(9); break;
            default: attr = cudaErrorInvalidValue; break;
        }
#undef FREE_PE_WIDE
        if (attr == cudaSuccess) return free_check_launch();
        (void)cudaGetLastError();                         // other widths: the kernels below
    }
    if (pd == 16 && D <= 5 * 256) {                   // the DiT */2 models: 4 channels, 2 x 2 patches
        const unsigned grid = (unsigned)(n_items < 148 * 4 ? n_items : 148 * 4);
        const int cpt = (D + 255) / 256;
        switch (cpt) {
            case 1: patch_embed_kernel<T, 16, 1><<<grid, 256, 0, s>>>(n_items, G, C, H, W, p, D, x_in, x_stride, pe_w, pe_b, pos, out); break;
            case 2: patch_embed_kernel<T, 16, 2><<<grid, 256, 0, s>>>(n_items, G, C, H, W, p, D, x_in, x_stride, pe_w, pe_b, pos, out); break;
            case 3: patch_embed_kernel<T, 16, 3><<<grid, 256, 0, s>>>(n_items, G, C, H, W, p, D, x_in, x_stride, pe_w, pe_b, pos, out); break;
            case 4: patch_embed_kernel<T, 16, 4><<<grid, 256, 0, s>>>(n_items, G, C, H, W, p, D, x_in, x_stride, pe_w, pe_b, pos, out); break;
            default: patch_embed_kernel<T, 16, 5><<<grid, 256, 0, s>>>(n_items, G, C, H, W, p, D, x_in, x_stride, pe_w, pe_b, pos, out); break;
        }
    } else {
        patch_embed_generic_kernel<T><<<(unsigned)n_items, 128, (size_t)pd * sizeof(float), s>>>(G, C, H, W, p, D, x_in, x_stride, pe_w, pe_b, pos, out);
    }
    return free_check_launch();
}

int patch_embed(int out_dtype, int n_states, int G, int C, int H, int W, int p, int D,
                const float* x_in, long long x_stride, const float* pe_w, const float* pe_b, const float* pos,
                void* out, cudaStream_t s) {
    return out_dtype == FREE_FP32
        ? patch_embed_launch<float>(n_states, G, C, H, W, p, D, x_in, x_stride, pe_w, pe_b, pos, (float*)out, s)
        : patch_embed_launch<__nv_bfloat16>(n_states, G, C, H, W, p, D, x_in, x_stride, pe_w, pe_b, pos, (__nv_bfloat16*)out, s);
}

template <typename T>
static int ln_launch(int M, int D, int rps, const float* x, const float* sh, const float* sc, long long ms, T* y, cudaStream_t s) {
    const bool vec = (D % 128 == 0) && (ms % 4 == 0) && free_aligned16(sh) && free_aligned16(sc) && free_aligned16(x) && free_aligned16(y);
    const int vpl = vec ? D / 128 : 0;
    // one warp per row at a time; persistent: 2 CTAs of 8 warps per SM, or 1 CTA of 12 warps for the widest rows
    const int wpc = vpl == 9 ? 12 : 8;
    const unsigned need = (unsigned)((M + wpc - 1) / wpc), cap = vpl == 9 ? 148u : 148u * 2u;
    const unsigned grid = need < cap ? need : cap;
    switch (vpl) {
        case 3: return free_launch(free_overlap_for_rows(M), ln_modulate_kernel<T, 3>, dim3(grid), dim3(256), 0, s, M, D, rps, x, sh, sc, ms, y);    // D = 384
        case 9: return free_launch(free_overlap_for_rows(M), ln_modulate_kernel<T, 9>, dim3(grid), dim3(384), 0, s, M, D, rps, x, sh, sc, ms, y);    // D = 1152
        default: return free_launch(free_overlap_for_rows(M), ln_modulate_kernel<T, 0>, dim3(grid), dim3(256), 0, s, M, D, rps, x, sh, sc, ms, y);
    }
}

int ln_modulate(int out_dtype, int M, int D, int rows_per_seq, const float* x, const float* shift, const float* scale,
                long long mod_stride, void* y, cudaStream_t s) {
    if (M < 1 || D < 1 || rows_per_seq < 1 || !x || !shift || !scale || !y) return FREE_ERR_ARG;
    return out_dtype == FREE_FP32 ? ln_launch<float>(M, D, rows_per_seq, x, shift, scale, mod_stride, (float*)y, s)
                                  : ln_launch<__nv_bfloat16>(M, D, rows_per_seq, x, shift, scale, mod_stride, (__nv_bfloat16*)y, s);
}

// bf16 hi / lo planes of the modulated LayerNorm (hi at y, lo at y + M*D elements)
int ln_modulate_split(int M, int D, int rows_per_seq, const float* x, const float* shift, const float* scale,
                      long long mod_stride, void* y, cudaStream_t s) {
    if (M < 1 || D < 1 || rows_per_seq < 1 || !x || !shift || !scale || !y) return FREE_ERR_ARG;
    __nv_bfloat16* yb = (__nv_bfloat16*)y;
    const bool vec = (D % 128 == 0) && (mod_stride % 4 == 0) && free_aligned16(shift) && free_aligned16(scale) && free_aligned16(x) &&
                     free_aligned16(y) && ((long long)M * D) % 8 == 0;
    const int vpl = vec ? D / 128 : 0;
    const int wpc = vpl == 9 ? 12 : 8;
    const unsigned need = (unsigned)((M + wpc - 1) / wpc), cap = vpl == 9 ? 148u : 148u * 2u;
    const unsigned grid = need < cap ? need : cap;
    switch (vpl) {
        case 3: ln_modulate_kernel<__nv_bfloat16, 3, true><<<grid, 256, 0, s>>>(M, D, rows_per_seq, x, shift, scale, mod_stride, yb); break;
        case 9: ln_modulate_kernel<__nv_bfloat16, 9, true><<<grid, 384, 0, s>>>(M, D, rows_per_seq, x, shift, scale, mod_stride, yb); break;
        default: ln_modulate_kernel<__nv_bfloat16, 0, true><<<grid, 256, 0, s>>>(M, D, rows_per_seq, x, shift, scale, mod_stride, yb); break;
    }
    return free_check_launch();
}

int head_weights(bool split, int p, int c_out, int D, const float* w, const float* b, void* out0, void* lo, float* b_out, cudaStream_t s) {
    const long long n = (long long)p * p * c_out * D;
    const unsigned grid = (unsigned)((n + 255) / 256 > 148 * 8 ? 148 * 8 : (n + 255) / 256);
    if (split) head_weights_kernel<true><<<grid, 256, 0, s>>>(p, c_out, D, w, b, out0, (__nv_bfloat16*)lo, b_out);
    else head_weights_kernel<false><<<grid, 256, 0, s>>>(p, c_out, D, w, b, out0, nullptr, b_out);
    return free_check_launch();
}

int convert_rows(int out_dtype, long long n, const float* x, void* y, cudaStream_t s) {
    const unsigned grid = (unsigned)((n + 255) / 256 > 148 * 16 ? 148 * 16 : (n + 255) / 256);
    if (out_dtype == FREE_FP32) convert_kernel<float><<<grid, 256, 0, s>>>(n, x, (float*)y);
    else convert_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>(n, x, (__nv_bfloat16*)y);
    return free_check_launch();
}

int head_to_mean(int n_states, int G, int d, float cfg_scale, int N_sched,
                 const float* head_out, const float* x_in, long long x_stride,
                 const int32_t* t_idx, const float* coef_x, const float* coef_eps, const float* sigma2,
                 float* mean_out, long long mean_stride, float* eps_out, long long eps_stride,
                 const float* noise, long long noise_stride, float* sample_out, long long sample_stride,
                 float* sample_out2, long long sample2_stride, const int32_t* sample2_mask, cudaStream_t s) {
    TailArgs a{n_states, G, d, N_sched, cfg_scale, head_out, x_in, x_stride, t_idx, coef_x, coef_eps, sigma2,
               mean_out, mean_stride, eps_out, eps_stride, noise, noise_stride, sample_out, sample_stride,
               sample_out2, sample2_stride, sample2_mask};
    const long long total = (long long)n_states * d;
    const unsigned grid = (unsigned)((total + 255) / 256 > 148 * 8 ? 148 * 8 : (total + 255) / 256);
    head_to_mean_kernel<<<grid, 256, 0, s>>>(a);
    return free_check_launch();
}

extern "C" int free_op_ln_modulate(int out_dtype, int M, int D, int rows_per_seq, const float* x,
                                   const float* shift, const float* scale, int64_t mod_stride, void* y, void* stream) {
    if (out_dtype != FREE_FP32 && out_dtype != FREE_BF16) return FREE_ERR_ARG;
    return ln_modulate(out_dtype, M, D, rows_per_seq, x, shift, scale, mod_stride, y, reinterpret_cast<cudaStream_t>(stream));
}
