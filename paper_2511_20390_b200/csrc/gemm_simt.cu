// fp32 linear layers on CUDA cores (the exact-arithmetic mode used for small models and for checking
// the data flow): 64x64 output tile per CTA, 4x4 outputs per thread, K staged 16 at a time through
// shared memory.  Any M, N, K; every global access is bounds-checked.
#include "internal.h"

namespace {

constexpr int TM = 64, TN = 64, TK = 16;

struct SimtArgs {
    int M, N, K;
    const float* A; long long lda;
    const float* W; long long ldw;
    const float* bias;
    int epi, out_dtype;
    void* out; long long ldo;
    float* resid; const float* gate; long long gate_stride; int rows_per_seq;
    const float* emb; const int32_t* emb_idx;
    int n_tok, img_C, img_H, img_W, img_p;
};

__global__ void __launch_bounds__(256) linear_fp32_kernel(SimtArgs a) {
    __shared__ float As[TK][TM + 1];
    __shared__ float Ws[TK][TN + 1];
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    const int m0 = blockIdx.y * TM, n0 = blockIdx.x * TN;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < a.K; k0 += TK) {
        for (int i = threadIdx.x; i < TM * TK; i += 256) {
            int r = i / TK, c = i % TK;
            int gm = m0 + r, gk = k0 + c;
            As[c][r] = (gm < a.M && gk < a.K) ? a.A[(long long)gm * a.lda + gk] : 0.f;
            int gn = n0 + r;
            Ws[c][r] = (gn < a.N && gk < a.K) ? a.W[(long long)gn * a.ldw + gk] : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < TK; ++kk) {
            float av[4], wv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { av[i] = As[kk][ty * 4 + i]; wv[i] = Ws[kk][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], wv[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int gm = m0 + ty * 4 + i;
        if (gm >= a.M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int gn = n0 + tx * 4 + j;
            if (gn >= a.N) continue;
            float v = acc[i][j] + (a.bias ? a.bias[gn] : 0.f);
            if (a.epi == EPI_GATE_RESIDUAL) {
                float g = a.gate ? a.gate[(long long)(gm / a.rows_per_seq) * a.gate_stride + gn] : 1.f;
                a.resid[(long long)gm * a.N + gn] += g * v;
                continue;
            }
            if (a.epi == EPI_UNPATCH || a.epi == EPI_UNPATCH_ACC) {     // head: token vectors scattered into images
                const int p = a.img_p, gw = a.img_W / p, ch = gn / (p * p), pr = (gn % (p * p)) / p, pc = gn % p;
                if (ch >= a.img_C) continue;
                const int seq = gm / a.n_tok, tok = gm % a.n_tok;
                float* dst = reinterpret_cast<float*>(a.out) +
                             (((long long)seq * a.img_C + ch) * a.img_H + (tok / gw) * p + pr) * a.img_W + (tok % gw) * p + pc;
                *dst = (a.epi == EPI_UNPATCH_ACC ? *dst : 0.f) + v;
                continue;
            }
            if (a.epi == EPI_BIAS_GELU) v = free_gelu_tanh(v);
            else if (a.epi == EPI_BIAS_SILU) v = free_silu(v);
            else if (a.epi == EPI_BIAS_EMB_SILU) v = free_silu(v + a.emb[(long long)a.emb_idx[gm] * a.N + gn]);
            if (a.out_dtype == FREE_BF16) reinterpret_cast<__nv_bfloat16*>(a.out)[(long long)gm * a.ldo + gn] = __float2bfloat16(v);
            else reinterpret_cast<float*>(a.out)[(long long)gm * a.ldo + gn] = v;
        }
    }
}

}  // namespace

int linear_fp32(const LinearArgs& l, cudaStream_t s) {
    if (l.M < 1 || l.N < 1 || l.K < 1 || !l.A || !l.W) return FREE_ERR_ARG;
    if (l.epi == EPI_QKV_HEADS || l.epi == EPI_QKV_TOKV) return FREE_ERR_UNSUPPORTED;
    if ((l.epi == EPI_UNPATCH || l.epi == EPI_UNPATCH_ACC) &&
        (l.img_p < 1 || l.img_C < 1 || l.img_H % l.img_p || l.img_W % l.img_p || l.n_tok != (l.img_H / l.img_p) * (l.img_W / l.img_p) ||
         l.M % l.n_tok || l.out_dtype != FREE_FP32)) return FREE_ERR_ARG;
    if (l.epi == EPI_GATE_RESIDUAL ? !l.resid : !l.out) return FREE_ERR_ARG;
    if (l.epi == EPI_BIAS_EMB_SILU && (!l.emb || !l.emb_idx)) return FREE_ERR_ARG;
    SimtArgs a{l.M, l.N, l.K, (const float*)l.A, l.lda ? l.lda : l.K, (const float*)l.W, l.ldw ? l.ldw : l.K, l.bias,
               l.epi, l.out_dtype, l.out, l.ldo ? l.ldo : l.N, l.resid, l.gate, l.gate_stride,
               l.rows_per_seq > 0 ? l.rows_per_seq : 1, l.emb, l.emb_idx, l.n_tok, l.img_C, l.img_H, l.img_W, l.img_p};
    dim3 grid((l.N + TN - 1) / TN, (l.M + TM - 1) / TM);
    linear_fp32_kernel<<<grid, 256, 0, s>>>(a);
    return free_check_launch();
}
