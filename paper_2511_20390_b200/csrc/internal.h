// Internal interfaces between the translation units of libfree_b200 (not part of the public ABI).
#pragma once
#include "common.cuh"

// ---- linear layers ---------------------------------------------------------------------------
// out = epilogue(A[M,K] * W[N,K]^T + bias).  A has row stride lda, W row stride ldw (elements).
enum {
    EPI_BIAS = FREE_EPI_BIAS,
    EPI_BIAS_GELU = FREE_EPI_BIAS_GELU,
    EPI_BIAS_SILU = FREE_EPI_BIAS_SILU,
    EPI_GATE_RESIDUAL = FREE_EPI_GATE_RESIDUAL,   // resid += gate * (acc + bias); gate == nullptr means 1
    EPI_BIAS_EMB_SILU = 4,                        // out = silu(acc + bias + emb[emb_idx[row], n])
    EPI_QKV_HEADS = 5,                            // bf16 only: scatter (acc + bias) into head-major q, k and v^T
    EPI_QKV_TOKV = 6,                             // bf16 only (CTA-pair kernel): q and k token-major into out[M, 2D], v^T head-major
    EPI_UNPATCH = 7,                              // head: (acc + bias) of the first img_C channels scattered into images (see LinearArgs)
    EPI_UNPATCH_ACC = 8,                          // the same, added to what the images hold
};

struct LinearArgs {
    int M = 0, N = 0, K = 0;
    const void* A = nullptr; long long lda = 0;
    const void* W = nullptr; long long ldw = 0;
    const float* bias = nullptr;
    int epi = EPI_BIAS;
    int out_dtype = FREE_FP32;
    void* out = nullptr; long long ldo = 0;
    float* resid = nullptr;                       // [M, N] fp32, row stride N
    const float* gate = nullptr; long long gate_stride = 0; int rows_per_seq = 1;
    const float* emb = nullptr; const int32_t* emb_idx = nullptr;
    // EPI_QKV_HEADS
    int heads = 0, d_head = 0, d_pad = 0, n_tok = 0;
    void* q = nullptr; void* k = nullptr; void* vt = nullptr;
    // EPI_UNPATCH[_ACC]: row = seq * n_tok + token (tokens row-major over the patch grid), column = (ch * p + pr) * p + pc;
    // out is fp32 [n_seq, img_C, img_H, img_W], element (seq, ch, trow * p + pr, tcol * p + pc); columns with ch >= img_C are dropped
    int img_C = 0, img_H = 0, img_W = 0, img_p = 0;
    uint32_t* err = nullptr;                      // device error word (tensor-core path)
};

int linear_fp32(const LinearArgs& a, cudaStream_t s);   // CUDA cores, any sizes
int linear_bf16(const LinearArgs& a, cudaStream_t s);   // tcgen05; K % 64 == 0, N % 16 == 0
bool linear_bf16_supported(int N, int K);
bool linear_bf16_pair_eligible(const LinearArgs& a);    // large shapes run on CTA pairs (256 x BN tiles)
int linear_bf16_pair(const LinearArgs& a, cudaStream_t s);

// ---- attention -------------------------------------------------------------------------------
// token-major qkv [n_seq, n_tok, 3, heads, d_head] -> out [n_seq, n_tok, heads*d_head]
int attention_simt(int dtype, int n_seq, int n_tok, int heads, int d_head, const void* qkv, void* out, cudaStream_t s);
// head-major bf16 operands written by EPI_QKV_HEADS: q,k [n_seq, heads, n_tok, d_pad], vt [n_seq, heads, d_pad, n_tok]
int attention_tc(int n_seq, int n_tok, int heads, int d_head, int d_pad, const void* q, const void* k, const void* vt,
                 void* out, uint32_t* err, cudaStream_t s);
bool attention_tc_supported(int n_tok, int d_head);
int attention_tc_dpad(int d_head);
// Two query tiles per CTA; q and k read from a token-major matrix [n_seq*n_tok, ld] (first `width` columns valid),
// head h of q at column q_col0 + h*d_head, of k at k_col0 + h*d_head; vt [n_seq, heads, d_pad, n_tok].
int attention_tc2(int n_seq, int n_tok, int heads, int d_head, const void* qk, long long ld, int width, int q_col0, int k_col0,
                  const void* vt, void* out, uint32_t* err, cudaStream_t s);
bool attention_tc2_supported(int n_tok, int d_head);
int attention_tc2_dpad(int d_head);

// ---- elementwise / row kernels ----------------------------------------------------------------
int cond_setup(int dtype, int n_states, int G, int freq_dim, int n_classes, int N_sched,
               const int32_t* t_idx, const int32_t* labels, const float* t_embed_value,
               void* temb /*[S,freq_dim]*/, int32_t* lab_seq /*[S]*/, cudaStream_t s);
int patch_embed(int out_dtype, int n_states, int G, int C, int H, int W, int p, int D,
                const float* x_in, long long x_stride, const float* pe_w, const float* pe_b, const float* pos,
                void* out /*[S*n_tok, D]*/, cudaStream_t s);
int ln_modulate(int out_dtype, int M, int D, int rows_per_seq, const float* x, const float* shift, const float* scale,
                long long mod_stride, void* y, cudaStream_t s);
int convert_rows(int out_dtype, long long n, const float* x, void* y, cudaStream_t s);
// y = modulated LayerNorm as two bf16 planes: hi = bf16(y) at y_split[0 .. M*D), lo = bf16(y - hi) behind it
int ln_modulate_split(int M, int D, int rows_per_seq, const float* x, const float* shift, const float* scale,
                      long long mod_stride, void* y_split, cudaStream_t s);
// head matrix [p*p*c_out, D] and bias with rows regrouped to (channel, row-in-patch, column-in-patch); split: bf16 hi / lo
// planes into out0 / lo, else an fp32 copy into out0
int head_weights(bool split, int p, int c_out, int D, const float* w, const float* b, void* out0, void* lo, float* b_out, cudaStream_t s);
// head_out [n_states, G, d]: the noise prediction of every stream as images (written by the head's EPI_UNPATCH epilogue)
int head_to_mean(int n_states, int G, int d, float cfg_scale, int N_sched,
                 const float* head_out, const float* x_in, long long x_stride,
                 const int32_t* t_idx, const float* coef_x, const float* coef_eps, const float* sigma2,
                 float* mean_out, long long mean_stride, float* eps_out, long long eps_stride,
                 const float* noise, long long noise_stride, float* sample_out, long long sample_stride,
                 float* sample_out2, long long sample2_stride, const int32_t* sample2_mask, cudaStream_t s);

// ---- verification from the noise predictions (verify_fused.cu) ----------------------------------
// As the public spec_verify_fused, with a row stride (elements) for x_first.
int spec_verify_fused_launch(int B, int K, long long d, int G, float cfg_scale,
                             const float* eps, const float* x_first, long long x_first_stride,
                             const float* m_draft, const float* x_draft, const float* coef_x, const float* coef_eps,
                             const float* sigma2, const float* lambda, const float* u, const int32_t* n_valid, int chunk,
                             float* x_out, int32_t* n_accept, float* logratio_out, float* dist2_out, float* means_out, cudaStream_t s);
