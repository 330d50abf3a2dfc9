// Host orchestration: context, workspace layout, the packed target pass, the drafter step and the
// sampling loop (Algorithm 1).  Every numerical step is a kernel launch on the caller's stream.
#include "internal.h"
#include <math.h>
#include <new>
#include <string.h>
#include <vector>

enum { PC_COND = 0, PC_EMBED, PC_LN, PC_QKV, PC_ATTN, PC_PROJ, PC_FC1, PC_FC2, PC_HEAD, PC_TAIL, PC_DRAFT_FC,
       PC_VERIFY, PC_CTRL, PC_N };
static const char* const kProfNames[PC_N] = {
    "conditioning + modulation tables", "patch embed / feature copy", "layernorm + modulate", "linear qkv",
    "attention", "linear proj (gate + residual)", "linear fc1 + gelu", "linear fc2 (gate + residual)",
    "head (layernorm + projection)", "guidance + mean", "drafter fusion layer",
    "spec_verify_fused (guidance, mean, verify)",
    "round control"};

struct ProfRec { int cls; double work; cudaEvent_t e0, e1; };

struct free_ctx {
    mutable bool prof_on = false;
    mutable std::vector<ProfRec> prof;
    free_model_desc m;
    bool has_drafter;
    free_drafter_desc dr;
    int n_tok, d_latent, patch_dim, out_dim, d_head, F;
    bool tc_attn;        // bf16 mode: attention on the tensor cores (else the CUDA-core kernel)
    bool attn2;          // ... with the two-tile kernel that reads q and k token-major (needs D % 128 == 0, 64 <= d_head <= 96)
    int d_pad;
};

namespace {

// Brackets one kernel launch (or a short group) with CUDA events when profiling is on.
struct Scope {
    const free_ctx* c; cudaStream_t s; cudaEvent_t e1 = nullptr;
    Scope(const free_ctx* c_, int cls, double work, cudaStream_t s_) : c(c_), s(s_) {
        if (!c->prof_on) return;
        ProfRec r{cls, work, nullptr, nullptr};
        if (cudaEventCreate(&r.e0) != cudaSuccess || cudaEventCreate(&r.e1) != cudaSuccess) { (void)cudaGetLastError(); return; }
        cudaEventRecord(r.e0, s);
        e1 = r.e1;
        c->prof.push_back(r);
    }
    ~Scope() { if (e1) cudaEventRecord(e1, s); }
};

inline size_t act_size(int dtype) { return dtype == FREE_BF16 ? 2 : 4; }

struct Workspace {
    uint32_t* err;
    void *temb, *h1, *sc;
    int32_t* lab_seq;
    float *mod, *fmod, *x;
    void *hn, *qkv, *att, *hmlp, *emb, *fin_split;
    float* head_out;
    // sampling loop
    float* fin_bias;
    float *x_cur, *m_a, *pack_in, *x_draft, *m_draft, *sigma2_bk, *lam_bk, *u_bk, *cx_bk, *ce_bk, *ell_bk, *d2_bk;
    void *feat0, *feat1;
    int32_t *cur_a, *nv, *n_acc, *t_step, *t_pack, *lab_pack, *t_draft, *act_draft, *active;
    int32_t* report;           // what the host reads after a round, contiguous: error word, then active, nv, n_acc, cursor of every sample
    size_t total;
};

// Lays the buffers out for `n` states (S = 2n sequences at most).  base == nullptr only measures.
Workspace plan(const free_ctx* c, int n, void* base) {
    Workspace w;
    memset(&w, 0, sizeof(w));
    const free_model_desc& m = c->m;
    const size_t S = 2 * (size_t)n, M = S * c->n_tok, D = m.D, as = act_size(m.dtype);
    size_t off = 0;
    auto take = [&](size_t bytes) -> void* {
        void* p = base ? (char*)base + off : nullptr;
        off += free_round_up(bytes, 256);
        return p;
    };
    const int nb = c->has_drafter && c->dr.n_blocks > m.depth ? c->dr.n_blocks : m.depth;
    w.err = (uint32_t*)take(256);
    w.temb = take(S * m.freq_dim * as);
    w.h1 = take(S * D * as);
    w.sc = take(S * D * as);
    w.lab_seq = (int32_t*)take(S * 4);
    w.mod = (float*)take(S * (size_t)nb * 6 * D * 4);
    w.fmod = (float*)take(S * 2 * D * 4);
    w.x = (float*)take(M * D * 4);
    w.hn = take(M * D * 4);                       // fp32-sized: also holds the head's fp32 LayerNorm output
    const size_t qkv_tok = M * 3 * D * as;
    const size_t qkv_head = c->tc_attn ? 3 * S * m.heads * (size_t)c->n_tok * c->d_pad * 2 + 256 : 0;
    w.qkv = take(qkv_tok > qkv_head ? qkv_tok : qkv_head);
    w.att = take(M * D * as);
    w.hmlp = take(M * (size_t)c->F * as);
    w.emb = take(M * D * as);
    w.head_out = (float*)take(S * (size_t)c->d_latent * 4);     // noise prediction of every stream as images
    w.fin_split = take((size_t)c->out_dim * D * 2 * 2);       // regrouped head matrix: bf16 hi and lo planes, or one fp32 copy
    w.fin_bias = (float*)take((size_t)c->out_dim * 4);
    const size_t dl = c->d_latent;
    w.x_cur = (float*)take(n * dl * 4);
    w.m_a = (float*)take(n * dl * 4);
    w.pack_in = (float*)take(n * dl * 4);
    w.x_draft = (float*)take(n * dl * 4);
    w.m_draft = (float*)take(n * dl * 4);
    w.sigma2_bk = (float*)take(n * 4);
    w.lam_bk = (float*)take(n * 4);
    w.u_bk = (float*)take(n * 4);
    w.cx_bk = (float*)take(n * 4);
    w.ce_bk = (float*)take(n * 4);
    w.ell_bk = (float*)take(n * 4);
    w.d2_bk = (float*)take(n * 4);
    w.feat0 = take(M * D * as);
    w.feat1 = take(M * D * as);
    for (int32_t** p : {&w.cur_a, &w.nv, &w.n_acc, &w.t_step, &w.t_pack, &w.lab_pack, &w.t_draft, &w.act_draft, &w.active})
        *p = (int32_t*)take((size_t)n * 4 + 256);
    w.report = (int32_t*)take((4 + 4 * (size_t)n) * 4);
    w.total = off;
    return w;
}

int lin(const free_ctx* c, LinearArgs a, cudaStream_t s) {
    return c->m.dtype == FREE_FP32 ? linear_fp32(a, s) : linear_bf16(a, s);
}

struct Stack {                 // one stack of blocks + its head (target or drafter)
    free_block_weights bw;
    int n_blocks;
    const void* fada_w; const float* fada_b;
    const float* fin_w; const float* fin_b;
};

// conditioning: sc = SiLU(t-MLP(features(t)) + E[label]) for every sequence; then the modulation tables
int run_cond(const free_ctx* c, const Workspace& w, const Stack& st, int n_states, int G,
             const int32_t* t_idx, const int32_t* labels, const free_schedule* sch, cudaStream_t s) {
    const free_model_desc& m = c->m;
    const int S = n_states * G, D = m.D;
    Scope prof(c, PC_COND, 2.0 * S * D * ((double)m.freq_dim + D + st.n_blocks * 6.0 * D + 2.0 * D), s);
    FREE_TRY(cond_setup(m.dtype, n_states, G, m.freq_dim, m.n_classes, sch->N, t_idx, labels, sch->t_embed_value,
                        w.temb, w.lab_seq, s));
    LinearArgs a;
    a.err = w.err;
    a.M = S; a.N = D; a.K = m.freq_dim; a.A = w.temb; a.W = m.t_w1; a.bias = m.t_b1;
    a.epi = EPI_BIAS_SILU; a.out_dtype = m.dtype; a.out = w.h1;
    FREE_TRY(lin(c, a, s));
    a = LinearArgs(); a.err = w.err;
    a.M = S; a.N = D; a.K = D; a.A = w.h1; a.W = m.t_w2; a.bias = m.t_b2;
    a.epi = EPI_BIAS_EMB_SILU; a.emb = m.y_emb; a.emb_idx = w.lab_seq; a.out_dtype = m.dtype; a.out = w.sc;
    FREE_TRY(lin(c, a, s));
    // all blocks' (shift, scale, gate) x 2 in one GEMM: the conditioning does not depend on the tokens
    a = LinearArgs(); a.err = w.err;
    a.M = S; a.N = st.n_blocks * 6 * D; a.K = D; a.A = w.sc; a.W = st.bw.ada_w; a.bias = st.bw.ada_b;
    a.epi = EPI_BIAS; a.out_dtype = FREE_FP32; a.out = w.mod;
    FREE_TRY(lin(c, a, s));
    a = LinearArgs(); a.err = w.err;
    a.M = S; a.N = 2 * D; a.K = D; a.A = w.sc; a.W = st.fada_w; a.bias = st.fada_b;
    a.epi = EPI_BIAS; a.out_dtype = FREE_FP32; a.out = w.fmod;
    return lin(c, a, s);
}

// the transformer blocks on the residual stream w.x [S*n_tok, D] (fp32)
int run_blocks(const free_ctx* c, const Workspace& w, const Stack& st, int S, cudaStream_t s) {
    const free_model_desc& m = c->m;
    const int D = m.D, T = c->n_tok, M = S * T, F = c->F;
    const size_t as = act_size(m.dtype);
    const long long ms = (long long)st.n_blocks * 6 * D;
    for (int i = 0; i < st.n_blocks; ++i) {
        const float* mod = w.mod + (size_t)i * 6 * D;
        auto wmat = [&](const void* base, size_t rows) { return (const void*)((const char*)base + (size_t)i * rows * D * as); };
        // attention branch
        const double ln_bytes = (double)M * D * (4 + as);
        { Scope p(c, PC_LN, ln_bytes, s); FREE_TRY(ln_modulate(m.dtype, M, D, T, w.x, mod, mod + D, ms, w.hn, s)); }
        LinearArgs a; a.err = w.err;
        a.M = M; a.N = 3 * D; a.K = D; a.A = w.hn; a.W = wmat(st.bw.qkv_w, 3 * D); a.bias = st.bw.qkv_b + (size_t)i * 3 * D;
        a.out_dtype = m.dtype;
        if (c->attn2) {
            // q, k token-major [M, 2D]; v^T head-major behind them
            a.epi = EPI_QKV_TOKV; a.heads = m.heads; a.d_head = c->d_head; a.d_pad = c->d_pad; a.n_tok = T;
            a.out = w.qkv; a.ldo = 2LL * D; a.out_dtype = FREE_BF16;
            a.vt = (char*)w.qkv + free_round_up((size_t)M * 2 * D * 2, 256);
            { Scope p(c, PC_QKV, 2.0 * M * 3 * D * D, s); FREE_TRY(lin(c, a, s)); }
            { Scope p(c, PC_ATTN, 4.0 * S * m.heads * (double)T * T * c->d_head, s);
              FREE_TRY(attention_tc2(S, T, m.heads, c->d_head, w.qkv, 2LL * D, 2 * D, 0, D, a.vt, w.att, w.err, s)); }
        } else if (c->tc_attn) {
            a.epi = EPI_QKV_HEADS; a.heads = m.heads; a.d_head = c->d_head; a.d_pad = c->d_pad; a.n_tok = T;
            const size_t per = (size_t)S * m.heads * T * c->d_pad * 2;
            a.q = w.qkv; a.k = (char*)w.qkv + per; a.vt = (char*)w.qkv + 2 * per;
            { Scope p(c, PC_QKV, 2.0 * M * 3 * D * D, s); FREE_TRY(lin(c, a, s)); }
            { Scope p(c, PC_ATTN, 4.0 * S * m.heads * (double)T * T * c->d_head, s);
              FREE_TRY(attention_tc(S, T, m.heads, c->d_head, c->d_pad, a.q, a.k, a.vt, w.att, w.err, s)); }
        } else {
            a.epi = EPI_BIAS; a.out = w.qkv;
            { Scope p(c, PC_QKV, 2.0 * M * 3 * D * D, s); FREE_TRY(lin(c, a, s)); }
            { Scope p(c, PC_ATTN, 4.0 * S * m.heads * (double)T * T * c->d_head, s);
              FREE_TRY(attention_simt(m.dtype, S, T, m.heads, c->d_head, w.qkv, w.att, s)); }
        }
        a = LinearArgs(); a.err = w.err;
        a.M = M; a.N = D; a.K = D; a.A = w.att; a.W = wmat(st.bw.proj_w, D); a.bias = st.bw.proj_b + (size_t)i * D;
        a.epi = EPI_GATE_RESIDUAL; a.resid = w.x; a.gate = mod + 2 * D; a.gate_stride = ms; a.rows_per_seq = T;
        { Scope p(c, PC_PROJ, 2.0 * M * D * D, s); FREE_TRY(lin(c, a, s)); }
        // MLP branch
        { Scope p(c, PC_LN, ln_bytes, s); FREE_TRY(ln_modulate(m.dtype, M, D, T, w.x, mod + 3 * D, mod + 4 * D, ms, w.hn, s)); }
        a = LinearArgs(); a.err = w.err;
        a.M = M; a.N = F; a.K = D; a.A = w.hn; a.W = wmat(st.bw.fc1_w, F); a.bias = st.bw.fc1_b + (size_t)i * F;
        a.epi = EPI_BIAS_GELU; a.out_dtype = m.dtype; a.out = w.hmlp;
        { Scope p(c, PC_FC1, 2.0 * M * F * D, s); FREE_TRY(lin(c, a, s)); }
        a = LinearArgs(); a.err = w.err;
        a.M = M; a.N = D; a.K = F; a.A = w.hmlp; a.W = (const char*)st.bw.fc2_w + (size_t)i * D * F * as; a.bias = st.bw.fc2_b + (size_t)i * D;
        a.epi = EPI_GATE_RESIDUAL; a.resid = w.x; a.gate = mod + 5 * D; a.gate_stride = ms; a.rows_per_seq = T;
        { Scope p(c, PC_FC2, 2.0 * M * F * D, s); FREE_TRY(lin(c, a, s)); }
    }
    return FREE_OK;
}

// modulated head: LayerNorm + (shift, scale), then the narrow projection (N = p*p*c_out, 32 for the */2 models).
// fp32 mode: CUDA cores.  bf16 mode: tensor cores at fp32-level accuracy -- a plain bf16 head was measured to raise
// the error of the noise prediction from 1.1e-2 to 1.4e-2 of the 2e-2 bound, so activations and weights are each
// split into bf16 hi + lo planes and  y W^T ~ y_hi W_hi^T + y_lo W_hi^T + y_hi W_lo^T  (the dropped lo*lo term
// is 2^-16 relative) is accumulated in fp32 by three small GEMMs.
// Output: `out` fp32 [S, C, H, W]: the noise channels of every sequence as images.  The head matrix and bias are first
// copied with their rows regrouped to (channel, row-in-patch, column-in-patch); the GEMM's epilogue drops the
// remaining (variance) channels and scatters each token's vector into its patch (unpatchify fused into the store).
int run_head(const free_ctx* c, const Workspace& w, const Stack& st, int S, float* out, cudaStream_t s) {
    const free_model_desc& m = c->m;
    const int D = m.D, T = c->n_tok, M = S * T, N = c->out_dim;
    Scope prof(c, PC_HEAD, 2.0 * M * D * N, s);
    LinearArgs a;
    a.M = M; a.N = N; a.K = D; a.bias = w.fin_bias;
    a.epi = EPI_UNPATCH; a.out_dtype = FREE_FP32; a.out = out;
    a.n_tok = T; a.img_C = m.C; a.img_H = m.H; a.img_W = m.W; a.img_p = m.patch;
    if (m.dtype == FREE_BF16 && linear_bf16_supported(N, D)) {
        void* w_hi = w.fin_split;
        void* w_lo = (char*)w.fin_split + (size_t)N * D * 2;
        const void* y_hi = w.hn;
        const void* y_lo = (const char*)w.hn + (size_t)M * D * 2;
        FREE_TRY(head_weights(true, m.patch, m.c_out, D, st.fin_w, st.fin_b, w_hi, w_lo, w.fin_bias, s));
        FREE_TRY(ln_modulate_split(M, D, T, w.x, w.fmod, w.fmod + D, 2LL * D, w.hn, s));
        a.err = w.err;
        a.A = y_hi; a.W = w_hi;
        FREE_TRY(linear_bf16(a, s));                              // bias + y_hi W_hi^T
        a.epi = EPI_UNPATCH_ACC; a.bias = nullptr;
        a.A = y_lo; a.W = w_hi;
        FREE_TRY(linear_bf16(a, s));                              // += y_lo W_hi^T
        a.A = y_hi; a.W = w_lo;
        return linear_bf16(a, s);                                 // += y_hi W_lo^T
    }
    FREE_TRY(head_weights(false, m.patch, m.c_out, D, st.fin_w, st.fin_b, w.fin_split, nullptr, w.fin_bias, s));
    FREE_TRY(ln_modulate(FREE_FP32, M, D, T, w.x, w.fmod, w.fmod + D, 2LL * D, w.hn, s));
    a.A = w.hn; a.W = w.fin_split;
    return linear_fp32(a, s);
}

struct PassIO {
    const float* x_in; long long x_stride;
    const int32_t* t_idx; const int32_t* labels;
    float* mean_out; long long mean_stride;
    float* eps_out;
    void* feat_out;
    float* head_raw;            // if set: the pass ends with the noise prediction of every stream [S, C, H, W] written here
    // sampling (optional): sample = mean + sigma * noise
    const float* noise; long long noise_stride;
    float* sample_out; long long sample_stride;
    float* sample_out2; long long sample2_stride; const int32_t* sample2_mask;
};

Stack target_stack(const free_ctx* c) {
    return Stack{c->m.blocks, c->m.depth, c->m.fada_w, c->m.fada_b, c->m.fin_w, c->m.fin_b};
}
Stack drafter_stack(const free_ctx* c) {
    return Stack{c->dr.blocks, c->dr.n_blocks, c->dr.fada_w, c->dr.fada_b, c->dr.fin_w, c->dr.fin_b};
}

int tail(const free_ctx* c, const Workspace& w, int n_states, int G, float cfg, const free_schedule* sch,
         const PassIO& io, cudaStream_t s) {
    const free_model_desc& m = c->m;
    Scope prof(c, PC_TAIL, (double)n_states * c->d_latent * 4 * 3, s);
    return head_to_mean(n_states, G, c->d_latent, cfg, sch->N, w.head_out, io.x_in, io.x_stride,
                        io.t_idx, sch->coef_x, sch->coef_eps, sch->sigma2, io.mean_out, io.mean_stride,
                        io.eps_out, c->d_latent, io.noise, io.noise_stride, io.sample_out, io.sample_stride,
                        io.sample_out2, io.sample2_stride, io.sample2_mask, s);
}

int target_pass(const free_ctx* c, const Workspace& w, int n_states, float cfg, const free_schedule* sch,
                const PassIO& io, cudaStream_t s) {
    const free_model_desc& m = c->m;
    const int G = (cfg > 0.f && cfg != 1.f) ? 2 : 1, S = n_states * G;
    const Stack st = target_stack(c);
    FREE_TRY(run_cond(c, w, st, n_states, G, io.t_idx, io.labels, sch, s));
    { Scope p(c, PC_EMBED, (double)S * c->n_tok * m.D * 4, s);
      FREE_TRY(patch_embed(FREE_FP32, n_states, G, m.C, m.H, m.W, m.patch, m.D, io.x_in, io.x_stride, m.pe_w, m.pe_b, m.pos, w.x, s)); }
    FREE_TRY(run_blocks(c, w, st, S, s));
    if (io.feat_out) { Scope p(c, PC_EMBED, (double)S * c->n_tok * m.D * 6, s);
                       FREE_TRY(convert_rows(m.dtype, (long long)S * c->n_tok * m.D, w.x, io.feat_out, s)); }
    if (io.head_raw) return run_head(c, w, st, S, io.head_raw, s);
    FREE_TRY(run_head(c, w, st, S, w.head_out, s));
    return tail(c, w, n_states, G, cfg, sch, io, s);
}

int drafter_pass(const free_ctx* c, const Workspace& w, int n_states, float cfg, const free_schedule* sch,
                 const PassIO& io, const void* f_prev, cudaStream_t s) {
    const free_model_desc& m = c->m;
    const int G = (cfg > 0.f && cfg != 1.f) ? 2 : 1, S = n_states * G, D = m.D, M = S * c->n_tok;
    const size_t as = act_size(m.dtype);
    const Stack st = drafter_stack(c);
    FREE_TRY(run_cond(c, w, st, n_states, G, io.t_idx, io.labels, sch, s));
    { Scope p(c, PC_EMBED, (double)M * D * as, s);
      FREE_TRY(patch_embed(m.dtype, n_states, G, m.C, m.H, m.W, m.patch, D, io.x_in, io.x_stride, m.pe_w, m.pe_b, m.pos, w.emb, s)); }
    {   // g = W_fc [embed || f] + b  as two accumulating GEMMs over the two halves of W_fc (row stride 2D)
        Scope fc(c, PC_DRAFT_FC, 2.0 * M * D * 2 * D, s);
        LinearArgs a; a.err = w.err;
        a.M = M; a.N = D; a.K = D; a.A = w.emb; a.W = c->dr.fc_w; a.ldw = 2 * D; a.bias = c->dr.fc_b;
        a.epi = EPI_BIAS; a.out_dtype = FREE_FP32; a.out = w.x;
        FREE_TRY(lin(c, a, s));
        a = LinearArgs(); a.err = w.err;
        a.M = M; a.N = D; a.K = D; a.A = f_prev; a.W = (const char*)c->dr.fc_w + (size_t)D * as; a.ldw = 2 * D;
        a.epi = EPI_GATE_RESIDUAL; a.resid = w.x; a.gate = nullptr; a.rows_per_seq = c->n_tok;
        FREE_TRY(lin(c, a, s));
    }
    FREE_TRY(run_blocks(c, w, st, S, s));
    if (io.feat_out) { Scope p(c, PC_EMBED, (double)M * D * 6, s); FREE_TRY(convert_rows(m.dtype, (long long)M * D, w.x, io.feat_out, s)); }
    FREE_TRY(run_head(c, w, st, S, w.head_out, s));
    return tail(c, w, n_states, G, cfg, sch, io, s);
}

int check_common(const free_ctx* c, int n_states, const free_schedule* sch, void* ws, size_t ws_bytes) {
    if (!c || !sch) return FREE_ERR_ARG;
    if (n_states < 1 || sch->N < 1) return FREE_ERR_SHAPE;
    if (!sch->coef_x || !sch->coef_eps || !sch->sigma2 || !sch->t_embed_value) return FREE_ERR_ARG;
    if (!ws || ws_bytes < plan(c, n_states, nullptr).total) return FREE_ERR_WORKSPACE;
    if (!free_aligned16(ws)) return FREE_ERR_ALIGN;
    return FREE_OK;
}

// ------------------------------------------------------------------------------------------------
// round control of the sampling loop (per-sample cursors, Alg. 1)
struct RoundArgs {
    int B, K, N;
    const int32_t* labels; const float* sigma2; const float* lambda; const float* uniforms;
    const float *coef_x, *coef_eps;
    int32_t *cur_a, *nv, *t_step, *t_pack, *lab_pack, *t_draft, *act_draft, *active;
    float *sigma2_bk, *lam_bk, *u_bk, *cx_bk, *ce_bk;
};

// From the cursors a[b] (next transition, 1-based) derive this round's index tables.
__global__ void round_setup_kernel(RoundArgs r) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= r.B) return;
    const int a = r.cur_a[b], N = r.N, K = r.K;
    const bool act = a <= N;
    r.active[b] = act;
    auto clampi = [&](int s) { return s < 0 ? 0 : (s >= N ? N - 1 : s); };
    r.t_step[b] = clampi(N - a);
    int last = a + K < N - 1 ? a + K : N - 1;        // b = min(N-1, a+K): the sigma = 0 transition is never drafted
    int nv = act && last > a ? last - a : 0;
    r.nv[b] = nv;
    for (int i = 0; i < K; ++i) {
        const int t = a + i + 1;                     // transition drafted at step i+1 / verified as draft i
        const int s = clampi(N - t);
        r.t_pack[b * K + i] = s;
        r.lab_pack[b * K + i] = r.labels[b];
        r.t_draft[i * r.B + b] = s;
        r.act_draft[i * r.B + b] = i < nv;
        const bool in = i < nv;
        r.sigma2_bk[b * K + i] = in ? r.sigma2[s] : 1.f;
        r.lam_bk[b * K + i] = (in && r.lambda) ? r.lambda[t - 1] : 1.f;
        r.u_bk[b * K + i] = in ? r.uniforms[(long long)b * N + (t - 1)] : 0.f;
        r.cx_bk[b * K + i] = r.coef_x[s];
        r.ce_bk[b * K + i] = r.coef_eps[s];
    }
}

// x_a = m_a + sigma_a z for active samples (the target's own step), also seeding the pack buffer
__global__ void target_sample_kernel(int B, int K, int d, int N, const int32_t* cur_a, const int32_t* active,
                                     const int32_t* t_step, const float* sigma2, const float* m_a,
                                     const float* noise_target, float* x_cur, float* pack_in) {
    const long long total = (long long)B * d;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int b = (int)(i / d), e = (int)(i % d);
        if (!active[b]) continue;
        const int a = cur_a[b];
        const float sg = sqrtf(fmaxf(sigma2[t_step[b]], 0.f));
        const float v = m_a[i] + sg * noise_target[((long long)b * N + (a - 1)) * d + e];
        x_cur[i] = v;
        if (K > 0) pack_in[(long long)b * K * d + e] = v;
    }
}

// a <- a + 1 + (finalised drafts): accepted ones plus the reflected one if a rejection occurred
// Also gathers what the host needs after a round into one contiguous record (report[0] = device error word, then the
// B-long arrays active, nv, n_acc, cursor), so that the sampling loop reads it with a single copy.
__global__ void cursor_update_kernel(int B, const int32_t* active, const int32_t* nv, const int32_t* n_acc, int32_t* cur_a,
                                     const uint32_t* err, int32_t* report) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b == 0) report[0] = (int32_t)*err;
    if (b >= B) return;
    const int act = active[b], v = nv[b], na = n_acc[b];
    int a = cur_a[b];
    if (act) {
        int fin = 0;
        if (v > 0) fin = na < 0 ? 0 : (na + 1 < v ? na + 1 : v);
        a += 1 + fin;
        cur_a[b] = a;
    }
    report[4 + b] = act; report[4 + B + b] = v; report[4 + 2 * B + b] = na; report[4 + 3 * B + b] = a;
}

// x_hat_{a+i+1} = m_hat_{a+i+1} + sigma z_D (drafting step i).  Written as verifier operand i and, unless it is
// the last draft, as packed input i+1.  Samples that draft fewer than i+1 steps compute on clamped indices;
// their slots are never examined (n_valid masks them).
__global__ void draft_sample_kernel(int B, int K, int d, int N, int i, const int32_t* cur_a, const int32_t* t_draft,
                                    const float* sigma2, const float* m_draft, const float* noise_draft,
                                    float* x_draft, float* pack_in) {
    const long long total = (long long)B * d;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (long long)gridDim.x * blockDim.x) {
        const int b = (int)(idx / d), e = (int)(idx % d);
        int t = cur_a[b] + i + 1;
        t = t > N ? N : t;
        const float sg = sqrtf(fmaxf(sigma2[t_draft[b]], 0.f));
        const long long slot = ((long long)b * K + i) * d + e;
        const float v = m_draft[slot] + sg * noise_draft[((long long)b * N + (t - 1)) * d + e];
        x_draft[slot] = v;
        if (i + 1 < K) pack_in[slot + d] = v;
    }
}

__global__ void fill_i32_kernel(int n, int32_t v, int32_t* p) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) p[i] = v;
}

}  // namespace

// ------------------------------------------------------------------------------------------------
extern "C" int free_create(const free_model_desc* t, const free_drafter_desc* d, free_ctx** out) {
    if (!t || !out) return FREE_ERR_ARG;
    *out = nullptr;
    if (t->dtype != FREE_FP32 && t->dtype != FREE_BF16) return FREE_ERR_ARG;
    if (t->C < 1 || t->H < 1 || t->W < 1 || t->patch < 1 || t->D < 1 || t->depth < 1 || t->heads < 1 ||
        t->n_classes < 1 || t->c_out < t->C || t->freq_dim < 2 || t->mlp_ratio < 1) return FREE_ERR_SHAPE;
    if (t->H % t->patch || t->W % t->patch || t->D % t->heads || t->freq_dim % 2) return FREE_ERR_SHAPE;
    const void* ptrs[] = {t->t_w1, t->t_b1, t->t_w2, t->t_b2, t->y_emb, t->pe_w, t->pe_b, t->pos,
                          t->blocks.ada_w, t->blocks.ada_b, t->blocks.qkv_w, t->blocks.qkv_b, t->blocks.proj_w, t->blocks.proj_b,
                          t->blocks.fc1_w, t->blocks.fc1_b, t->blocks.fc2_w, t->blocks.fc2_b,
                          t->fada_w, t->fada_b, t->fin_w, t->fin_b};
    for (const void* p : ptrs) { if (!p) return FREE_ERR_ARG; if (!free_aligned16(p)) return FREE_ERR_ALIGN; }
    if (d) {
        if (d->n_blocks < 1) return FREE_ERR_SHAPE;
        const void* dp[] = {d->fc_w, d->fc_b, d->blocks.ada_w, d->blocks.ada_b, d->blocks.qkv_w, d->blocks.qkv_b,
                            d->blocks.proj_w, d->blocks.proj_b, d->blocks.fc1_w, d->blocks.fc1_b, d->blocks.fc2_w, d->blocks.fc2_b,
                            d->fada_w, d->fada_b, d->fin_w, d->fin_b};
        for (const void* p : dp) { if (!p) return FREE_ERR_ARG; if (!free_aligned16(p)) return FREE_ERR_ALIGN; }
    }
    free_ctx* c = new (std::nothrow) free_ctx;
    if (!c) return FREE_ERR_ARG;
    c->m = *t;
    c->has_drafter = d != nullptr;
    if (d) c->dr = *d; else memset(&c->dr, 0, sizeof(c->dr));
    c->n_tok = (t->H / t->patch) * (t->W / t->patch);
    c->d_latent = t->C * t->H * t->W;
    c->patch_dim = t->C * t->patch * t->patch;
    c->out_dim = t->c_out * t->patch * t->patch;
    c->d_head = t->D / t->heads;
    c->F = t->mlp_ratio * t->D;
    c->tc_attn = false;
    c->attn2 = false;
    c->d_pad = c->d_head;
    if (t->dtype == FREE_BF16) {
        // tensor-core tiles need K % 64 == 0 and N % 16 == 0 for every GEMM of the stack
        if (!linear_bf16_supported(t->D, t->freq_dim) || !linear_bf16_supported(3 * t->D, t->D) ||
            !linear_bf16_supported(c->F, t->D) || !linear_bf16_supported(t->D, c->F)) { delete c; return FREE_ERR_UNSUPPORTED; }
        c->tc_attn = attention_tc_supported(c->n_tok, c->d_head);
        if (c->tc_attn) c->d_pad = attention_tc_dpad(c->d_head);
        c->attn2 = c->tc_attn && attention_tc2_supported(c->n_tok, c->d_head) && t->D % 128 == 0;
    }
    *out = c;
    return FREE_OK;
}

extern "C" int free_destroy(free_ctx* c) {
    if (!c) return FREE_ERR_ARG;
    delete c;
    return FREE_OK;
}

extern "C" size_t free_workspace_bytes(const free_ctx* c, int max_states) {
    if (!c || max_states < 1) return 0;
    return plan(c, max_states, nullptr).total;
}

extern "C" int dit_verify_pass(free_ctx* c, int n_states, const float* x_in, const int32_t* t_idx, const int32_t* labels,
                               float cfg_scale, const free_schedule* sch, float* mean_out, float* eps_out, void* feat_out,
                               void* ws, size_t ws_bytes, void* stream) {
    if (!x_in || !t_idx || !labels || !mean_out) return FREE_ERR_ARG;
    FREE_TRY(check_common(c, n_states, sch, ws, ws_bytes));
    if (!free_aligned16(x_in) || !free_aligned16(mean_out) || !free_aligned16(eps_out) || !free_aligned16(feat_out)) return FREE_ERR_ALIGN;
    const Workspace w = plan(c, n_states, ws);
    FREE_CUDA_TRY(cudaMemsetAsync(w.err, 0, 4, reinterpret_cast<cudaStream_t>(stream)));
    PassIO io{};
    io.x_in = x_in; io.x_stride = c->d_latent; io.t_idx = t_idx; io.labels = labels;
    io.mean_out = mean_out; io.mean_stride = c->d_latent; io.eps_out = eps_out; io.feat_out = feat_out;
    return target_pass(c, w, n_states, cfg_scale, sch, io, reinterpret_cast<cudaStream_t>(stream));
}

extern "C" int dit_verify_pass_raw(free_ctx* c, int n_states, const float* x_in, const int32_t* t_idx, const int32_t* labels,
                                   int guidance, const free_schedule* sch, float* eps_out, void* feat_out,
                                   void* ws, size_t ws_bytes, void* stream) {
    if (!x_in || !t_idx || !labels || !eps_out) return FREE_ERR_ARG;
    FREE_TRY(check_common(c, n_states, sch, ws, ws_bytes));
    if (!free_aligned16(x_in) || !free_aligned16(eps_out) || !free_aligned16(feat_out)) return FREE_ERR_ALIGN;
    const Workspace w = plan(c, n_states, ws);
    FREE_CUDA_TRY(cudaMemsetAsync(w.err, 0, 4, reinterpret_cast<cudaStream_t>(stream)));
    PassIO io{};
    io.x_in = x_in; io.x_stride = c->d_latent; io.t_idx = t_idx; io.labels = labels;
    io.feat_out = feat_out; io.head_raw = eps_out;
    return target_pass(c, w, n_states, guidance ? 2.f : 0.f, sch, io, reinterpret_cast<cudaStream_t>(stream));
}

extern "C" int draft_step(free_ctx* c, int n_states, const float* x_prev, const void* f_prev, const int32_t* t_idx,
                          const int32_t* labels, float cfg_scale, const free_schedule* sch, const float* noise,
                          float* m_hat, float* x_hat, void* f_next, void* ws, size_t ws_bytes, void* stream) {
    if (!x_prev || !f_prev || !t_idx || !labels || !noise || !m_hat || !x_hat || !f_next) return FREE_ERR_ARG;
    FREE_TRY(check_common(c, n_states, sch, ws, ws_bytes));
    if (!c->has_drafter || f_prev == f_next) return FREE_ERR_ARG;
    if (!free_aligned16(x_prev) || !free_aligned16(f_prev) || !free_aligned16(noise) || !free_aligned16(m_hat) ||
        !free_aligned16(x_hat) || !free_aligned16(f_next)) return FREE_ERR_ALIGN;
    const Workspace w = plan(c, n_states, ws);
    FREE_CUDA_TRY(cudaMemsetAsync(w.err, 0, 4, reinterpret_cast<cudaStream_t>(stream)));
    PassIO io{};
    io.x_in = x_prev; io.x_stride = c->d_latent; io.t_idx = t_idx; io.labels = labels;
    io.mean_out = m_hat; io.mean_stride = c->d_latent; io.feat_out = f_next;
    io.noise = noise; io.noise_stride = c->d_latent; io.sample_out = x_hat; io.sample_stride = c->d_latent;
    return drafter_pass(c, w, n_states, cfg_scale, sch, io, f_prev, reinterpret_cast<cudaStream_t>(stream));
}

namespace {

struct RoundIO {
    int B, K;
    const int32_t* labels;
    const free_schedule* sch;
    float cfg;
    const float* lambda;
    const float *noise_target, *noise_draft, *uniforms;
};

// One round of Algorithm 1 for every sample whose cursor has not passed N, in three parts: (front) index tables, target
// step, K drafter steps; (pass) the packed target pass over a range of the B*K packed states; (back) verification and
// cursor update.  State (w.x_cur, w.cur_a) lives in the workspace.  A single GPU runs the pass over all states; with the
// packed states partitioned over several GPUs each runs front and back in full and the pass on its share.
int round_front(const free_ctx* c, const Workspace& w, const RoundIO& r, cudaStream_t s) {
    const int B = r.B, K = r.K, N = r.sch->N, d = c->d_latent;
    const free_schedule* sch = r.sch;
    RoundArgs ra{B, K, N, r.labels, sch->sigma2, r.lambda, r.uniforms, sch->coef_x, sch->coef_eps, w.cur_a, w.nv, w.t_step,
                 w.t_pack, w.lab_pack, w.t_draft, w.act_draft, w.active, w.sigma2_bk, w.lam_bk, w.u_bk, w.cx_bk, w.ce_bk};
    const unsigned egrid = (unsigned)(((long long)B * d + 255) / 256 > 148 * 8 ? 148 * 8 : ((long long)B * d + 255) / 256);
    { Scope p(c, PC_CTRL, 0, s);
      round_setup_kernel<<<(B + 127) / 128, 128, 0, s>>>(ra);
      FREE_TRY(free_check_launch()); }
    // (1) target step on the current state of every sample
    PassIO io{};
    io.x_in = w.x_cur; io.x_stride = d; io.t_idx = w.t_step; io.labels = r.labels;
    io.mean_out = w.m_a; io.mean_stride = d; io.feat_out = K > 0 ? w.feat0 : nullptr;
    FREE_TRY(target_pass(c, w, B, r.cfg, sch, io, s));
    { Scope p(c, PC_CTRL, 0, s);
      target_sample_kernel<<<egrid, 256, 0, s>>>(B, K, d, N, w.cur_a, w.active, w.t_step, sch->sigma2, w.m_a,
                                                  r.noise_target, w.x_cur, w.pack_in);
      FREE_TRY(free_check_launch()); }
    if (K > 0) {
        // (2) K drafter steps, each from the previous draft and feature
        void* f_prev = w.feat0; void* f_next = w.feat1;
        for (int i = 0; i < K; ++i) {
            PassIO di{};
            di.x_in = w.pack_in + (size_t)i * d; di.x_stride = (long long)K * d;         // x_hat_{a+i}
            di.t_idx = w.t_draft + (size_t)i * B; di.labels = r.labels;
            di.mean_out = w.m_draft + (size_t)i * d; di.mean_stride = (long long)K * d;
            di.feat_out = f_next;
            FREE_TRY(drafter_pass(c, w, B, r.cfg, sch, di, f_prev, s));
            { Scope p(c, PC_CTRL, 0, s);
              draft_sample_kernel<<<egrid, 256, 0, s>>>(B, K, d, N, i, w.cur_a, w.t_draft + (size_t)i * B, sch->sigma2,
                                                         w.m_draft, r.noise_draft, w.x_draft, w.pack_in);
              FREE_TRY(free_check_launch()); }
            void* tmp = f_prev; f_prev = f_next; f_next = tmp;
        }
    }
    return FREE_OK;
}

// (3) the packed target pass over states [lo, hi) of (x_a, x_hat_{a+1..a+K-1}) of every sample (state index b*K + k),
//     stopped at the head's output; eps_all is the [B*K, G, d] tensor of all states' noise predictions
int round_pass(const free_ctx* c, const Workspace& w, const RoundIO& r, int lo, int hi, float* eps_all, cudaStream_t s) {
    if (r.K < 1 || hi <= lo) return FREE_OK;
    const int d = c->d_latent, G = (r.cfg > 0.f && r.cfg != 1.f) ? 2 : 1;
    PassIO pi{};
    pi.x_in = w.pack_in + (size_t)lo * d; pi.x_stride = d; pi.t_idx = w.t_pack + lo; pi.labels = w.lab_pack + lo;
    pi.head_raw = eps_all + (size_t)lo * G * d;
    return target_pass(c, w, hi - lo, r.cfg, r.sch, pi, s);
}

// (4) guidance, the means m_{a+1..a+K} and the sequential verification with the first-rejection break in one kernel; the
//     finalised state replaces x_cur; then the cursors move
int round_back(const free_ctx* c, const Workspace& w, const RoundIO& r, const float* eps_all, cudaStream_t s) {
    const int B = r.B, K = r.K, d = c->d_latent;
    if (K > 0) {
        const int G = (r.cfg > 0.f && r.cfg != 1.f) ? 2 : 1;
        Scope p(c, PC_VERIFY, (double)B * ((2.0 + G) * K + 2) * d * 4, s);
        FREE_TRY(spec_verify_fused_launch(B, K, d, G, r.cfg, eps_all, w.pack_in, (long long)K * d,
                                          w.m_draft, w.x_draft, w.cx_bk, w.ce_bk, w.sigma2_bk, w.lam_bk, w.u_bk, w.nv, 0,
                                          w.x_cur, w.n_acc, w.ell_bk, w.d2_bk, nullptr, s));
    }
    Scope p(c, PC_CTRL, 0, s);
    cursor_update_kernel<<<(B + 127) / 128, 128, 0, s>>>(B, w.active, w.nv, w.n_acc, w.cur_a, w.err, w.report);
    return free_check_launch();
}

int one_round(const free_ctx* c, const Workspace& w, const RoundIO& r, cudaStream_t s) {
    FREE_TRY(round_front(c, w, r, s));
    FREE_TRY(round_pass(c, w, r, 0, r.B * r.K, w.head_out, s));
    return round_back(c, w, r, w.head_out, s);
}

int check_round_args(const free_ctx* c, int B, int K, const free_schedule* sch, void* ws, size_t ws_bytes,
                     const float* noise_draft, const float* uniforms) {
    if (B < 1) return FREE_ERR_SHAPE;
    if (K < 0 || K > FREE_MAX_K) return FREE_ERR_SHAPE;
    if (K > 0 && (!noise_draft || !uniforms)) return FREE_ERR_ARG;
    FREE_TRY(check_common(c, B * (K > 0 ? K : 1), sch, ws, ws_bytes));
    if (K > 0 && !c->has_drafter) return FREE_ERR_ARG;
    return FREE_OK;
}

}  // namespace

extern "C" int free_spec_round(free_ctx* c, int B, const float* x_cur, const int32_t* cursor, const int32_t* labels,
                               const free_schedule* sch, const free_spec_params* prm,
                               const float* noise_target, const float* noise_draft, const float* uniforms,
                               float* x_next, int32_t* cursor_next, int32_t* n_accept,
                               void* ws, size_t ws_bytes, void* stream) {
    if (!x_cur || !cursor || !labels || !prm || !noise_target || !x_next || !cursor_next) return FREE_ERR_ARG;
    FREE_TRY(check_round_args(c, B, prm->K, sch, ws, ws_bytes, noise_draft, uniforms));
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const int K = prm->K, d = c->d_latent;
    const Workspace w = plan(c, B * (K > 0 ? K : 1), ws);
    FREE_CUDA_TRY(cudaMemsetAsync(w.err, 0, 4, s));
    FREE_CUDA_TRY(cudaMemcpyAsync(w.x_cur, x_cur, (size_t)B * d * 4, cudaMemcpyDeviceToDevice, s));
    FREE_CUDA_TRY(cudaMemcpyAsync(w.cur_a, cursor, (size_t)B * 4, cudaMemcpyDeviceToDevice, s));
    RoundIO r{B, K, labels, sch, prm->cfg_scale, prm->lambda, noise_target, noise_draft, uniforms};
    FREE_TRY(one_round(c, w, r, s));
    FREE_CUDA_TRY(cudaMemcpyAsync(x_next, w.x_cur, (size_t)B * d * 4, cudaMemcpyDeviceToDevice, s));
    FREE_CUDA_TRY(cudaMemcpyAsync(cursor_next, w.cur_a, (size_t)B * 4, cudaMemcpyDeviceToDevice, s));
    if (n_accept && K > 0) FREE_CUDA_TRY(cudaMemcpyAsync(n_accept, w.n_acc, (size_t)B * 4, cudaMemcpyDeviceToDevice, s));
    return FREE_OK;
}

extern "C" int free_split_range(int n_states, int world, int rank, int* lo, int* hi) {
    if (!lo || !hi) return FREE_ERR_ARG;
    if (n_states < 0 || world < 1 || rank < 0 || rank >= world || n_states % world) return FREE_ERR_SHAPE;
    const int per = n_states / world;
    *lo = rank * per; *hi = *lo + per;
    return FREE_OK;
}

extern "C" int free_spec_round_begin(free_ctx* c, int B, const float* x_cur, const int32_t* cursor, const int32_t* labels,
                                     const free_schedule* sch, const free_spec_params* prm,
                                     const float* noise_target, const float* noise_draft, const float* uniforms,
                                     int rank, int world, float* eps_all, void* ws, size_t ws_bytes, void* stream) {
    if (!x_cur || !cursor || !labels || !prm || !noise_target || !eps_all) return FREE_ERR_ARG;
    if (prm->K < 1) return FREE_ERR_SHAPE;
    FREE_TRY(check_round_args(c, B, prm->K, sch, ws, ws_bytes, noise_draft, uniforms));
    if (!free_aligned16(eps_all)) return FREE_ERR_ALIGN;
    int lo = 0, hi = 0;
    FREE_TRY(free_split_range(B * prm->K, world, rank, &lo, &hi));
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const int d = c->d_latent;
    const Workspace w = plan(c, B * prm->K, ws);
    FREE_CUDA_TRY(cudaMemsetAsync(w.err, 0, 4, s));
    FREE_CUDA_TRY(cudaMemcpyAsync(w.x_cur, x_cur, (size_t)B * d * 4, cudaMemcpyDeviceToDevice, s));
    FREE_CUDA_TRY(cudaMemcpyAsync(w.cur_a, cursor, (size_t)B * 4, cudaMemcpyDeviceToDevice, s));
    RoundIO r{B, prm->K, labels, sch, prm->cfg_scale, prm->lambda, noise_target, noise_draft, uniforms};
    FREE_TRY(round_front(c, w, r, s));
    return round_pass(c, w, r, lo, hi, eps_all, s);
}

extern "C" int free_spec_round_finish(free_ctx* c, int B, const int32_t* labels, const free_schedule* sch, const free_spec_params* prm,
                                      const float* noise_target, const float* noise_draft, const float* uniforms,
                                      const float* eps_all, float* x_next, int32_t* cursor_next, int32_t* n_accept,
                                      void* ws, size_t ws_bytes, void* stream) {
    if (!labels || !prm || !eps_all || !x_next || !cursor_next) return FREE_ERR_ARG;
    if (prm->K < 1) return FREE_ERR_SHAPE;
    FREE_TRY(check_round_args(c, B, prm->K, sch, ws, ws_bytes, noise_draft, uniforms));
    if (!free_aligned16(eps_all) || !free_aligned16(x_next)) return FREE_ERR_ALIGN;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const int d = c->d_latent;
    const Workspace w = plan(c, B * prm->K, ws);
    RoundIO r{B, prm->K, labels, sch, prm->cfg_scale, prm->lambda, noise_target, noise_draft, uniforms};
    FREE_TRY(round_back(c, w, r, eps_all, s));
    FREE_CUDA_TRY(cudaMemcpyAsync(x_next, w.x_cur, (size_t)B * d * 4, cudaMemcpyDeviceToDevice, s));
    FREE_CUDA_TRY(cudaMemcpyAsync(cursor_next, w.cur_a, (size_t)B * 4, cudaMemcpyDeviceToDevice, s));
    if (n_accept) FREE_CUDA_TRY(cudaMemcpyAsync(n_accept, w.n_acc, (size_t)B * 4, cudaMemcpyDeviceToDevice, s));
    return FREE_OK;
}

namespace {

// Per-transition sums of what the verifier saw (Sec. 3.4: prediction deviation and acceptance probability).
struct Diag { double* dev_sum; double* acc_sum; int64_t* count; };

// Algorithm 1 for B samples: rounds until every cursor has passed N.  Host side of a round: cursors (loop control),
// statistics and, when asked, the per-transition records of every examined draft.
int run_trajectory(free_ctx* c, int B, const float* x0, const int32_t* labels, const free_schedule* sch,
                   const free_spec_params* prm, const float* noise_target, const float* noise_draft,
                   const float* uniforms, float* x_final, free_traj_stats* stats, const Diag* diag,
                   void* ws, cudaStream_t s) {
    const int K = prm->K;
    const Workspace w = plan(c, B * (K > 0 ? K : 1), ws);
    const int N = sch->N, d = c->d_latent;
    if (stats) memset(stats, 0, sizeof(*stats));

    FREE_CUDA_TRY(cudaMemsetAsync(w.err, 0, 4, s));
    FREE_CUDA_TRY(cudaMemcpyAsync(w.x_cur, x0, (size_t)B * d * 4, cudaMemcpyDeviceToDevice, s));
    fill_i32_kernel<<<(B + 127) / 128, 128, 0, s>>>(B, 1, w.cur_a);
    FREE_TRY(free_check_launch());
    std::vector<int32_t> h_a(B, 1), h_prev(B, 1), h_nv(B), h_acc(B), h_act(B);
    // one pinned record per round instead of five pageable copies (each of which the driver stages and waits for)
    struct Pinned {
        int32_t* p = nullptr;
        ~Pinned() { if (p) cudaFreeHost(p); }
    } rep;
    const size_t rep_words = 4 + 4 * (size_t)B;
    FREE_CUDA_TRY(cudaHostAlloc((void**)&rep.p, rep_words * 4, cudaHostAllocDefault));
    std::vector<float> h_ell, h_d2, h_ce(N);
    if (diag && K > 0) {
        h_ell.resize((size_t)B * K); h_d2.resize((size_t)B * K);
        FREE_CUDA_TRY(cudaMemcpyAsync(h_ce.data(), sch->coef_eps, (size_t)N * 4, cudaMemcpyDeviceToHost, s));
    }
    RoundIO r{B, K, labels, sch, prm->cfg_scale, prm->lambda, noise_target, noise_draft, uniforms};

    // Every round launches the same kernels with the same arguments (cursors and states live in the workspace), so on
    // request the second round is recorded into a CUDA graph and the later ones are single graph launches.
    struct GraphHolder {
        cudaGraphExec_t exec = nullptr;
        ~GraphHolder() { if (exec) cudaGraphExecDestroy(exec); }
    } gh;
    bool want_graph = prm->use_graph && !c->prof_on;
    for (long long round = 0; round < 2LL * N + 2; ++round) {
        bool any = false;
        for (int b = 0; b < B; ++b) any |= h_a[b] <= N;
        if (!any) break;
        h_prev = h_a;
        if (!gh.exec && want_graph && round == 1) {          // round 0 ran eagerly: one-time function attributes are set
            if (cudaStreamBeginCapture(s, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
                (void)cudaGetLastError();                  // e.g. the legacy default stream cannot be captured: stay eager
                want_graph = false;
            } else {
                cudaGraph_t graph = nullptr;
                const int rc = one_round(c, w, r, s);
                const cudaError_t ce = cudaStreamEndCapture(s, &graph);
                if (rc != FREE_OK || ce != cudaSuccess || !graph) {
                    if (graph) cudaGraphDestroy(graph);
                    (void)cudaGetLastError();
                    return rc != FREE_OK ? rc : FREE_ERR_CUDA;
                }
                const cudaError_t ie = cudaGraphInstantiate(&gh.exec, graph, 0);
                cudaGraphDestroy(graph);
                if (ie != cudaSuccess) { gh.exec = nullptr; (void)cudaGetLastError(); return FREE_ERR_CUDA; }
            }
        }
        if (gh.exec) {
            FREE_CUDA_TRY(cudaGraphLaunch(gh.exec, s));
            if (stats) stats->graph_rounds += 1;
        } else {
            FREE_TRY(one_round(c, w, r, s));
        }
        FREE_CUDA_TRY(cudaMemcpyAsync(rep.p, w.report, rep_words * 4, cudaMemcpyDeviceToHost, s));
        if (diag && K > 0) {
            FREE_CUDA_TRY(cudaMemcpyAsync(h_ell.data(), w.ell_bk, (size_t)B * K * 4, cudaMemcpyDeviceToHost, s));
            FREE_CUDA_TRY(cudaMemcpyAsync(h_d2.data(), w.d2_bk, (size_t)B * K * 4, cudaMemcpyDeviceToHost, s));
        }
        FREE_CUDA_TRY(cudaStreamSynchronize(s));
        FREE_TRY(free_device_error_code((uint32_t)rep.p[0]));
        for (int b = 0; b < B; ++b) {
            h_act[b] = rep.p[4 + b]; h_nv[b] = rep.p[4 + B + b]; h_acc[b] = rep.p[4 + 2 * B + b]; h_a[b] = rep.p[4 + 3 * B + b];
        }
        for (int b = 0; b < B; ++b) {
            if (!h_act[b]) continue;
            if (K > 0 && h_nv[b] > 0 && h_acc[b] < 0) return h_acc[b];
            if (diag && K > 0 && h_nv[b] > 0) {
                // examined drafts: the accepted ones and the rejected one; draft i verifies transition a + i + 1
                const int seen = h_acc[b] < h_nv[b] ? h_acc[b] + 1 : h_nv[b];
                for (int i = 0; i < seen; ++i) {
                    const int t = h_prev[b] + i + 1;
                    const double ell = (double)h_ell[(size_t)b * K + i], d2 = (double)h_d2[(size_t)b * K + i];
                    const double ce = (double)h_ce[N - t];
                    diag->dev_sum[t - 1] += ce != 0.0 ? sqrt(d2) / fabs(ce) : 0.0;
                    diag->acc_sum[t - 1] += ell < 0.0 ? exp(ell) : 1.0;
                    diag->count[t - 1] += 1;
                }
            }
            if (!stats) continue;
            stats->target_calls += 1;
            if (h_nv[b] > 0) {
                stats->target_calls += 1;
                stats->draft_calls += h_nv[b];
                stats->accepted += h_acc[b];
                if (h_acc[b] < h_nv[b]) stats->rejected += 1;
                stats->accept_hist[h_acc[b]] += 1;
            }
        }
        if (stats) stats->rounds += 1;
    }
    if (x_final) FREE_CUDA_TRY(cudaMemcpyAsync(x_final, w.x_cur, (size_t)B * d * 4, cudaMemcpyDeviceToDevice, s));
    FREE_CUDA_TRY(cudaStreamSynchronize(s));
    if (stats && stats->target_calls > 0) stats->parallel_efficiency = (double)B * N / (double)stats->target_calls;
    return FREE_OK;
}

}  // namespace

extern "C" int sample_trajectory(free_ctx* c, int B, const float* x0, const int32_t* labels, const free_schedule* sch,
                                 const free_spec_params* prm, const float* noise_target, const float* noise_draft,
                                 const float* uniforms, float* x_final, free_traj_stats* stats,
                                 void* ws, size_t ws_bytes, void* stream) {
    if (!x0 || !labels || !prm || !noise_target || !x_final) return FREE_ERR_ARG;
    FREE_TRY(check_round_args(c, B, prm->K, sch, ws, ws_bytes, noise_draft, uniforms));
    return run_trajectory(c, B, x0, labels, sch, prm, noise_target, noise_draft, uniforms, x_final, stats, nullptr, ws,
                          reinterpret_cast<cudaStream_t>(stream));
}

extern "C" int free_uncertainty_profile(free_ctx* c, int B, const float* x0, const int32_t* labels, const free_schedule* sch,
                                        const free_spec_params* prm, const float* noise_target, const float* noise_draft,
                                        const float* uniforms, double* eps_delta, double* accept_prob, int64_t* count,
                                        void* ws, size_t ws_bytes, void* stream) {
    if (!x0 || !labels || !prm || !noise_target || !eps_delta || !accept_prob || !count) return FREE_ERR_ARG;
    if (prm->K < 1) return FREE_ERR_SHAPE;
    FREE_TRY(check_round_args(c, B, prm->K, sch, ws, ws_bytes, noise_draft, uniforms));
    const int N = sch->N;
    for (int n = 0; n < N; ++n) { eps_delta[n] = 0.0; accept_prob[n] = 0.0; count[n] = 0; }
    const Diag diag{eps_delta, accept_prob, count};
    FREE_TRY(run_trajectory(c, B, x0, labels, sch, prm, noise_target, noise_draft, uniforms, nullptr, nullptr, &diag, ws,
                            reinterpret_cast<cudaStream_t>(stream)));
    for (int n = 0; n < N; ++n)
        if (count[n] > 0) { eps_delta[n] /= (double)count[n]; accept_prob[n] /= (double)count[n]; }
    return FREE_OK;
}

// ------------------------------------------------------------------------------------------------ profiling
extern "C" int free_profile_begin(free_ctx* c) {
    if (!c) return FREE_ERR_ARG;
    for (ProfRec& r : c->prof) { cudaEventDestroy(r.e0); cudaEventDestroy(r.e1); }
    c->prof.clear();
    c->prof_on = true;
    return FREE_OK;
}

extern "C" int free_profile_end(free_ctx* c, free_prof_entry* out, int max_entries, int* n_entries) {
    if (!c || !out || !n_entries || max_entries < 1) return FREE_ERR_ARG;
    c->prof_on = false;
    double ms[PC_N] = {}, work[PC_N] = {};
    long long cnt[PC_N] = {};
    int rc = FREE_OK;
    for (ProfRec& r : c->prof) {
        float t = 0.f;
        if (cudaEventSynchronize(r.e1) != cudaSuccess || cudaEventElapsedTime(&t, r.e0, r.e1) != cudaSuccess) { (void)cudaGetLastError(); rc = FREE_ERR_CUDA; }
        ms[r.cls] += t; work[r.cls] += r.work; cnt[r.cls] += 1;
        cudaEventDestroy(r.e0); cudaEventDestroy(r.e1);
    }
    c->prof.clear();
    int n = 0;
    for (int k = 0; k < PC_N && n < max_entries; ++k) {
        if (!cnt[k]) continue;
        strncpy(out[n].name, kProfNames[k], sizeof(out[n].name) - 1);
        out[n].name[sizeof(out[n].name) - 1] = 0;
        out[n].launches = cnt[k]; out[n].ms = ms[k]; out[n].work = work[k];
        ++n;
    }
    *n_entries = n;
    return rc;
}
