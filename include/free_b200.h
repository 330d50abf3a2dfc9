/*
 * free_b200 -- C ABI of the packed parallel-verification path of FREE
 * ("Uncertainty-Aware Autoregression for Parallel Diffusion Transformers") for one B200 GPU.
 *
 * Conventions shared by every call
 *   - Return value: 0 (FREE_OK) or a negative FREE_ERR_* code; free_strerror() names it.
 *     No call throws, aborts or prints.
 *   - Pointers marked DEVICE are addresses in the current CUDA device's global memory and must be
 *     16-byte aligned; pointers marked HOST are ordinary host memory.  The caller owns every buffer.
 *     The library allocates no device memory: scratch space is the caller's workspace `ws`, sized by
 *     free_workspace_bytes().  Tensors are dense, row-major, innermost index last.
 *   - Device-side waits are bounded.  If one gives up, the kernels stop early and OR a non-zero code into the
 *     first 4 bytes of the workspace (the "device error word", cleared at the start of every call that takes a
 *     workspace); results are then invalid.  sample_trajectory() returns FREE_ERR_DEVICE_TIMEOUT itself;
 *     for the asynchronous calls the caller reads the word after synchronising.
 *   - `stream` is a cudaStream_t passed as void*.  Work is enqueued on it and the call returns
 *     without waiting, except sample_trajectory(), which synchronises once per round.
 *   - No random numbers are drawn inside: noise and uniforms are inputs, so that a run can be
 *     reproduced by another implementation.
 *   - "sequence" = one DiT forward of one latent state; with classifier-free guidance every state
 *     costs G = 2 sequences (conditional, then unconditional with the null label), else G = 1.
 *   - dtype FREE_FP32: all arithmetic in fp32 on CUDA cores (small models, exactness checks).
 *     dtype FREE_BF16: GEMMs and attention on the tensor cores (tcgen05, bf16 operands, fp32
 *     accumulation); residual stream, LayerNorm statistics, modulation and softmax in fp32.
 */
#ifndef FREE_B200_H
#define FREE_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define FREE_OK                   0
#define FREE_ERR_ARG            (-1)   /* null pointer, negative count, bad enum                     */
#define FREE_ERR_SHAPE          (-2)   /* dimensions inconsistent with the model or with each other  */
#define FREE_ERR_ALIGN          (-3)   /* a DEVICE pointer is not 16-byte aligned                    */
#define FREE_ERR_UNSUPPORTED    (-4)   /* valid request outside what the kernels implement           */
#define FREE_ERR_SIGMA          (-5)   /* a variance was <= 0 or not finite                          */
#define FREE_ERR_WORKSPACE      (-6)   /* workspace missing or smaller than free_workspace_bytes()   */
#define FREE_ERR_CUDA           (-7)   /* a CUDA runtime / driver call failed                        */
#define FREE_ERR_DEVICE_TIMEOUT (-8)   /* a bounded device-side wait gave up (pipeline fault)        */

#define FREE_FP32 0
#define FREE_BF16 1

#define FREE_MAX_K 64                  /* most drafts per sample the verifier accepts */

const char* free_strerror(int code);

/* Weights of `n` stacked transformer blocks.  Matrices are [n, out, in] in the model's dtype
 * (fp32 or bf16), biases are fp32 [n, out].  adaLN rows are ordered
 * (shift1, scale1, gate1, shift2, scale2, gate2), each D wide.  All DEVICE. */
typedef struct free_block_weights {
    const void*  ada_w;  const float* ada_b;    /* [n, 6D, D], [n, 6D] */
    const void*  qkv_w;  const float* qkv_b;    /* [n, 3D, D], [n, 3D]; output split as (3, heads, d_head) */
    const void*  proj_w; const float* proj_b;   /* [n, D, D],  [n, D]  */
    const void*  fc1_w;  const float* fc1_b;    /* [n, rD, D], [n, rD], r = mlp_ratio */
    const void*  fc2_w;  const float* fc2_b;    /* [n, D, rD], [n, D]  */
} free_block_weights;

/* Target DiT (the paper uses DiT-XL/2 as published, Sec. 3.1 / Sec. 4; adaLN-Zero blocks). */
typedef struct free_model_desc {
    int32_t dtype;                       /* FREE_FP32 or FREE_BF16: type of the `void*` matrices and of features */
    int32_t C, H, W, patch;              /* latent channels, height, width; patch size */
    int32_t D, depth, heads;             /* hidden width, blocks, attention heads (D % heads == 0) */
    int32_t n_classes;                   /* label n_classes is the null class */
    int32_t c_out;                       /* output channels of the head (2C with learned variance; first C = noise) */
    int32_t freq_dim, mlp_ratio;         /* sinusoidal timestep features (even), MLP expansion */
    const void*  t_w1;  const float* t_b1;   /* [D, freq_dim], [D]   timestep MLP, layer 1 (then SiLU) */
    const void*  t_w2;  const float* t_b2;   /* [D, D], [D]          timestep MLP, layer 2 */
    const float* y_emb;                      /* [n_classes+1, D]     class embedding table */
    const float* pe_w;  const float* pe_b;   /* [D, C*p*p], [D]      patch embedding, patch vector order (c, row, col) */
    const float* pos;                        /* [n_tok, D]           fixed position table */
    free_block_weights blocks;               /* n = depth */
    const void*  fada_w; const float* fada_b;/* [2D, D], [2D]        final modulation (shift, scale) */
    const float* fin_w;  const float* fin_b; /* [p*p*c_out, D], [..] head; output vector order (row, col, channel) */
} free_model_desc;

/* Drafter (Sec. 3.1): reuses the target's embedding tables; g = W_fc [embed(x) || f] + b_fc, then
 * n_blocks DiT blocks (the paper uses one) and its own modulated head. */
typedef struct free_drafter_desc {
    int32_t n_blocks;
    const void*  fc_w;   const float* fc_b;  /* [D, 2D], [D] */
    free_block_weights blocks;
    const void*  fada_w; const float* fada_b;
    const float* fin_w;  const float* fin_b;
} free_drafter_desc;

/* Reverse-process tables indexed by schedule index s = 0..N-1 (s = N-1 is the noisiest), all DEVICE
 * fp32 [N].  mean = coef_x[s] * x - coef_eps[s] * eps (Eq. ddpm_update, Appendix C);
 * sigma2[s] is the fixed posterior variance (Sec. 4); t_embed_value[s] is fed to the timestep embedder. */
typedef struct free_schedule {
    int32_t N;
    const float* coef_x;
    const float* coef_eps;
    const float* sigma2;
    const float* t_embed_value;
} free_schedule;

/*
 * free_schedule_linear / free_schedule_respaced -- the reverse-process tables of a DDPM noise schedule, in fp64,
 * HOST-only (no CUDA call; any thread).  The caller rounds them to fp32 and uploads them for `free_schedule`.
 *   beta_s linear from beta_first (s = 0) to beta_last (s = N-1); alpha_s = 1 - beta_s; abar_s = prod_{r<=s} alpha_r.
 *   Reverse step of Eq. ddpm_update (Appendix "Variance Setting"):
 *       coef_x[s] = 1 / sqrt(alpha_s),   coef_eps[s] = beta_s / (sqrt(1 - abar_s) sqrt(alpha_s)).
 *   variance_mode selects the fixed variance (the Appendix allows any predefined sigma_t):
 *       FREE_VAR_POSTERIOR  sigma2 = beta~_s = beta_s (1 - abar_{s-1}) / (1 - abar_s), abar_{-1} = 1   (Sec. 4)
 *       FREE_VAR_BETA       sigma2 = beta_s
 *       FREE_VAR_INTERP     sigma2 = beta_s^v beta~_s^(1-v), v = variance_weight in [0, 1]
 *   stochasticity >= 0 replaces the step by one Euler-Maruyama step of the epsilon-family of reverse processes
 *   (Appendix "Stochasticity Hyperparameter", Eq. mean_var_gamma) for the variance-preserving process, with
 *   e = stochasticity:  coef_x = 1 + beta_s / 2,  coef_eps = (1 + e^2)/2 beta_s / sqrt(1 - abar_s),
 *   sigma2 = e^2 beta_s  (variance_mode is then ignored).  Pass a negative value for the DDPM step above.
 *   In every variant sigma2[0] = 0: the last transition adds no noise.
 *   free_schedule_respaced keeps abar of the n_full-step linear schedule at the N evenly spaced indices
 *   round_half_even(i (n_full-1)/(N-1)), recomputes beta from consecutive ratios of abar, and reports those original
 *   indices in t_embed_value (what the timestep embedder sees); free_schedule_linear reports s itself.
 *   coef_x, coef_eps, sigma2, t_embed_value   HOST double [N], written
 * Errors: ARG (null pointer, bad mode), SHAPE (N < 2, n_full < N, betas outside (0, 1), weight outside [0, 1]).
 */
#define FREE_VAR_POSTERIOR 0
#define FREE_VAR_BETA      1
#define FREE_VAR_INTERP    2
int free_schedule_linear(int N, double beta_first, double beta_last,
                         int variance_mode, double variance_weight, double stochasticity,
                         double* coef_x, double* coef_eps, double* sigma2, double* t_embed_value);
int free_schedule_respaced(int N, int n_full, double beta_first, double beta_last,
                           int variance_mode, double variance_weight, double stochasticity,
                           double* coef_x, double* coef_eps, double* sigma2, double* t_embed_value);

typedef struct free_ctx free_ctx;

/* Validate the descriptors, record them (weights are NOT copied: they must outlive the context) and
 * prepare the tensor maps of the weight matrices.  `drafter` may be NULL.  HOST structs. */
int free_create(const free_model_desc* target, const free_drafter_desc* drafter, free_ctx** out);
int free_destroy(free_ctx* ctx);

/* Bytes of workspace needed by dit_verify_pass / draft_step / sample_trajectory when at
 * most `max_states` latent states are processed per call with guidance on (the larger case). */
size_t free_workspace_bytes(const free_ctx* ctx, int max_states);

/*
 * dit_verify_pass -- the packed parallel target pass (Alg. 1, "compute means m_{a+1:b+1} in parallel";
 * Sec. 3.3; Fig. 1a): ONE batched forward over n_states latent states, each with its own schedule
 * index and label, followed by guidance and the reverse-transition mean (Eq. ddpm_update).
 *   x_in      DEVICE fp32 [n_states, C, H, W]
 *   t_idx     DEVICE int32 [n_states], schedule index of the transition each state undergoes
 *   labels    DEVICE int32 [n_states] in 0..n_classes
 *   cfg_scale guidance scale w: eps = eps_u + w (eps_c - eps_u); w <= 0 or w == 1 disables guidance (G = 1)
 *   mean_out  DEVICE fp32 [n_states, C, H, W]          (required)
 *   eps_out   DEVICE fp32 [n_states, C, H, W] or NULL  guided noise prediction
 *   feat_out  DEVICE model dtype [n_states, G, n_tok, D] or NULL: top-block feature (token matrix after
 *             the last block, Sec. 3.1), conditional stream first
 * Errors: ARG, SHAPE (n_states < 1), ALIGN, WORKSPACE, UNSUPPORTED (model dims the kernels cannot tile), CUDA.
 */
int dit_verify_pass(free_ctx* ctx, int n_states,
                         const float* x_in, const int32_t* t_idx, const int32_t* labels, float cfg_scale,
                         const free_schedule* sched,
                         float* mean_out, float* eps_out, void* feat_out,
                         void* ws, size_t ws_bytes, void* stream);

/*
 * dit_verify_pass_raw -- the packed target pass stopped at the network's output: no guidance, no mean.  Feeds
 * spec_verify_fused(), which applies guidance and Eq. ddpm_update itself (Alg. 1, parallel-means line + verification).
 *   guidance  0: one sequence per state (G = 1); non-zero: conditional and unconditional sequences (G = 2)
 *   eps_out   DEVICE fp32 [n_states, G, C, H, W]: the noise prediction of every stream as an image (the head's first C
 *             output channels, un-patchified by the head GEMM's own epilogue; the variance channels are not stored);
 *             conditional stream first
 *   other arguments and errors as for dit_verify_pass.
 */
int dit_verify_pass_raw(free_ctx* ctx, int n_states,
                        const float* x_in, const int32_t* t_idx, const int32_t* labels, int guidance,
                        const free_schedule* sched, float* eps_out, void* feat_out,
                        void* ws, size_t ws_bytes, void* stream);

/*
 * spec_verify -- Algorithm 2 (reflection maximal coupling) applied to K drafts per sample in order,
 * stopping at the first rejection (Alg. 1, verification loop), with the relaxed acceptance of
 * Eq. acc_relax as a mode.  For draft k of sample b, with d = m_hat - m and r = x_hat - m_hat:
 *     ell = -lambda (d.r + |d|^2 / 2) / sigma2      (= lambda (m - m_hat).(x_hat - mid) / sigma2, Eq. qp)
 *     accept iff log u <= min(0, ell)               (u <= min(1, e^ell); u = 0 always accepts)
 * At the first rejected draft j: x_out = m_j + r_j - 2 d_j (d_j.r_j) / |d_j|^2 (x_out = x_hat_j if d_j = 0).
 * If all n_valid drafts are accepted x_out = x_hat of the last one.  Sums are accumulated in fp64.
 *   B, K, d   samples, drafts per sample (1..FREE_MAX_K), elements per state
 *   m_target, m_draft, x_draft  DEVICE fp32 [B, K, d]
 *   sigma2    DEVICE fp32 [B, K]  variance of each transition (> 0)
 *   lambda    DEVICE fp32 [B, K] relaxation scale in [0, 1], or NULL for the strict rule (lambda = 1)
 *   u         DEVICE fp32 [B, K] uniforms in [0, 1]
 *   n_valid   DEVICE int32 [B] number of drafts present (0..K), or NULL for K
 *   x_out     DEVICE fp32 [B, d]; row b is left untouched when n_valid[b] == 0 or on a variance error
 *   n_accept  DEVICE int32 [B]: number of accepted drafts (0..n_valid[b]); if < n_valid[b], draft
 *             n_accept[b] (0-based) was the rejected one.  Set to FREE_ERR_SIGMA if a present draft
 *             of that sample has sigma2 <= 0 or NaN.
 *   logratio_out DEVICE fp32 [B, K] or NULL: ell of every present draft (NaN for absent ones)
 * No workspace.  Errors: ARG, SHAPE (K out of range, d < 1), ALIGN, CUDA.
 */
int spec_verify(int B, int K, int64_t d,
                     const float* m_target, const float* m_draft, const float* x_draft,
                     const float* sigma2, const float* lambda, const float* u, const int32_t* n_valid,
                     float* x_out, int32_t* n_accept, float* logratio_out, void* stream);

/*
 * spec_verify_fused -- spec_verify() fed by the noise predictions of the packed pass instead of by means: per draft k
 * of sample b the kernel forms eps = eps_u + w (eps_c - eps_u) (eps = eps_c when G = 1) and the target mean
 * m_k = coef_x[b,k] x_k - coef_eps[b,k] eps (Eq. ddpm_update) in fp64 registers, and then proceeds exactly as
 * spec_verify.  The packed state x_k is x_first[b] for k = 0 and the previous draft x_draft[b,k-1] after that (Alg. 1:
 * the pass sees the current state and the first K-1 drafts), so the drafts are fetched once for both roles and the
 * [B,K,d] tensor of target means is never written or read.
 *   B, K, d    samples, drafts per sample (1..FREE_MAX_K), elements per state
 *   G, cfg_scale   streams per state (1 or 2) and the guidance scale w (used when G = 2)
 *   eps        DEVICE fp32 [B, K, G, d], layout of dit_verify_pass_raw
 *   x_first    DEVICE fp32 [B, d]
 *   m_draft, x_draft        DEVICE fp32 [B, K, d]
 *   coef_x, coef_eps, sigma2, u   DEVICE fp32 [B, K]; lambda DEVICE fp32 [B, K] or NULL; n_valid DEVICE int32 [B] or NULL
 *   chunk      0: all present drafts are examined (same outputs as spec_verify).  c > 0: early exit -- drafts are
 *              examined c at a time and the rows after the chunk holding the first rejection are never read;
 *              x_out and n_accept are unchanged by this, logratio_out is NaN for drafts that were not examined, and
 *              FREE_ERR_SIGMA is reported only for examined drafts.
 *   x_out, n_accept, logratio_out   as for spec_verify (x_out may not alias x_first or x_draft)
 *   dist2_out  DEVICE fp32 [B, K] or NULL: |m_hat - m|^2 of every examined draft (NaN for the others).  Both means come
 *              from the same packed state, so |eps_pred - eps_ref| = sqrt(dist2) / coef_eps: the prediction deviation
 *              that Sec. 3.4 tracks.
 *   means_out  DEVICE fp32 [B, K, d] or NULL: the target means of the examined drafts, rounded to fp32 (diagnostic)
 * No workspace.  Errors: ARG (null pointer, G not 1 or 2), SHAPE, ALIGN, CUDA.
 */
int spec_verify_fused(int B, int K, int64_t d, int G, float cfg_scale,
                      const float* eps, const float* x_first, const float* m_draft, const float* x_draft,
                      const float* coef_x, const float* coef_eps, const float* sigma2, const float* lambda,
                      const float* u, const int32_t* n_valid, int chunk,
                      float* x_out, int32_t* n_accept, float* logratio_out, float* dist2_out, float* means_out, void* stream);

/*
 * draft_step -- one step of feature-level autoregression (Sec. 3.1; Alg. 1, drafting loop) for
 * n_states states:  (m_hat, f_next) = p(. | x_prev, f_prev);  x_hat = m_hat + sqrt(sigma2[t]) * noise.
 *   x_prev  DEVICE fp32 [n_states, C, H, W]
 *   f_prev  DEVICE model dtype [n_states, G, n_tok, D]
 *   t_idx, labels, cfg_scale, sched: as for dit_verify_pass (t_idx = the transition being predicted)
 *   noise   DEVICE fp32 [n_states, C, H, W] standard normal draws
 *   m_hat, x_hat  DEVICE fp32 [n_states, C, H, W]
 *   f_next  DEVICE model dtype [n_states, G, n_tok, D] (may not alias f_prev)
 * Errors: as dit_verify_pass, plus ARG if the context has no drafter.
 */
int draft_step(free_ctx* ctx, int n_states,
                    const float* x_prev, const void* f_prev,
                    const int32_t* t_idx, const int32_t* labels, float cfg_scale,
                    const free_schedule* sched, const float* noise,
                    float* m_hat, float* x_hat, void* f_next,
                    void* ws, size_t ws_bytes, void* stream);

typedef struct free_spec_params {
    int32_t K;                 /* drafts per round (0 = plain sequential sampler) */
    float   cfg_scale;
    const float* lambda;       /* DEVICE fp32 [N] relaxation table indexed by transition n-1 (n = 1 first), or NULL = strict */
    int32_t use_graph;         /* sample_trajectory / free_uncertainty_profile only.  Non-zero: the second round is recorded
                                  by stream capture into a CUDA graph and every later round is one graph launch (the rounds
                                  of a trajectory launch the same kernels with the same arguments; what changes lives in the
                                  workspace).  Removes the launch overhead that shows at small batches (4% per round at
                                  B = 1 on XL/2 512^2).  The graph and its executable are driver objects created and
                                  destroyed inside the call; `stream` must not be capturing already.  Ignored while
                                  free_profile_begin() is active and on streams that cannot be captured (the legacy
                                  default stream): the rounds are then launched one kernel at a time as usual.  free_spec_round() ignores the field: it can itself be
                                  captured by the caller once it has run eagerly once. */
} free_spec_params;

typedef struct free_traj_stats {     /* HOST, filled on return */
    int64_t rounds;                  /* batch rounds executed */
    int64_t target_calls;            /* target invocations summed over samples (single steps + packed passes) */
    int64_t draft_calls;             /* drafter steps summed over samples */
    int64_t accepted, rejected;      /* drafts accepted / rejected, summed over samples */
    int64_t accept_hist[FREE_MAX_K + 1];   /* rounds that accepted exactly i drafts */
    double  parallel_efficiency;     /* B * N / target_calls (Sec. 4, metric 1) */
    int64_t graph_rounds;            /* rounds launched as a CUDA graph (0 unless params->use_graph took effect) */
} free_traj_stats;

/*
 * sample_trajectory -- Algorithm 1 for B samples with per-sample cursors.  N = sched->N transitions;
 * transition n = 1..N uses schedule index N - n.  Each round: target step on the current state, K
 * drafter steps, one packed target pass over (state, first K-1 drafts), sequential verification;
 * the cursor moves past the last finalised state.  The final transition (sigma = 0) is never drafted.
 *   x0            DEVICE fp32 [B, C, H, W]   initial latents ~ N(0, I)
 *   labels        DEVICE int32 [B]
 *   noise_target  DEVICE fp32 [B, N, C*H*W]  noise of transition n when taken by the target
 *   noise_draft   DEVICE fp32 [B, N, C*H*W]  noise of transition n when proposed by the drafter
 *   uniforms      DEVICE fp32 [B, N]         acceptance uniform of transition n
 *   x_final       DEVICE fp32 [B, C, H, W]
 *   stats         HOST, may be NULL
 * Blocks until done.  Errors: as above; SIGMA if a drafted transition has sigma2 <= 0.
 */
int sample_trajectory(free_ctx* ctx, int B,
                           const float* x0, const int32_t* labels,
                           const free_schedule* sched, const free_spec_params* params,
                           const float* noise_target, const float* noise_draft, const float* uniforms,
                           float* x_final, free_traj_stats* stats,
                           void* ws, size_t ws_bytes, void* stream);

/*
 * free_uncertainty_profile -- the offline run of Sec. 3.4: Algorithm 1 (as sample_trajectory, strict or with the given
 * lambda) with the context's drafter proposing and the target verifying, recording for every EXAMINED draft (the
 * accepted ones and the rejected one of each round) the prediction deviation |eps_pred - eps_ref|_2 and the acceptance
 * probability min(1, e^ell), averaged per transition.  Both noise predictions refer to the same packed state, so the
 * deviation is |m_hat - m| / coef_eps, taken from the verifier's own sums.  (The paper runs the DiT against itself; a
 * DiT has no feature input, so here the proposer is whatever drafter the context holds.)
 *   eps_delta, accept_prob   HOST double [N], index n-1 for transition n; 0 where count is 0
 *   count                    HOST int64 [N]: examined drafts per transition (transition 1 and the last are never drafted)
 *   params->K >= 1; other arguments as for sample_trajectory.  Blocks until done.
 */
int free_uncertainty_profile(free_ctx* ctx, int B, const float* x0, const int32_t* labels,
                             const free_schedule* sched, const free_spec_params* params,
                             const float* noise_target, const float* noise_draft, const float* uniforms,
                             double* eps_delta, double* accept_prob, int64_t* count,
                             void* ws, size_t ws_bytes, void* stream);

/*
 * free_fit_lambda_profile -- relaxation table lambda_n from measured deviations (Sec. 3.4: a smooth, monotonically
 * increasing curve fitted to eps_delta, inverted and rescaled to [0, 1]).  Host-only.  Steps: transitions without a
 * measurement (count == 0, NaN or negative) take the nearest measured value; weighted least-squares non-decreasing fit
 * (pool adjacent violators, weights = count, or 1 when count is NULL); centred moving average over 2*window+1 points
 * with the ends held (keeps the curve non-decreasing); lambda_n = g_1 / g_n, which is 1 at the first transition,
 * non-increasing, in (0, 1], and makes lambda_n * g_n constant (a uniform scaled discrepancy).  g_n = 0 gives 1.
 *   eps_delta HOST double [N]; count HOST int64 [N] or NULL; lambda_out HOST fp32 [N] (the table of free_spec_params)
 * Errors: ARG, SHAPE (N < 1, window < 0, nothing measured).
 */
int free_fit_lambda_profile(const double* eps_delta, const int64_t* count, int N, int window, float* lambda_out);

/*
 * spec_round -- the body of Algorithm 1's loop, once: for every sample b whose cursor[b] <= N (cursor = index of
 * the next transition, 1-based), target step on x_cur[b], K drafter steps, packed target pass, verification;
 * x_next[b] is the last finalised state and cursor_next[b] points past it.  sample_trajectory is this call
 * repeated until every cursor exceeds N.  The packed pass ends at the noise predictions and spec_verify_fused() does the rest.
 * Asynchronous.  Arguments as for sample_trajectory;
 *   x_cur, x_next DEVICE fp32 [B, C, H, W] (may alias); cursor, cursor_next DEVICE int32 [B] (may alias);
 *   n_accept DEVICE int32 [B] or NULL: drafts accepted this round (undefined for samples that drafted nothing).
 */
int free_spec_round(free_ctx* ctx, int B, const float* x_cur, const int32_t* cursor, const int32_t* labels,
                    const free_schedule* sched, const free_spec_params* params,
                    const float* noise_target, const float* noise_draft, const float* uniforms,
                    float* x_next, int32_t* cursor_next, int32_t* n_accept,
                    void* ws, size_t ws_bytes, void* stream);

/*
 * free_spec_round_begin / free_spec_round_finish -- one round of Algorithm 1 with the packed target pass partitioned over
 * `world` GPUs, the deployment the paper measures (Sec. 4, wall-clock protocol: the drafts of a round are verified on
 * parallel GPUs, one draft per GPU when the speculation length equals the number of GPUs).  Every rank holds the same
 * weights, inputs, noise and uniforms and calls both functions with the same arguments except `rank`:
 *   begin   target step on the current states and the K drafter steps (replicated: they are the sequential part of a
 *           round), then the packed target pass over THIS RANK'S share of the B*K packed states (state index b*K + k;
 *           rank r owns the contiguous range given by free_split_range); their noise predictions are written into
 *           eps_all at the states' own positions
 *   (caller) all-gather eps_all over the ranks, in place: every rank contributes the slice it wrote.  The library makes
 *           no collective call itself; the exchange is the caller's (NCCL all-gather into local memory).  No kernel of
 *           the library reads another GPU's memory.
 *   finish  guidance, means, verification and cursor update on the gathered predictions, replicated on every rank: all
 *           ranks take the same decisions from the same bytes, so nothing has to be sent back.
 * With world == 1 the pair is free_spec_round() in two halves (bit-identical results).  Between the two calls the round's
 * state lives in the workspace: the same `ws` must be passed and nothing else may use it.
 *   rank, world   0 <= rank < world; B*K must be a multiple of world (FREE_ERR_SHAPE otherwise)
 *   eps_all       DEVICE fp32 [B*K, G, C, H, W] (layout of dit_verify_pass_raw), caller-owned
 *   other arguments as for free_spec_round(); params->K >= 1.  Both calls are asynchronous.
 * free_split_range: HOST-only; the states [lo, hi) that `rank` owns.
 */
int free_split_range(int n_states, int world, int rank, int* lo, int* hi);
int free_spec_round_begin(free_ctx* ctx, int B, const float* x_cur, const int32_t* cursor, const int32_t* labels,
                          const free_schedule* sched, const free_spec_params* params,
                          const float* noise_target, const float* noise_draft, const float* uniforms,
                          int rank, int world, float* eps_all, void* ws, size_t ws_bytes, void* stream);
int free_spec_round_finish(free_ctx* ctx, int B, const int32_t* labels, const free_schedule* sched, const free_spec_params* params,
                           const float* noise_target, const float* noise_draft, const float* uniforms,
                           const float* eps_all, float* x_next, int32_t* cursor_next, int32_t* n_accept,
                           void* ws, size_t ws_bytes, void* stream);

/*
 * Per-kernel timing (measurement aid; the paper has no counterpart).  Between free_profile_begin() and
 * free_profile_end() every kernel launched by the context's passes is bracketed by CUDA events on the caller's
 * stream.  free_profile_end() waits for them and returns one entry per kernel class: launches, summed device time
 * and summed algorithmic work (FLOPs for linear layers and attention, bytes for the bandwidth-bound kernels).
 * `out` is HOST memory with room for max_entries entries.
 */
typedef struct free_prof_entry {
    char    name[48];
    int64_t launches;
    double  ms;
    double  work;
} free_prof_entry;
int free_profile_begin(free_ctx* ctx);
int free_profile_end(free_ctx* ctx, free_prof_entry* out, int max_entries, int* n_entries);

/*
 * free_set_launch_overlap -- process-wide switch for programmatic dependent launch (a CUDA stream feature; the paper has no
 * counterpart).  When on (the default) the kernels of a pass are launched so that each may be brought onto the SMs and
 * do its set-up while its predecessor on the stream is still finishing; it reads and writes global memory only after the
 * predecessor has completed, so results are identical.  It shortens a step where kernels are short and is applied to
 * launches over at most 16384 token rows (on longer kernels it measured slightly slower).
 * Returns the previous setting.  HOST-only; takes effect for launches made afterwards.
 */
int free_set_launch_overlap(int on);

/*
 * Device error word (safety aid; the paper has no counterpart).  free_device_error_code() maps a HOST copy of a device
 * error word to the library's return code: 0 -> FREE_OK, anything else -> FREE_ERR_DEVICE_TIMEOUT.  It is the mapping
 * sample_trajectory() applies after every round.
 * free_selftest_bounded_wait() runs the bounded wait of the tensor-core pipelines once on a barrier that nothing ever
 * signals: one warp, no copies, tensor memory or clusters involved.  The wait gives up after `limit_cycles` SM clock
 * cycles (1 .. 1e8, i.e. at most about 50 ms), ORs a non-zero code into *device_error exactly as the pipelines do, and
 * the kernel returns; the context stays usable.  It shows that an expired wait ends in an error status, not in a stuck
 * launch.
 *   device_error   DEVICE uint32, OR-ed into (clear it first)
 *   waited_cycles  DEVICE int64 or NULL: SM cycles the wait took
 * Asynchronous.  Errors: ARG, SHAPE (limit out of range), ALIGN, CUDA.
 */
int free_device_error_code(uint32_t word);
int free_selftest_bounded_wait(uint32_t* device_error, int64_t limit_cycles, int64_t* waited_cycles, void* stream);

/*
 * free_drafter_loss -- the drafter's training objectives (Sec. 3.2), forward values, as one fused reduction:
 *   L_noise  = mean over all elements of (eps_pred - eps_ref)^2                                   (Eq. mse)
 *   L_feat   = mean over sequences and tokens of 1 - <p, r> / (|p| |r| + eps_cos)                 (Eq. cos)
 *   L_smooth = mean over sequences, tokens and channels of phi_beta(p - r)                        (Eqs. smooth, huber)
 *   L_total  = L_noise + lambda_f L_feat + lambda_s L_smooth                                      (Eq. free_loss)
 *   dtype            FREE_FP32 or FREE_BF16: type of the features
 *   eps_pred, eps_ref   DEVICE fp32 [n_seq, d_eps]
 *   f_pred, f_ref       DEVICE `dtype` [n_seq, n_tok, D] (top-block features)
 *   beta > 0, eps_cos >= 0
 *   out              DEVICE double [4]: L_noise, L_feat, L_smooth, L_total
 *   ws               DEVICE, >= free_drafter_loss_workspace_bytes(): per-CTA partial sums (added in a fixed order)
 * Asynchronous.  Errors: ARG, SHAPE, WORKSPACE, ALIGN, CUDA.
 */
size_t free_drafter_loss_workspace_bytes(void);
int free_drafter_loss(int dtype, int n_seq, int n_tok, int D, int64_t d_eps,
                      const float* eps_pred, const float* eps_ref, const void* f_pred, const void* f_ref,
                      float lambda_f, float lambda_s, float beta, float eps_cos,
                      double* out, void* ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Building blocks, exported so that each kernel can be checked against the CPU oracle on its own.
 * They are the same kernels the calls above launch.
 * ------------------------------------------------------------------------------------------------ */

#define FREE_EPI_BIAS            0   /* out = acc + bias                                   */
#define FREE_EPI_BIAS_GELU       1   /* out = gelu_tanh(acc + bias)                        */
#define FREE_EPI_BIAS_SILU       2   /* out = silu(acc + bias)                             */
#define FREE_EPI_GATE_RESIDUAL   3   /* resid[row, n] += gate[row / rows_per_seq, n] * (acc + bias), fp32 in place */

/* out[M, N] = epilogue(A[M, K] * W[N, K]^T + bias[N]).  A, W in `dtype`; bias fp32 or NULL.
 * out_dtype FREE_FP32 or FREE_BF16 (ignored for GATE_RESIDUAL, whose output is the fp32 `resid`).
 * gate: DEVICE fp32, element (seq, n) at gate[seq * gate_stride + n].
 * BF16 path (tcgen05): K % 64 == 0, N % 32 == 0; FP32 path (CUDA cores): any sizes.
 * `ws` (>= free_op_linear_workspace_bytes()) holds the device error word of the pipeline. */
size_t free_op_linear_workspace_bytes(void);
int free_op_linear(int dtype, int epilogue, int out_dtype, int M, int N, int K,
                   const void* A, const void* W, const float* bias, void* out,
                   float* resid, const float* gate, int64_t gate_stride, int rows_per_seq,
                   void* ws, size_t ws_bytes, void* stream);

/* LayerNorm (no affine, eps 1e-6, biased variance) of each row of x fp32 [M, D], then
 * y = ln * (1 + scale[seq]) + shift[seq], seq = row / rows_per_seq; shift/scale element (seq, c) at
 * ptr[seq * mod_stride + c].  y in `out_dtype` [M, D]. */
int free_op_ln_modulate(int out_dtype, int M, int D, int rows_per_seq, const float* x,
                        const float* shift, const float* scale, int64_t mod_stride, void* y, void* stream);

/* Non-causal multi-head self-attention of n_seq sequences: qkv [n_seq, n_tok, 3, heads, d_head] in
 * `dtype`, out [n_seq, n_tok, heads * d_head] in `dtype`; softmax(q k^T / sqrt(d_head)) v per head. */
int free_op_attention(int dtype, int n_seq, int n_tok, int heads, int d_head,
                      const void* qkv, void* out, void* ws, size_t ws_bytes, void* stream);
size_t free_op_attention_workspace_bytes(int dtype, int n_seq, int n_tok, int heads, int d_head);

/*
 * free_op_attention_static -- bf16 tensor-core attention that allocates nothing and takes no workspace.
 * (The paper has no counterpart: this serves callers that are not allowed to allocate device memory -- code that
 * runs under a frozen memory plan, plugins whose host application owns the memory pool, loops that must not hit
 * the device-wide synchronisation of cudaMalloc / cudaFree.)  Same result as free_op_attention(FREE_BF16, ...).
 * The scratch (head-major copies of q, k, v^T) is a 12 MiB array built into the library's device image: every
 * GPU that loads the library holds it until the process ends.
 *   Limit: n_seq * heads * n_tok * d_pad <= FREE_STATIC_ATTN_MAX_ELEMS, d_pad = d_head rounded up to 64/80/96/128;
 *          larger problems return FREE_ERR_WORKSPACE.  n_tok % 128 == 0, d_head % 8 == 0, d_head <= 128, else
 *          FREE_ERR_UNSUPPORTED.
 *   qkv, out     DEVICE bf16, as for free_op_attention
 *   device_error DEVICE uint32 (caller's): 0 after the call completes unless a bounded device-side wait gave up
 * The first call on each device looks up the array's device address (with that device current); make that first
 * call outside any stream capture.  All calls share the one array, which keeps the previous call's contents:
 * each call rewrites everything it reads, but two calls that overlap on the GPU (different streams) race.
 */
#define FREE_STATIC_ATTN_MAX_ELEMS (1u << 21)
int free_op_attention_static(int n_seq, int n_tok, int heads, int d_head, const void* qkv, void* out,
                             uint32_t* device_error, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* FREE_B200_H */
