// Non-causal multi-head self-attention on the 5th-generation tensor cores, two query tiles per CTA.
//
// A work item is 256 queries of one (sequence, head): two tiles of 128 queries that alternate on the tensor core and on
// the exp2 unit, so that the softmax of one tile runs while the MMAs of the other execute.  CTAs are persistent (one
// per SM) and walk over the items: at d_head 72 and 1024 tokens an item is only 8 key blocks long, and launching,
// allocating TMEM, loading Q and filling the pipeline once per item cost a quarter of the time.  The producer loads the
// next item's Q (as soon as the last S of the current item has read the old one), K and V, and the next item's first S
// is issued, while the softmax warps still finish, normalise and store the current item.
// Phases.  The exp2 phases of the two tiles must alternate: when they coincide each takes 2200 clocks instead of 1350
// and nothing overlaps the rest of a block (4000 clocks per block instead of 3300).  Nothing restores the alternation
// once it is lost, and the end of an item leaves the tiles skewed, so every item starts with a hand-over: tile 1 takes
// its first block after tile 0's first, and tile 0 its second block after tile 1's first.
//   warps 0-7   softmax of query tile 0: a query row (= one TMEM lane) is shared by two threads, warp w and warp
//               w + 4, which take the two halves of 64 keys of every block (four softmax warps per scheduler keep
//               the exp2 unit, which bounds this kernel at d_head 72, fed while others wait on TMEM or barriers)
//   warps 8-15  the same for query tile 1
//   warp 16     TMA producer: per item the Q tiles (whose padding columns it zeroes itself), then K and V^T blocks of
//               128 keys into double buffers
//   warps 17-18 MMA issuers, one per query tile (each runs converged, one elected lane issues; a barrier poll costs
//               ~200 clocks and an MMA issue ~50-100, so one warp serving both tiles was the bottleneck):
//               S_t = Q_t K^T (128 x 128 x d_pad) into TMEM, O_t = P_t V (128 x d_pad x 128) into TMEM
// Per block of 128 keys and per tile, a softmax thread pulls its half row of S out of TMEM in one round trip and
// releases S at once (the next block's S is issued while this softmax still runs), takes the row maximum, turns the
// row into exp2 probabilities (row sum in fp32, P rounded to bf16 into shared memory in the MMA operand layout) and
// signals P; the two threads of a row exchange their half-row maxima through shared memory (named barrier of their two
// warps) so that both use the same exponent offset, and add their partial row sums at the end.  O_t accumulates in TMEM across all key blocks: the exponent offset of a row is only moved when the row
// maximum has grown by more than 8 (a factor 256), in which case the row's O and running sum are rescaled in place
// before that block's P V is issued; numerator and denominator always share the offset, so the result is exact.
// Issue order per block and tile: S(next), then P V; at an item's last block P V first (the next S waits for the next
// item's operands).  The finished rows are normalised into a dense copy of the tile in shared memory (the tile's P
// buffer) and leave by one TMA store per 32 rows.
//
// Operands.  q and k are read straight from a token-major bf16 matrix [n_seq * n_tok, ld] (the output of the QKV
// linear layer): head h of q starts at column q_col0 + h * d_head, of k at k_col0 + h * d_head.  d_pad is 64 plus a
// tail of 0 / 16 / 32 columns (its own 32- / 64-byte swizzle).  When d_head is not 64 + tail, the tail's last columns
// belong to the next head: they are zeroed in the Q tiles after loading (the matching K columns then multiply
// zeros).  v^T is head-major [n_seq * heads, d_pad, n_tok] (rows past d_head are never used: they only feed
// output columns that are not stored).  Output: [n_seq * n_tok, heads * d_head] bf16.
#include "internal.h"
#include "tc_common.cuh"
#include <mutex>

namespace {

constexpr int BQ = 128, BKV = 128;
constexpr int kThreads = 608;
constexpr uint32_t kCtrlBytes = 8192;          // barriers (1 KB), row-maximum exchange (4 KB), row-sum exchange (2 KB)
constexpr uint32_t kTmemCols = 512;           // S_0 [0,128), S_1 [128,256), O_0 [256,384), O_1 [384,512)

struct Attn2Args {
    int n_tok, heads, d_head;
    int n_items, qblocks;                    // work items = (sequence * heads + head, block of 256 queries)
    int q_col0, k_col0;
    float scale_log2e;
    uint32_t* err;
};

template <int DP> struct Geo2 {
    static constexpr int W1 = DP - 64;                                  // tail chunk: 0, 16 or 32 columns
    static constexpr uint32_t LAY1 = W1 == 32 ? 4 : 6;                  // 64- or 32-byte swizzle
    static constexpr uint32_t ROW1 = W1 * 2;                            // bytes per row of the tail chunk
    static constexpr uint32_t QK0_BYTES = 128 * 128;
    static constexpr uint32_t QK1_BYTES = 128 * ROW1;
    static constexpr uint32_t QK_BYTES = QK0_BYTES + QK1_BYTES;         // one Q or K tile (multiple of 1024)
    static constexpr uint32_t V_HALF = DP * 128;                        // DP rows x 64 keys
    static constexpr uint32_t V_BYTES = 2 * V_HALF;
    static constexpr uint32_t P_HALF = 128 * 128;
    static constexpr uint32_t P_BYTES = 2 * P_HALF;
    static constexpr uint32_t OFF_Q = 0;                                // two tiles
    static constexpr uint32_t OFF_K = OFF_Q + 2 * QK_BYTES;             // two buffers
    static constexpr uint32_t OFF_V = OFF_K + 2 * QK_BYTES;             // two buffers
    static constexpr uint32_t OFF_P = OFF_V + 2 * V_BYTES;              // two tiles
    static constexpr uint32_t TILE_BYTES = OFF_P + 2 * P_BYTES;
    static constexpr uint32_t SMEM = 1024 /*align*/ + kCtrlBytes + TILE_BYTES;
    static_assert(QK_BYTES % 1024 == 0 && V_HALF % 1024 == 0, "tiles must keep the swizzle alignment");
    static_assert(SMEM <= 227 * 1024, "does not fit in shared memory");
};

__device__ __forceinline__ float ex2(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }

template <int DP>
__global__ void __launch_bounds__(kThreads, 1)
attention_tc2_kernel(const __grid_constant__ CUtensorMap mapQK0, const __grid_constant__ CUtensorMap mapQK1,
                     const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapO, const Attn2Args a) {
    using G = Geo2<DP>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* bar_q = reinterpret_cast<uint64_t*>(smem);
    uint64_t* bar_qz = bar_q + 1;       // Q tiles fixed up (padding columns zeroed): the producer warp arrives after its fix-up
    uint64_t* k_full = bar_q + 2;       // [2]
    uint64_t* k_empty = bar_q + 4;      // [2]
    uint64_t* v_full = bar_q + 6;       // [2]
    uint64_t* v_empty = bar_q + 8;      // [2]
    uint64_t* s_full = bar_q + 10;      // [2] per tile: S complete
    uint64_t* p_ready = bar_q + 12;     // [2] per tile: P stored and S consumed (4 warp arrivals)
    uint64_t* o_full = bar_q + 14;      // [2] per tile: O_j complete
    uint64_t* s_free = bar_q + 16;      // [2] per tile: S_j read out of TMEM (4 warp arrivals)
    uint64_t* q_free = bar_q + 18;      // the last S of an item has read Q (one commit per tile): the next item's Q may land
    uint64_t* o_free = bar_q + 19;      // [2] per tile: the finished O has been read out of TMEM (8 warp arrivals)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_q + 21);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    float* mx_x = reinterpret_cast<float*>(smem + 1024);       // [parity][tile][half][row]
    float* l_x = reinterpret_cast<float*>(smem + 5120);        // [tile][half][row]
    uint8_t* tiles = smem + kCtrlBytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int T = a.n_tok, nb = T / BKV;
    // The CTA walks over work items first, first + step, ...  All its items have the same number of query tiles: the
    // host launches one CTA per item when the last block of 256 queries is half empty.
    const int first = blockIdx.x, step = gridDim.x;
    const int nq = ((first % a.qblocks) * 2 * BQ + BQ < T) ? 2 : 1;
    const int my_items = first < a.n_items ? (a.n_items - first + step - 1) / step : 0;
    const uint32_t total = (uint32_t)my_items * (uint32_t)nb;          // key blocks this CTA goes through

    if (threadIdx.x == 0) {
        tc::mbar_init(bar_q, 1); tc::mbar_init(bar_qz, 1); tc::mbar_init(q_free, nq);
        for (int i = 0; i < 2; ++i) {
            tc::mbar_init(&k_full[i], 1); tc::mbar_init(&k_empty[i], nq); tc::mbar_init(&v_full[i], 1); tc::mbar_init(&v_empty[i], nq);
            tc::mbar_init(&s_full[i], 1); tc::mbar_init(&p_ready[i], 8); tc::mbar_init(&o_full[i], 1); tc::mbar_init(&s_free[i], 8);
            tc::mbar_init(&o_free[i], 8);
        }
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::fence_proxy_async();
    }
    if (warp == 17) { tc::tmem_alloc(tmem_slot, kTmemCols); tc::tmem_relinquish(); }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    auto fail = [&]() { *abort_flag = 1; atomicOr(a.err, FREE_DEV_ERR_ATTN); };
    // everything above touched only this CTA's shared and tensor memory: from here on q, k, v are read
    free_grid_dep_wait();
    free_grid_dep_launch();
    // warp-uniform bounded wait; false = give up
    auto wait = [&](uint64_t* bar, uint32_t parity) -> bool { return tc::wait_uniform(bar, parity, abort_flag); };
    // two barriers polled together (their poll latencies overlap)
    auto wait2 = [&](uint64_t* b0, uint32_t p0, uint64_t* b1, uint32_t p1) -> bool {
        bool r0 = tc::mbar_try_wait(b0, p0), r1 = tc::mbar_try_wait(b1, p1);
        if (!(r0 && r1)) {
            if (*abort_flag) return false;
            if (!r0) r0 = tc::mbar_wait(b0, p0);
            if (!r1) r1 = tc::mbar_wait(b1, p1);
        }
        return __all_sync(0xffffffffu, r0 && r1);
    };

    if (warp == 16) {
        // ------------------------------------------------------------------ TMA producer (and Q fix-up)
        if (lane == 0) { tc::tma_prefetch_desc(&mapQK0); tc::tma_prefetch_desc(&mapV); }
        bool ok = true;
        uint32_t g = 0;                                     // running key-block count: buffer g & 1, phase (g >> 1) & 1
        int it = 0;
        for (int w = first; ok && w < a.n_items; w += step, ++it) {
            const int sh = w / a.qblocks, q0 = (w % a.qblocks) * 2 * BQ;       // sh = sequence * heads + head
            const int seq = sh / a.heads, head = sh % a.heads;
            const int row_q = seq * T + q0;                 // row of the first query in the token-major matrix
            const int xq = a.q_col0 + head * a.d_head, xk = a.k_col0 + head * a.d_head;
            const int v_row = sh * DP;
            if (it > 0) {                                   // the previous item's last S has read the Q tiles
                ok = wait(q_free, (uint32_t)(it - 1) & 1u);
                if (!ok) break;
            }
            if (tc::elect_one()) {
                tc::mbar_expect_tx(bar_q, (uint32_t)nq * G::QK_BYTES);
                for (int t = 0; t < nq; ++t) {
                    uint8_t* sQ = tiles + G::OFF_Q + t * G::QK_BYTES;
                    tc::tma_load_2d(sQ, &mapQK0, bar_q, xq, row_q + t * BQ);
                    if (G::W1 > 0) tc::tma_load_2d(sQ + G::QK0_BYTES, &mapQK1, bar_q, xq + 64, row_q + t * BQ);
                }
            }
            __syncwarp();
            for (int j = 0; ok && j < nb; ++j, ++g) {
                const int b = (int)(g & 1u);
                const uint32_t ph = (g >> 1) & 1u;
                ok = wait(&k_empty[b], ph ^ 1u);
                if (!ok) break;
                if (tc::elect_one()) {
                    uint8_t* sK = tiles + G::OFF_K + b * G::QK_BYTES;
                    tc::mbar_expect_tx(&k_full[b], G::QK_BYTES);
                    tc::tma_load_2d(sK, &mapQK0, &k_full[b], xk, seq * T + j * BKV);
                    if (G::W1 > 0) tc::tma_load_2d(sK + G::QK0_BYTES, &mapQK1, &k_full[b], xk + 64, seq * T + j * BKV);
                }
                __syncwarp();
                if (j == 0) {
                    // Q has landed: zero its columns [d_head, d_pad) (they belong to the next head), then release it to
                    // the MMA warps.  Done here so that the next item's first S can be issued while the softmax warps
                    // still finish the previous item.
                    ok = wait(bar_q, (uint32_t)it & 1u);
                    if (!ok) break;
                    if constexpr (G::W1 > 0) {
                        constexpr int units = G::ROW1 / 16, rows_per_128 = 128 / G::ROW1;
                        for (int t = 0; t < nq; ++t) {
                            uint8_t* sQ = tiles + G::OFF_Q + t * G::QK_BYTES;
                            for (int r = lane; r < BQ; r += 32)
                                for (int u = (a.d_head - 64) / 8; u < units; ++u) {
                                    const int su = u ^ ((r / rows_per_128) & (units - 1));
                                    *reinterpret_cast<uint4*>(sQ + G::QK0_BYTES + r * G::ROW1 + su * 16) = make_uint4(0u, 0u, 0u, 0u);
                                }
                        }
                    }
                    tc::fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) tc::mbar_arrive(bar_qz);
                }
                ok = wait(&v_empty[b], ph ^ 1u);
                if (!ok) break;
                if (tc::elect_one()) {
                    uint8_t* sV = tiles + G::OFF_V + b * G::V_BYTES;
                    tc::mbar_expect_tx(&v_full[b], G::V_BYTES);
                    tc::tma_load_2d(sV, &mapV, &v_full[b], j * BKV, v_row);
                    tc::tma_load_2d(sV + G::V_HALF, &mapV, &v_full[b], j * BKV + 64, v_row);
                }
                __syncwarp();
            }
        }
        if (!ok) {
            if (lane == 0) fail();
            const long long t0 = clock64();                 // loads in flight land within microseconds
            while (clock64() - t0 < 400000ll) { }
        }
        __syncwarp();
    } else if (warp >= 17) {
        // ------------------------------------------------------------------ MMA issuer of query tile t
        const int t = warp - 17;
        if (t < nq) {
            const uint32_t idesc_s = tc::idesc_bf16(BQ, BKV), idesc_o = tc::idesc_bf16(BQ, DP);
            const uint32_t qa = tc::smem_u32(tiles + G::OFF_Q) + t * G::QK_BYTES, k_base = tc::smem_u32(tiles + G::OFF_K);
            const uint32_t v_base = tc::smem_u32(tiles + G::OFF_V), pa = tc::smem_u32(tiles + G::OFF_P) + t * G::P_BYTES;
            const uint32_t d_s = tmem_base + t * 128, d_o = tmem_base + 256 + t * 128;
            // operand descriptors are fixed per buffer: built once
            constexpr int KS = DP / 16;
            uint64_t qd[KS], kd[2][KS], pd[8], vd[2][8];
#pragma unroll
            for (int k = 0; k < KS; ++k) {
                if (k < 4) {
                    qd[k] = tc::smem_desc(qa + k * 32, 1024, 2);
                    kd[0][k] = tc::smem_desc(k_base + k * 32, 1024, 2);
                    kd[1][k] = tc::smem_desc(k_base + G::QK_BYTES + k * 32, 1024, 2);
                } else {
                    qd[k] = tc::smem_desc(qa + G::QK0_BYTES + (k - 4) * 32, 8 * G::ROW1, G::LAY1);
                    kd[0][k] = tc::smem_desc(k_base + G::QK0_BYTES + (k - 4) * 32, 8 * G::ROW1, G::LAY1);
                    kd[1][k] = tc::smem_desc(k_base + G::QK_BYTES + G::QK0_BYTES + (k - 4) * 32, 8 * G::ROW1, G::LAY1);
                }
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const uint32_t half = k >> 2, ko = (k & 3) * 32;
                pd[k] = tc::smem_desc(pa + half * G::P_HALF + ko, 1024, 2);
                vd[0][k] = tc::smem_desc(v_base + half * G::V_HALF + ko, 1024, 2);
                vd[1][k] = tc::smem_desc(v_base + G::V_BYTES + half * G::V_HALF + ko, 1024, 2);
            }
            // The whole warp runs the issue sequences; the instructions are predicated on the elected lane `el`.
            auto issue_s = [&](uint32_t el, int kb, bool last_of_item) {   // S_t = Q_t K^T over d_pad in steps of 16
#pragma unroll
                for (int k = 0; k < KS; ++k) tc::mma_bf16_if(el, d_s, qd[k], kb ? kd[1][k] : kd[0][k], idesc_s, k != 0);
                tc::mma_commit_if(el, &s_full[t]);
                tc::mma_commit_if(el, &k_empty[kb]);            // one arrival per tile
                if (last_of_item) tc::mma_commit_if(el, q_free);   // Q is no longer needed once this S has executed
            };
            auto issue_o = [&](uint32_t el, int vb, uint32_t accumulate) {   // O_t (+)= P_t V over the 128 keys in steps of 16
#pragma unroll
                for (int k = 0; k < 8; ++k) tc::mma_bf16_if(el, d_o, pd[k], vb ? vd[1][k] : vd[0][k], idesc_o, (accumulate | (uint32_t)k) != 0 ? 1u : 0u);
                tc::mma_commit_if(el, &o_full[t]);
                tc::mma_commit_if(el, &v_empty[vb]);
            };
            bool ok = total > 0 && wait2(bar_q, 0, bar_qz, 0) && wait(&k_full[0], 0);
            if (ok) {
                tc::tc_fence_after();
                issue_s(tc::elect_one() ? 1u : 0u, 0, nb == 1);
                __syncwarp();
            }
            int j = 0, it = 0;                                  // block within the item, item count
            for (uint32_t g = 0; ok && g < total; ++g) {
                const int b = (int)(g & 1u);
                const uint32_t ph = g & 1u, bph = (g >> 1) & 1u;
                const bool new_item = j + 1 == nb;
                // Order within a block: the next block's S first (its operands are there long before this block's P).  At
                // an item's last block the other way round: the next S needs the next item's Q and K, and this item's
                // last P V must not wait for them.
#pragma unroll 1
                for (int stepi = 0; ok && stepi < 2; ++stepi) {
                    const bool do_s = (stepi == 0) != new_item;
                    if (do_s) {
                        if (g + 1 < total) {
                            // S_t of the next block (of this item or of the next one) as soon as this tile's softmax has
                            // pulled S_t of this block out of TMEM
                            ok = wait2(&s_free[t], ph, &k_full[b ^ 1], ((g + 1) >> 1) & 1u);
                            if (!ok) break;
                            if (new_item) {
                                ok = wait2(bar_q, (uint32_t)(it + 1) & 1u, bar_qz, (uint32_t)(it + 1) & 1u);
                                if (!ok) break;
                            }
                            tc::tc_fence_after();
                            issue_s(tc::elect_one() ? 1u : 0u, b ^ 1, new_item ? nb == 1 : j + 2 == nb);
                            __syncwarp();
                        }
                    } else {
                        ok = wait2(&p_ready[t], ph, &v_full[b], bph);
                        if (!ok) break;
                        if (j == 0 && it > 0) {                 // the previous item's O has been read out
                            ok = wait(&o_free[t], (uint32_t)(it - 1) & 1u);
                            if (!ok) break;
                        }
                        tc::tc_fence_after();
                        issue_o(tc::elect_one() ? 1u : 0u, b, j > 0 ? 1u : 0u);
                        __syncwarp();
                    }
                }
                if (!ok) break;
                if (++j == nb) { j = 0; ++it; }
            }
            if (!ok && lane == 0) fail();
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ softmax + output accumulation
        const int t = warp >> 3, hf = (warp >> 2) & 1, wq = warp & 3;
        if (t < nq) {
            const int r = wq * 32 + lane;                          // query row within the tile = TMEM lane
            const uint32_t lane_sel = (uint32_t)(wq * 32) << 16;
            const uint32_t tmem_S = tmem_base + t * 128 + hf * 64 + lane_sel, tmem_O = tmem_base + 256 + t * 128 + lane_sel;
            uint8_t* prow = tiles + G::OFF_P + t * G::P_BYTES + hf * G::P_HALF + r * 128;   // this thread's 64 keys of P
            constexpr int NCH = DP / 16;                            // 16-column chunks of O: the two threads of a row split them
            const int ch0 = hf == 0 ? 0 : (NCH + 1) / 2, ch1 = hf == 0 ? (NCH + 1) / 2 : NCH;
            bool ok = true;
            float m_used = -INFINITY, l_run = 0.f;                  // exponent offset of this row; sum over this thread's keys
            const float cs = a.scale_log2e;
            const int pair_id = 1 + t * 4 + wq;                     // named barrier of the two warps that share these rows
            auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(pair_id) : "memory"); };
            // The pair barrier is a hardware barrier (cheap, but unbounded): both warps therefore run it in every
            // iteration whatever happened before, and a warp whose bounded wait gave up only stops doing work.
            bool s_polled = false;                                  // an early poll already saw this block's S complete
            int j = 0, w = first;                                   // block within the item, the item
            for (uint32_t g = 0; g < total; ++g) {
                const uint32_t ph = g & 1u;
                uint32_t sv[64];                                    // this thread's half row of S
                float m_half = 0.f;
                bool o_polled = false;
                float* xs = mx_x + (((int)(g & 1u) * 2 + t) * 2) * 128;
                if (j == 0) { m_used = -INFINITY; l_run = 0.f; }
                if (ok && !s_polled) ok = wait(&s_full[t], ph);
                if (ok) {
                    tc::tc_fence_after();
                    tc::tmem_ld64(tmem_S, sv);                      // one TMEM round trip
                    tc::tmem_wait_ld();
                    tc::tc_fence_before();
                    __syncwarp();
                    if (lane == 0) tc::mbar_arrive(&s_free[t]);     // the next block's S may overwrite TMEM now
                    // poll early for the previous P V (its latency hides behind the maximum and the pair barrier)
                    if (g > 0) o_polled = tc::mbar_try_wait(&o_full[t], ph ^ 1u);
                    float m0 = __uint_as_float(sv[0]), m1 = __uint_as_float(sv[1]), m2 = __uint_as_float(sv[2]), m3 = __uint_as_float(sv[3]);
#pragma unroll
                    for (int i = 4; i < 64; i += 4) {
                        m0 = fmaxf(m0, __uint_as_float(sv[i])); m1 = fmaxf(m1, __uint_as_float(sv[i + 1]));
                        m2 = fmaxf(m2, __uint_as_float(sv[i + 2])); m3 = fmaxf(m3, __uint_as_float(sv[i + 3]));
                    }
                    m_half = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
                    xs[hf * 128 + r] = m_half;                      // for the thread that holds the other 64 keys of this row
                }
                pair_sync();
                if (j == 0 && w != first) {
                    // The previous item's rows were staged in the tile's P buffer: every store of the tile has read its
                    // rows before any warp writes this item's P (the stores had the whole first part of this block to
                    // do so; hardware barrier of the tile's 8 warps, run unconditionally like pair_sync).
                    if (hf == 0 && lane == 0) tc::bulk_wait_read<0>();
                    asm volatile("bar.sync %0, 256;" ::"r"(9 + t) : "memory");
                }
                // the previous P V has read P and O_t is complete up to the previous block: P may be overwritten, O rescaled
                // (within an item; at an item's first block the previous P V was awaited before O was read out)
                if (ok && j > 0 && !__all_sync(0xffffffffu, o_polled)) ok = wait(&o_full[t], ph ^ 1u);
                if (ok) {
                    const float m_new = fmaxf(m_used, fmaxf(m_half, xs[(hf ^ 1) * 128 + r]));
                    if (__any_sync(0xffffffffu, (m_new - m_used) * cs > 8.f)) {
                        // move the exponent offset of the rows of this warp (always on the first block); the partner
                        // warp takes the same decision from the same values and rescales the other columns of O
                        if (j > 0) {
                            tc::tc_fence_after();
                            const float alpha = ex2((m_used - m_new) * cs);
                            for (int ch = ch0; ch < ch1; ++ch) {
                                uint32_t ov[16];
                                tc::tmem_ld16(tmem_O + ch * 16, ov);
                                tc::tmem_wait_ld();
#pragma unroll
                                for (int i = 0; i < 16; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha);
                                tc::tmem_st16(tmem_O + ch * 16, ov);
                            }
                            tc::tmem_wait_st();
                            l_run *= alpha;
                        }
                        m_used = m_new;
                    }
                    // on the first block of every item: tile 1 starts its exponentials when tile 0 has finished its own,
                    // so that from then on one tile is in its exp2 phase (the unit both tiles share) while the other
                    // loads, exchanges and stores
                    if (j == 0 && t == 1) ok = wait(&p_ready[0], ph);
                    // and tile 0 takes its second block after tile 1's first: whatever skew the previous item left
                    // between the tiles, they leave the item's start in opposite phases
                    if (j == 1 && t == 0 && nq == 2) ok = wait(&p_ready[1], ph ^ 1u);
                }
                if (ok) {
                    const float mc = m_used * cs;
                    float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
                    for (int c0 = 0; c0 < 64; c0 += 32) {
                        uint32_t pk[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const float p0 = ex2(fmaf(__uint_as_float(sv[c0 + 2 * i]), cs, -mc));
                            const float p1 = ex2(fmaf(__uint_as_float(sv[c0 + 2 * i + 1]), cs, -mc));
                            sum0 += p0; sum1 += p1;
                            __nv_bfloat162 bb = __floats2bfloat162_rn(p0, p1);
                            pk[i] = *reinterpret_cast<uint32_t*>(&bb);
                        }
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int unit = (c0 >> 3) + u;         // 16-byte unit within the 128-byte row
                            *reinterpret_cast<uint4*>(prow + ((unit ^ (r & 7)) << 4)) = make_uint4(pk[4 * u], pk[4 * u + 1], pk[4 * u + 2], pk[4 * u + 3]);
                        }
                    }
                    l_run += sum0 + sum1;
                    // poll early for the next block's S (issued long ago): the answer arrives while P is published
                    const bool s_next = j + 1 < nb && tc::mbar_try_wait(&s_full[t], ph ^ 1u);
                    tc::tc_fence_before();
                    tc::fence_proxy_async();                        // P (generic-proxy stores) visible to the tensor core
                    __syncwarp();
                    if (lane == 0) tc::mbar_arrive(&p_ready[t]);
                    s_polled = __all_sync(0xffffffffu, s_next);
                }
                if (++j < nb) continue;
                // ---- the item's last block is done: normalise and store its rows, then hand O back
                j = 0;
                // row sum = this thread's keys + the partner's (both were kept at the same exponent offset)
                l_x[(t * 2 + hf) * 128 + r] = l_run;
                pair_sync();
                if (ok) ok = wait(&o_full[t], ph);
                const uint32_t row_bytes = (uint32_t)a.d_head * 2u;
                uint8_t* stage = tiles + G::OFF_P + t * G::P_BYTES;
                if (ok) {
                    tc::tc_fence_after();
                    const float inv = 1.f / (l_run + l_x[(t * 2 + (hf ^ 1)) * 128 + r]);
                    const int dh = a.d_head;                            // multiple of 8
                    uint8_t* srow = stage + (uint32_t)r * row_bytes;
                    for (int ch = ch0; ch < ch1; ++ch) {
                        const int c0 = ch * 16;
                        uint32_t ov[16];
                        tc::tmem_ld16(tmem_O + c0, ov);
                        tc::tmem_wait_ld();
#pragma unroll
                        for (int h8 = 0; h8 < 16; h8 += 8) {
                            if (c0 + h8 < dh) {
                                uint32_t wv[4];
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    __nv_bfloat162 bb = __floats2bfloat162_rn(__uint_as_float(ov[h8 + 2 * i]) * inv, __uint_as_float(ov[h8 + 2 * i + 1]) * inv);
                                    wv[i] = *reinterpret_cast<uint32_t*>(&bb);
                                }
                                *reinterpret_cast<uint4*>(srow + (c0 + h8) * 2) = make_uint4(wv[0], wv[1], wv[2], wv[3]);
                            }
                        }
                    }
                    tc::tc_fence_before();
                    tc::fence_proxy_async();                            // the staged rows are read by the TMA unit
                    __syncwarp();
                    if (lane == 0) tc::mbar_arrive(&o_free[t]);         // the next item's first P V may overwrite O
                }
                pair_sync();                                            // both column halves of these 32 rows are in place
                if (ok && hf == 0 && lane == 0) {
                    const int sh = w / a.qblocks, q0 = (w % a.qblocks) * 2 * BQ;
                    const int seq = sh / a.heads, head = sh % a.heads;
                    tc::tma_store_2d(&mapO, tc::smem_u32(stage + (uint32_t)(wq * 32) * row_bytes), head * a.d_head, seq * T + q0 + t * BQ + wq * 32);
                    tc::bulk_commit();                                  // read back before the next item's first P store
                }
                w += step;
            }
            if (hf == 0 && lane == 0) tc::bulk_wait_read<0>();          // shared memory is given back when the CTA ends
            if (!ok && lane == 0) fail();
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 17) { tc::tc_fence_after(); tc::tmem_dealloc(tmem_base, kTmemCols); }
}

template <int DP>
int launch(int n_seq, int n_tok, int heads, int d_head, const void* qk, long long ld, int width, int q_col0, int k_col0,
           const void* vt, void* out, uint32_t* err, cudaStream_t s) {
    using G = Geo2<DP>;
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [&] {
        attr_err = cudaFuncSetAttribute(attention_tc2_kernel<DP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)G::SMEM);
    });
    if (attr_err != cudaSuccess) return FREE_ERR_CUDA;
    const uint64_t rows = (uint64_t)n_seq * n_tok, rows_v = (uint64_t)n_seq * heads * DP;
    if (rows > 0x7fffffffull || rows_v > 0x7fffffffull) return FREE_ERR_SHAPE;
    CUtensorMap mQK0, mQK1, mV, mO;
    FREE_TRY(free_tensor_map_2d(&mQK0, qk, (uint64_t)width, rows, (uint64_t)ld * 2, 64, 128, 128));
    if (G::W1 > 0) FREE_TRY(free_tensor_map_2d(&mQK1, qk, (uint64_t)width, rows, (uint64_t)ld * 2, G::W1, 128, (int)G::ROW1));
    else mQK1 = mQK0;
    FREE_TRY(free_tensor_map_2d(&mV, vt, (uint64_t)n_tok, rows_v, (uint64_t)n_tok * 2, 64, DP, 128));
    FREE_TRY(free_tensor_map_2d(&mO, out, (uint64_t)heads * d_head, rows, (uint64_t)heads * d_head * 2, (uint32_t)d_head, 32, 0));
    const int qblocks = (n_tok + 2 * BQ - 1) / (2 * BQ);
    const long long n_items = (long long)qblocks * n_seq * heads;
    if (n_items > 0x7fffffffll) return FREE_ERR_SHAPE;
    Attn2Args a{n_tok, heads, d_head, (int)n_items, qblocks, q_col0, k_col0, 1.4426950408889634f / sqrtf((float)d_head), err};
    // persistent CTAs, one per SM, when every item has two query tiles; else one CTA per item (they then differ)
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) { (void)cudaGetLastError(); sms = 148; }
    const bool uniform = n_tok % (2 * BQ) == 0;
    const unsigned grid = (unsigned)((uniform && n_items > sms) ? sms : n_items);
    return free_launch(free_overlap_for_rows((long long)rows), attention_tc2_kernel<DP>, dim3(grid), dim3(kThreads), (size_t)G::SMEM, s, mQK0, mQK1, mV, mO, a);
}

}  // namespace

int attention_tc2_dpad(int d) { return d <= 64 ? 64 : (d <= 80 ? 80 : 96); }

bool attention_tc2_supported(int n_tok, int d_head) {
    return n_tok >= 128 && n_tok % 128 == 0 && d_head >= 64 && d_head % 8 == 0 && d_head <= 96;
}

int attention_tc2(int n_seq, int n_tok, int heads, int d_head, const void* qk, long long ld, int width, int q_col0, int k_col0,
                  const void* vt, void* out, uint32_t* err, cudaStream_t s) {
    if (n_seq < 1 || heads < 1 || !qk || !vt || !out || !err) return FREE_ERR_ARG;
    if (!attention_tc2_supported(n_tok, d_head)) return FREE_ERR_UNSUPPORTED;
    if (ld % 8 || q_col0 % 8 || k_col0 % 8 || width > ld || !free_aligned16(qk) || !free_aligned16(vt) || !free_aligned16(out)) return FREE_ERR_ALIGN;
    const int dp = attention_tc2_dpad(d_head);
    switch (dp) {
        case 64: return launch<64>(n_seq, n_tok, heads, d_head, qk, ld, width, q_col0, k_col0, vt, out, err, s);
        case 80: return launch<80>(n_seq, n_tok, heads, d_head, qk, ld, width, q_col0, k_col0, vt, out, err, s);
        case 96: return launch<96>(n_seq, n_tok, heads, d_head, qk, ld, width, q_col0, k_col0, vt, out, err, s);
        default: return FREE_ERR_UNSUPPORTED;
    }
}
