// Non-causal multi-head self-attention on the 5th-generation tensor cores (bf16 operands, fp32 softmax).
//
// One CTA per (sequence, head, block of 128 queries); two CTAs share an SM so that one CTA's softmax
// overlaps the other's MMAs.  Per block of 128 keys:
//   S = Q K^T        tcgen05.mma, operands from shared memory (TMA, swizzled), S in TMEM (128 columns)
//   softmax          128 threads, one query row each: tcgen05.ld of S, running max / sum (online softmax),
//                    P = exp2(..) rounded to bf16 and stored to shared memory in the MMA operand layout
//   O_j = P V        tcgen05.mma, V^T from shared memory, O_j in TMEM (d_pad columns)
//   acc = acc * alpha + O_j   in registers (fp32)
// Operand layouts (written by the QKV GEMM's epilogue): q, k [seq*heads, n_tok, d_pad] and
// v^T [seq*heads, d_pad, n_tok], bf16, zero padded from d_head to d_pad.  d_pad is 64 plus a tail of
// 0 / 16 / 32 / 64 elements; the tail chunk uses the 32 / 64 / 128-byte swizzle of its own width.
// Output: [seq * n_tok, heads * d_head] bf16 (the A operand of the projection GEMM).
#include "internal.h"
#include "tc_common.cuh"
#include <mutex>

namespace {

constexpr int BQ = 128, BKV = 128;
constexpr int kThreads = 160;                 // warps 0-3: softmax (one TMEM lane quarter each); warp 4: TMA + MMA issue
constexpr uint32_t kTmemCols = 256;           // S: columns [0,128); O_j: columns [128, 128 + d_pad)

struct AttnArgs {
    int n_tok, heads, d_head;
    float scale_log2e;
    __nv_bfloat16* out;
    uint32_t* err;
};

template <int DP> struct Geo {
    static constexpr int W0 = 64;                               // first K chunk (elements)
    static constexpr int W1 = DP - 64;                          // tail chunk: 0, 16, 32 or 64
    static constexpr uint32_t LAY0 = 2;                         // 128-byte swizzle
    static constexpr uint32_t LAY1 = W1 == 64 ? 2 : (W1 == 32 ? 4 : 6);
    static constexpr uint32_t ROW1 = W1 * 2;                    // bytes per row of the tail chunk
    static constexpr uint32_t QK0_BYTES = 128 * 128;            // 128 rows x 128 bytes
    static constexpr uint32_t QK1_BYTES = 128 * ROW1;
    static constexpr uint32_t QK_BYTES = QK0_BYTES + QK1_BYTES; // one Q or K tile
    static constexpr uint32_t V_HALF = DP * 128;                // DP rows x 64 keys x 2 bytes
    static constexpr uint32_t V_BYTES = 2 * V_HALF;
    static constexpr uint32_t P_HALF = 128 * 128;
    static constexpr uint32_t P_BYTES = 2 * P_HALF;
    static constexpr uint32_t OFF_Q = 0;
    static constexpr uint32_t OFF_K = (QK_BYTES + 1023) / 1024 * 1024;
    static constexpr uint32_t OFF_V = OFF_K + (QK_BYTES + 1023) / 1024 * 1024;
    static constexpr uint32_t OFF_P = OFF_V + (V_BYTES + 1023) / 1024 * 1024;
    static constexpr uint32_t TILE_BYTES = OFF_P + P_BYTES;
    static constexpr uint32_t SMEM = 1024 /*align*/ + 1024 /*barriers*/ + TILE_BYTES;
};

__device__ __forceinline__ float ex2(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }

template <int DP>
__global__ void __launch_bounds__(kThreads, 2)
attention_tc_kernel(const __grid_constant__ CUtensorMap mapQ0, const __grid_constant__ CUtensorMap mapQ1,
                    const __grid_constant__ CUtensorMap mapK0, const __grid_constant__ CUtensorMap mapK1,
                    const __grid_constant__ CUtensorMap mapV, const AttnArgs a) {
    using G = Geo<DP>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* bar_q = reinterpret_cast<uint64_t*>(smem);
    uint64_t* bar_k = bar_q + 1;
    uint64_t* bar_v = bar_q + 2;
    uint64_t* bar_s = bar_q + 3;      // S = Q K^T complete
    uint64_t* bar_p = bar_q + 4;      // P stored, S consumed (4 warp arrivals)
    uint64_t* bar_o = bar_q + 5;      // O_j = P V complete
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_q + 8);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    uint8_t* tiles = smem + 1024;
    uint8_t *sQ = tiles + G::OFF_Q, *sK = tiles + G::OFF_K, *sV = tiles + G::OFF_V, *sP = tiles + G::OFF_P;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sh = blockIdx.y;                         // sequence * heads + head
    const int q0 = blockIdx.x * BQ;
    const int T = a.n_tok, nb = T / BKV;

    if (threadIdx.x == 0) {
        tc::mbar_init(bar_q, 1); tc::mbar_init(bar_k, 1); tc::mbar_init(bar_v, 1);
        tc::mbar_init(bar_s, 1); tc::mbar_init(bar_p, 4); tc::mbar_init(bar_o, 1);
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::fence_proxy_async();
    }
    if (warp == 4) { tc::tmem_alloc(tmem_slot, kTmemCols); tc::tmem_relinquish(); }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_S = tmem_base, tmem_O = tmem_base + 128;
    auto fail = [&]() { *abort_flag = 1; atomicOr(a.err, FREE_DEV_ERR_ATTN); };

    if (warp == 4) {
        // ------------------------------------------------------------------ TMA + MMA issuer
        if (lane == 0) {
            const long long qk_row = (long long)sh * T;            // row of token 0 in the [seq*heads*n_tok, d_pad] view
            const int v_row = sh * DP;                              // row of channel 0 in the [seq*heads*d_pad, n_tok] view
            auto load_k = [&](int j) {
                tc::mbar_expect_tx(bar_k, G::QK_BYTES);
                tc::tma_load_2d(sK, &mapK0, bar_k, 0, (int)(qk_row + (long long)j * BKV));
                if (G::W1 > 0) tc::tma_load_2d(sK + G::QK0_BYTES, &mapK1, bar_k, 64, (int)(qk_row + (long long)j * BKV));
            };
            auto load_v = [&](int j) {
                tc::mbar_expect_tx(bar_v, G::V_BYTES);
                tc::tma_load_2d(sV, &mapV, bar_v, j * BKV, v_row);
                tc::tma_load_2d(sV + G::V_HALF, &mapV, bar_v, j * BKV + 64, v_row);
            };
            auto mma_s = [&]() {                                    // S = Q K^T over d_pad in steps of 16
                const uint32_t qa = tc::smem_u32(sQ), ka = tc::smem_u32(sK);
                const uint32_t idesc = tc::idesc_bf16(BQ, BKV);
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    tc::mma_bf16(tmem_S, tc::smem_desc(qa + k * 32, 1024, G::LAY0), tc::smem_desc(ka + k * 32, 1024, G::LAY0), idesc, k != 0);
#pragma unroll
                for (int k = 0; k < G::W1 / 16; ++k)
                    tc::mma_bf16(tmem_S, tc::smem_desc(qa + G::QK0_BYTES + k * 32, 8 * G::ROW1, G::LAY1),
                                 tc::smem_desc(ka + G::QK0_BYTES + k * 32, 8 * G::ROW1, G::LAY1), idesc, 1u);
                tc::mma_commit(bar_s);
            };
            auto mma_o = [&]() {                                    // O_j = P V over the 128 keys in steps of 16
                const uint32_t pa = tc::smem_u32(sP), va = tc::smem_u32(sV);
                const uint32_t idesc = tc::idesc_bf16(BQ, DP);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const uint32_t half = k >> 2, ko = (k & 3) * 32;
                    tc::mma_bf16(tmem_O, tc::smem_desc(pa + half * G::P_HALF + ko, 1024, 2),
                                 tc::smem_desc(va + half * G::V_HALF + ko, 1024, 2), idesc, k != 0);
                }
                tc::mma_commit(bar_o);
            };
            bool ok = true;
            tc::mbar_expect_tx(bar_q, G::QK_BYTES);
            tc::tma_load_2d(sQ, &mapQ0, bar_q, 0, (int)(qk_row + q0));
            if (G::W1 > 0) tc::tma_load_2d(sQ + G::QK0_BYTES, &mapQ1, bar_q, 64, (int)(qk_row + q0));
            load_k(0);
            load_v(0);
            ok = tc::mbar_wait(bar_q, 0) && tc::mbar_wait(bar_k, 0);
            if (ok) { tc::tc_fence_after(); mma_s(); }
            for (int j = 0; ok && j < nb; ++j) {
                const uint32_t ph = j & 1u;
                if (j == 0 && nb > 1) {                             // K buffer is free once S_0 is complete
                    ok = tc::mbar_wait(bar_s, 0);
                    if (!ok) break;
                    load_k(1);
                }
                ok = !*abort_flag && tc::mbar_wait(bar_p, ph) && tc::mbar_wait(bar_v, ph);
                if (!ok) break;
                tc::tc_fence_after();
                mma_o();
                if (j + 1 < nb) {
                    ok = tc::mbar_wait(bar_k, ph ^ 1u);             // K_{j+1} landed
                    if (!ok) break;
                    tc::tc_fence_after();
                    mma_s();                                        // S_{j+1}: softmax has finished reading S_j
                }
                ok = tc::mbar_wait(bar_o, ph);                      // P V done: V and P buffers are free
                if (!ok) break;
                if (j + 1 < nb) load_v(j + 1);
                if (j + 2 < nb) {
                    ok = tc::mbar_wait(bar_s, ph ^ 1u);             // S_{j+1} done: K buffer is free
                    if (!ok) break;
                    load_k(j + 2);
                }
            }
            if (!ok) {
                fail();
                // let loads in flight land before shared memory is released
                tc::mbar_wait(bar_k, 0, 40000000ll); tc::mbar_wait(bar_k, 1, 40000000ll);
                tc::mbar_wait(bar_v, 0, 40000000ll); tc::mbar_wait(bar_v, 1, 40000000ll);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ softmax + output accumulation
        const uint32_t lane_sel = (uint32_t)(warp * 32) << 16;
        const int r = warp * 32 + lane;                            // query row within the block
        float acc[DP];
#pragma unroll
        for (int c = 0; c < DP; ++c) acc[c] = 0.f;
        float m_run = -INFINITY, l_run = 0.f;
        const float cs = a.scale_log2e;
        uint8_t* prow = sP + r * 128;
        bool ok = true;
        for (int j = 0; j < nb; ++j) {
            const uint32_t ph = j & 1u;
            bool bad = *abort_flag || !tc::mbar_wait(bar_s, ph);
            if (__any_sync(0xffffffffu, bad)) { ok = false; break; }
            tc::tc_fence_after();
            // pass 1: block maximum of this row
            float mx = m_run;
#pragma unroll
            for (int c0 = 0; c0 < BKV; c0 += 32) {
                uint32_t v[32];
                tc::tmem_ld32(tmem_S + lane_sel + c0, v);
                tc::tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) mx = fmaxf(mx, __uint_as_float(v[i]));
            }
            const float alpha = ex2((m_run - mx) * cs);            // 0 on the first block (m_run = -inf)
            const float mxc = mx * cs;
            m_run = mx;
            // pass 2: probabilities, row sum, bf16 P into shared memory (128-byte swizzled rows)
            float sum = 0.f;
#pragma unroll
            for (int c0 = 0; c0 < BKV; c0 += 32) {
                uint32_t v[32];
                tc::tmem_ld32(tmem_S + lane_sel + c0, v);
                tc::tmem_wait_ld();
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float p0 = ex2(fmaf(__uint_as_float(v[2 * i]), cs, -mxc));
                    const float p1 = ex2(fmaf(__uint_as_float(v[2 * i + 1]), cs, -mxc));
                    sum += p0 + p1;
                    __nv_bfloat162 b = __floats2bfloat162_rn(p0, p1);
                    pk[i] = *reinterpret_cast<uint32_t*>(&b);
                }
                uint8_t* base = prow + (c0 >> 6) * G::P_HALF;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int unit = ((c0 & 63) >> 3) + u;           // 16-byte unit within the 128-byte row
                    *reinterpret_cast<uint4*>(base + ((unit ^ (r & 7)) << 4)) = make_uint4(pk[4 * u], pk[4 * u + 1], pk[4 * u + 2], pk[4 * u + 3]);
                }
            }
            l_run = l_run * alpha + sum;
            tc::tc_fence_before();
            tc::fence_proxy_async();                               // P (generic-proxy stores) visible to the tensor core
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(bar_p);
            // accumulate O_j
            bad = !tc::mbar_wait(bar_o, ph);
            if (__any_sync(0xffffffffu, bad)) { ok = false; break; }
            tc::tc_fence_after();
#pragma unroll
            for (int c0 = 0; c0 < DP; c0 += 16) {
                uint32_t v[16];
                tc::tmem_ld16(tmem_O + lane_sel + c0, v);
                tc::tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 16; ++i) acc[c0 + i] = fmaf(acc[c0 + i], alpha, __uint_as_float(v[i]));
            }
            tc::tc_fence_before();
        }
        if (ok) {
            const float inv = 1.f / l_run;
            const int seq = sh / a.heads, head = sh % a.heads;
            __nv_bfloat16* dst = a.out + ((long long)seq * T + q0 + r) * ((long long)a.heads * a.d_head) + (long long)head * a.d_head;
            const int dh = a.d_head;                                // multiple of 8
#pragma unroll
            for (int c0 = 0; c0 < DP; c0 += 8) {
                if (c0 < dh) {
                    uint32_t w[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        __nv_bfloat162 b = __floats2bfloat162_rn(acc[c0 + 2 * i] * inv, acc[c0 + 2 * i + 1] * inv);
                        w[i] = *reinterpret_cast<uint32_t*>(&b);
                    }
                    *reinterpret_cast<uint4*>(dst + c0) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
        } else if (lane == 0) {
            fail();
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 4) { tc::tc_fence_after(); tc::tmem_dealloc(tmem_base, kTmemCols); }
}

template <int DP>
int launch(int n_seq, int n_tok, int heads, int d_head, const void* q, const void* k, const void* vt, void* out,
           uint32_t* err, cudaStream_t s) {
    using G = Geo<DP>;
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [&] {
        attr_err = cudaFuncSetAttribute(attention_tc_kernel<DP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)G::SMEM);
    });
    if (attr_err != cudaSuccess) return FREE_ERR_CUDA;
    const uint64_t rows_qk = (uint64_t)n_seq * heads * n_tok, rows_v = (uint64_t)n_seq * heads * DP;
    if (rows_qk > 0x7fffffffull) return FREE_ERR_SHAPE;
    CUtensorMap mQ0, mQ1, mK0, mK1, mV;
    FREE_TRY(free_tensor_map_2d(&mQ0, q, DP, rows_qk, (uint64_t)DP * 2, 64, 128, 128));
    FREE_TRY(free_tensor_map_2d(&mK0, k, DP, rows_qk, (uint64_t)DP * 2, 64, 128, 128));
    if (G::W1 > 0) {
        FREE_TRY(free_tensor_map_2d(&mQ1, q, DP, rows_qk, (uint64_t)DP * 2, G::W1, 128, (int)G::ROW1));
        FREE_TRY(free_tensor_map_2d(&mK1, k, DP, rows_qk, (uint64_t)DP * 2, G::W1, 128, (int)G::ROW1));
    } else { mQ1 = mQ0; mK1 = mK0; }
    FREE_TRY(free_tensor_map_2d(&mV, vt, (uint64_t)n_tok, rows_v, (uint64_t)n_tok * 2, 64, DP, 128));
    AttnArgs a{n_tok, heads, d_head, 1.4426950408889634f / sqrtf((float)d_head), (__nv_bfloat16*)out, err};
    dim3 grid(n_tok / BQ, n_seq * heads);
    attention_tc_kernel<DP><<<grid, kThreads, G::SMEM, s>>>(mQ0, mQ1, mK0, mK1, mV, a);
    return free_check_launch();
}

}  // namespace

int attention_tc_dpad(int d) { return d <= 64 ? 64 : (d <= 80 ? 80 : (d <= 96 ? 96 : 128)); }

bool attention_tc_supported(int n_tok, int d_head) {
    return n_tok >= 128 && n_tok % 128 == 0 && d_head >= 8 && d_head % 8 == 0 && d_head <= 128;
}

int attention_tc(int n_seq, int n_tok, int heads, int d_head, int d_pad, const void* q, const void* k, const void* vt,
                 void* out, uint32_t* err, cudaStream_t s) {
    if (n_seq < 1 || heads < 1 || !q || !k || !vt || !out || !err) return FREE_ERR_ARG;
    if (!attention_tc_supported(n_tok, d_head) || d_pad != attention_tc_dpad(d_head)) return FREE_ERR_UNSUPPORTED;
    if ((long long)n_seq * heads > 65535) {
        // grid.y limit: split the batch of (sequence, head) pairs
        const int per = 65535 / heads;
        for (int s0 = 0; s0 < n_seq; s0 += per) {
            const int ns = n_seq - s0 < per ? n_seq - s0 : per;
            const size_t qo = (size_t)s0 * heads * n_tok * d_pad * 2;
            FREE_TRY(attention_tc(ns, n_tok, heads, d_head, d_pad, (const char*)q + qo, (const char*)k + qo, (const char*)vt + qo,
                                  (char*)out + (size_t)s0 * n_tok * heads * d_head * 2, err, s));
        }
        return FREE_OK;
    }
    switch (d_pad) {
        case 64: return launch<64>(n_seq, n_tok, heads, d_head, q, k, vt, out, err, s);
        case 80: return launch<80>(n_seq, n_tok, heads, d_head, q, k, vt, out, err, s);
        case 96: return launch<96>(n_seq, n_tok, heads, d_head, q, k, vt, out, err, s);
        case 128: return launch<128>(n_seq, n_tok, heads, d_head, q, k, vt, out, err, s);
        default: return FREE_ERR_UNSUPPORTED;
    }
}
