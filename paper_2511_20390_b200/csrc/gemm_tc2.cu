// bf16 linear layers on CTA pairs (tcgen05 cta_group::2): the kernel behind the large GEMMs of the DiT blocks.
//
//   out = epilogue(A[M,K] * W[N,K]^T + bias),   A and W bf16 (K contiguous), fp32 accumulation in TMEM.
//
// Why pairs: a 128 x 256 tile per SM needs 48 KB of operands per 64-wide K step, and the L2 -> SM path
// (about 48 B per clock per SM) then holds the tensor core to half rate.  Two CTAs of a cluster that share
// one 256 x 256 tile each load their own 128 rows of A and only HALF of the W rows (32 KB per K step); the
// MMA reads both halves across the pair.  No multicast loads are used anywhere.
//
// Persistent kernel, one CTA per SM, clusters of two, 192 threads per CTA:
//   warp 0     TMA producer (both CTAs): its A rows and its W half into a ring of stages; completion is
//              counted on the even CTA's mbarrier, which expects the bytes of both CTAs;
//   warp 1     MMA issuer (even CTA only): tcgen05.mma.cta_group::2, 256 x 256 x 16 per instruction, two TMEM
//              accumulators per CTA; stage-release and accumulator-ready barriers are signalled in both CTAs.
//              The whole warp runs the issue loop converged and one elected lane issues: measured on B200, a
//              single-lane (divergent) loop of wait + 4 MMAs + commit takes ~660 clocks per K step, the converged
//              loop ~508 (= the 4 x 128 clocks the instructions take to execute).  Issuing an MMA costs the thread
//              10-20 clocks; what a K step costs besides is its wait, fence and election, so tiles are 256 wide (128
//              clocks of tensor work per instruction) wherever there are enough row blocks; a ragged last column block
//              (N = 1152 = 4.5 tiles) is computed only as wide as it is (its own tensor map of half as many W rows per
//              CTA, its own instruction shape): it then runs at the shared-memory limit, 0.73 of a full tile's time
//              instead of all of it.  With few row blocks all column blocks are 128 wide (see linear_bf16_pair);
//   warps 2-5  epilogue (both CTAs, each on its own 128 rows): tcgen05.ld, fused bias / GELU / gate, then
//              through swizzled shared-memory staging to a TMA store, or a TMA add-reduction for the gated
//              residual update (the fp32 residual stream is never read by the SM).  QKV variants: HEADS scatters
//              straight into head-major q, k, v^T; TOKV stores the q and k column blocks token-major like any
//              other bf16 output and, for the v column blocks, stages groups of 8 columns transposed for all
//              128 rows of the CTA and writes each group with one 2 KB TMA store into head-major v^T.
// Tile order: N fastest, so the clusters in flight share a few row blocks of A while W stays in L2.
#include "internal.h"
#include "tc_common.cuh"
#include <mutex>

namespace {

constexpr int BK = 64;
constexpr int kThreads = 192;
constexpr int kMaxStages = 8;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kABytes = 128 * BK * 2;              // one CTA's A tile of a stage
constexpr uint32_t kCtrlBytes = 1024;
constexpr uint32_t kStageBufBytes = 4096;               // 32 rows x 128 bytes
constexpr int kBufsPerWarp = 4;                         // staging buffers per epilogue warp: stores in flight per warp
constexpr uint32_t kStagingBytes = 4 * kBufsPerWarp * kStageBufBytes;
constexpr uint32_t kVBufBytes = 8192;                   // v^T staging: 3 buffers of 4 groups x (8 columns x 128 tokens)
static_assert(3 * kVBufBytes <= kStagingBytes, "v^T staging must fit");
constexpr uint32_t kSmemBudget = 227 * 1024;

struct Tc2Args {
    int M, N, K, num_m, num_n, stages;
    int last_n;                             // valid columns of the last column block (BN when N is a multiple of BN)
    const float* bias;
    const float* gate; long long gate_stride; int rows_per_seq;
    int heads, d_head, d_pad, n_tok;
    __nv_bfloat16 *q, *k, *vt;
    uint32_t* err;
};

__device__ __forceinline__ float tanh_fast(float x) { float y; asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ float gelu_fast(float a) {
    return 0.5f * a * (1.0f + tanh_fast(0.7978845608028654f * (a + 0.044715f * a * a * a)));
}
__device__ __forceinline__ uint4 pack8(const float* v) {
    __nv_bfloat162 p0 = __floats2bfloat162_rn(v[0], v[1]), p1 = __floats2bfloat162_rn(v[2], v[3]);
    __nv_bfloat162 p2 = __floats2bfloat162_rn(v[4], v[5]), p3 = __floats2bfloat162_rn(v[6], v[7]);
    uint4 u;
    u.x = *reinterpret_cast<uint32_t*>(&p0); u.y = *reinterpret_cast<uint32_t*>(&p1);
    u.z = *reinterpret_cast<uint32_t*>(&p2); u.w = *reinterpret_cast<uint32_t*>(&p3);
    return u;
}

// Head-major scatter of one row's 32 columns [n0, n0+32) of the QKV output (d_head % 8 == 0).
__device__ __forceinline__ void scatter_qkv(const Tc2Args& a, int row, int n0, const float* v) {
    const int D = a.heads * a.d_head, dh = a.d_head, dp = a.d_pad, T = a.n_tok;
    const int seq = row / T, tok = row % T;
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        const int n = n0 + 8 * g;
        const int which = n / D, hd = (n % D) / dh, c = n % dh;
        const long long sh = (long long)seq * a.heads + hd;
        if (which < 2) {
            __nv_bfloat16* dst = (which == 0 ? a.q : a.k) + (sh * T + tok) * dp + c;
            *reinterpret_cast<uint4*>(dst) = pack8(v + 8 * g);
            if (c + 8 == dh)
                for (int z = dh; z < dp; z += 8) *reinterpret_cast<uint4*>(dst + (z - c)) = zero;
        } else {
            __nv_bfloat16* dst = a.vt + (sh * dp + c) * T + tok;
#pragma unroll
            for (int i = 0; i < 8; ++i) dst[(long long)i * T] = __float2bfloat16(v[8 * g + i]);
            if (c + 8 == dh)
                for (int z = dh; z < dp; ++z) a.vt[(sh * dp + z) * T + tok] = __float2bfloat16(0.f);
        }
    }
}

template <int EPI, bool OUT_BF16, int BN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
linear_tc2_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapW,
                  const __grid_constant__ CUtensorMap mapWl, const __grid_constant__ CUtensorMap mapO, const __grid_constant__ CUtensorMap mapV, const Tc2Args a) {
    constexpr uint32_t kBBytes = (BN / 2) * BK * 2;          // one CTA's half of the W tile of a stage
    constexpr uint32_t kStageBytes = kABytes + kBBytes;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem);      // used in the even CTA only
    uint64_t* empty = full + kMaxStages;
    uint64_t* accf = empty + kMaxStages;
    uint64_t* acce = accf + 2;                               // used in the even CTA only
    uint64_t* ebar = acce + 2;                               // TOKV variant: meeting point of the four epilogue warps
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ebar + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    uint8_t* staging = smem + kCtrlBytes;
    uint8_t* tiles = staging + kStagingBytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = tc::cluster_ctarank();
    const int stages = a.stages, nk = a.K / BK;
    const long long total = (long long)a.num_m * a.num_n;
    const long long first = tc::cluster_id_x(), step = tc::num_clusters_x();

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], 1); }
        for (int i = 0; i < 2; ++i) { tc::mbar_init(&accf[i], 1); tc::mbar_init(&acce[i], 8); }
        tc::mbar_init(ebar, 4);
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::fence_proxy_async();
    }
    if (warp == 1) { tc::tmem_alloc_pair(tmem_slot, kTmemCols); tc::tmem_relinquish_pair(); }
    tc::tc_fence_before();
    tc::cluster_sync_all();                                  // barriers of both CTAs initialised before any remote use
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    auto fail = [&](uint32_t code) { *abort_flag = 1; atomicOr(a.err, code); };
    // everything above touched only this cluster's shared and tensor memory: from here on the operands are read
    free_grid_dep_wait();
    free_grid_dep_launch();

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) { tc::tma_prefetch_desc(&mapA); tc::tma_prefetch_desc(&mapW); tc::tma_prefetch_desc(&mapWl); }
        const uint32_t full0 = tc::mapa(tc::smem_u32(&full[0]), 0);          // the even CTA's stage barriers
        int s = 0;                                           // stage and its phase advance by counting (no divisions in the loop)
        uint32_t ph = 0;
        bool ok = true;
        for (long long t = first; ok && t < total; t += step) {
            const int m_blk = (int)(t / a.num_n), n_blk = (int)(t % a.num_n);
            // a ragged last column block is computed only as wide as it is: each CTA loads half of its valid W rows
            const bool narrow = n_blk == a.num_n - 1 && a.last_n < BN;
            const int half = narrow ? a.last_n / 2 : BN / 2;
            const int a_row = m_blk * 256 + (int)rank * 128, w_row = n_blk * BN + (int)rank * half;
            const uint32_t tx = 2u * (kABytes + (uint32_t)half * BK * 2u);
            for (int kb = 0; kb < nk; ++kb) {
                ok = tc::wait_uniform(&empty[s], ph ^ 1u, abort_flag);
                if (!ok) { if (lane == 0) fail(FREE_DEV_ERR_EMPTY_WAIT); break; }
                if (tc::elect_one()) {
                    const uint32_t dst = tc::smem_u32(tiles + (size_t)s * kStageBytes);
                    if (rank == 0) tc::mbar_expect_tx(&full[s], tx);
                    tc::tma_load_2d_pair(dst, &mapA, full0 + 8u * s, kb * BK, a_row);
                    tc::tma_load_2d_pair(dst + kABytes, narrow ? &mapWl : &mapW, full0 + 8u * s, kb * BK, w_row);
                }
                __syncwarp();
                if (++s == stages) { s = 0; ph ^= 1u; }
            }
        }
        if (!ok || *abort_flag) {
            // loads in flight must land before the shared memory is given back: they take microseconds
            const long long t0 = clock64();
            while (clock64() - t0 < 400000ll) { }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (even CTA only)
        if (rank == 0) {
            const uint32_t idesc_full = tc::idesc_bf16(256, BN), idesc_last = tc::idesc_bf16(256, a.last_n);
            uint32_t tl = 0, ph = 0;
            int s = 0;
            bool ok = true;
            for (long long t = first; ok && t < total; t += step, ++tl) {
                const uint32_t acc = tl & 1u, aph = (tl >> 1) & 1u;
                ok = tc::wait_uniform(&acce[acc], aph ^ 1u, abort_flag);
                if (!ok) { if (lane == 0) fail(FREE_DEV_ERR_ACC_EMPTY); break; }
                tc::tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * (uint32_t)BN;
                const uint32_t idesc = (int)(t % a.num_n) == a.num_n - 1 ? idesc_last : idesc_full;
                for (int kb = 0; kb < nk; ++kb) {
                    ok = tc::wait_uniform(&full[s], ph, abort_flag);
                    if (!ok) { if (lane == 0) fail(FREE_DEV_ERR_FULL_WAIT); break; }
                    tc::tc_fence_after();
                    if (tc::elect_one()) {
                        const uint32_t a_addr = tc::smem_u32(tiles + (size_t)s * kStageBytes), b_addr = a_addr + kABytes;
#pragma unroll
                        for (int k = 0; k < BK / 16; ++k)
                            tc::mma_bf16_pair(d_tmem, tc::smem_desc(a_addr + k * 32, 1024, 2), tc::smem_desc(b_addr + k * 32, 1024, 2),
                                              idesc, (kb | k) != 0 ? 1u : 0u);
                        tc::mma_commit_pair(&empty[s]);      // both CTAs may refill the stage once these MMAs have read it
                    }
                    __syncwarp();
                    if (++s == stages) { s = 0; ph ^= 1u; }
                }
                if (ok && tc::elect_one()) tc::mma_commit_pair(&accf[acc]);   // accumulators complete in both CTAs
                __syncwarp();
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue (both CTAs)
        const int q = warp & 3;                              // TMEM lanes [32q, 32q+32) belong to this warp
        const uint32_t acce0 = tc::mapa(tc::smem_u32(&acce[0]), 0);
        uint8_t* my_stage = staging + (size_t)q * kBufsPerWarp * kStageBufBytes;
        constexpr int CH = OUT_BF16 ? 64 : 32;               // columns per staging buffer (128 bytes per row)
        uint32_t tl = 0, nst = 0, eph = 0;
        bool meet_ok = true;
        auto meet = [&]() -> bool {                          // the four epilogue warps, bounded (unlike a named barrier)
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(ebar);
            const bool met = tc::mbar_wait(ebar, eph);
            eph ^= 1u;
            return !__any_sync(0xffffffffu, !met);
        };
        for (long long t = first; t < total; t += step, ++tl) {
            const int m_blk = (int)(t / a.num_n), n_blk = (int)(t % a.num_n);
            const uint32_t acc = tl & 1u, aph = (tl >> 1) & 1u;
            if (!tc::wait_uniform(&accf[acc], aph, abort_flag)) { if (lane == 0) fail(FREE_DEV_ERR_ACC_FULL); break; }
            tc::tc_fence_after();
            const int row0 = m_blk * 256 + (int)rank * 128 + q * 32;
            const int row = row0 + lane;
            const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16) + acc * (uint32_t)BN;
            if (EPI == EPI_QKV_HEADS) {
#pragma unroll 1
                for (int c0 = 0; c0 < BN && n_blk * BN + c0 < a.N; c0 += 32) {
                    uint32_t r[32];
                    tc::tmem_ld32(t_addr + (uint32_t)c0, r);
                    tc::tmem_wait_ld();
                    if (row < a.M) {
                        const int n0 = n_blk * BN + c0;
                        float v[32];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const float4 b = __ldg(reinterpret_cast<const float4*>(a.bias + n0) + i);
                            v[4 * i + 0] = __uint_as_float(r[4 * i + 0]) + b.x; v[4 * i + 1] = __uint_as_float(r[4 * i + 1]) + b.y;
                            v[4 * i + 2] = __uint_as_float(r[4 * i + 2]) + b.z; v[4 * i + 3] = __uint_as_float(r[4 * i + 3]) + b.w;
                        }
                        scatter_qkv(a, row, n0, v);
                    }
                }
            } else if (EPI == EPI_QKV_TOKV && n_blk * BN >= 2 * a.heads * a.d_head) {
                // ---- a column block of v: transposed through shared memory into v^T [seq*heads*d_pad, n_tok]
                // (mapV: box 128 tokens x 8 rows).  The CTA's 128 rows are 128 consecutive tokens of one sequence.
                const int etid = q * 32 + lane;                         // row of the CTA tile = TMEM lane
                const int row_base = m_blk * 256 + (int)rank * 128;
                const bool live = row_base < a.M;
                const int seq = live ? row_base / a.n_tok : 0, tok0 = live ? row_base % a.n_tok : 0;
                // stores of the previous tile (which may have used the per-warp buffers) must have read their source
                if (lane == 0) tc::bulk_wait_read<0>();
                meet_ok = meet();
                if (!meet_ok) { if (lane == 0) fail(FREE_DEV_ERR_ACC_FULL); break; }
#pragma unroll 1
                for (int c0 = 0; c0 < BN && n_blk * BN + c0 < a.N; c0 += 32) {
                    const int n0 = n_blk * BN + c0;
                    uint32_t r[32];
                    tc::tmem_ld32(t_addr + (uint32_t)c0, r);
                    tc::tmem_wait_ld();
                    uint8_t* buf = staging + (nst % 3u) * kVBufBytes;   // rewritten three chunks later, after two meetings
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float4 b = __ldg(reinterpret_cast<const float4*>(a.bias + n0) + i);
                        const float v0 = __uint_as_float(r[4 * i + 0]) + b.x, v1 = __uint_as_float(r[4 * i + 1]) + b.y;
                        const float v2 = __uint_as_float(r[4 * i + 2]) + b.z, v3 = __uint_as_float(r[4 * i + 3]) + b.w;
                        uint8_t* gp = buf + (i >> 1) * 2048 + (i & 1) * 1024 + etid * 2;      // [group][column][token]
                        *reinterpret_cast<__nv_bfloat16*>(gp) = __float2bfloat16(v0);
                        *reinterpret_cast<__nv_bfloat16*>(gp + 256) = __float2bfloat16(v1);
                        *reinterpret_cast<__nv_bfloat16*>(gp + 512) = __float2bfloat16(v2);
                        *reinterpret_cast<__nv_bfloat16*>(gp + 768) = __float2bfloat16(v3);
                    }
                    tc::fence_proxy_async();
                    meet_ok = meet();
                    if (!meet_ok) { if (lane == 0) fail(FREE_DEV_ERR_ACC_FULL); break; }
                    if (lane == 0) {                                    // each warp issues one of the four groups
                        if (live) {
                            const int g = warp - 2;
                            const int vc = n0 + 8 * g - 2 * a.heads * a.d_head;
                            const int hd = vc / a.d_head, c = vc % a.d_head;
                            tc::tma_store_2d(&mapV, tc::smem_u32(buf + g * 2048), tok0, (seq * a.heads + hd) * a.d_pad + c);
                        }
                        tc::bulk_commit();
                        tc::bulk_wait_read<1>();
                    }
                    ++nst;
                }
                if (!meet_ok) break;
                // the next tile may use the per-warp buffers: this tile's stores must have read theirs first
                if (lane == 0) tc::bulk_wait_read<0>();
                meet_ok = meet();
                if (!meet_ok) { if (lane == 0) fail(FREE_DEV_ERR_ACC_FULL); break; }
            } else {
                const int rowc = row < a.M ? row : a.M - 1;
                const float* gp = (EPI == EPI_GATE_RESIDUAL && a.gate) ? a.gate + (long long)(rowc / a.rows_per_seq) * a.gate_stride : nullptr;
#pragma unroll 1
                for (int c0 = 0; c0 < BN && n_blk * BN + c0 < a.N; c0 += CH) {
                    const int n0 = n_blk * BN + c0;
                    float v[CH];
#pragma unroll
                    for (int h = 0; h < CH / 32; ++h) {
                        uint32_t r[32];
                        tc::tmem_ld32(t_addr + (uint32_t)(c0 + 32 * h), r);
                        tc::tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[32 * h + i] = __uint_as_float(r[i]);
                    }
                    if (a.bias) {
#pragma unroll
                        for (int i = 0; i < CH / 4; ++i) {
                            const float4 b = __ldg(reinterpret_cast<const float4*>(a.bias + n0) + i);
                            v[4 * i + 0] += b.x; v[4 * i + 1] += b.y; v[4 * i + 2] += b.z; v[4 * i + 3] += b.w;
                        }
                    }
                    if (EPI == EPI_BIAS_GELU) {
#pragma unroll
                        for (int i = 0; i < CH; ++i) v[i] = gelu_fast(v[i]);
                    }
                    if (EPI == EPI_GATE_RESIDUAL && gp) {
                        const bool gvec = (reinterpret_cast<uintptr_t>(gp + n0) & 15u) == 0;
#pragma unroll
                        for (int i = 0; i < CH / 4; ++i) {
                            float4 g;
                            if (gvec) g = __ldg(reinterpret_cast<const float4*>(gp + n0) + i);
                            else g = make_float4(__ldg(gp + n0 + 4 * i), __ldg(gp + n0 + 4 * i + 1), __ldg(gp + n0 + 4 * i + 2), __ldg(gp + n0 + 4 * i + 3));
                            v[4 * i + 0] *= g.x; v[4 * i + 1] *= g.y; v[4 * i + 2] *= g.z; v[4 * i + 3] *= g.w;
                        }
                    }
                    // stage the 32 x 128-byte block (16-byte units XOR-swizzled by row, as the tensor map expects)
                    uint8_t* buf = my_stage + (nst % kBufsPerWarp) * kStageBufBytes;
                    if (lane == 0) tc::bulk_wait_read<kBufsPerWarp - 1>();   // the store issued from this buffer kBufsPerWarp chunks ago has read it
                    __syncwarp();
                    uint8_t* rowp = buf + lane * 128;
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        uint4 w;
                        if (OUT_BF16) w = pack8(v + 8 * u);
                        else w = make_uint4(__float_as_uint(v[4 * u]), __float_as_uint(v[4 * u + 1]), __float_as_uint(v[4 * u + 2]), __float_as_uint(v[4 * u + 3]));
                        *reinterpret_cast<uint4*>(rowp + ((u ^ (lane & 7)) << 4)) = w;
                    }
                    tc::fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) {
                        if (row0 < a.M) {                                // rows past M inside the box are clipped by the TMA unit
                            if (EPI == EPI_GATE_RESIDUAL) tc::tma_reduce_add_2d(&mapO, tc::smem_u32(buf), n0, row0);
                            else tc::tma_store_2d(&mapO, tc::smem_u32(buf), n0, row0);
                        }
                        tc::bulk_commit();
                    }
                    ++nst;
                }
            }
            tc::tc_fence_before();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive_cluster(acce0 + 8u * acc);
        }
        if (lane == 0) tc::bulk_wait<0>();                   // every store of this warp complete before the CTA ends
        __syncwarp();
    }
    // ---------------------------------------------------------------------- teardown
    tc::tc_fence_before();
    tc::cluster_sync_all();                                  // the peer may still read this CTA's shared memory until here
    if (warp == 1) { tc::tc_fence_after(); tc::tmem_dealloc_pair(tmem_base, kTmemCols); }
}

int sm_count() {
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 2) n = 148;
    }
    return n;
}

template <int EPI, bool OUT_BF16, int BN>
int launch(const CUtensorMap& mA, const CUtensorMap& mW, const CUtensorMap& mWl, const CUtensorMap& mO, const CUtensorMap& mV,
           const Tc2Args& a, size_t smem, cudaStream_t s) {
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [&] {
        attr_err = cudaFuncSetAttribute(linear_tc2_kernel<EPI, OUT_BF16, BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget);
    });
    if (attr_err != cudaSuccess) return FREE_ERR_CUDA;
    const long long tiles = (long long)a.num_m * a.num_n;
    const long long pairs = sm_count() / 2;
    const int grid = 2 * (int)(tiles < pairs ? tiles : pairs);
    return free_launch(free_overlap_for_rows(a.M), linear_tc2_kernel<EPI, OUT_BF16, BN>, dim3(grid), dim3(kThreads), smem, s, mA, mW, mWl, mO, mV, a);
}

template <int BN>
int dispatch(const LinearArgs& l, Tc2Args a, cudaStream_t s) {
    constexpr uint32_t stage_bytes = kABytes + (BN / 2) * BK * 2;
    a.stages = (int)((kSmemBudget - 1024 - kCtrlBytes - kStagingBytes) / stage_bytes);
    if (a.stages > kMaxStages) a.stages = kMaxStages;
    a.num_m = (l.M + 255) / 256; a.num_n = (l.N + BN - 1) / BN;
    const size_t smem = 1024 + kCtrlBytes + kStagingBytes + (size_t)a.stages * stage_bytes;
    const long long lda = l.lda ? l.lda : l.K, ldw = l.ldw ? l.ldw : l.K, ldo = l.ldo ? l.ldo : l.N;
    CUtensorMap mA, mW, mO;
    FREE_TRY(free_tensor_map_2d(&mA, l.A, (uint64_t)l.K, (uint64_t)l.M, (uint64_t)lda * 2, BK, 128, 128));
    FREE_TRY(free_tensor_map_2d(&mW, l.W, (uint64_t)l.K, (uint64_t)l.N, (uint64_t)ldw * 2, BK, BN / 2, 128));
    a.last_n = l.N - (a.num_n - 1) * BN;                 // 64, 128, 192 or BN (N is a multiple of 64)
    CUtensorMap mWl = mW;
    if (a.last_n < BN) FREE_TRY(free_tensor_map_2d(&mWl, l.W, (uint64_t)l.K, (uint64_t)l.N, (uint64_t)ldw * 2, BK, (uint32_t)a.last_n / 2, 128));
    const bool ob = l.out_dtype == FREE_BF16;
    switch (l.epi) {
        case EPI_BIAS:
            FREE_TRY(free_tensor_map_2d_typed(&mO, ob ? 2 : 4, l.out, (uint64_t)l.N, (uint64_t)l.M, (uint64_t)ldo * (ob ? 2 : 4), ob ? 64 : 32, 32, 128));
            return ob ? launch<EPI_BIAS, true, BN>(mA, mW, mWl, mO, mO, a, smem, s) : launch<EPI_BIAS, false, BN>(mA, mW, mWl, mO, mO, a, smem, s);
        case EPI_BIAS_GELU:
            FREE_TRY(free_tensor_map_2d_typed(&mO, 2, l.out, (uint64_t)l.N, (uint64_t)l.M, (uint64_t)ldo * 2, 64, 32, 128));
            return launch<EPI_BIAS_GELU, true, BN>(mA, mW, mWl, mO, mO, a, smem, s);
        case EPI_GATE_RESIDUAL:
            FREE_TRY(free_tensor_map_2d_typed(&mO, 4, l.resid, (uint64_t)l.N, (uint64_t)l.M, (uint64_t)l.N * 4, 32, 32, 128));
            return launch<EPI_GATE_RESIDUAL, false, BN>(mA, mW, mWl, mO, mO, a, smem, s);
        case EPI_QKV_HEADS:
            mO = mA;                                         // unused by this variant
            return launch<EPI_QKV_HEADS, true, BN>(mA, mW, mWl, mO, mO, a, smem, s);
        case EPI_QKV_TOKV: {
            CUtensorMap mV;
            const int qk_cols = 2 * l.heads * l.d_head;
            FREE_TRY(free_tensor_map_2d_typed(&mO, 2, l.out, (uint64_t)qk_cols, (uint64_t)l.M, (uint64_t)ldo * 2, 64, 32, 128));
            FREE_TRY(free_tensor_map_2d_typed(&mV, 2, l.vt, (uint64_t)l.n_tok, (uint64_t)(l.M / l.n_tok) * l.heads * l.d_pad,
                                              (uint64_t)l.n_tok * 2, 128, 8, 0));
            return launch<EPI_QKV_TOKV, true, BN>(mA, mW, mWl, mO, mV, a, smem, s);
        }
        default:
            return FREE_ERR_UNSUPPORTED;
    }
}

}  // namespace

// Shapes and epilogues the pair kernel takes; everything else stays on the single-CTA kernel.
bool linear_bf16_pair_eligible(const LinearArgs& l) {
    if ((l.M <= 128 && l.epi != EPI_QKV_TOKV) || l.K < BK || l.K % BK) return false;
    if (l.N < 256 || l.N % 64) return false;            // column chunks of the epilogue are 64 wide
    switch (l.epi) {
        case EPI_BIAS: return l.out != nullptr;
        case EPI_BIAS_GELU: return l.out != nullptr && l.out_dtype == FREE_BF16;
        case EPI_GATE_RESIDUAL: return l.resid != nullptr;
        case EPI_QKV_HEADS: return l.bias != nullptr;
        case EPI_QKV_TOKV:                                   // column blocks are wholly q/k or wholly v; 128-row blocks lie in one sequence
            return l.bias != nullptr && (2 * l.heads * l.d_head) % 256 == 0 && l.n_tok % 128 == 0;
        default: return false;
    }
}

// Arguments have been validated by linear_bf16().
int linear_bf16_pair(const LinearArgs& l, cudaStream_t s) {
    Tc2Args a{};
    a.M = l.M; a.N = l.N; a.K = l.K;
    a.bias = l.bias;
    a.gate = l.gate; a.gate_stride = l.gate_stride; a.rows_per_seq = l.rows_per_seq > 0 ? l.rows_per_seq : 1;
    a.heads = l.heads; a.d_head = l.d_head; a.d_pad = l.d_pad; a.n_tok = l.n_tok;
    a.q = (__nv_bfloat16*)l.q; a.k = (__nv_bfloat16*)l.k; a.vt = (__nv_bfloat16*)l.vt;
    a.err = l.err;
    // Column blocks of 256 keep the tensor core busiest, but few row blocks leave clusters idle in the last (or only) wave:
    // 2048 rows x 1152 columns are 40 tiles on 74 clusters.  Blocks of 128 columns make twice as many tiles.  A narrow
    // tile's K loop runs at the shared-memory limit (0.73 of a wide tile's, measured) and its epilogue takes half as long;
    // with the epilogue of a wide tile worth about 1024 elements of K, the relative time of a narrow tile is
    // (0.73 K + 0.5 * 1024) / (K + 1024): 0.62 at K = 1152, 0.69 at K = 4608 (measured: 12288 x 1152 x 1152 is 8% faster
    // narrow, 24576 x 1152 x 1152 5% slower, 12288 x 1152 x 4608 9% slower, 2048 and 4096 x 1152 x 4608 23% faster).
    // Narrow blocks are taken when waves x relative tile time is shorter; only
    // for the epilogues whose column chunks do not care about the block width.
    const bool narrow_ok = (l.epi == EPI_GATE_RESIDUAL || l.epi == EPI_BIAS || l.epi == EPI_BIAS_GELU) && l.N % 128 == 0;
    if (narrow_ok) {
        const long long pairs = sm_count() / 2, num_m = (l.M + 255) / 256;
        const long long wide = num_m * ((l.N + 255) / 256), narrow = num_m * (l.N / 128);
        const double rel = (0.73 * l.K + 0.5 * 1024.0) / ((double)l.K + 1024.0);
        const double t_wide = (double)((wide + pairs - 1) / pairs), t_narrow = rel * (double)((narrow + pairs - 1) / pairs);
        if (t_narrow < t_wide) return dispatch<128>(l, a, s);
    }
    return dispatch<256>(l, a, s);
}
