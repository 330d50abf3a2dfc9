// bf16 linear layers on the 5th-generation tensor cores.
//
//   out = epilogue(A[M,K] * W[N,K]^T + bias),   A and W bf16 (K contiguous), fp32 accumulation in TMEM.
//
// Persistent, warp-specialised kernel, one CTA per SM:
//   warp 0     TMA producer: 128 x 64 tiles of A and BN x 64 tiles of W into a ring of shared-memory
//              stages (128-byte swizzle), completion counted on an mbarrier per stage;
//   warp 1     MMA issuer: one thread issues tcgen05.mma (128 x BN x 16 per instruction) straight from shared
//              memory into one of two TMEM accumulators, and commits stage-release / accumulator-ready barriers;
//   warps 2-5  epilogue: tcgen05.ld of the finished accumulator (each warp owns one 32-lane quarter of TMEM),
//              fused bias / GELU / SiLU / gated residual / head-major QKV scatter, direct global stores.
//              It overlaps the MMAs of the next tile through the second accumulator.
// Tile order: each CTA keeps one 128-row block of A and walks the N blocks, so the A rows of a band of
// SM-count row blocks stay in L2 while the (small) weight matrix is re-read from L2.
#include "internal.h"
#include "tc_common.cuh"
#include <mutex>

namespace {

constexpr int BM = 128, BK = 64;
constexpr int kThreads = 192;
constexpr int kMaxStages = 8;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kABytes = BM * BK * 2;
constexpr uint32_t kCtrlBytes = 1024;
constexpr uint32_t kSmemBudget = 227 * 1024;

struct TcArgs {
    int M, N, K, BN, stages, num_m, num_n;
    const float* bias;
    void* out; long long ldo;
    float* resid; const float* gate; long long gate_stride; int rows_per_seq;
    const float* emb; const int32_t* emb_idx;
    int heads, d_head, d_pad, n_tok;
    __nv_bfloat16 *q, *k, *vt;
    int img_C, img_H, img_W, img_p;
    uint32_t* err;
};

struct TileIter {            // static schedule shared by the three roles
    int num_m, num_n, G, full_bands, rem;
    long long total, full_tiles;
    __device__ TileIter(int nm, int nn, int g) : num_m(nm), num_n(nn), G(g) {
        full_bands = nm / g; rem = nm % g;
        full_tiles = (long long)full_bands * g * nn;
        total = (long long)nm * nn;
    }
    __device__ void coords(long long t, int& m_blk, int& n_blk) const {
        if (t < full_tiles) {
            const long long per = (long long)G * num_n;
            const int band = (int)(t / per), r = (int)(t % per);
            n_blk = r / G; m_blk = band * G + r % G;
        } else {
            const int r = (int)(t - full_tiles);
            n_blk = r / rem; m_blk = full_bands * G + r % rem;
        }
    }
};

__device__ __forceinline__ float tanh_fast(float x) { float y; asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ float gelu_fast(float a) {
    return 0.5f * a * (1.0f + tanh_fast(0.7978845608028654f * (a + 0.044715f * a * a * a)));
}
__device__ __forceinline__ float silu_fast(float a) { return a / (1.0f + __expf(-a)); }

__device__ __forceinline__ uint4 pack8(const float* v) {
    __nv_bfloat162 p0 = __floats2bfloat162_rn(v[0], v[1]), p1 = __floats2bfloat162_rn(v[2], v[3]);
    __nv_bfloat162 p2 = __floats2bfloat162_rn(v[4], v[5]), p3 = __floats2bfloat162_rn(v[6], v[7]);
    uint4 u;
    u.x = *reinterpret_cast<uint32_t*>(&p0); u.y = *reinterpret_cast<uint32_t*>(&p1);
    u.z = *reinterpret_cast<uint32_t*>(&p2); u.w = *reinterpret_cast<uint32_t*>(&p3);
    return u;
}

// One thread: row `row`, columns [n0, n0 + 32) of the output tile, accumulator values in r.
template <int EPI, bool OUT_BF16>
__device__ __forceinline__ void epilogue_chunk(const TcArgs& a, int row, int n0, const uint32_t (&r)[32]) {
    if (row >= a.M) return;
    float v[32];
    if (a.bias) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float4 b = __ldg(reinterpret_cast<const float4*>(a.bias + n0) + i);
            v[4 * i + 0] = __uint_as_float(r[4 * i + 0]) + b.x; v[4 * i + 1] = __uint_as_float(r[4 * i + 1]) + b.y;
            v[4 * i + 2] = __uint_as_float(r[4 * i + 2]) + b.z; v[4 * i + 3] = __uint_as_float(r[4 * i + 3]) + b.w;
        }
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
    }
    if (EPI == EPI_GATE_RESIDUAL) {
        float* rp = a.resid + (long long)row * a.N + n0;
        const float* gp = a.gate ? a.gate + (long long)(row / a.rows_per_seq) * a.gate_stride + n0 : nullptr;
        const bool gvec = gp && ((reinterpret_cast<uintptr_t>(gp) & 15u) == 0);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float4 x = reinterpret_cast<float4*>(rp)[i];
            float4 g = make_float4(1.f, 1.f, 1.f, 1.f);
            if (gvec) g = __ldg(reinterpret_cast<const float4*>(gp) + i);
            else if (gp) g = make_float4(__ldg(gp + 4 * i), __ldg(gp + 4 * i + 1), __ldg(gp + 4 * i + 2), __ldg(gp + 4 * i + 3));
            x.x = fmaf(g.x, v[4 * i + 0], x.x); x.y = fmaf(g.y, v[4 * i + 1], x.y);
            x.z = fmaf(g.z, v[4 * i + 2], x.z); x.w = fmaf(g.w, v[4 * i + 3], x.w);
            reinterpret_cast<float4*>(rp)[i] = x;
        }
        return;
    }
    if (EPI == EPI_QKV_HEADS) {
        const int D = a.heads * a.d_head, dh = a.d_head, dp = a.d_pad, T = a.n_tok;
        const int seq = row / T, tok = row % T;
        const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int g = 0; g < 4; ++g) {                   // groups of 8 columns never straddle a head (d_head % 8 == 0)
            const int n = n0 + 8 * g;
            const int which = n / D, hd = (n % D) / dh, c = n % dh;
            const long long sh = (long long)seq * a.heads + hd;
            if (which < 2) {
                __nv_bfloat16* dst = (which == 0 ? a.q : a.k) + (sh * T + tok) * dp + c;
                *reinterpret_cast<uint4*>(dst) = pack8(v + 8 * g);
                if (c + 8 == dh)
                    for (int z = dh; z < dp; z += 8) *reinterpret_cast<uint4*>(dst + (z - c)) = zero;   // zero the K padding
            } else {
                __nv_bfloat16* dst = a.vt + (sh * dp + c) * T + tok;
#pragma unroll
                for (int i = 0; i < 8; ++i) dst[(long long)i * T] = __float2bfloat16(v[8 * g + i]);
                if (c + 8 == dh)
                    for (int z = dh; z < dp; ++z) a.vt[(sh * dp + z) * T + tok] = __float2bfloat16(0.f);
            }
        }
        return;
    }
    if (EPI == EPI_UNPATCH || EPI == EPI_UNPATCH_ACC) {
        // the thread's token: its patch is p rows of p pixels per channel; consecutive threads hold consecutive tokens of a
        // patch row, so that the stores of a warp to one image row are contiguous
        const int p = a.img_p, gw = a.img_W / p, pp = p * p;
        const int seq = row / a.n_tok, tok = row % a.n_tok, trow = tok / gw, tcol = tok % gw;
        float* img = reinterpret_cast<float*>(a.out) + (long long)seq * a.img_C * a.img_H * a.img_W;
        if (p == 2) {
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
                const int n = n0 + i, ch = n >> 2, pr = (n >> 1) & 1;
                if (ch < a.img_C) {
                    float2* dst = reinterpret_cast<float2*>(img + ((long long)ch * a.img_H + trow * 2 + pr) * a.img_W + tcol * 2);
                    float2 o = make_float2(v[i], v[i + 1]);
                    if (EPI == EPI_UNPATCH_ACC) { const float2 old = *dst; o.x += old.x; o.y += old.y; }
                    *dst = o;
                }
            }
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const int n = n0 + i, ch = n / pp, pr = (n % pp) / p, pc = n % p;
                if (ch < a.img_C) {
                    float* dst = img + ((long long)ch * a.img_H + trow * p + pr) * a.img_W + tcol * p + pc;
                    *dst = (EPI == EPI_UNPATCH_ACC ? *dst : 0.f) + v[i];
                }
            }
        }
        return;
    }
    if (EPI == EPI_BIAS_GELU) {
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = gelu_fast(v[i]);
    } else if (EPI == EPI_BIAS_SILU) {
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = silu_fast(v[i]);
    } else if (EPI == EPI_BIAS_EMB_SILU) {
        const float* e = a.emb + (long long)a.emb_idx[row] * a.N + n0;
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = silu_fast(v[i] + __ldg(e + i));
    }
    if (OUT_BF16) {
        uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(a.out) + (long long)row * a.ldo + n0);
#pragma unroll
        for (int g = 0; g < 4; ++g) dst[g] = pack8(v + 8 * g);
    } else {
        float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(a.out) + (long long)row * a.ldo + n0);
#pragma unroll
        for (int g = 0; g < 8; ++g) dst[g] = make_float4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
    }
}

template <int EPI, bool OUT_BF16>
__global__ void __launch_bounds__(kThreads, 1)
linear_tc_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapW, const TcArgs a) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem);
    uint64_t* empty = full + kMaxStages;
    uint64_t* accf = empty + kMaxStages;
    uint64_t* acce = accf + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acce + 2);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    uint8_t* tiles = smem + kCtrlBytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int BN = a.BN, stages = a.stages, nk = a.K / BK;
    const uint32_t b_bytes = (uint32_t)BN * BK * 2, stage_bytes = kABytes + b_bytes;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], 1); }
        for (int i = 0; i < 2; ++i) { tc::mbar_init(&accf[i], 1); tc::mbar_init(&acce[i], 4); }
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::fence_proxy_async();
    }
    if (warp == 1) { tc::tmem_alloc(tmem_slot, kTmemCols); tc::tmem_relinquish(); }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const TileIter sched(a.num_m, a.num_n, (int)gridDim.x);
    auto fail = [&](uint32_t code) { *abort_flag = 1; atomicOr(a.err, code); };

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            tc::tma_prefetch_desc(&mapA);
            tc::tma_prefetch_desc(&mapW);
            uint32_t it = 0;
            bool ok = true;
            for (long long t = blockIdx.x; ok && t < sched.total; t += gridDim.x) {
                int m_blk, n_blk;
                sched.coords(t, m_blk, n_blk);
                for (int kb = 0; kb < nk; ++kb, ++it) {
                    const int s = it % stages;
                    const uint32_t ph = (it / stages) & 1u;
                    if (*abort_flag || !tc::mbar_wait(&empty[s], ph ^ 1u)) { fail(FREE_DEV_ERR_EMPTY_WAIT); ok = false; break; }
                    uint8_t* st = tiles + (size_t)s * stage_bytes;
                    tc::mbar_expect_tx(&full[s], stage_bytes);
                    tc::tma_load_2d(st, &mapA, &full[s], kb * BK, m_blk * BM);
                    tc::tma_load_2d(st + kABytes, &mapW, &full[s], kb * BK, n_blk * BN);
                }
            }
            if (!ok || *abort_flag) {
                // loads already issued must land before the shared memory is given back
                const uint32_t n_back = it < (uint32_t)stages ? it : (uint32_t)stages;
                for (uint32_t j = it - n_back; j < it; ++j) tc::mbar_wait(&full[j % stages], (j / stages) & 1u, 100000000ll);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = tc::idesc_bf16(BM, BN);
            uint32_t it = 0, tl = 0;
            bool ok = true;
            for (long long t = blockIdx.x; ok && t < sched.total; t += gridDim.x, ++tl) {
                const uint32_t acc = tl & 1u, aph = (tl >> 1) & 1u;
                if (*abort_flag || !tc::mbar_wait(&acce[acc], aph ^ 1u)) { fail(FREE_DEV_ERR_ACC_EMPTY); ok = false; break; }
                tc::tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * (uint32_t)BN;
                for (int kb = 0; kb < nk; ++kb, ++it) {
                    const int s = it % stages;
                    const uint32_t ph = (it / stages) & 1u;
                    if (*abort_flag || !tc::mbar_wait(&full[s], ph)) { fail(FREE_DEV_ERR_FULL_WAIT); ok = false; break; }
                    tc::tc_fence_after();
                    const uint32_t a_addr = tc::smem_u32(tiles + (size_t)s * stage_bytes), b_addr = a_addr + kABytes;
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        tc::mma_bf16(d_tmem, tc::smem_desc(a_addr + k * 32, 1024, 2), tc::smem_desc(b_addr + k * 32, 1024, 2),
                                     idesc, (kb | k) != 0 ? 1u : 0u);
                    tc::mma_commit(&empty[s]);           // stage reusable once these MMAs have read it
                }
                if (ok) tc::mma_commit(&accf[acc]);      // accumulator complete
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue
        const int q = warp & 3;                          // TMEM lanes [32q, 32q+32) belong to this warp
        uint32_t tl = 0;
        for (long long t = blockIdx.x; t < sched.total; t += gridDim.x, ++tl) {
            int m_blk, n_blk;
            sched.coords(t, m_blk, n_blk);
            const uint32_t acc = tl & 1u, aph = (tl >> 1) & 1u;
            const bool bad = *abort_flag || !tc::mbar_wait(&accf[acc], aph);
            if (__any_sync(0xffffffffu, bad)) { if (lane == 0) fail(FREE_DEV_ERR_ACC_FULL); break; }   // warp-uniform exit
            tc::tc_fence_after();
            const int row = m_blk * BM + q * 32 + lane;
            const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16) + acc * (uint32_t)BN;
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t r[32];
                tc::tmem_ld32(t_addr + (uint32_t)c0, r);
                tc::tmem_wait_ld();
                epilogue_chunk<EPI, OUT_BF16>(a, row, n_blk * BN + c0, r);
            }
            tc::tc_fence_before();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&acce[acc]);
        }
    }
    // ---------------------------------------------------------------------- teardown
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 1) { tc::tc_fence_after(); tc::tmem_dealloc(tmem_base, kTmemCols); }
}

int pick_bn(int N) {
    for (int bn : {256, 192, 128, 224, 160, 96, 64, 32})
        if (N % bn == 0) return bn;
    return 0;
}

int sm_count() {
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
    }
    return n;
}

template <int EPI, bool OUT_BF16>
int launch(const CUtensorMap& mA, const CUtensorMap& mW, const TcArgs& a, size_t smem, cudaStream_t s) {
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [&] {
        attr_err = cudaFuncSetAttribute(linear_tc_kernel<EPI, OUT_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget);
    });
    if (attr_err != cudaSuccess) return FREE_ERR_CUDA;
    const long long tiles = (long long)a.num_m * a.num_n;
    const int grid = (int)(tiles < sm_count() ? tiles : sm_count());
    linear_tc_kernel<EPI, OUT_BF16><<<grid, kThreads, smem, s>>>(mA, mW, a);
    return free_check_launch();
}

}  // namespace

bool linear_bf16_supported(int N, int K) { return N >= 32 && N % 32 == 0 && K >= 64 && K % 64 == 0; }

// Per-epilogue argument checks shared by the single-CTA and the CTA-pair kernels.
static int validate_epilogue(const LinearArgs& l, long long ldo) {
    switch (l.epi) {
        case EPI_BIAS: case EPI_BIAS_GELU: case EPI_BIAS_SILU:
            return (!l.out || !free_aligned16(l.out) || ldo % 8) ? FREE_ERR_ARG : FREE_OK;
        case EPI_BIAS_EMB_SILU:
            return (!l.out || !l.emb || !l.emb_idx || !free_aligned16(l.out) || ldo % 8) ? FREE_ERR_ARG : FREE_OK;
        case EPI_GATE_RESIDUAL:
            return (!l.resid || !free_aligned16(l.resid)) ? FREE_ERR_ARG : FREE_OK;
        case EPI_QKV_HEADS:
            return (!l.q || !l.k || !l.vt || l.heads < 1 || l.d_head % 8 || l.d_pad % 8 || l.d_pad < l.d_head || l.n_tok < 1 ||
                    l.N != 3 * l.heads * l.d_head || l.M % l.n_tok) ? FREE_ERR_ARG : FREE_OK;
        case EPI_QKV_TOKV:
            return (!l.out || !l.vt || !free_aligned16(l.out) || ldo % 8 || l.heads < 1 || l.d_head % 8 || l.d_pad % 8 || l.d_pad < l.d_head ||
                    l.n_tok < 1 || l.N != 3 * l.heads * l.d_head || l.M % l.n_tok) ? FREE_ERR_ARG : FREE_OK;
        case EPI_UNPATCH: case EPI_UNPATCH_ACC:
            return (!l.out || !free_aligned16(l.out) || l.out_dtype != FREE_FP32 || l.img_p < 1 || l.img_C < 1 || l.img_H % l.img_p ||
                    l.img_W % l.img_p || l.n_tok != (l.img_H / l.img_p) * (l.img_W / l.img_p) || l.M % l.n_tok ||
                    l.N < l.img_C * l.img_p * l.img_p) ? FREE_ERR_ARG : FREE_OK;
        default:
            return FREE_ERR_ARG;
    }
}

int linear_bf16(const LinearArgs& l, cudaStream_t s) {
    if (l.M < 1 || !l.A || !l.W || !l.err) return FREE_ERR_ARG;
    if (!linear_bf16_supported(l.N, l.K)) return FREE_ERR_UNSUPPORTED;
    const long long lda = l.lda ? l.lda : l.K, ldw = l.ldw ? l.ldw : l.K, ldo = l.ldo ? l.ldo : l.N;
    if (lda % 8 || ldw % 8 || !free_aligned16(l.A) || !free_aligned16(l.W)) return FREE_ERR_ALIGN;
    if (l.bias && !free_aligned16(l.bias)) return FREE_ERR_ALIGN;
    FREE_TRY(validate_epilogue(l, ldo));
    if (linear_bf16_pair_eligible(l)) return linear_bf16_pair(l, s);       // the large GEMMs: 256 x BN tiles on CTA pairs
    if (l.epi == EPI_QKV_TOKV) return FREE_ERR_UNSUPPORTED;                // only the pair kernel has this epilogue
    TcArgs a{};
    a.M = l.M; a.N = l.N; a.K = l.K;
    a.BN = pick_bn(l.N);
    if (a.BN == 0) return FREE_ERR_UNSUPPORTED;
    const uint32_t stage_bytes = kABytes + (uint32_t)a.BN * BK * 2;
    a.stages = (int)((kSmemBudget - 1024 - kCtrlBytes) / stage_bytes);
    if (a.stages > kMaxStages) a.stages = kMaxStages;
    if (a.stages < 2) return FREE_ERR_UNSUPPORTED;
    a.num_m = (l.M + BM - 1) / BM; a.num_n = l.N / a.BN;
    a.bias = l.bias; a.out = l.out; a.ldo = ldo;
    a.resid = l.resid; a.gate = l.gate; a.gate_stride = l.gate_stride; a.rows_per_seq = l.rows_per_seq > 0 ? l.rows_per_seq : 1;
    a.emb = l.emb; a.emb_idx = l.emb_idx;
    a.heads = l.heads; a.d_head = l.d_head; a.d_pad = l.d_pad; a.n_tok = l.n_tok;
    a.q = (__nv_bfloat16*)l.q; a.k = (__nv_bfloat16*)l.k; a.vt = (__nv_bfloat16*)l.vt;
    a.img_C = l.img_C; a.img_H = l.img_H; a.img_W = l.img_W; a.img_p = l.img_p;
    a.err = l.err;
    const size_t smem = 1024 + kCtrlBytes + (size_t)a.stages * stage_bytes;

    CUtensorMap mA, mW;
    FREE_TRY(free_tensor_map_2d(&mA, l.A, (uint64_t)l.K, (uint64_t)l.M, (uint64_t)lda * 2, BK, BM, 128));
    FREE_TRY(free_tensor_map_2d(&mW, l.W, (uint64_t)l.K, (uint64_t)l.N, (uint64_t)ldw * 2, BK, (uint32_t)a.BN, 128));

    const bool ob = l.out_dtype == FREE_BF16;
    switch (l.epi) {
        case EPI_BIAS:
            return ob ? launch<EPI_BIAS, true>(mA, mW, a, smem, s) : launch<EPI_BIAS, false>(mA, mW, a, smem, s);
        case EPI_BIAS_GELU:
            return ob ? launch<EPI_BIAS_GELU, true>(mA, mW, a, smem, s) : launch<EPI_BIAS_GELU, false>(mA, mW, a, smem, s);
        case EPI_BIAS_SILU:
            return ob ? launch<EPI_BIAS_SILU, true>(mA, mW, a, smem, s) : launch<EPI_BIAS_SILU, false>(mA, mW, a, smem, s);
        case EPI_BIAS_EMB_SILU:
            return ob ? launch<EPI_BIAS_EMB_SILU, true>(mA, mW, a, smem, s) : launch<EPI_BIAS_EMB_SILU, false>(mA, mW, a, smem, s);
        case EPI_GATE_RESIDUAL:
            return launch<EPI_GATE_RESIDUAL, false>(mA, mW, a, smem, s);
        case EPI_QKV_HEADS:
            return launch<EPI_QKV_HEADS, true>(mA, mW, a, smem, s);
        case EPI_UNPATCH:
            return launch<EPI_UNPATCH, false>(mA, mW, a, smem, s);
        case EPI_UNPATCH_ACC:
            return launch<EPI_UNPATCH_ACC, false>(mA, mW, a, smem, s);
        default:
            return FREE_ERR_ARG;
    }
}
