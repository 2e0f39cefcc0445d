// S2-Attn forward for sm_100a.
//
// One CTA computes one 128-row query tile of one (batch, head, group): steps "roll", "group",
// "attention" and "roll back" of Algorithm 1 collapse into the choice of TMA coordinates.  Query
// tile i of rolled group g in a head with shift s covers ORIGINAL tokens
// ((g*G + i*128 + s) mod N) .. +127 (s and G are multiples of 128, so a tile never straddles the
// sequence end); its keys are tiles 0..i of the same group, fetched at their own original
// positions -- for the wrapped last group of a shifted head that is the range [N-G/2, N) followed
// by [0, G/2).  Outputs are stored at the original token rows, which is the roll back.
//
// Warp roles (192 threads): warp 0 issues TMA loads, warp 1 owns tensor memory and issues the
// tcgen05 MMAs, warps 2-5 hold one score row per thread (tcgen05.ld 32x32b) and run the online
// softmax.  S = Q K^T accumulates in tensor memory, P (bf16) is written back over S and used as the
// tensor-memory A operand of O += P V; O stays in tensor memory until the epilogue.  Two CTAs fit
// on one SM, so one CTA's softmax overlaps the other CTA's MMAs.
#include "s2a_params.h"
#include "sm100_ptx.cuh"

namespace s2a {

namespace {

template <int HD>
struct FwdCfg {
    static constexpr int kThreads = 192;
    static constexpr int kBoxes = HD / 64;                      // 64-column TMA boxes per tile
    static constexpr int kBoxBytes = kTile * 128;               // 128 rows x 128 bytes
    static constexpr int kTileBytes = kBoxes * kBoxBytes;       // one Q, K or V tile
    static constexpr int kStages = (HD == 128) ? 1 : 2;         // K/V ring depth
    static constexpr int kBarBytes = 256;
    static constexpr int kSmemBytes = 1024 /* alignment slack */ + (1 + 2 * kStages) * kTileBytes + kBarBytes;
    static constexpr int kTmemCols = 256;                       // S: [0,128)  O: [128, 128+HD)
    static constexpr int kColS = 0;
    static constexpr int kColO = 128;
};

// Threshold (in log2 units) below which a larger running maximum is ignored: P then grows by at
// most 2^8, which bf16 and the fp32 row sum absorb, and O needs no rescale.
constexpr float kLazyRescale = 8.0f;

template <int HD>
__global__ void __launch_bounds__(FwdCfg<HD>::kThreads, 2) s2a_fwd_kernel(const __grid_constant__ FwdParams p) {
    using C = FwdCfg<HD>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem;
    uint8_t* sK = sQ + C::kTileBytes;
    uint8_t* sV = sK + C::kStages * C::kTileBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(sV + C::kStages * C::kTileBytes);
    uint64_t* q_full = bars + 0;
    uint64_t* s_full = bars + 1;
    uint64_t* p_full = bars + 2;
    uint64_t* o_full = bars + 3;
    uint64_t* drain = bars + 4;
    uint64_t* k_full = bars + 5;                 // [kStages]
    uint64_t* k_empty = k_full + C::kStages;     // [kStages]
    uint64_t* v_full = k_empty + C::kStages;     // [kStages]
    uint64_t* v_empty = v_full + C::kStages;     // [kStages]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(v_empty + C::kStages);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    // A bounded wait that expired earlier (in any kernel) leaves the status word set: later CTAs
    // then return at once instead of each running into its own time limit.
    __shared__ int s_poisoned;
    if (threadIdx.x == 0) s_poisoned = *reinterpret_cast<volatile int*>(p.status);
    __syncthreads();
    if (s_poisoned != 0) return;

    // ---- which tile: heaviest query tiles of a group first, groups of one head adjacent -------
    const int Tg = p.geo.tiles_per_group;
    const int it = blockIdx.x % Tg;
    const int unit = blockIdx.x / Tg;
    const int i = Tg - 1 - it;                 // query tile inside the group
    const int g = unit % p.geo.groups;
    const int h = (unit / p.geo.groups) % p.geo.H;
    const int b = unit / (p.geo.groups * p.geo.H);
    const int hk = h / (p.geo.H / p.geo.Hkv);
    const int s = (h < p.geo.n_unshifted) ? 0 : p.geo.shift;
    const int n_kv = i + 1;                    // causal: key tiles 0..i of the same group
    // original token of rolled position x:  (x + s) mod N
    auto orig_token = [&](int rolled) {
        int t = (rolled + s) % p.geo.N;
        return t < 0 ? t + p.geo.N : t;
    };
    const int tq0 = orig_token(g * p.geo.G + i * kTile);

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        mbar_init(s_full, 1);
        mbar_init(p_full, 128);
        mbar_init(o_full, 1);
        mbar_init(drain, 1);
        for (int st = 0; st < C::kStages; ++st) {
            mbar_init(k_full + st, 1);
            mbar_init(k_empty + st, 1);
            mbar_init(v_full + st, 1);
            mbar_init(v_empty + st, 1);
        }
        *abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&p.tm_q);
        tma_prefetch_desc(&p.tm_k);
        tma_prefetch_desc(&p.tm_v);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, C::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const WaitCtx ctx{abort_flag, p.status};

    if (warp == 0) {
        // =========================== TMA producer ============================================
        if (lane == 0) {
            mbar_expect_tx(q_full, C::kTileBytes);
            for (int bx = 0; bx < C::kBoxes; ++bx)
                tma_load_4d(sQ + bx * C::kBoxBytes, &p.tm_q, q_full, bx * 64, h, tq0, b);
            int j = 0;
            for (; j < n_kv; ++j) {
                const int st = j % C::kStages;
                const uint32_t ph = (j / C::kStages) & 1;
                const int tk0 = orig_token(g * p.geo.G + j * kTile);
                if (!mbar_wait(k_empty + st, ph ^ 1, ctx, kWaitFwd + 1)) break;
                mbar_expect_tx(k_full + st, C::kTileBytes);
                for (int bx = 0; bx < C::kBoxes; ++bx)
                    tma_load_4d(sK + st * C::kTileBytes + bx * C::kBoxBytes, &p.tm_k, k_full + st, bx * 64, hk, tk0, b);
                if (!mbar_wait(v_empty + st, ph ^ 1, ctx, kWaitFwd + 2)) break;
                mbar_expect_tx(v_full + st, C::kTileBytes);
                for (int bx = 0; bx < C::kBoxes; ++bx)
                    tma_load_4d(sV + st * C::kTileBytes + bx * C::kBoxBytes, &p.tm_v, v_full + st, bx * 64, hk, tk0, b);
            }
            if (*abort_flag != 0) {
                // let loads that are still in flight land before the CTA gives its memory back
                mbar_wait_drain(q_full, 0);
                for (int jj = (j > C::kStages ? j - C::kStages : 0); jj < j; ++jj) {
                    mbar_wait_drain(k_full + jj % C::kStages, (jj / C::kStages) & 1);
                    mbar_wait_drain(v_full + jj % C::kStages, (jj / C::kStages) & 1);
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // =========================== MMA issuer ==============================================
        if (lane == 0) {
            constexpr uint32_t idesc_s = idesc_bf16(128, 128, 0, 0);  // S = Q K^T   (both K-major)
            constexpr uint32_t idesc_o = idesc_bf16(128, HD, 0, 1);   // O += P V    (V is MN-major)
            const uint32_t tS = tmem_base + C::kColS;
            const uint32_t tO = tmem_base + C::kColO;
            const uint32_t aQ = smem_u32(sQ);
            bool ok = mbar_wait(q_full, 0, ctx, kWaitFwd + 3);
            for (int j = 0; ok && j < n_kv; ++j) {
                const int st = j % C::kStages;
                const uint32_t ph = (j / C::kStages) & 1;
                const uint32_t aK = smem_u32(sK + st * C::kTileBytes);
                const uint32_t aV = smem_u32(sV + st * C::kTileBytes);
                if (!mbar_wait(k_full + st, ph, ctx, kWaitFwd + 4)) break;
                tc_fence_after();
                // The previous P (aliased on S) was consumed by the previous P.V, which precedes
                // this MMA in issue order; the softmax warps finished reading S before that.
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {
                    const uint32_t off = (kk >> 2) * C::kBoxBytes + (kk & 3) * 32;
                    mma_ss(tS, desc_k_major(aQ + off), desc_k_major(aK + off), idesc_s, kk > 0);
                }
                mma_commit(k_empty + st);
                mma_commit(s_full);
                if (!mbar_wait(p_full, j & 1, ctx, kWaitFwd + 5)) break;
                if (!mbar_wait(v_full + st, ph, ctx, kWaitFwd + 6)) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < kTile / 16; ++kk) {
                    mma_ts(tO, tS + kk * 8, desc_mn_major(aV + kk * 2048, C::kBoxBytes), idesc_o, (j > 0) || (kk > 0));
                }
                mma_commit(v_empty + st);
                if (j == n_kv - 1) mma_commit(o_full);
            }
            if (*abort_flag != 0) {
                // MMAs already issued must finish before tensor memory is released
                mma_commit(drain);
                mbar_wait_drain(drain, 0);
            }
        }
        __syncwarp();
    } else {
        // =========================== softmax + epilogue ======================================
        const int quad = warp & 3;             // tensor-memory lane quadrant this warp may access
        const int row = quad * 32 + lane;      // row of the query tile owned by this thread
        const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
        const float c2 = p.scale_log2;
        float m_used = -INFINITY;              // running maximum, already scaled to log2 units
        float l = 0.f;                         // running sum of exp2(s*c2 - m_used)
        bool ok = true;
        for (int j = 0; j < n_kv; ++j) {
            if (!mbar_wait(s_full, j & 1, ctx, kWaitFwd + 7)) { ok = false; break; }
            tc_fence_after();
            uint32_t sreg[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld_32x32(t_row + C::kColS + c * 32, sreg[c]);
            tmem_wait_ld();
            if (j == i) {
                // diagonal tile: key x of the tile is visible to query row r iff x <= r
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (c * 32 + e > row) sreg[c][e] = 0xff800000u;  // -inf
            }
            float mx = -INFINITY;
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
                for (int e = 0; e < 32; ++e) mx = fmaxf(mx, __uint_as_float(sreg[c][e]));
            const float m_new = fmaxf(m_used, mx * c2);
            if (j == 0) {
                m_used = m_new;
            } else {
                const bool need = (m_new - m_used) > kLazyRescale;
                if (__any_sync(0xffffffffu, need)) {
                    // s_full(j) also covers the previous P.V, so O is quiescent here
                    const float alpha = need ? fast_exp2(m_used - m_new) : 1.0f;
                    l *= alpha;
#pragma unroll
                    for (int c = 0; c < HD / 32; ++c) {
                        uint32_t oreg[32];
                        tmem_ld_32x32(t_row + C::kColO + c * 32, oreg);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) oreg[e] = __float_as_uint(__uint_as_float(oreg[e]) * alpha);
                        tmem_st_32x32(t_row + C::kColO + c * 32, oreg);
                    }
                    if (need) m_used = m_new;
                }
            }
            float sum = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t preg[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const float p0 = fast_exp2(fmaf(__uint_as_float(sreg[c][2 * e]), c2, -m_used));
                    const float p1 = fast_exp2(fmaf(__uint_as_float(sreg[c][2 * e + 1]), c2, -m_used));
                    sum += p0 + p1;
                    preg[e] = pack_bf16(p0, p1);
                }
                tmem_st_32x16(t_row + C::kColS + c * 16, preg);
            }
            l += sum;
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(p_full);
        }
        if (ok && mbar_wait(o_full, 0, ctx, kWaitFwd + 8)) {
            tc_fence_after();
            const float inv_l = 1.0f / l;
            const int t = tq0 + row;
            __nv_bfloat16* orow = p.o + ((static_cast<size_t>(b) * p.geo.N + t) * p.geo.H + h) * HD;
#pragma unroll
            for (int c = 0; c < HD / 32; ++c) {
                uint32_t oreg[32];
                tmem_ld_32x32(t_row + C::kColO + c * 32, oreg);
                tmem_wait_ld();
                uint4* dst = reinterpret_cast<uint4*>(orow + c * 32);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    uint4 pk;
                    pk.x = pack_bf16(__uint_as_float(oreg[8 * e + 0]) * inv_l, __uint_as_float(oreg[8 * e + 1]) * inv_l);
                    pk.y = pack_bf16(__uint_as_float(oreg[8 * e + 2]) * inv_l, __uint_as_float(oreg[8 * e + 3]) * inv_l);
                    pk.z = pack_bf16(__uint_as_float(oreg[8 * e + 4]) * inv_l, __uint_as_float(oreg[8 * e + 5]) * inv_l);
                    pk.w = pack_bf16(__uint_as_float(oreg[8 * e + 6]) * inv_l, __uint_as_float(oreg[8 * e + 7]) * inv_l);
                    dst[e] = pk;
                }
            }
            // natural-log sum-exp of the scaled scores
            p.lse[(static_cast<size_t>(b) * p.geo.H + h) * p.geo.N + t] = (m_used + log2f(l)) * 0.6931471805599453f;
        }
    }

    // ---- teardown ------------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, C::kTmemCols);
    }
}

}  // namespace

cudaError_t configure_fwd() {
    cudaError_t e = cudaFuncSetAttribute(s2a_fwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         FwdCfg<64>::kSmemBytes);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(s2a_fwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                FwdCfg<128>::kSmemBytes);
}

cudaError_t launch_fwd(const FwdParams& p, int d, cudaStream_t stream) {
    const long long n_cta = static_cast<long long>(p.geo.B) * p.geo.H * p.geo.groups * p.geo.tiles_per_group;
    const dim3 grid(static_cast<unsigned>(n_cta));
    if (d == 64) {
        s2a_fwd_kernel<64><<<grid, FwdCfg<64>::kThreads, FwdCfg<64>::kSmemBytes, stream>>>(p);
    } else {
        s2a_fwd_kernel<128><<<grid, FwdCfg<128>::kThreads, FwdCfg<128>::kSmemBytes, stream>>>(p);
    }
    return cudaGetLastError();
}

}  // namespace s2a
