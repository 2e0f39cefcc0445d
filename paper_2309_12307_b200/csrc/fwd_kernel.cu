// S2-Attn forward for sm_100a.
//
// One CTA computes one 128-row query tile of one (batch, head, group): steps "roll", "group",
// "attention" and "roll back" of Algorithm 1 collapse into the choice of TMA coordinates.  Query
// tile i of rolled group g in a head with shift s covers the ORIGINAL tokens given by tile_ref():
// a group is one run of original tokens starting at (g*G + s) mod N, or, where it wraps past the
// sequence end, two runs ([N-G/2, N) followed by [0, G/2) in Algorithm 1), and each run is tiled from
// its own start, so a tile never straddles the sequence end.  Its keys are tiles 0..i of the same
// group, fetched at their own original positions.  When G or s is not a multiple of 128 the last
// tile of a run has fewer than 128 valid rows: the rest of the box holds neighbouring tokens (or
// zero fill), masked as key columns and not stored as query rows.  Outputs are stored at the
// original token rows, which is the roll back.
//
// Warp roles (320 threads): warp 0 issues TMA loads, warp 1 owns tensor memory and issues the
// tcgen05 MMAs, warps 2-9 run the online softmax: a score row lives in one tensor-memory lane
// (tcgen05.ld 32x32b) and is shared by two threads, one per 64-column half, which exchange their
// partial row maxima through shared memory.  S = Q K^T accumulates in tensor memory, P (bf16) is written back over S and used as the
// tensor-memory A operand of O += P V; O stays in tensor memory until the epilogue.  Two CTAs fit
// on one SM, so one CTA's softmax overlaps the other CTA's MMAs.
#include "s2a_params.h"
#include "sm100_ptx.cuh"

namespace s2a {

namespace {

template <int HD>
struct FwdCfg {
    static constexpr int kThreads = 320;
    static constexpr int kBoxes = HD / 64;                      // 64-column TMA boxes per tile
    static constexpr int kBoxBytes = kTile * 128;               // 128 rows x 128 bytes
    static constexpr int kTileBytes = kBoxes * kBoxBytes;       // one Q, K or V tile
    static constexpr int kStages = (HD == 128) ? 1 : 2;         // K/V ring depth
    static constexpr int kBarBytes = 256 + 2 * 2 * 128 * 8;  // barriers + row-max exchange slots
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
    // exchange slots between the two threads of a row: [2 parities][2 halves][128 rows] x {value, sequence}
    volatile float2* xch = reinterpret_cast<volatile float2*>(reinterpret_cast<uint8_t*>(bars) + 256);

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
    int unit, it;
    decode_block(blockIdx.x, p.geo.B * p.geo.H * p.geo.groups, Tg, &unit, &it);
    const int g = unit % p.geo.groups;
    const int h = (unit / p.geo.groups) % p.geo.H;
    const int b = unit / (p.geo.groups * p.geo.H);
    const int hk = h / (p.geo.H / p.geo.Hkv);
    const int s = (h < p.geo.n_unshifted) ? 0 : p.geo.shift;
    const GroupLayout L = group_layout(p.geo, s, g);
    const int i = L.nTiles - 1 - it;           // query tile inside the group
    if (i < 0) return;                         // this group has fewer tiles than the largest one
    const int j_begin = first_key_tile(L, i);
    const int n_kv = i + 1 - j_begin;          // causal: key tiles j_begin..i of the same group (j_begin = 0 by default)
    const TileRef tq = tile_ref(L, i);
    const int tq0 = tq.tok0;

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        mbar_init(s_full, 1);
        mbar_init(p_full, 256);
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
    for (int idx = threadIdx.x; idx < 2 * 2 * 128; idx += C::kThreads) {  // sequence 0 = "nothing published"
        const_cast<float2*>(xch)[idx] = make_float2(0.f, 0.f);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, C::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const WaitCtx ctx{abort_flag, p.status, p.host_status};

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
                const int tk0 = tile_ref(L, j_begin + j).tok0;
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
        // The whole warp walks the loop so that addresses and descriptors stay warp-uniform values;
        // only the MMA and commit instructions themselves are issued by one elected lane.
        constexpr uint32_t idesc_s = idesc_bf16(128, 128, 0, 0);  // S = Q K^T   (both K-major)
        constexpr uint32_t idesc_o = idesc_bf16(128, HD, 0, 1);   // O += P V    (V is MN-major)
        const uint32_t tS = tmem_base + C::kColS;
        const uint32_t tO = tmem_base + C::kColO;
        const uint32_t dQ = desc_lo_k_major(smem_u32(sQ));
        bool ok = mbar_wait_uniform(q_full, 0, ctx, kWaitFwd + 3);
        for (int j = 0; ok && j < n_kv; ++j) {
            const int st = j % C::kStages;
            const uint32_t ph = (j / C::kStages) & 1;
            const uint32_t dK = desc_lo_k_major(smem_u32(sK + st * C::kTileBytes));
            const uint32_t dV = desc_lo_mn_major(smem_u32(sV + st * C::kTileBytes), C::kBoxBytes);
            if (!mbar_wait_uniform(k_full + st, ph, ctx, kWaitFwd + 4)) break;
            tc_fence_after();
            // The previous P (aliased on S) was consumed by the previous P.V, which precedes
            // this MMA in issue order; the softmax warps finished reading S before that.
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {
                    constexpr uint32_t kBox = C::kBoxBytes;
                    mma_ss(tS, dQ + desc_step_k_major(kk, kBox), dK + desc_step_k_major(kk, kBox), idesc_s, kk > 0);
                }
                mma_commit(k_empty + st);
                mma_commit(s_full);
            }
            __syncwarp();
            if (!mbar_wait_uniform(p_full, j & 1, ctx, kWaitFwd + 5)) break;
            if (!mbar_wait_uniform(v_full + st, ph, ctx, kWaitFwd + 6)) break;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kTile / 16; ++kk) {
                    mma_ts(tO, tS + (kk >> 2) * 64 + (kk & 3) * 8, dV + kk * kDescStepMn, idesc_o, (j > 0) || (kk > 0));
                }
                mma_commit(v_empty + st);
                if (j == n_kv - 1) mma_commit(o_full);
            }
            __syncwarp();
        }
        if (__any_sync(0xffffffffu, *abort_flag != 0)) {
            // MMAs already issued must finish before tensor memory is released
            if (elect_one()) {
                mma_commit(drain);
                mbar_wait_drain(drain, 0);
            }
        }
        __syncwarp();
    } else {
        // =========================== softmax + epilogue ======================================
        // Thread (quad, lane, half) owns columns [64*half, +64) of score row 32*quad + lane.  Its
        // bf16 P values go over the first 32 of its own columns, so the two halves never write
        // into columns the other half still has to read: P's 128 K values sit at packed columns
        // [0,32) and [64,96).
        const int quad = warp & 3;             // tensor-memory lane quadrant this warp may access
        const int half = (warp - 2) >> 2;
        const int row = quad * 32 + lane;
        const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
        const uint32_t t_mine = t_row + C::kColS + half * 64;
        const float c2 = p.scale_log2;
        float m_used = -INFINITY;              // running maximum in use, already scaled to log2 units
        float l = 0.f;                         // this half's part of the running sum of exp2(s*c2 - m_used)
        bool ok = true;
        // Publish `v` to the thread that owns the other half of this row and fetch its value.
        // One 8-byte store carries the value together with a sequence number, the reader polls
        // (bounded) until the number matches.  Slots alternate with the parity of `seq`; a thread
        // cannot run two exchanges ahead of its partner, so a slot is never overwritten unread.
        auto pair_exchange = [&](float v, int seq, float& other) -> bool {
            const uint32_t slot = smem_u32(const_cast<float2*>(xch)) + (seq & 1) * 2048;
            const uint32_t mine = slot + (half * 128 + row) * 8;
            const uint32_t theirs = slot + ((half ^ 1) * 128 + row) * 8;
            asm volatile("st.volatile.shared.v2.b32 [%0], {%1, %2};" ::"r"(mine), "r"(__float_as_uint(v)), "r"(seq + 1)
                         : "memory");
            const long long t0 = clock64();
            for (uint32_t spins = 1;; ++spins) {
                uint32_t val, tag;
                asm volatile("ld.volatile.shared.v2.b32 {%0, %1}, [%2];" : "=r"(val), "=r"(tag) : "r"(theirs) : "memory");
                if (tag == static_cast<uint32_t>(seq + 1)) {
                    other = __uint_as_float(val);
                    return true;
                }
                if ((spins & 255u) == 0) {
                    if (*abort_flag != 0) return false;
                    if (clock64() - t0 > kWaitLimitCycles) {
                        report_expiry(ctx, kWaitFwd + 9);
                        return false;
                    }
                }
            }
        };
        for (int j = 0; j < n_kv; ++j) {
            if (!mbar_wait(s_full, j & 1, ctx, kWaitFwd + 7)) { ok = false; break; }
            tc_fence_after();
            // pass 1: row maximum of this thread's 64 columns (the scores are read again in pass 2,
            // 32 at a time, which keeps the register footprint small enough for two CTAs per SM)
            // Key x of the tile is visible to query row r iff it is one of the tile's valid rows and,
            // on the diagonal tile, x <= r.  Off the diagonal a full tile needs no mask at all.
            const int k_valid = tile_ref(L, j_begin + j).valid;
            const bool last = (j == n_kv - 1);
            const bool diagonal = last || k_valid < kTile;   // "this tile is masked"
            const int vis = (last && row < k_valid) ? row : k_valid - 1;
            const int lim = vis - half * 64;   // visible iff (column within this half) <= lim
            float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t sreg[32];
                tmem_ld_32x32(t_mine + c * 32, sreg);
                tmem_wait_ld();
                if (diagonal) {
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (c * 32 + e > lim) sreg[e] = 0xff800000u;  // -inf
                }
#pragma unroll
                for (int e = 0; e < 32; ++e) mx4[e & 3] = fmaxf(mx4[e & 3], __uint_as_float(sreg[e]));
            }
            const float mx_own = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
            float mx_other;
            if (!pair_exchange(mx_own, j, mx_other)) { ok = false; break; }
            const float mx = fmaxf(mx_own, mx_other);
            const float m_new = fmaxf(m_used, mx * c2);
            if (j == 0) {
                m_used = m_new;
            } else {
                const bool need = (m_new - m_used) > kLazyRescale;
                if (__any_sync(0xffffffffu, need)) {
                    // s_full(j) also covers the previous P.V, so O is quiescent here; each half
                    // rescales its own half of O's columns
                    const float alpha = need ? fast_exp2(m_used - m_new) : 1.0f;
                    l *= alpha;
#pragma unroll
                    for (int c = 0; c < HD / 64; ++c) {
                        uint32_t oreg[32];
                        const uint32_t t_o = t_row + C::kColO + half * (HD / 2) + c * 32;
                        tmem_ld_32x32(t_o, oreg);
                        tmem_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) oreg[e] = __float_as_uint(__uint_as_float(oreg[e]) * alpha);
                        tmem_st_32x32(t_o, oreg);
                    }
                    if (need) m_used = m_new;
                }
            }
            float sum4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t sreg[32];
                tmem_ld_32x32(t_mine + c * 32, sreg);
                tmem_wait_ld();
                if (diagonal) {
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (c * 32 + e > lim) sreg[e] = 0xff800000u;
                }
                uint32_t preg[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const float p0 = fast_exp2(fmaf(__uint_as_float(sreg[2 * e]), c2, -m_used));
                    const float p1 = fast_exp2(fmaf(__uint_as_float(sreg[2 * e + 1]), c2, -m_used));
                    sum4[e & 3] += p0 + p1;
                    preg[e] = pack_bf16(p0, p1);
                }
                // packed columns [16c, 16c+16) overlay score columns [16c, 16c+16) of this half, which
                // pass 2 has already consumed (c = 1 writes over columns 16..31, read when c was 0)
                tmem_st_32x16(t_mine + c * 16, preg);
            }
            l += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(p_full);
        }
        if (ok && mbar_wait(o_full, 0, ctx, kWaitFwd + 8)) {
            tc_fence_after();
            // total row sum = this half's part + the other half's
            float l_other = 0.f;
            pair_exchange(l, n_kv, l_other);
            const float l_row = l + l_other;
            const float inv_l = 1.0f / l_row;
            const int t = tq0 + row;
            const bool row_valid = row < tq.valid;   // rows past the end of a ragged tile are not part of the group
            __nv_bfloat16* orow = p.o + ((static_cast<size_t>(b) * p.geo.N + t) * p.geo.H + h) * HD + half * (HD / 2);
#pragma unroll
            for (int c = 0; c < HD / 64; ++c) {
                uint32_t oreg[32];
                tmem_ld_32x32(t_row + C::kColO + half * (HD / 2) + c * 32, oreg);
                tmem_wait_ld();
                uint4* dst = reinterpret_cast<uint4*>(orow + c * 32);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    uint4 pk;
                    pk.x = pack_bf16(__uint_as_float(oreg[8 * e + 0]) * inv_l, __uint_as_float(oreg[8 * e + 1]) * inv_l);
                    pk.y = pack_bf16(__uint_as_float(oreg[8 * e + 2]) * inv_l, __uint_as_float(oreg[8 * e + 3]) * inv_l);
                    pk.z = pack_bf16(__uint_as_float(oreg[8 * e + 4]) * inv_l, __uint_as_float(oreg[8 * e + 5]) * inv_l);
                    pk.w = pack_bf16(__uint_as_float(oreg[8 * e + 6]) * inv_l, __uint_as_float(oreg[8 * e + 7]) * inv_l);
                    if (row_valid) dst[e] = pk;
                }
            }
            // natural-log sum-exp of the scaled scores
            if (half == 0 && row_valid)
                p.lse[(static_cast<size_t>(b) * p.geo.H + h) * p.geo.N + t] = (m_used + log2f(l_row)) * 0.6931471805599453f;
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
