// S2-Attn backward for sm_100a, head dim 128: dK, dV and dQ from ONE pass over the attended tile pairs
// (five matrix products per pair instead of the seven that separate dK/dV and dQ kernels execute).
//
// One CTA owns a 128-row key tile (b, hk, original tokens tk0..tk0+127) and walks, for every query
// head of that KV head, the 128-row query tiles i >= j of the tile's group (roll and grouping folded
// into TMA coordinates as everywhere else).  Per step, with keys along tensor-memory lanes:
//     S^T  = K Q^T                      (SS MMA)      P^T  = exp2(S^T c2 - lse)        (elementwise)
//     dP^T = V dO^T                     (SS MMA)      dS^T = P^T o (dP^T - D)          (elementwise)
//     dV  += P^T dO                     (TS MMA, P^T bf16 in tensor memory over S^T)
//     dK  += dS^T Q                     (SS MMA, dS^T bf16 written to shared memory by the elementwise warps)
//     dQ^T = K^T dS^T                   (SS MMA from the same shared-memory tile; both operands MN-major)
// dQ^T (head dim along lanes, queries along columns) is added to an fp32 accumulator in global
// memory with coalesced red.global.add (a warp instruction covers 32 consecutive head-dim elements
// of one query row); a small kernel then scales it and rounds it to bf16.  dQ's summation order
// over key tiles is therefore not fixed (results vary in the last bits from run to run); dK and dV
// never leave the CTA's tensor memory and stay deterministic.
//
// Tensor memory (512 columns): S^T / P^T [0,128)   dP^T then dQ^T [128,256)   dV [256,384)   dK [384,512)
// Shared memory: K 32 KB, V 32 KB, two stages of (Q 32 KB + dO 32 KB + lse, D 1 KB), dS^T 32 KB.
#include "s2a_params.h"
#include "sm100_ptx.cuh"

namespace s2a {

namespace {

constexpr float kLog2eF = 1.4426950408889634f;
constexpr int kHD = 128;
constexpr int kFThreads = 640;                 // TMA warp, MMA warp, two spare warps, 2 x 8 elementwise warps
constexpr int kFBox = kTile * 128;             // one 64-column TMA box of 128 rows
constexpr int kFTile = 2 * kFBox;              // a 128 x 128 bf16 tile
constexpr int kFStages = 2;
constexpr int kFStat = 2 * kTile * 4;          // lse[128] and D[128] of a stage
constexpr int kFOffK = 0;
constexpr int kFOffV = kFTile;
constexpr int kFOffStage = 2 * kFTile;                       // per stage: Q then dO
constexpr int kFOffDS = kFOffStage + kFStages * 2 * kFTile;
constexpr int kFOffStat = kFOffDS + kFTile;
constexpr int kFOffBars = kFOffStat + kFStages * kFStat;
constexpr int kFPayload = kFOffBars + 256;
constexpr int kFSmemBytes = 232448;            // everything an SM offers to one CTA
static_assert(kFPayload <= kFSmemBytes, "shared memory layout too large");

struct FusedBars {
    uint64_t res_full, acc_full, drain;
    uint64_t s_full, dp_full, p_ready, p_taken, ds_ready, ds_free, dq_full, dq_drained;
    uint64_t st_full[kFStages], st_empty[kFStages];
    uint32_t tmem_slot;
    int abort_flag;
    int poisoned;
};

__device__ __forceinline__ int mod_pos_f(int x, int n) {
    int r = x % n;
    return r < 0 ? r + n : r;
}

__device__ __forceinline__ float4 lds_f4(uint32_t saddr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(saddr));
    return v;
}

// query tiles that attend key tile tk0 in head hq: tiles j .. Tg-1 of group g (rolled order)
struct TileWalk {
    int s, g, j;
};
__device__ __forceinline__ TileWalk tile_walk(const Geometry& geo, int hq, int tk0) {
    TileWalk w;
    w.s = (hq < geo.n_unshifted) ? 0 : geo.shift;
    const int pos = mod_pos_f(tk0 - w.s, geo.N);
    w.g = pos / geo.G;
    w.j = (pos % geo.G) / kTile;
    return w;
}

__global__ void __launch_bounds__(kFThreads, 1) s2a_bwd_fused_kernel(const __grid_constant__ BwdFusedParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sK = smem + kFOffK;
    uint8_t* sV = smem + kFOffV;
    uint8_t* sStage = smem + kFOffStage;
    uint8_t* sDS = smem + kFOffDS;
    float* sStat = reinterpret_cast<float*>(smem + kFOffStat);
    FusedBars* bars = reinterpret_cast<FusedBars*>(smem + kFOffBars);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const Geometry& geo = p.geo;
    const int rep = geo.H / geo.Hkv;

    // The layout uses all but a few hundred bytes of the SM's shared memory: give up cleanly if
    // the 1024-byte alignment of the window left too little room.  A bounded wait that expired
    // earlier (in any kernel) leaves the status word set: later CTAs then return at once.
    if (threadIdx.x == 0) {
        const bool fits = (smem + kFPayload) <= (smem_raw + kFSmemBytes);
        int poisoned = *reinterpret_cast<volatile int*>(p.status);
        if (!fits && poisoned == 0) {
            atomicCAS(p.status, 0, kWaitBwdFused + 99);
            poisoned = 1;
        }
        *reinterpret_cast<volatile int*>(smem_raw) = poisoned;  // first word of the window, always inside it
    }
    __syncthreads();
    if (*reinterpret_cast<volatile int*>(smem_raw) != 0) return;
    __syncthreads();

    // key tile: enumerate in the rolled order of the first query head of the KV head, heaviest
    // (earliest in the group) first
    const int Tg = geo.tiles_per_group;
    const int j0 = static_cast<int>(blockIdx.x % Tg);
    const int unit = blockIdx.x / Tg;
    const int g0 = unit % geo.groups;
    const int hk = (unit / geo.groups) % geo.Hkv;
    const int b = unit / (geo.groups * geo.Hkv);
    const int hq0 = hk * rep;
    const int s0 = (hq0 < geo.n_unshifted) ? 0 : geo.shift;
    const int tk0 = mod_pos_f(g0 * geo.G + j0 * kTile + s0, geo.N);

    int total_steps = 0;
    for (int hq = hq0; hq < hq0 + rep; ++hq) total_steps += Tg - tile_walk(geo, hq, tk0).j;

    if (threadIdx.x == 0) {
        mbar_init(&bars->res_full, 1);
        mbar_init(&bars->acc_full, 1);
        mbar_init(&bars->drain, 1);
        mbar_init(&bars->s_full, 1);
        mbar_init(&bars->dp_full, 1);
        mbar_init(&bars->p_ready, 256);
        mbar_init(&bars->p_taken, 256);
        mbar_init(&bars->ds_free, 1);
        mbar_init(&bars->ds_ready, 256);
        mbar_init(&bars->dq_full, 1);
        mbar_init(&bars->dq_drained, 256);
        for (int st = 0; st < kFStages; ++st) {
            mbar_init(&bars->st_full[st], 1);
            mbar_init(&bars->st_empty[st], 1);
        }
        bars->abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&p.tm_q);
        tma_prefetch_desc(&p.tm_do);
        tma_prefetch_desc(&p.tm_k);
        tma_prefetch_desc(&p.tm_v);
    }
    if (warp == 3) {
        tmem_alloc(&bars->tmem_slot, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_slot;
    const WaitCtx ctx{&bars->abort_flag, p.status};
    constexpr uint32_t kColS = 0, kColP2 = 128, kColDV = 256, kColDK = 384;

    if (warp == 0) {
        // =========================== TMA producer ============================================
        if (lane == 0) {
            mbar_expect_tx(&bars->res_full, 2 * kFTile);
            for (int bx = 0; bx < 2; ++bx) {
                tma_load_4d(sK + bx * kFBox, &p.tm_k, &bars->res_full, bx * 64, hk, tk0, b);
                tma_load_4d(sV + bx * kFBox, &p.tm_v, &bars->res_full, bx * 64, hk, tk0, b);
            }
            int it = 0;
            bool ok = true;
            for (int hq = hq0; ok && hq < hq0 + rep; ++hq) {
                const TileWalk w = tile_walk(geo, hq, tk0);
                for (int i = w.j; i < Tg; ++i, ++it) {
                    const int st = it % kFStages;
                    const uint32_t ph = (it / kFStages) & 1;
                    const int tq0 = mod_pos_f(w.g * geo.G + i * kTile + w.s, geo.N);
                    if (!mbar_wait(&bars->st_empty[st], ph ^ 1, ctx, kWaitBwdFused + 1)) { ok = false; break; }
                    mbar_expect_tx(&bars->st_full[st], 2 * kFTile + kFStat);
                    uint8_t* sQ = sStage + st * 2 * kFTile;
                    uint8_t* sDO = sQ + kFTile;
                    for (int bx = 0; bx < 2; ++bx) {
                        tma_load_4d(sQ + bx * kFBox, &p.tm_q, &bars->st_full[st], bx * 64, hq, tq0, b);
                        tma_load_4d(sDO + bx * kFBox, &p.tm_do, &bars->st_full[st], bx * 64, hq, tq0, b);
                    }
                    const size_t stat_idx = (static_cast<size_t>(b) * geo.H + hq) * geo.N + tq0;
                    bulk_load_1d(sStat + st * 2 * kTile, p.lse + stat_idx, kTile * 4, &bars->st_full[st]);
                    bulk_load_1d(sStat + st * 2 * kTile + kTile, p.Dsum + stat_idx, kTile * 4, &bars->st_full[st]);
                }
            }
            if (bars->abort_flag != 0) {
                mbar_wait_drain(&bars->res_full, 0);
                for (int nn = (it > kFStages ? it - kFStages : 0); nn < it; ++nn)
                    mbar_wait_drain(&bars->st_full[nn % kFStages], (nn / kFStages) & 1);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // =========================== MMA issuer ==============================================
        // The whole warp walks the loop (warp-uniform addresses); one elected lane issues.  All five
        // products of a step come from this one warp, in an order that keeps tensor-memory reuse safe:
        //   S^T(n+1) after dV(n) (same columns hold P^T(n)) and after group B has copied P^T(n) out,
        //   dP^T(n)  after the draining of dQ^T(n-1) (same columns).
        constexpr uint32_t idesc_kk = idesc_bf16(128, 128, 0, 0);   // both operands K-major
        constexpr uint32_t idesc_kn = idesc_bf16(128, 128, 0, 1);   // B MN-major
        constexpr uint32_t idesc_nn = idesc_bf16(128, 128, 1, 1);   // A and B MN-major
        const uint32_t aK = smem_u32(sK), aV = smem_u32(sV), aDS = smem_u32(sDS);
        const uint32_t dK_k = desc_lo_k_major(aK), dV_k = desc_lo_k_major(aV);
        const uint32_t dK_mn = desc_lo_mn_major(aK, kFBox);
        const uint32_t dDS_k = desc_lo_k_major(aDS), dDS_mn = desc_lo_mn_major(aDS, kFBox);
        const uint32_t tS = tmem_base + kColS, tP2 = tmem_base + kColP2;
        auto issue_scores = [&](int n) -> bool {   // S^T(n) = K Q(n)^T
            const int st = n % kFStages;
            if (!mbar_wait_uniform(&bars->st_full[st], (n / kFStages) & 1, ctx, kWaitBwdFused + 3)) return false;
            tc_fence_after();
            const uint32_t dQ_k = desc_lo_k_major(smem_u32(sStage + st * 2 * kFTile));
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    mma_ss(tS, dK_k + desc_step_k_major(kk, kFBox), dQ_k + desc_step_k_major(kk, kFBox), idesc_kk, kk > 0);
                mma_commit(&bars->s_full);
            }
            __syncwarp();
            return true;
        };
        bool ok = mbar_wait_uniform(&bars->res_full, 0, ctx, kWaitBwdFused + 2);
        ok = ok && issue_scores(0);
        for (int n = 0; ok && n < total_steps; ++n) {
            const int st = n % kFStages;
            const uint32_t par = n & 1;
            const uint32_t aQ = smem_u32(sStage + st * 2 * kFTile), aDO = aQ + kFTile;
            const uint32_t dDO_k = desc_lo_k_major(aDO);
            const uint32_t dQ_mn = desc_lo_mn_major(aQ, kFBox), dDO_mn = desc_lo_mn_major(aDO, kFBox);
            if (n > 0 && !mbar_wait_uniform(&bars->dq_drained, par ^ 1, ctx, kWaitBwdFused + 4)) break;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    mma_ss(tP2, dV_k + desc_step_k_major(kk, kFBox), dDO_k + desc_step_k_major(kk, kFBox), idesc_kk, kk > 0);
                mma_commit(&bars->dp_full);
            }
            __syncwarp();
            if (!mbar_wait_uniform(&bars->p_ready, par, ctx, kWaitBwdFused + 5)) break;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)   // bf16 P^T: 128 query values at packed columns [0,32) and [64,96)
                    mma_ts(tmem_base + kColDV, tS + (kk >> 2) * 64 + (kk & 3) * 8, dDO_mn + kk * kDescStepMn, idesc_kn,
                           (n > 0) || (kk > 0));
            }
            __syncwarp();
            if (n + 1 < total_steps) {
                // the next scores overwrite P^T(n): dV(n) precedes them in issue order, and group B must have
                // taken its copy of P^T(n)
                if (!mbar_wait_uniform(&bars->p_taken, par, ctx, kWaitBwdFused + 12)) break;
                if (!issue_scores(n + 1)) break;
            }
            if (!mbar_wait_uniform(&bars->ds_ready, par, ctx, kWaitBwdFused + 6)) break;
            tc_fence_after();
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)   // dQ^T = K^T dS^T first: its columns have to be drained before the next dP^T
                    mma_ss(tP2, dK_mn + kk * kDescStepMn, dDS_mn + kk * kDescStepMn, idesc_nn, kk > 0);
                mma_commit(&bars->dq_full);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)   // dK += dS^T Q: A = dS^T tile (keys x queries, K-major), B = Q MN-major
                    mma_ss(tmem_base + kColDK, dDS_k + desc_step_k_major(kk, kFBox), dQ_mn + kk * kDescStepMn, idesc_kn,
                           (n > 0) || (kk > 0));
                mma_commit(&bars->ds_free);
                mma_commit(&bars->st_empty[st]);
                if (n == total_steps - 1) mma_commit(&bars->acc_full);
            }
            __syncwarp();
        }
        if (__any_sync(0xffffffffu, bars->abort_flag != 0)) {
            if (elect_one()) {
                mma_commit(&bars->drain);
                mbar_wait_drain(&bars->drain, 0);
            }
        }
        __syncwarp();
    } else if (warp < 4) {
        // spare warps (warp 3 owns the tensor-memory allocation)
    } else if (warp < 12) {
        // =========================== elementwise group A: P^T ================================
        // Thread (quad, hf, lane): key row r = 32 quad + lane, queries [64 hf, +64).  Its 64 bf16
        // P^T values (32 packed columns) go over the first half of its own S^T columns.
        const int quad = warp & 3;
        const int hf = (warp - 4) >> 2;
        const int r = quad * 32 + lane;
        const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
        const uint32_t tS = t_row + kColS + hf * 64;
        const float c2 = p.scale_log2;
        const uint64_t c2x2 = f2_pack(c2, c2), nl2e = f2_pack(-kLog2eF, -kLog2eF);
        bool ok = true;
        int n = 0;
        for (int hq = hq0; ok && hq < hq0 + rep; ++hq) {
            const TileWalk w = tile_walk(geo, hq, tk0);
            for (int i = w.j; i < Tg; ++i, ++n) {
                const int st = n % kFStages;
                const uint32_t par = n & 1;
                if (!mbar_wait(&bars->st_full[st], (n / kFStages) & 1, ctx, kWaitBwdFused + 8)) { ok = false; break; }
                if (!mbar_wait(&bars->s_full, par, ctx, kWaitBwdFused + 9)) { ok = false; break; }
                tc_fence_after();
                const uint32_t stat_sa = smem_u32(sStat + st * 2 * kTile) + hf * 256;  // lse of my 64 queries
                const bool diagonal = (i == w.j);   // query x of the tile sees key row r iff r <= x
                uint32_t sr[2][32];
                tmem_ld_32x32(tS, sr[0]);
                tmem_ld_32x32(tS + 32, sr[1]);
                tmem_wait_ld();
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t pk[16];
#pragma unroll
                    for (int e4 = 0; e4 < 8; ++e4) {
                        const float4 l = lds_f4(stat_sa + (c * 32 + e4 * 4) * 4);
                        const uint64_t lp[2] = {f2_pack(l.x, l.y), f2_pack(l.z, l.w)};
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            const int e = e4 * 4 + 2 * u;
                            float x0, x1;
                            f2_unpack(f2_fma(f2_pack(__uint_as_float(sr[c][e]), __uint_as_float(sr[c][e + 1])), c2x2,
                                             f2_mul(lp[u], nl2e)),
                                      x0, x1);
                            float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
                            if (diagonal) {
                                const int x = hf * 64 + c * 32 + e;
                                if (r > x) p0 = 0.f;
                                if (r > x + 1) p1 = 0.f;
                            }
                            pk[e >> 1] = pack_bf16(p0, p1);
                        }
                    }
                    tmem_st_32x16(tS + c * 16, pk);
                }
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(&bars->p_ready);
            }
        }
    } else {
        // =========================== elementwise group B: dS^T and the dQ^T drain ============
        // Same (quad, hf, lane) geometry: lane r is a key row for P^T / dP^T and a head-dim index
        // for dQ^T; columns [64 hf, +64) are queries.
        const int quad = warp & 3;
        const int hf = (warp - 12) >> 2;
        const int r = quad * 32 + lane;
        const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
        const uint32_t tPt = t_row + kColS + hf * 64;     // bf16 P^T written by group A (32 packed columns)
        const uint32_t tP2 = t_row + kColP2 + hf * 64;
        const uint32_t ds_row = smem_u32(sDS) + hf * kFBox + r * 128;
        const size_t col_stride = static_cast<size_t>(geo.H) * kHD;
        bool ok = true;
        int n = 0;
        for (int hq = hq0; ok && hq < hq0 + rep; ++hq) {
            const TileWalk w = tile_walk(geo, hq, tk0);
            for (int i = w.j; i < Tg; ++i, ++n) {
                const int st = n % kFStages;
                const uint32_t par = n & 1;
                const int tq0 = mod_pos_f(w.g * geo.G + i * kTile + w.s, geo.N);
                const uint32_t stat_sa = smem_u32(sStat + st * 2 * kTile) + hf * 256 + 512;  // D of my 64 queries
                // ---- take a copy of P^T(n) ---------------------------------------------------------
                if (!mbar_wait(&bars->p_ready, par, ctx, kWaitBwdFused + 13)) { ok = false; break; }
                tc_fence_after();
                uint32_t pk[32];
                tmem_ld_32x32(tPt, pk);
                tmem_wait_ld();
                tc_fence_before();
                mbar_arrive(&bars->p_taken);
                // ---- dS^T(n) -------------------------------------------------------------------------
                if (!mbar_wait(&bars->dp_full, par, ctx, kWaitBwdFused + 10)) { ok = false; break; }
                // the previous step's dK / dQ^T MMAs still read the dS^T tile until they are done
                if (n > 0 && !mbar_wait(&bars->ds_free, par ^ 1, ctx, kWaitBwdFused + 14)) { ok = false; break; }
                tc_fence_after();
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t pr[32];
                    tmem_ld_32x32(tP2 + c * 32, pr);
                    tmem_wait_ld();
                    uint32_t dsw[16];
#pragma unroll
                    for (int e4 = 0; e4 < 8; ++e4) {
                        const float4 dd = lds_f4(stat_sa + (c * 32 + e4 * 4) * 4);
                        const uint64_t dp2[2] = {f2_pack(dd.x, dd.y), f2_pack(dd.z, dd.w)};
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            const int e = e4 * 4 + 2 * u;
                            const uint32_t pw = pk[c * 16 + (e >> 1)];
                            const uint64_t pp = f2_pack(__uint_as_float(pw << 16), __uint_as_float(pw & 0xffff0000u));
                            const uint64_t t = f2_sub(f2_pack(__uint_as_float(pr[e]), __uint_as_float(pr[e + 1])), dp2[u]);
                            float d0, d1;
                            f2_unpack(f2_mul(pp, t), d0, d1);
                            dsw[e >> 1] = pack_bf16(d0, d1);
                        }
                    }
                    // my row of the dS^T tile: box hf, row r, eight 16-byte chunks whose position is permuted
                    // by (r & 7) -- the layout a 128-byte-swizzle TMA box would have
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        const int chunk = c * 4 + q4;  // 8 queries per chunk
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(ds_row + ((chunk ^ (r & 7)) << 4)),
                                     "r"(dsw[4 * q4]), "r"(dsw[4 * q4 + 1]), "r"(dsw[4 * q4 + 2]), "r"(dsw[4 * q4 + 3])
                                     : "memory");
                    }
                }
                fence_proxy_async_smem();   // the MMAs read this tile through the async proxy
                tc_fence_before();
                mbar_arrive(&bars->ds_ready);
                // ---- drain dQ^T(n): head-dim index r, queries 64 hf .. --------------------------------
                if (!mbar_wait(&bars->dq_full, par, ctx, kWaitBwdFused + 7)) { ok = false; break; }
                tc_fence_after();
                float* base = p.dq_acc + ((static_cast<size_t>(b) * geo.N + tq0 + hf * 64) * geo.H + hq) * kHD + r;
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t v[32];
                    tmem_ld_32x32(tP2 + c * 32, v);
                    tmem_wait_ld();
                    if (c == 1) {   // all of my columns are in registers: the next dP^T may overwrite them
                        tc_fence_before();
                        mbar_arrive(&bars->dq_drained);
                    }
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        asm volatile("red.global.add.f32 [%0], %1;" ::"l"(base + (c * 32 + e) * col_stride),
                                     "f"(__uint_as_float(v[e]))
                                     : "memory");
                }
            }
        }
        // ---- epilogue: dV and dK (group B's 256 threads: 64 columns of each per thread) ------------
        if (ok && mbar_wait(&bars->acc_full, 0, ctx, kWaitBwdFused + 11)) {
            tc_fence_after();
            const size_t out_row = ((static_cast<size_t>(b) * geo.N + tk0 + r) * geo.Hkv + hk) * kHD + hf * 64;
#pragma unroll
            for (int m = 0; m < 2; ++m) {          // m = 0: dV, m = 1: dK
                const uint32_t t_acc = t_row + (m == 0 ? kColDV : kColDK) + hf * 64;
                const float mul = (m == 0) ? 1.0f : p.scale;
                __nv_bfloat16* dst_row = (m == 0 ? p.dv : p.dk) + out_row;
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t a[32];
                    tmem_ld_32x32(t_acc + c * 32, a);
                    tmem_wait_ld();
                    uint4* dst = reinterpret_cast<uint4*>(dst_row + c * 32);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        uint4 o;
                        o.x = pack_bf16(__uint_as_float(a[8 * e + 0]) * mul, __uint_as_float(a[8 * e + 1]) * mul);
                        o.y = pack_bf16(__uint_as_float(a[8 * e + 2]) * mul, __uint_as_float(a[8 * e + 3]) * mul);
                        o.z = pack_bf16(__uint_as_float(a[8 * e + 4]) * mul, __uint_as_float(a[8 * e + 5]) * mul);
                        o.w = pack_bf16(__uint_as_float(a[8 * e + 6]) * mul, __uint_as_float(a[8 * e + 7]) * mul);
                        dst[e] = o;
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 3) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

__global__ void __launch_bounds__(256) s2a_dq_convert_kernel(const DqConvertParams p) {
    const long long i = (static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x) * 8;
    if (i >= p.n) return;
    const float4 a = *reinterpret_cast<const float4*>(p.dq_acc + i);
    const float4 c = *reinterpret_cast<const float4*>(p.dq_acc + i + 4);
    uint4 o;
    o.x = pack_bf16(a.x * p.scale, a.y * p.scale);
    o.y = pack_bf16(a.z * p.scale, a.w * p.scale);
    o.z = pack_bf16(c.x * p.scale, c.y * p.scale);
    o.w = pack_bf16(c.z * p.scale, c.w * p.scale);
    *reinterpret_cast<uint4*>(p.dq + i) = o;
}

}  // namespace

cudaError_t configure_bwd_fused() {
    return cudaFuncSetAttribute(s2a_bwd_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kFSmemBytes);
}

cudaError_t launch_bwd_fused(const BwdFusedParams& p, cudaStream_t stream) {
    const Geometry& g = p.geo;
    const unsigned grid = static_cast<unsigned>(static_cast<long long>(g.B) * g.Hkv * g.groups * g.tiles_per_group);
    s2a_bwd_fused_kernel<<<grid, kFThreads, kFSmemBytes, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_dq_convert(const DqConvertParams& p, cudaStream_t stream) {
    const long long threads = (p.n + 7) / 8;
    s2a_dq_convert_kernel<<<static_cast<unsigned>((threads + 255) / 256), 256, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace s2a
