// S2-Attn backward for sm_100a: the derivative of Algorithm 1 (with Eq. 1 inside each group).
//
// With P = exp(scale * Q K^T - lse) on the attended pairs and D_t = dO_t . o_t:
//     dV = P^T dO          dP = dO V^T          dS = P o (dP - D)
//     dQ = scale * dS K    dK = scale * dS^T Q
// Four kernels:
//   1. preprocess: D[b,h,t] = sum_c dO[b,t,h,c] * o[b,t,h,c]                     (memory bound)
//   2. dQ, recomputing: one CTA per 128-row query tile, walks the 128-key tiles of its group (keys <=
//            query) and computes S, dP, dS again
//   3. dK,dV: persistent; a work item is one 128-row key tile, against which the 64-query sub-tiles of
//            every query head that shares the KV head (queries >= key) are streamed, so the sum over
//            those heads stays in tensor memory and needs no atomics.  It works on the transposed
//            scores S^T = K Q^T so that P^T and dS^T come out with keys along tensor-memory lanes, which
//            is the layout the A operand of dV += P^T dO and dK += dS^T Q needs.  Optionally it also
//            leaves dS^T in global memory,
//   4. dQ from spilled dS^T: persistent; a chain of plain products dQ_i = scale * sum_j dS_ij K_j that
//            replaces kernel 2 when the caller's workspace has room for the spill.
// The roll of the shifted heads and the group boundaries are folded into TMA coordinates exactly
// as in the forward kernel; all results are stored at original token rows.
//
// Kernels 2 and 3 use the same warp roles (384 threads, one CTA per SM, all 512 tensor-memory columns):
// warp 0 loads with TMA; warp 1 issues the score MMAs and warp 2 the gradient MMAs (a single issuing
// warp spends so long on its own barrier waits that the tensor pipe runs dry in between; with two, one
// can issue while the other waits); warp 3 owns the tensor-memory allocation; warps 4-11 do the
// elementwise work with one tensor-memory lane and half of the columns per thread.  dP (dP^T) has a
// single buffer: the elementwise warps copy their part of it into registers and release it at once,
// which leaves the columns for two score buffers (and, in kernel 3, for K as a tensor-memory operand),
// so that the score products of the next step run while the elementwise warps work on the current one.
#include "s2a_params.h"
#include "sm100_ptx.cuh"

namespace s2a {

namespace {

constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ int mod_pos(int x, int n) {
    int r = x % n;
    return r < 0 ? r + n : r;
}

// ------------------------------------------------------------------------------------------------
// 1. preprocess
// ------------------------------------------------------------------------------------------------
// Each row of d bf16 values is read by d/8 threads with 16-byte loads.
template <int HD>
__global__ void __launch_bounds__(256) s2a_bwd_preprocess_kernel(const PreParams p) {
    constexpr int kThreadsPerRow = HD / 8;
    const long long n_rows = static_cast<long long>(p.B) * p.N * p.H;
    const long long gtid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    const long long row = gtid / kThreadsPerRow;  // (b * N + t) * H + h
    const int part = static_cast<int>(gtid % kThreadsPerRow);
    float acc = 0.f;
    if (row < n_rows) {
        const uint4 a = reinterpret_cast<const uint4*>(p.o + row * HD)[part];
        const uint4 c = reinterpret_cast<const uint4*>(p.dO + row * HD)[part];
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w};
        const uint32_t cw[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            // a bf16 is the upper half of an fp32
            acc = fmaf(__uint_as_float(aw[e] << 16), __uint_as_float(cw[e] << 16), acc);
            acc = fmaf(__uint_as_float(aw[e] & 0xffff0000u), __uint_as_float(cw[e] & 0xffff0000u), acc);
        }
    }
#pragma unroll
    for (int off = kThreadsPerRow / 2; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (row < n_rows && part == 0) {
        const int h = static_cast<int>(row % p.H);
        const long long bt = row / p.H;
        const int t = static_cast<int>(bt % p.N);
        const long long b = bt / p.N;
        p.Dsum[(b * p.H + h) * p.N + t] = acc;
    }
}

// ------------------------------------------------------------------------------------------------
// shared configuration of the two tensor-core kernels
// ------------------------------------------------------------------------------------------------
template <int HD>
struct BwdCfg {
    static constexpr int kThreads = 384;  // TMA warp, two MMA warps, one spare, 8 elementwise warps
    static constexpr int kBoxes = HD / 64;
    static constexpr int kBigBoxBytes = kTile * 128;            // 128-row box
    static constexpr int kSubBoxBytes = kSubTile * 128;         // 64-row box
    static constexpr int kBigTileBytes = kBoxes * kBigBoxBytes; // resident operand tile
    static constexpr int kSubTileBytes = kBoxes * kSubBoxBytes; // streamed operand tile
    static constexpr int kStages = 4;
    static constexpr int kStatBytes = kSubTile * 4;             // lse or D of one streamed tile
    static constexpr int kStageBytes = 2 * kSubTileBytes;       // two streamed operands per stage
    static constexpr int kBarBytes = 512;
    static constexpr int kNeeded = 1024 + 2 * kBigTileBytes + kStages * kStageBytes + kStages * 2 * kStatBytes + kBarBytes;
    // at least 120 KB so that only one CTA fits on an SM: each CTA allocates all of tensor memory
    static constexpr int kSmemBytes = kNeeded > 120 * 1024 ? kNeeded : 120 * 1024;
    static constexpr int kTmemCols = 512;
};

// Store COLS consecutive fp32 accumulator columns of this thread's tensor-memory lane (times `mul`)
// as bf16 to `dst`.
template <int COLS>
__device__ __forceinline__ void store_acc_cols(uint32_t t_addr, float mul, __nv_bfloat16* dst_row, bool row_valid) {
#pragma unroll
    for (int c = 0; c < COLS / 32; ++c) {
        uint32_t r[32];
        tmem_ld_32x32(t_addr + c * 32, r);
        tmem_wait_ld();
        uint4* dst = reinterpret_cast<uint4*>(dst_row + c * 32);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            uint4 pk;
            pk.x = pack_bf16(__uint_as_float(r[8 * e + 0]) * mul, __uint_as_float(r[8 * e + 1]) * mul);
            pk.y = pack_bf16(__uint_as_float(r[8 * e + 2]) * mul, __uint_as_float(r[8 * e + 3]) * mul);
            pk.z = pack_bf16(__uint_as_float(r[8 * e + 4]) * mul, __uint_as_float(r[8 * e + 5]) * mul);
            pk.w = pack_bf16(__uint_as_float(r[8 * e + 6]) * mul, __uint_as_float(r[8 * e + 7]) * mul);
            if (row_valid) dst[e] = pk;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// 2. dQ
// ------------------------------------------------------------------------------------------------
// One CTA per 128-row query tile; it walks the 128-key tiles j_begin..i of its group (keys <= query).
// Per key tile n:  S_n = Q K_n^T,  dP_n = dO V_n^T,  dS_n = P_n o (dP_n - D) as bf16 written over the
// start of S_n's columns,  dQ += dS_n K_n  (K_n is MN-major in the tile that served Q K_n^T).
// Full 128x128 score products: a 64-column product re-reads the 128-row A operand from shared memory
// for half the work and runs at 48 instead of 32 clocks per K step.
//
// Tensor memory columns: dQ [0,HD)   S buffers [128,256) [256,384)   dP [384,512)
// Only one dP buffer fits, so the elementwise warps copy their part of dP_{n+1} into registers as soon
// as they are done with step n and release the buffer at once: dP_{n+2} (and S_{n+2}, into the S
// buffer that the dQ MMAs of step n give back) run while they work on step n+1.  Shared memory: Q_i and dO_i resident, a ring of three K tiles and a ring of two V tiles.
template <int HD>
struct DqCfg {
    static constexpr int kThreads = 384;  // TMA warp, two MMA warps, one spare, 8 elementwise warps
    static constexpr int kBoxes = HD / 64;
    static constexpr int kBoxBytes = kTile * 128;          // 128 rows x 128 bytes
    static constexpr int kTileBytes = kBoxes * kBoxBytes;  // one Q, dO, K or V tile
    // K_n serves S_n early in step n-1 and the dQ MMAs at the end of step n: three K tiles are live
    // around the issue of S_{n+1}, V_n only until dP_n is done.
    static constexpr int kRingK = 3;
    static constexpr int kRingV = 2;
    static constexpr int kBarBytes = 512;
    static constexpr int kNeeded = 1024 + (2 + kRingK + kRingV) * kTileBytes + kBarBytes;
    // at least 120 KB so that only one CTA fits on an SM: each CTA allocates all of tensor memory
    static constexpr int kSmemBytes = kNeeded > 120 * 1024 ? kNeeded : 120 * 1024;
    static constexpr int kTmemCols = 512;
};

struct DqBars {
    uint64_t res_full;     // Q_i and dO_i landed
    uint64_t acc_full;     // all dQ MMAs done
    uint64_t drain;        // abort path only (gradient MMA warp)
    uint64_t drain2;       // abort path only (score MMA warp)
    uint64_t dp_ready;     // dP_n is in tensor memory
    uint64_t s_ready[2];   // S_n is in tensor memory (buffer n & 1)
    uint64_t dp_free;      // every elementwise thread holds its part of dP_n in registers
    uint64_t p_full[2];    // bf16 dS_n is in tensor memory
    uint64_t buf_free[2];  // the dQ MMAs that read an S buffer's bf16 dS are done
    uint64_t k_full[3], k_empty[3], v_full[2], v_empty[2];
    uint32_t tmem_slot;
    int abort_flag;
};

template <int HD>
__global__ void __launch_bounds__(DqCfg<HD>::kThreads, 1) s2a_bwd_dq_kernel(const __grid_constant__ BwdDqParams p) {
    using C = DqCfg<HD>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem;                                // resident: Q_i
    uint8_t* sDO = sQ + C::kTileBytes;                 // resident: dO_i
    uint8_t* sK = sDO + C::kTileBytes;                 // ring of K tiles
    uint8_t* sV = sK + C::kRingK * C::kTileBytes;      // ring of V tiles
    DqBars* bars = reinterpret_cast<DqBars*>(sV + C::kRingV * C::kTileBytes);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    // A bounded wait that expired earlier (in any kernel) leaves the status word set: later CTAs
    // then return at once instead of each running into its own time limit.
    __shared__ int s_poisoned;
    if (threadIdx.x == 0) s_poisoned = *reinterpret_cast<volatile int*>(p.status);
    __syncthreads();
    if (s_poisoned != 0) return;
    const Geometry& geo = p.geo;

    const int Tg = geo.tiles_per_group;
    int unit, rank;
    decode_block(blockIdx.x, geo.B * geo.H * geo.groups, Tg, &unit, &rank);
    const int g = unit % geo.groups;
    const int h = (unit / geo.groups) % geo.H;
    const int b = unit / (geo.groups * geo.H);
    const int hk = h / (geo.H / geo.Hkv);
    const int s = (h < geo.n_unshifted) ? 0 : geo.shift;
    const GroupLayout L = group_layout(geo, s, g);
    const int i = L.nTiles - 1 - rank;  // heaviest query tiles first
    if (i < 0) return;                  // this group has fewer tiles than the largest one
    const int j_begin = first_key_tile(L, i);
    const int n_steps = i + 1 - j_begin;  // key tiles j_begin .. i of the group (j_begin = 0 by default)
    const TileRef tq = tile_ref(L, i);
    const int tq0 = tq.tok0;

    if (threadIdx.x == 0) {
        mbar_init(&bars->res_full, 1);
        mbar_init(&bars->acc_full, 1);
        mbar_init(&bars->drain, 1);
        mbar_init(&bars->drain2, 1);
        mbar_init(&bars->dp_ready, 1);
        mbar_init(&bars->dp_free, 256);
        for (int x = 0; x < 2; ++x) {
            mbar_init(&bars->s_ready[x], 1);
            mbar_init(&bars->p_full[x], 256);
            mbar_init(&bars->buf_free[x], 1);
            mbar_init(&bars->v_full[x], 1);
            mbar_init(&bars->v_empty[x], 1);
        }
        for (int x = 0; x < C::kRingK; ++x) {
            mbar_init(&bars->k_full[x], 1);
            mbar_init(&bars->k_empty[x], 1);
        }
        bars->abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&p.tm_q);
        tma_prefetch_desc(&p.tm_do);
        tma_prefetch_desc(&p.tm_k);
        tma_prefetch_desc(&p.tm_v);
    }
    if (warp == 3) {
        tmem_alloc(&bars->tmem_slot, C::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_slot;
    const WaitCtx ctx{&bars->abort_flag, p.status, p.host_status};
    constexpr uint32_t kColAcc = 0, kColS = 128, kColP = 384;

    if (warp == 0) {
        if (lane == 0) {
            mbar_expect_tx(&bars->res_full, 2 * C::kTileBytes);
            for (int bx = 0; bx < C::kBoxes; ++bx) {
                tma_load_4d(sQ + bx * C::kBoxBytes, &p.tm_q, &bars->res_full, bx * 64, h, tq0, b);
                tma_load_4d(sDO + bx * C::kBoxBytes, &p.tm_do, &bars->res_full, bx * 64, h, tq0, b);
            }
            int n = 0;
            for (; n < n_steps; ++n) {
                const int st = n & 1;
                const uint32_t ph = (n >> 1) & 1;
                const int tk0 = tile_ref(L, j_begin + n).tok0;
                if (!mbar_wait(&bars->v_empty[st], ph ^ 1, ctx, kWaitBwdDq + 1)) break;
                mbar_expect_tx(&bars->v_full[st], C::kTileBytes);
                for (int bx = 0; bx < C::kBoxes; ++bx)
                    tma_load_4d(sV + st * C::kTileBytes + bx * C::kBoxBytes, &p.tm_v, &bars->v_full[st], bx * 64, hk, tk0, b);
                const int sk = n % C::kRingK;
                const uint32_t phk = (n / C::kRingK) & 1;
                if (!mbar_wait(&bars->k_empty[sk], phk ^ 1, ctx, kWaitBwdDq + 8)) {
                    mbar_wait_drain(&bars->v_full[st], ph);
                    break;
                }
                mbar_expect_tx(&bars->k_full[sk], C::kTileBytes);
                for (int bx = 0; bx < C::kBoxes; ++bx)
                    tma_load_4d(sK + sk * C::kTileBytes + bx * C::kBoxBytes, &p.tm_k, &bars->k_full[sk], bx * 64, hk, tk0, b);
            }
            if (bars->abort_flag != 0) {
                // let loads that are still in flight land before the CTA gives its memory back
                mbar_wait_drain(&bars->res_full, 0);
                for (int nn = (n > C::kRingK ? n - C::kRingK : 0); nn < n; ++nn)
                    mbar_wait_drain(&bars->k_full[nn % C::kRingK], (nn / C::kRingK) & 1);
                for (int nn = (n > C::kRingV ? n - C::kRingV : 0); nn < n; ++nn)
                    mbar_wait_drain(&bars->v_full[nn & 1], (nn >> 1) & 1);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---- score MMAs: dP_n = dO V_n^T first (its buffer is free as soon as the elementwise warps
        // hold dP_{n-1} in registers), then S_n = Q K_n^T into S buffer n & 1 (free once the dQ MMAs
        // of step n-2 are done).  The whole warp walks the loop so that addresses and descriptors
        // stay warp-uniform values; only the MMA and commit instructions are issued by one elected lane.
        constexpr uint32_t idesc_sc = idesc_bf16(128, kTile, 0, 0);
        const uint32_t dQ = desc_lo_k_major(smem_u32(sQ)), dDO = desc_lo_k_major(smem_u32(sDO));
        const uint32_t tP = tmem_base + kColP;
        bool ok = mbar_wait_uniform(&bars->res_full, 0, ctx, kWaitBwdDq + 3);
        for (int n = 0; ok && n < n_steps; ++n) {
            const int st = n & 1;
            const uint32_t ph = (n >> 1) & 1;
            const int sk = n % C::kRingK;
            // the two TMA barriers first: they have usually completed long ago, and every wait that sits
            // between the two groups of MMAs below is time the tensor pipe idles
            if (!mbar_wait_uniform(&bars->v_full[st], ph, ctx, kWaitBwdDq + 2)) break;
            if (!mbar_wait_uniform(&bars->k_full[sk], (n / C::kRingK) & 1, ctx, kWaitBwdDq + 10)) break;
            if (n >= 1 && !mbar_wait_uniform(&bars->dp_free, (n - 1) & 1, ctx, kWaitBwdDq + 9)) break;
            tc_fence_after();
            const uint32_t dV = desc_lo_k_major(smem_u32(sV + st * C::kTileBytes));
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk)
                    mma_ss(tP, dDO + desc_step_k_major(kk, C::kBoxBytes), dV + desc_step_k_major(kk, C::kBoxBytes), idesc_sc, kk > 0);
                mma_commit(&bars->v_empty[st]);
                mma_commit(&bars->dp_ready);
            }
            __syncwarp();
            if (n >= 2 && !mbar_wait_uniform(&bars->buf_free[st], ph ^ 1, ctx, kWaitBwdDq + 7)) break;
            tc_fence_after();
            const uint32_t dK = desc_lo_k_major(smem_u32(sK + sk * C::kTileBytes));
            const uint32_t tS = tmem_base + kColS + st * kTile;
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk)
                    mma_ss(tS, dQ + desc_step_k_major(kk, C::kBoxBytes), dK + desc_step_k_major(kk, C::kBoxBytes), idesc_sc, kk > 0);
                mma_commit(&bars->s_ready[st]);
            }
            __syncwarp();
        }
        if (__any_sync(0xffffffffu, bars->abort_flag != 0)) {
            if (elect_one()) {
                mma_commit(&bars->drain2);
                mbar_wait_drain(&bars->drain2, 0);
            }
        }
        __syncwarp();
    } else if (warp == 2) {
        // ---- gradient MMAs: dQ += dS_n K_n
        constexpr uint32_t idesc_acc = idesc_bf16(128, HD, 0, 1);
        for (int n = 0; n < n_steps; ++n) {
            const int st = n & 1;
            if (!mbar_wait_uniform(&bars->p_full[st], (n >> 1) & 1, ctx, kWaitBwdDq + 4)) break;
            tc_fence_after();
            const int sk = n % C::kRingK;
            const uint32_t dKmn = desc_lo_mn_major(smem_u32(sK + sk * C::kTileBytes), C::kBoxBytes);
            const uint32_t tdS = tmem_base + kColS + st * kTile;  // bf16 dS over the S buffer
            if (elect_one()) {
#pragma unroll
                for (int kk = 0; kk < kTile / 16; ++kk)
                    mma_ts(tmem_base + kColAcc, tdS + (kk >> 2) * 64 + (kk & 3) * 8, dKmn + kk * kDescStepMn, idesc_acc,
                           (n > 0) || (kk > 0));
                mma_commit(&bars->k_empty[sk]);
                mma_commit(&bars->buf_free[st]);
                if (n == n_steps - 1) mma_commit(&bars->acc_full);
            }
            __syncwarp();
        }
        if (__any_sync(0xffffffffu, bars->abort_flag != 0)) {
            // MMAs already issued (by either MMA warp) must finish before tensor memory is released
            if (elect_one()) {
                mma_commit(&bars->drain);
                mbar_wait_drain(&bars->drain, 0);
            }
        }
        __syncwarp();
    } else if (warp == 3) {
        // spare warp: owns the tensor-memory allocation only
    } else {
        // ---- elementwise: thread (quad, lane, half) owns columns [64 half, +64) of score row
        // 32 quad + lane.  Its 64 bf16 dS values (32 packed columns) go over the first 32 of its own
        // columns, so the two halves never write into columns the other half still has to read: the
        // 128 K values of the dS operand sit at packed columns [0,32) and [64,96) of the S buffer.
        const int quad = warp & 3;
        const int half = (warp - 4) >> 2;
        const int row = quad * 32 + lane;
        const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
        // rows past the end of a ragged tile are not part of the group: they are computed on whatever
        // the box holds there and never stored
        const bool row_valid = row < tq.valid;
        const size_t stat_idx = (static_cast<size_t>(b) * geo.H + h) * geo.N + tq0 + row;
        const float neg_lse2 = row_valid ? -p.lse[stat_idx] * kLog2e : 0.f;
        const float Drow = row_valid ? p.Dsum[stat_idx] : 0.f;
        const float c2 = p.scale_log2;
        const uint64_t c2x2 = f2_pack(c2, c2), nlx2 = f2_pack(neg_lse2, neg_lse2), Dx2 = f2_pack(Drow, Drow);
        bool ok = true;
        uint32_t dp[64];  // this thread's part of dP_n
        // Copy dP_m out of tensor memory and release its buffer.  Done for step 0 up front and for step
        // n+1 at the END of step n (dP_{n+1} has been complete for a long time by then), so that dP_{n+2}
        // and S_{n+2} can be issued while step n+1 is still being worked on.
        auto fetch_dp = [&](int m) -> bool {
            if (!mbar_wait(&bars->dp_ready, m & 1, ctx, kWaitBwdDq + 5)) return false;
            tc_fence_after();
            tmem_ld_32x32(t_row + kColP + half * 64, *reinterpret_cast<uint32_t(*)[32]>(&dp[0]));
            tmem_ld_32x32(t_row + kColP + half * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&dp[32]));
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(&bars->dp_free);
            return true;
        };
        ok = fetch_dp(0);
        for (int n = 0; ok && n < n_steps; ++n) {
            const int st = n & 1;
            if (!mbar_wait(&bars->s_ready[st], (n >> 1) & 1, ctx, kWaitBwdDq + 11)) { ok = false; break; }
            tc_fence_after();
            // Key x of the tile is visible to query row r iff it is one of the tile's valid rows and,
            // in the diagonal tile, x <= r.  Off the diagonal a full tile needs no mask at all.
            const int k_valid = tile_ref(L, j_begin + n).valid;
            const bool last = (n == n_steps - 1);
            const bool masked = last || k_valid < kTile;
            const int vis = (last && row < k_valid) ? row : k_valid - 1;
            const int lim = vis - half * 64;  // visible iff (column within this half) <= lim
            const uint32_t tS = t_row + kColS + st * kTile + half * 64;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t sr[32];
                tmem_ld_32x32(tS + c * 32, sr);
                tmem_wait_ld();
                uint32_t pk[16];
                if (masked) {
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        float pe0 = fast_exp2(fmaf(__uint_as_float(sr[2 * e]), c2, neg_lse2));
                        float pe1 = fast_exp2(fmaf(__uint_as_float(sr[2 * e + 1]), c2, neg_lse2));
                        if (c * 32 + 2 * e > lim) pe0 = 0.f;
                        if (c * 32 + 2 * e + 1 > lim) pe1 = 0.f;
                        pk[e] = pack_bf16(pe0 * (__uint_as_float(dp[c * 32 + 2 * e]) - Drow),
                                          pe1 * (__uint_as_float(dp[c * 32 + 2 * e + 1]) - Drow));
                    }
                } else {
                    // two columns per instruction for the multiply-adds
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        const uint64_t x = f2_fma(f2_pack(__uint_as_float(sr[2 * e]), __uint_as_float(sr[2 * e + 1])), c2x2, nlx2);
                        float x0, x1;
                        f2_unpack(x, x0, x1);
                        // part of the exponentials goes to the FMA pipe (see poly_exp2_x2)
                        const uint64_t pe = ((kPolyExpMask >> e) & 1u) ? poly_exp2_x2(x) : f2_pack(fast_exp2(x0), fast_exp2(x1));
                        const uint64_t t = f2_sub(f2_pack(__uint_as_float(dp[c * 32 + 2 * e]), __uint_as_float(dp[c * 32 + 2 * e + 1])), Dx2);
                        float d0, d1;
                        f2_unpack(f2_mul(pe, t), d0, d1);
                        pk[e] = pack_bf16(d0, d1);
                    }
                }
                // packed columns [16c, 16c+16) overlay score columns [16c, 16c+16) of this half, which
                // have been read already (c = 1 writes over columns 16..31, read when c was 0)
                tmem_st_32x16(tS + c * 16, pk);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(&bars->p_full[st]);
            if (n + 1 < n_steps && !fetch_dp(n + 1)) { ok = false; break; }
        }
        if (ok && mbar_wait(&bars->acc_full, 0, ctx, kWaitBwdDq + 6)) {
            tc_fence_after();
            __nv_bfloat16* dst = p.dq + (static_cast<size_t>(b) * geo.N + tq0 + row) * p.dq_tok_stride + static_cast<size_t>(h) * HD;
            store_acc_cols<HD / 2>(t_row + kColAcc + half * (HD / 2), p.scale, dst + half * (HD / 2), row_valid);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 3) {
        tc_fence_after();
        tmem_dealloc(tmem_base, C::kTmemCols);
    }
}

// ------------------------------------------------------------------------------------------------
// 3. dK, dV
// ------------------------------------------------------------------------------------------------
// Tensor memory columns: dV [0,HD)  dK [128,128+HD)  S^T buffers [256,320) [320,384)  dP^T [384,448)
//                        K (bf16, the A operand of the score products) [448,448+HD/2)
// One dP^T buffer is enough because the elementwise warps copy their part of it into registers at the
// start of a step and release the buffer at once; that leaves room for a third S^T
// buffer, and with three steps in flight the chain scores -> elementwise -> gradient MMAs of one
// buffer no longer leaves the tensor pipe idle.
//
// The CTA owns key tile (b, hk, original tokens tk0 .. tk0+127).  For every query head hq that
// reads KV head hk (shift s): the tile sits at rolled position (tk0 - s) mod N, i.e. in group g at
// key tile j, and is attended by query sub-tiles (64 rows) 2j .. 2*nTiles-1 of that group.  (When the
// tiles are ragged the host only admits KV heads whose query heads all have the same shift, so the
// key tile is a tile of every head's partition.)
struct HeadWalk {
    GroupLayout L;
    int g, j, n_begin, n_end;
};
__device__ __forceinline__ HeadWalk head_walk(const Geometry& geo, int hq, int tk0) {
    HeadWalk w;
    const int s = (hq < geo.n_unshifted) ? 0 : geo.shift;
    const int pos = mod_pos(tk0 - s, geo.N);
    w.g = pos / geo.G;
    w.L = group_layout(geo, s, w.g);
    const int in_group = pos % geo.G;
    const int nB = w.L.nTiles - w.L.nA;
    w.j = in_group < w.L.lenA ? (w.L.swapped ? nB : 0) + in_group / kTile
                              : (w.L.swapped ? 0 : w.L.nA) + (in_group - w.L.lenA) / kTile;
    w.n_begin = 2 * w.j;
    w.n_end = 2 * end_query_tile(w.L, w.j);
    return w;
}

// A work item of the dK,dV kernel: key tile `j0` (in the partition of the KV head's first query head) of
// unit (b, hk, g0), in the block order shared by all kernels.  total_steps = 0 marks a slot of a group
// that has fewer tiles than the largest one.
struct DkDvItem {
    int b, hk, tk0, k_valid, total_steps;
};
__device__ __forceinline__ DkDvItem dkdv_item(const Geometry& geo, const SpillPass& pass, long long id) {
    DkDvItem t;
    int unit, j0;
    decode_block(id, geo.B * pass.nk * geo.groups, geo.tiles_per_group, &unit, &j0);
    const int g0 = unit % geo.groups;
    const int rep = geo.H / geo.Hkv;
    t.hk = pass.hk0 + (unit / geo.groups) % pass.nk;
    t.b = unit / (geo.groups * pass.nk);
    const int hq0 = t.hk * rep;
    const int s0 = (hq0 < geo.n_unshifted) ? 0 : geo.shift;
    const GroupLayout L0 = group_layout(geo, s0, g0);
    t.total_steps = 0;
    t.tk0 = 0, t.k_valid = 0;
    if (j0 >= L0.nTiles) return t;
    const TileRef tk = tile_ref(L0, j0);
    t.tk0 = tk.tok0;
    t.k_valid = tk.valid;
    for (int hq = hq0; hq < hq0 + rep; ++hq) {
        const HeadWalk w = head_walk(geo, hq, t.tk0);
        t.total_steps += w.n_end - w.n_begin;
    }
    return t;
}

// Barriers of the persistent dK,dV kernel.  Steps are counted through all items of the CTA (`it`), so
// the rings of stages and score buffers simply carry on from one item to the next.
template <int kStages>
struct DkDvBars {
    uint64_t res_full;            // K and V of an item landed (one phase per item)
    uint64_t kt_full;             // K of an item has been copied into tensor memory
    uint64_t kv_empty;            // the score products of an item are done: K and V may be overwritten
    uint64_t acc_full;            // all gradient MMAs of an item are done
    uint64_t acc_empty;           // the accumulators of an item have been read out
    uint64_t drain;               // abort path only (gradient MMA warp)
    uint64_t drain2;              // abort path only (score MMA warp)
    uint64_t s_full[3];           // S^T of a step is in tensor memory (buffer it % 3)
    uint64_t p_full[3];           // bf16 P^T and dS^T of a step are in tensor memory
    uint64_t buf_free[3];         // gradient MMAs that read a score buffer's bf16 operands are done
    uint64_t dp_free;             // the elementwise threads of a step hold their dP^T in registers
    uint64_t st_full[kStages];    // streamed operands of a stage landed
    uint64_t st_empty[kStages];   // MMAs reading a stage are done
    uint64_t sched_full[8];       // a work item id has been published
    long long item[8];
    uint32_t tmem_slot;
    int abort_flag;
};

// kSpill: every step's dS^T also goes to global memory (see SpillPass) for s2a_bwd_dq_spill_kernel.
//
// Persistent: one CTA per SM draws key tiles, heaviest first, from a counter in global memory.  The TMA
// warp runs ahead across items (the K and V of the next item are fetched as soon as the last score
// product of the current one has been issued and completed, its first query sub-tiles right behind),
// so that barrier set-up, tensor-memory allocation, the first loads and the pipeline fill are paid
// once per SM instead of once per key tile, and the score products of the next item run while the
// accumulators of the finished one are written out.
template <int HD, bool kSpill>
__global__ void __launch_bounds__(BwdCfg<HD>::kThreads, 1) s2a_bwd_dkdv_kernel(const __grid_constant__ BwdDkDvParams p) {
    using C = BwdCfg<HD>;
    using Bars = DkDvBars<C::kStages>;
    constexpr int kBufs = 2;   // S^T buffers in flight
    constexpr int kCols = 32;  // query columns per elementwise thread and step: two threads share a key row
    constexpr int kChunks = kCols / 16;
    constexpr int kSched = 8;  // item ids in flight: the TMA warp is at most five items ahead of the read-out
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sK = smem;                                // resident: K_j
    uint8_t* sV = sK + C::kBigTileBytes;               // resident: V_j
    uint8_t* sStage = sV + C::kBigTileBytes;           // per stage: Q_n then dO_n
    float* sStat = reinterpret_cast<float*>(sStage + C::kStages * C::kStageBytes);  // per stage: lse[64], D[64]
    Bars* bars = reinterpret_cast<Bars*>(reinterpret_cast<uint8_t*>(sStat) + C::kStages * 2 * C::kStatBytes);
    static_assert(sizeof(Bars) <= C::kBarBytes, "barrier block");

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    // A bounded wait that expired earlier (in any kernel) leaves the status word set: later CTAs
    // then return at once instead of each running into its own time limit.
    __shared__ int s_poisoned;
    if (threadIdx.x == 0) s_poisoned = *reinterpret_cast<volatile int*>(p.status);
    __syncthreads();
    if (s_poisoned != 0) return;
    const Geometry& geo = p.geo;
    const int rep = geo.H / geo.Hkv;
    const int Tg = geo.tiles_per_group;
    const long long n_items = static_cast<long long>(geo.B) * p.pass.nk * geo.groups * Tg;

    if (threadIdx.x == 0) {
        mbar_init(&bars->res_full, 1);
        mbar_init(&bars->kt_full, 256);
        mbar_init(&bars->kv_empty, 1);
        mbar_init(&bars->acc_full, 1);
        mbar_init(&bars->acc_empty, 256);
        mbar_init(&bars->drain, 1);
        mbar_init(&bars->drain2, 1);
        for (int x = 0; x < kBufs; ++x) {
            mbar_init(&bars->s_full[x], 1);
            mbar_init(&bars->p_full[x], 256);
            mbar_init(&bars->buf_free[x], 1);
        }
        mbar_init(&bars->dp_free, 256);
        for (int st = 0; st < C::kStages; ++st) {
            mbar_init(&bars->st_full[st], 1);
            mbar_init(&bars->st_empty[st], 1);
        }
        for (int x = 0; x < kSched; ++x) mbar_init(&bars->sched_full[x], 1);
        bars->abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&p.tm_q);
        tma_prefetch_desc(&p.tm_do);
        tma_prefetch_desc(&p.tm_k);
        tma_prefetch_desc(&p.tm_v);
    }
    if (warp == 3) {
        tmem_alloc(&bars->tmem_slot, C::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_slot;
    const WaitCtx ctx{&bars->abort_flag, p.status, p.host_status};
    constexpr uint32_t kColDV = 0, kColDK = 128, kColS = 256, kColP = 384, kColKt = 448;

    // Every consumer role walks the same sequence of items: wait for the k-th id, stop at the end marker.
    auto next_item = [&](int k, int where, long long* id) -> bool {
        if (!mbar_wait(&bars->sched_full[k % kSched], (k / kSched) & 1, ctx, where)) return false;
        *id = bars->item[k % kSched];
        return *id < n_items;
    };

    if (warp == 0) {
        if (lane == 0) {
            int it = 0;
            int last_res = -1;  // newest item whose K and V were requested
            bool ok = true;
            for (int k = 0; ok; ++k) {
                // draw the next item that has work; the other warps only see real items and the end marker
                long long id;
                DkDvItem t;
                do {
                    id = static_cast<long long>(atomicAdd(p.counter, 1));
                    if (id >= n_items) break;
                    t = dkdv_item(geo, p.pass, id);
                } while (t.total_steps == 0);
                bars->item[k % kSched] = id;
                mbar_arrive(&bars->sched_full[k % kSched]);  // release: the id is visible to whoever sees the phase
                if (id >= n_items) break;
                // K and V of the item: their buffers are free once the score products of the previous item are done
                if (k > 0 && !mbar_wait(&bars->kv_empty, (k - 1) & 1, ctx, kWaitBwdDkDv + 10)) break;
                mbar_expect_tx(&bars->res_full, 2 * C::kBigTileBytes);
                for (int bx = 0; bx < C::kBoxes; ++bx) {
                    tma_load_4d(sK + bx * C::kBigBoxBytes, &p.tm_k, &bars->res_full, bx * 64, t.hk, t.tk0, t.b);
                    tma_load_4d(sV + bx * C::kBigBoxBytes, &p.tm_v, &bars->res_full, bx * 64, t.hk, t.tk0, t.b);
                }
                last_res = k;
                const int hq0 = t.hk * rep;
                for (int hq = hq0; ok && hq < hq0 + rep; ++hq) {
                    const HeadWalk w = head_walk(geo, hq, t.tk0);
                    for (int n = w.n_begin; n < w.n_end; ++n, ++it) {
                        const int st = it % C::kStages;
                        const uint32_t ph = (it / C::kStages) & 1;
                        const TileRef tq = subtile_ref(w.L, n);
                        const int tq0 = tq.tok0;
                        // statistics of the valid rows only (a multiple of 4 rows, so of 16 bytes): a ragged
                        // sub-tile must not read past the end of the arrays
                        const uint32_t stat_bytes = static_cast<uint32_t>(tq.valid) * 4u;
                        if (!mbar_wait(&bars->st_empty[st], ph ^ 1, ctx, kWaitBwdDkDv + 1)) { ok = false; break; }
                        mbar_expect_tx(&bars->st_full[st], C::kStageBytes + 2 * stat_bytes);
                        uint8_t* sQ = sStage + st * C::kStageBytes;
                        uint8_t* sDO = sQ + C::kSubTileBytes;
                        for (int bx = 0; bx < C::kBoxes; ++bx) {
                            tma_load_4d(sQ + bx * C::kSubBoxBytes, &p.tm_q, &bars->st_full[st], bx * 64, hq, tq0, t.b);
                            tma_load_4d(sDO + bx * C::kSubBoxBytes, &p.tm_do, &bars->st_full[st], bx * 64, hq, tq0, t.b);
                        }
                        const size_t stat_idx = (static_cast<size_t>(t.b) * geo.H + hq) * geo.N + tq0;
                        if (stat_bytes != 0) {
                            bulk_load_1d(sStat + st * 2 * kSubTile, p.lse + stat_idx, stat_bytes, &bars->st_full[st]);
                            bulk_load_1d(sStat + st * 2 * kSubTile + kSubTile, p.Dsum + stat_idx, stat_bytes, &bars->st_full[st]);
                        }
                    }
                }
            }
            if (bars->abort_flag != 0) {
                // let loads that are still in flight land before the CTA gives its memory back: K and V of
                // the newest item and the stages issued last
                if (last_res >= 0) mbar_wait_drain(&bars->res_full, last_res & 1);
                for (int nn = (it > C::kStages ? it - C::kStages : 0); nn < it; ++nn)
                    mbar_wait_drain(&bars->st_full[nn % C::kStages], (nn / C::kStages) & 1);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---- score MMAs of step `it`: dP^T = V dO^T into the single dP^T buffer (free as soon as the
        // elementwise warps hold the previous one in registers), then S^T = K Q^T into buffer it % 3
        // (warp-uniform loop, one elected lane issues; see the dQ kernel)
        constexpr uint32_t idesc_sc = idesc_bf16(128, kSubTile, 0, 0);
        const uint32_t dV = desc_lo_k_major(smem_u32(sV));
        const uint32_t tP = tmem_base + kColP, tKt = tmem_base + kColKt;
        int it = 0;
        bool ok = true;
        for (int k = 0; ok; ++k) {
            long long id = n_items;
            if (!__all_sync(0xffffffffu, next_item(k, kWaitBwdDkDv + 11, &id) ? 1 : 0)) break;  // warp-uniform outcome
            const DkDvItem t = dkdv_item(geo, p.pass, id);
            if (!mbar_wait_uniform(&bars->res_full, k & 1, ctx, kWaitBwdDkDv + 3)) break;
            if (!mbar_wait_uniform(&bars->kt_full, k & 1, ctx, kWaitBwdDkDv + 16)) break;
            for (int x = 0; x < t.total_steps; ++x, ++it) {
                const int st = it % C::kStages;
                const int bf = it % kBufs;
                if (!mbar_wait_uniform(&bars->st_full[st], (it / C::kStages) & 1, ctx, kWaitBwdDkDv + 2)) { ok = false; break; }
                if (it >= 1 && !mbar_wait_uniform(&bars->dp_free, (it - 1) & 1, ctx, kWaitBwdDkDv + 9)) { ok = false; break; }
                tc_fence_after();
                const uint32_t aQ = smem_u32(sStage + st * C::kStageBytes);
                const uint32_t dQ = desc_lo_k_major(aQ), dDO = desc_lo_k_major(aQ + C::kSubTileBytes);
                if (elect_one()) {
#pragma unroll
                    for (int kk = 0; kk < HD / 16; ++kk)
                        mma_ss(tP, dV + desc_step_k_major(kk, C::kBigBoxBytes), dDO + desc_step_k_major(kk, C::kSubBoxBytes),
                               idesc_sc, kk > 0);
                }
                __syncwarp();
                if (it >= kBufs && !mbar_wait_uniform(&bars->buf_free[bf], ((it / kBufs) & 1) ^ 1, ctx, kWaitBwdDkDv + 8)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tS = tmem_base + kColS + bf * kSubTile;
                if (elect_one()) {
#pragma unroll
                    for (int kk = 0; kk < HD / 16; ++kk)
                        mma_ts(tS, tKt + 8 * kk, dQ + desc_step_k_major(kk, C::kSubBoxBytes), idesc_sc, kk > 0);
                    mma_commit(&bars->s_full[bf]);
                    if (x == t.total_steps - 1) mma_commit(&bars->kv_empty);  // nothing reads this item's K and V any more
                }
                __syncwarp();
            }
        }
        if (__any_sync(0xffffffffu, bars->abort_flag != 0)) {
            if (elect_one()) {
                mma_commit(&bars->drain2);
                mbar_wait_drain(&bars->drain2, 0);
            }
        }
        __syncwarp();
    } else if (warp == 2) {
        // ---- gradient MMAs: dV += P^T dO and dK += dS^T Q of step `it`; both bf16 operands sit in
        // the step's S^T buffer
        constexpr uint32_t idesc_acc = idesc_bf16(128, HD, 0, 1);
        int it = 0;
        bool ok = true;
        for (int k = 0; ok; ++k) {
            long long id = n_items;
            if (!__all_sync(0xffffffffu, next_item(k, kWaitBwdDkDv + 12, &id) ? 1 : 0)) break;  // warp-uniform outcome
            const DkDvItem t = dkdv_item(geo, p.pass, id);
            for (int x = 0; x < t.total_steps; ++x, ++it) {
                const int st = it % C::kStages;
                const int bf = it % kBufs;
                if (!mbar_wait_uniform(&bars->p_full[bf], (it / kBufs) & 1, ctx, kWaitBwdDkDv + 4)) { ok = false; break; }
                // the first products of an item overwrite the accumulators: the previous item's must have been read out
                if (x == 0 && k > 0 && !mbar_wait_uniform(&bars->acc_empty, (k - 1) & 1, ctx, kWaitBwdDkDv + 13)) { ok = false; break; }
                tc_fence_after();
                const uint32_t aQ = smem_u32(sStage + st * C::kStageBytes);
                const uint32_t dQmn = desc_lo_mn_major(aQ, C::kSubBoxBytes);
                const uint32_t dDOmn = desc_lo_mn_major(aQ + C::kSubTileBytes, C::kSubBoxBytes);
                // the 16 queries of K slice kk: P^T in packed columns [16 kk, +8) of the buffer, dS^T in [16 kk + 8, +8)
                const uint32_t tPt = tmem_base + kColS + bf * kSubTile;
                if (elect_one()) {
#pragma unroll
                    for (int kk = 0; kk < kSubTile / 16; ++kk)
                        mma_ts(tmem_base + kColDV, tPt + 16 * kk, dDOmn + kk * kDescStepMn, idesc_acc, (x > 0) || (kk > 0));
#pragma unroll
                    for (int kk = 0; kk < kSubTile / 16; ++kk)
                        mma_ts(tmem_base + kColDK, tPt + 16 * kk + 8, dQmn + kk * kDescStepMn, idesc_acc, (x > 0) || (kk > 0));
                    mma_commit(&bars->st_empty[st]);
                    mma_commit(&bars->buf_free[bf]);
                    if (x == t.total_steps - 1) mma_commit(&bars->acc_full);
                }
                __syncwarp();
            }
        }
        if (__any_sync(0xffffffffu, bars->abort_flag != 0)) {
            if (elect_one()) {
                mma_commit(&bars->drain);
                mbar_wait_drain(&bars->drain, 0);
            }
        }
        __syncwarp();
    } else if (warp == 3) {
        // spare warp: owns the tensor-memory allocation only
    } else {
        // ---- elementwise.  Thread (quad, lane, group) owns key row 32 quad + lane and the query columns
        // [32 group, +32) of every step.  (Letting the two groups of four warps take alternate steps with a
        // whole row per thread was measured too: with two S^T buffers the chain S^T -> elementwise ->
        // gradient MMAs of a buffer is what a step waits for, and half the columns per thread halve its
        // elementwise part: 3.33 against 3.53 ms on the Llama2-7B 32k shape.)
        const int quad = warp & 3;
        const int group = (warp - 4) >> 2;
        const int row = quad * 32 + lane;  // key row of the tile owned by this thread
        const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
        const float c2 = p.scale_log2;
        bool ok = true;
        int it = 0;
        auto lds4 = [](uint32_t a) {
            // explicit shared-memory loads: through a generic pointer they cost far more latency
            float4 r;
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w) : "r"(a));
            return r;
        };
        // K of item k goes from its shared-memory tile into tensor memory, where it is the A operand of
        // S^T = K Q^T: an A operand in shared memory would be read again by every step (4 KB per MMA
        // against 2 KB of B), and shared-memory bandwidth is what bounds this kernel.  Row `row`, columns
        // [64 group, +64) of d: eight 16-byte chunks of the 128-byte-swizzled row, 32 packed columns.
        auto copy_k = [&](int k) -> bool {
            if (!mbar_wait(&bars->res_full, k & 1, ctx, kWaitBwdDkDv + 17)) return false;
            if (group * 64 < HD) {
                const uint32_t src = smem_u32(sK) + group * C::kBigBoxBytes + row * 128;
                uint32_t kr[32];
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                                 : "=r"(kr[4 * c]), "=r"(kr[4 * c + 1]), "=r"(kr[4 * c + 2]), "=r"(kr[4 * c + 3])
                                 : "r"(src + ((c ^ (row & 7)) << 4)));
                }
                tmem_st_32x32(t_row + kColKt + group * 32, kr);
                tmem_wait_st();
            }
            tc_fence_before();
            mbar_arrive(&bars->kt_full);
            return true;
        };
        for (int k = 0; ok; ++k) {
            long long id;
            if (!next_item(k, kWaitBwdDkDv + 14, &id)) break;
            if (k == 0 && !copy_k(0)) break;   // later items: copied at the end of the item before
            const DkDvItem t = dkdv_item(geo, p.pass, id);
            const bool key_valid = row < t.k_valid;  // rows past the end of a ragged tile belong to other tiles
            const int hq0 = t.hk * rep;
            for (int hq = hq0; ok && hq < hq0 + rep; ++hq) {
                const HeadWalk w = head_walk(geo, hq, t.tk0);
                // where this thread's dS^T values go when they are spilled: key row `row` of block (j, n) of the
                // spill unit (b, hq, g).  A block is stored chunk-major (16-byte chunk c of row r at uint4 index
                // c * 128 + r), so the 32 lanes of a warp write 512 contiguous bytes at a time.
                uint4* spill_head = nullptr;
                if constexpr (kSpill) {
                    const long long su = (static_cast<long long>(t.b) * (p.pass.nk * rep) + (hq - p.pass.hk0 * rep)) * geo.groups + w.g;
                    spill_head = reinterpret_cast<uint4*>(p.spill + spill_block(su, Tg, w.j, w.n_begin) * kSpillBlockElems) + row;
                }
                for (int n = w.n_begin; n < w.n_end; ++n, ++it) {
                    const int cg0 = 2 * group;   // first 16-column chunk of this thread
                    const int st = it % C::kStages;
                    const int bf = it % kBufs;
                    // The statistics of this step travel with its stage.  s_full covers dP^T of this step as
                    // well: its MMAs were issued before those of S^T by the same thread, and a commit completes
                    // after everything issued before it.
                    if (!mbar_wait(&bars->st_full[st], (it / C::kStages) & 1, ctx, kWaitBwdDkDv + 5) ||
                        !mbar_wait(&bars->s_full[bf], (it / kBufs) & 1, ctx, kWaitBwdDkDv + 6)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    // copy this thread's part of dP^T into registers and release the single dP^T buffer as soon
                    // as the copy has landed, so that the dP^T product of the next step runs while this step is
                    // worked on
                    uint32_t pr[kCols];
                    tmem_ld_32x32(t_row + kColP + 16 * cg0, pr);
                    // S^T in two chunks of 16 columns; the bf16 results of a chunk go back over its 16 columns:
                    // P^T into the first 8 (packed), dS^T into the other 8
                    const uint32_t tS = t_row + kColS + bf * kSubTile;
                    uint32_t sbuf[2][16];
                    tmem_ld_32x16(tS + 16 * cg0, sbuf[0]);
                    tmem_ld_32x16(tS + 16 * (cg0 + 1), sbuf[1]);
                    tmem_wait_ld();
                    tc_fence_before();
                    mbar_arrive(&bars->dp_free);
                    const uint32_t stat_sa = smem_u32(sStat + st * 2 * kSubTile);  // lse[64] then D[64] of this stage
                    // query x of this sub-tile sees key row r iff x is a valid row of the sub-tile and, in the
                    // diagonal tile, 128 j + r <= 64 n + x
                    const int q_valid = subtile_ref(w.L, n).valid;
                    const bool masked = (n < w.n_begin + 2) || (q_valid < kSubTile);
                    const int lim = (n < w.n_begin + 2) ? row - (n & 1) * kSubTile : -64;  // visible iff lim <= x < q_valid
                    uint4* spill_dst = nullptr;
                    if constexpr (kSpill) spill_dst = spill_head + static_cast<size_t>(n - w.n_begin) * (kSpillBlockElems / 8);
#pragma unroll
                    for (int c = 0; c < kChunks; ++c) {
                        const int cg = cg0 + c;   // chunk within the sub-tile: queries [16 cg, +16)
                        const uint32_t (&sr)[16] = sbuf[c];
                        uint32_t pkP[8], pkS[8];
                        if (masked) {
                            // masked sub-tiles: scalar path.  Statistics of rows that are not valid were never
                            // loaded, so a masked entry is set to zero, never multiplied by zero.
#pragma unroll
                            for (int e4 = 0; e4 < 4; ++e4) {
                                const float4 l = lds4(stat_sa + (16 * cg + 4 * e4) * 4);
                                const float4 dd = lds4(stat_sa + kSubTile * 4 + (16 * cg + 4 * e4) * 4);
                                const float lv[4] = {l.x, l.y, l.z, l.w};
                                const float dv[4] = {dd.x, dd.y, dd.z, dd.w};
                                float pt[4], ds[4];
#pragma unroll
                                for (int u = 0; u < 4; ++u) {
                                    const int x = 16 * cg + 4 * e4 + u;   // query within the sub-tile
                                    const bool visible = (x >= lim) && (x < q_valid);
                                    const float pe = fast_exp2(fmaf(__uint_as_float(sr[4 * e4 + u]), c2, -lv[u] * kLog2e));
                                    pt[u] = visible ? pe : 0.f;
                                    ds[u] = visible ? pe * (__uint_as_float(pr[16 * c + 4 * e4 + u]) - dv[u]) : 0.f;
                                }
                                pkP[2 * e4] = pack_bf16(pt[0], pt[1]), pkP[2 * e4 + 1] = pack_bf16(pt[2], pt[3]);
                                pkS[2 * e4] = pack_bf16(ds[0], ds[1]), pkS[2 * e4 + 1] = pack_bf16(ds[2], ds[3]);
                            }
                        } else {
                            // two columns per instruction for the multiply-adds
                            const uint64_t c2x2 = f2_pack(c2, c2), nl2e = f2_pack(-kLog2e, -kLog2e);
#pragma unroll
                            for (int e4 = 0; e4 < 4; ++e4) {
                                const float4 l = lds4(stat_sa + (16 * cg + 4 * e4) * 4);
                                const float4 dd = lds4(stat_sa + kSubTile * 4 + (16 * cg + 4 * e4) * 4);
                                const uint64_t lp[2] = {f2_pack(l.x, l.y), f2_pack(l.z, l.w)};
                                const uint64_t dp[2] = {f2_pack(dd.x, dd.y), f2_pack(dd.z, dd.w)};
#pragma unroll
                                for (int u = 0; u < 2; ++u) {
                                    const int e = 4 * e4 + 2 * u;   // column within the chunk
                                    const int x = 16 * c + e;       // column among this thread's
                                    const uint64_t xs = f2_fma(f2_pack(__uint_as_float(sr[e]), __uint_as_float(sr[e + 1])), c2x2,
                                                               f2_mul(lp[u], nl2e));
                                    float x0, x1;
                                    f2_unpack(xs, x0, x1);
                                    const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
                                    pkP[e >> 1] = pack_bf16(p0, p1);
                                    const uint64_t tt = f2_sub(f2_pack(__uint_as_float(pr[x]), __uint_as_float(pr[x + 1])), dp[u]);
                                    float d0, d1;
                                    f2_unpack(f2_mul(f2_pack(p0, p1), tt), d0, d1);
                                    pkS[e >> 1] = pack_bf16(d0, d1);
                                }
                            }
                        }
                        tmem_st_32x8(tS + 16 * cg, pkP);
                        tmem_st_32x8(tS + 16 * cg + 8, pkS);
                        if constexpr (kSpill) {
                            // streaming stores: written once, read once by the dQ kernel much later
#pragma unroll
                            for (int cc = 0; cc < 2; ++cc) {
                                uint4 x = make_uint4(pkS[4 * cc], pkS[4 * cc + 1], pkS[4 * cc + 2], pkS[4 * cc + 3]);
                                if (!key_valid) x = make_uint4(0u, 0u, 0u, 0u);
                                __stcs(spill_dst + (2 * cg + cc) * kTile, x);
                            }
                        }
                    }
                    tmem_wait_st();
                    tc_fence_before();
                    mbar_arrive(&bars->p_full[bf]);
                }
            }
            if (!ok) break;
            // K of the next item, if there is one, while the last gradient MMAs of this one run: the TMA
            // warp fetched it as soon as the last score product of this item was done (which also means that
            // nothing reads the old copy any more)
            {
                long long next_id;
                if (next_item(k + 1, kWaitBwdDkDv + 18, &next_id)) {
                    if (!copy_k(k + 1)) break;
                } else if (bars->abort_flag != 0) {
                    break;
                }
            }
            if (!mbar_wait(&bars->acc_full, k & 1, ctx, kWaitBwdDkDv + 7)) break;
            tc_fence_after();
            const size_t out_row = (static_cast<size_t>(t.b) * geo.N + t.tk0 + row) * p.dkv_tok_stride + static_cast<size_t>(t.hk) * HD;
            if (group == 0) store_acc_cols<HD>(t_row + kColDV, 1.0f, p.dv + out_row, key_valid);
            else store_acc_cols<HD>(t_row + kColDK, p.scale, p.dk + out_row, key_valid);
            tc_fence_before();
            mbar_arrive(&bars->acc_empty);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 3) {
        tc_fence_after();
        tmem_dealloc(tmem_base, C::kTmemCols);
    }
}

// ------------------------------------------------------------------------------------------------
// 4. dQ from spilled dS^T
// ------------------------------------------------------------------------------------------------
// dQ_i = scale * sum_j dS_ij K_j over the key tiles j_begin..i of the group, with dS_ij read back from
// the blocks the spilling dK,dV kernel wrote: nothing is recomputed, the kernel is a chain of
// 128x128x128 products whose A operand streams from global memory once (memory bound).
//
// Persistent: one CTA per SM takes (unit, query tile) work items, heaviest first, from a counter in
// global memory.  Warp 0 draws the items and loads with TMA (it runs ahead across item boundaries, so
// the ring never drains between items), warp 1 issues the MMAs into one of two accumulators in tensor
// memory, warps 2-5 write the finished accumulator out while the next item is being multiplied.
// A block (j, n) is copied to shared memory as it lies in global memory (one bulk copy for the blocks
// (j, 2i) and (j, 2i+1), which are neighbours): chunk-major, i.e. the 16-byte chunk c (8 queries) of
// key row r at byte (c * 128 + r) * 16.  Eight key rows of one chunk are 128 contiguous bytes: the
// "core matrix" of an MN-major operand without swizzle (M = queries, K = keys), with 2048 bytes
// between chunks along M and 128 bytes between groups of 8 keys along K; the two blocks side by side
// are the 128-query A operand.  B is the K tile, MN-major (N = d) with the 128-byte swizzle TMA
// leaves, as in the recomputing dQ kernel.
template <int HD>
struct DqSpillCfg {
    static constexpr int kThreads = 192;  // TMA warp, MMA warp, four epilogue warps
    static constexpr int kBoxes = HD / 64;
    static constexpr int kKBoxBytes = kTile * 128;
    static constexpr int kKBytes = kBoxes * kKBoxBytes;
    static constexpr int kDsBlockBytes = kSpillBlockElems * 2;
    static constexpr int kStageBytes = 2 * kDsBlockBytes + kKBytes;
    static constexpr int kStages = 3;
    static constexpr int kSched = 8;  // work items the producer can be ahead of the epilogue: at most 5
    static constexpr int kBarBytes = 512;
    static constexpr int kSmemBytes = 1024 + kStages * kStageBytes + kBarBytes;
    static constexpr int kTmemCols = 256;  // two accumulators of 128 columns
};

struct DqSpillBars {
    uint64_t full[3], empty[3];
    uint64_t acc_full[2], acc_empty[2];
    uint64_t sched_full[8];
    uint64_t drain;
    long long item[8];
    uint32_t tmem_slot;
    int abort_flag;
};

struct DqSpillItem {
    int b, h, hk, i, j_begin, n_steps, tq0, q_valid;
    long long unit;
    GroupLayout L;
};
// Work item `id` (heaviest query tiles of a chunk of units first, as in the other kernels).  n_steps = 0
// marks a slot of a group that has fewer tiles than the largest one.
__device__ __forceinline__ DqSpillItem dq_spill_item(const Geometry& geo, const SpillPass& pass, long long id) {
    DqSpillItem t;
    const int rep = geo.H / geo.Hkv;
    const int heads = pass.nk * rep;
    int unit, rank;
    decode_block(id, geo.B * heads * geo.groups, geo.tiles_per_group, &unit, &rank);
    const int g = unit % geo.groups;
    t.h = pass.hk0 * rep + (unit / geo.groups) % heads;
    t.b = unit / (geo.groups * heads);
    t.hk = t.h / rep;
    t.unit = unit;
    const int s = (t.h < geo.n_unshifted) ? 0 : geo.shift;
    t.L = group_layout(geo, s, g);
    t.i = t.L.nTiles - 1 - rank;
    if (t.i < 0) {
        t.n_steps = 0;
        t.j_begin = 0, t.tq0 = 0, t.q_valid = 0;
        return t;
    }
    t.j_begin = first_key_tile(t.L, t.i);
    t.n_steps = t.i + 1 - t.j_begin;
    const TileRef tq = tile_ref(t.L, t.i);
    t.tq0 = tq.tok0;
    t.q_valid = tq.valid;
    return t;
}

template <int HD>
__global__ void __launch_bounds__(DqSpillCfg<HD>::kThreads, 1) s2a_bwd_dq_spill_kernel(const __grid_constant__ BwdDqSpillParams p) {
    using C = DqSpillCfg<HD>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    DqSpillBars* bars = reinterpret_cast<DqSpillBars*>(smem + C::kStages * C::kStageBytes);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    __shared__ int s_poisoned;
    if (threadIdx.x == 0) s_poisoned = *reinterpret_cast<volatile int*>(p.status);
    __syncthreads();
    if (s_poisoned != 0) return;
    const Geometry& geo = p.geo;
    const int Tg = geo.tiles_per_group;
    const long long n_items = static_cast<long long>(geo.B) * p.pass.nk * (geo.H / geo.Hkv) * geo.groups * Tg;

    if (threadIdx.x == 0) {
        for (int x = 0; x < C::kStages; ++x) {
            mbar_init(&bars->full[x], 1);
            mbar_init(&bars->empty[x], 1);
        }
        for (int x = 0; x < 2; ++x) {
            mbar_init(&bars->acc_full[x], 1);
            mbar_init(&bars->acc_empty[x], 128);
        }
        for (int x = 0; x < C::kSched; ++x) mbar_init(&bars->sched_full[x], 1);
        mbar_init(&bars->drain, 1);
        bars->abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&p.tm_k);
    }
    if (warp == 1) {
        tmem_alloc(&bars->tmem_slot, C::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_slot;
    const WaitCtx ctx{&bars->abort_flag, p.status, p.host_status};

    if (warp == 0) {
        // ---- scheduler + TMA producer -------------------------------------------------------------
        if (lane == 0) {
            long long it = 0;  // stage uses so far
            bool ok = true;
            for (int k = 0; ok; ++k) {
                // draw the next item that has work (slots of groups with fewer tiles than the largest are
                // skipped here, so the other warps only ever see real items and the end marker)
                long long id;
                DqSpillItem t;
                do {
                    id = static_cast<long long>(atomicAdd(p.counter, 1));
                    if (id >= n_items) break;
                    t = dq_spill_item(geo, p.pass, id);
                } while (t.n_steps == 0);
                bars->item[k % C::kSched] = id;
                mbar_arrive(&bars->sched_full[k % C::kSched]);  // release: the id is visible to whoever sees the phase
                if (id >= n_items) break;
                for (int n = 0; n < t.n_steps; ++n, ++it) {
                    const int st = static_cast<int>(it % C::kStages);
                    const uint32_t ph = static_cast<uint32_t>(it / C::kStages) & 1u;
                    if (!mbar_wait(&bars->empty[st], ph ^ 1, ctx, kWaitBwdDqSpill + 1)) { ok = false; break; }
                    const int j = t.j_begin + n;
                    uint8_t* sDs = smem + st * C::kStageBytes;
                    uint8_t* sK = sDs + 2 * C::kDsBlockBytes;
                    mbar_expect_tx(&bars->full[st], C::kStageBytes);
                    const long long blk = spill_block(t.unit, Tg, j, 2 * t.i);
                    bulk_load_1d(sDs, p.spill + blk * kSpillBlockElems, 2 * C::kDsBlockBytes, &bars->full[st]);
                    const int tk0 = tile_ref(t.L, j).tok0;
                    for (int bx = 0; bx < C::kBoxes; ++bx)
                        tma_load_4d(sK + bx * C::kKBoxBytes, &p.tm_k, &bars->full[st], bx * 64, t.hk, tk0, t.b);
                }
            }
            if (bars->abort_flag != 0) {
                for (long long nn = (it > C::kStages ? it - C::kStages : 0); nn < it; ++nn)
                    mbar_wait_drain(&bars->full[nn % C::kStages], static_cast<uint32_t>(nn / C::kStages) & 1u);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---- MMA issuer (warp-uniform loop, one elected lane issues) ------------------------------
        constexpr uint32_t idesc = idesc_bf16(128, HD, 1, 1);
        long long it = 0;
        bool ok = true;
        int used = 0;  // accumulator uses so far
        for (int k = 0; ok; ++k) {
            if (!mbar_wait_uniform(&bars->sched_full[k % C::kSched], (k / C::kSched) & 1, ctx, kWaitBwdDqSpill + 2)) break;
            const long long id = bars->item[k % C::kSched];
            if (id >= n_items) break;
            const DqSpillItem t = dq_spill_item(geo, p.pass, id);
            const int buf = used & 1;
            if (!mbar_wait_uniform(&bars->acc_empty[buf], ((used >> 1) & 1) ^ 1, ctx, kWaitBwdDqSpill + 3)) break;
            tc_fence_after();
            const uint32_t tAcc = tmem_base + buf * 128;
            for (int n = 0; n < t.n_steps; ++n, ++it) {
                const int st = static_cast<int>(it % C::kStages);
                if (!mbar_wait_uniform(&bars->full[st], static_cast<uint32_t>(it / C::kStages) & 1u, ctx, kWaitBwdDqSpill + 4)) { ok = false; break; }
                tc_fence_after();
                const uint32_t aDs = smem_u32(smem + st * C::kStageBytes);
                const uint32_t dA = desc_lo_mn_major_plain(aDs, 128);
                const uint32_t dB = desc_lo_mn_major(aDs + 2 * C::kDsBlockBytes, C::kKBoxBytes);
                if (elect_one()) {
#pragma unroll
                    for (int kk = 0; kk < kTile / 16; ++kk)
                        mma_ss_hi(tAcc, dA + kk * (256u >> 4), desc_hi_plain(2048), dB + kk * kDescStepMn, kDescHi, idesc,
                                  (n > 0) || (kk > 0));
                    mma_commit(&bars->empty[st]);
                    if (n == t.n_steps - 1) mma_commit(&bars->acc_full[buf]);
                }
                __syncwarp();
            }
            ++used;
        }
        if (__any_sync(0xffffffffu, bars->abort_flag != 0)) {
            if (elect_one()) {
                mma_commit(&bars->drain);
                mbar_wait_drain(&bars->drain, 0);
            }
        }
        __syncwarp();
    } else {
        // ---- epilogue: thread owns accumulator row 32 * quad + lane -------------------------------
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
        int used = 0;
        for (int k = 0;; ++k) {
            if (!mbar_wait(&bars->sched_full[k % C::kSched], (k / C::kSched) & 1, ctx, kWaitBwdDqSpill + 5)) break;
            const long long id = bars->item[k % C::kSched];
            if (id >= n_items) break;
            const DqSpillItem t = dq_spill_item(geo, p.pass, id);
            const int buf = used & 1;
            if (!mbar_wait(&bars->acc_full[buf], (used >> 1) & 1, ctx, kWaitBwdDqSpill + 6)) break;
            tc_fence_after();
            __nv_bfloat16* dst = p.dq + (static_cast<size_t>(t.b) * geo.N + t.tq0 + row) * p.dq_tok_stride + static_cast<size_t>(t.h) * HD;
            store_acc_cols<HD>(t_row + buf * 128, p.scale, dst, row < t.q_valid);
            tc_fence_before();
            mbar_arrive(&bars->acc_empty[buf]);
            ++used;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, C::kTmemCols);
    }
}

}  // namespace

cudaError_t configure_bwd() {
    cudaError_t e;
    e = cudaFuncSetAttribute(s2a_bwd_dq_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, DqCfg<64>::kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(s2a_bwd_dq_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, DqCfg<128>::kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(s2a_bwd_dkdv_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg<64>::kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(s2a_bwd_dkdv_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg<128>::kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(s2a_bwd_dkdv_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg<64>::kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(s2a_bwd_dkdv_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg<128>::kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(s2a_bwd_dq_spill_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, DqSpillCfg<64>::kSmemBytes);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(s2a_bwd_dq_spill_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                DqSpillCfg<128>::kSmemBytes);
}

cudaError_t launch_bwd_preprocess(const PreParams& p, int d, cudaStream_t stream) {
    const long long threads = static_cast<long long>(p.B) * p.N * p.H * (d / 8);
    const unsigned grid = static_cast<unsigned>((threads + 255) / 256);
    if (d == 64) s2a_bwd_preprocess_kernel<64><<<grid, 256, 0, stream>>>(p);
    else s2a_bwd_preprocess_kernel<128><<<grid, 256, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_bwd_dq(const BwdDqParams& p, int d, cudaStream_t stream) {
    const Geometry& g = p.geo;
    const unsigned grid = static_cast<unsigned>(static_cast<long long>(g.B) * g.H * g.groups * g.tiles_per_group);
    if (d == 64) s2a_bwd_dq_kernel<64><<<grid, DqCfg<64>::kThreads, DqCfg<64>::kSmemBytes, stream>>>(p);
    else s2a_bwd_dq_kernel<128><<<grid, DqCfg<128>::kThreads, DqCfg<128>::kSmemBytes, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_bwd_dkdv(const BwdDkDvParams& p, int d, int n_sm, cudaStream_t stream) {
    const Geometry& g = p.geo;
    const long long items = static_cast<long long>(g.B) * p.pass.nk * g.groups * g.tiles_per_group;
    const unsigned grid = static_cast<unsigned>(items < n_sm ? items : n_sm);
    if (p.spill != nullptr) {
        if (d == 64) s2a_bwd_dkdv_kernel<64, true><<<grid, BwdCfg<64>::kThreads, BwdCfg<64>::kSmemBytes, stream>>>(p);
        else s2a_bwd_dkdv_kernel<128, true><<<grid, BwdCfg<128>::kThreads, BwdCfg<128>::kSmemBytes, stream>>>(p);
    } else {
        if (d == 64) s2a_bwd_dkdv_kernel<64, false><<<grid, BwdCfg<64>::kThreads, BwdCfg<64>::kSmemBytes, stream>>>(p);
        else s2a_bwd_dkdv_kernel<128, false><<<grid, BwdCfg<128>::kThreads, BwdCfg<128>::kSmemBytes, stream>>>(p);
    }
    return cudaGetLastError();
}

cudaError_t launch_bwd_dq_spill(const BwdDqSpillParams& p, int d, int n_sm, cudaStream_t stream) {
    const Geometry& g = p.geo;
    const long long items = static_cast<long long>(g.B) * p.pass.nk * (g.H / g.Hkv) * g.groups * g.tiles_per_group;
    const unsigned grid = static_cast<unsigned>(items < n_sm ? items : n_sm);
    if (d == 64) s2a_bwd_dq_spill_kernel<64><<<grid, DqSpillCfg<64>::kThreads, DqSpillCfg<64>::kSmemBytes, stream>>>(p);
    else s2a_bwd_dq_spill_kernel<128><<<grid, DqSpillCfg<128>::kThreads, DqSpillCfg<128>::kSmemBytes, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace s2a
