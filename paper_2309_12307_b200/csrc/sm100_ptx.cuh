// Thin wrappers over the sm_100a instructions the S2-Attn kernels are built from:
// mbarrier, TMA (cp.async.bulk[.tensor]), tensor memory (tcgen05.alloc/ld/st) and the
// 5th-generation tensor-core MMA (tcgen05.mma) with its shared-memory / instruction descriptors.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace s2a {

// Longest a single wait may take (SM clock cycles, ~1 s) before the kernel gives up.
constexpr long long kWaitLimitCycles = 2000000000LL;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---------------------------------------------------------------------------------------------
// mbarrier
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Where bounded waits report: `abort_flag` lives in the CTA's shared memory (non-zero = this CTA is
// giving up), `status` is the device-wide status word (0 = fine, otherwise the code of the first
// wait that expired), `host_status` its mirror in mapped host memory, which the host entry points
// read without synchronising.
struct WaitCtx {
    volatile int* abort_flag;
    int* status;
    volatile int* host_status;
};

// Record that the wait `where` expired: in the CTA's abort flag, in the device status word (first
// code wins) and in its host-visible mirror.
__device__ __forceinline__ void report_expiry(const WaitCtx& ctx, int where) {
    *ctx.abort_flag = where;
    if (atomicCAS(ctx.status, 0, where) == 0) {
        *ctx.host_status = where;
        __threadfence_system();
    }
}

// Bounded wait.  Returns false if the CTA is aborting (another thread's wait expired) or if this
// wait expired (after `limit` SM clock cycles); in the latter case the expiry is reported.
// Callers leave their loop and go to the common teardown.
__device__ __forceinline__ bool mbar_wait_limit(uint64_t* bar, uint32_t parity, const WaitCtx& ctx, int where,
                                                long long limit) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 63u) == 0) {
            if (*ctx.abort_flag != 0) return false;
            if (clock64() - t0 > limit) {
                report_expiry(ctx, where);
                return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, const WaitCtx& ctx, int where) {
    return mbar_wait_limit(bar, parity, ctx, where, kWaitLimitCycles);
}
// All 32 lanes wait; the outcome is made warp-uniform so the warp can keep executing warp-wide
// instructions (or leave its loop) together.
__device__ __forceinline__ bool mbar_wait_uniform(uint64_t* bar, uint32_t parity, const WaitCtx& ctx, int where) {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, ctx, where) ? 1 : 0) != 0;
}
// One lane of a fully active warp (the same lane every time for a given warp).
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "elect.sync _|p, 0xffffffff;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(pred));
    return pred != 0;
}

// Teardown helper for an aborting CTA: wait (time-limited, ignoring the abort flag) for an
// operation that is still in flight so that it cannot land after the CTA's resources are reused.
__device__ __forceinline__ void mbar_wait_drain(uint64_t* bar, uint32_t parity) {
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > kWaitLimitCycles / 8) return;
    }
}

// ---------------------------------------------------------------------------------------------
// TMA
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* tmap) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(tmap) : "memory");
}
// 4-D tiled load global -> shared, completion counted in bytes on `bar`.
// Coordinates are (c0 = innermost ... c3 = outermost); c0 * element size must be a multiple of 16 B.
__device__ __forceinline__ void tma_load_4d(void* smem_dst, const CUtensorMap* tmap, uint64_t* bar, int c0, int c1,
                                            int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(tmap), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
// 1-D bulk copy global -> shared (addresses 16-byte aligned, size a multiple of 16 bytes).
__device__ __forceinline__ void bulk_load_1d(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(smem_dst)),
                 "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// ---------------------------------------------------------------------------------------------
// Tensor memory
// ---------------------------------------------------------------------------------------------
// Allocation / deallocation are warp-wide (.sync.aligned): call from one full warp.
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_slot, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_slot)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// A tensor-memory address is (lane << 16) | column.  A warp may only touch the 32 lanes of its own
// quadrant (warp index within the warpgroup): lanes [32 * (warp % 4), +32).

// 32 lanes x 32 consecutive 32-bit columns: thread i of the warp receives lane (lane0 + i),
// register j holds column (col0 + j).
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st_32x32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]),
          "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]),
          "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st_32x8(uint32_t taddr, const uint32_t (&r)[8]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
        : "memory");
}
__device__ __forceinline__ void tmem_st_32x16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}

// ---------------------------------------------------------------------------------------------
// MMA descriptors (bf16 operands, fp32 accumulation)
// ---------------------------------------------------------------------------------------------
// Shared-memory operand tiles are what a TMA box of 64 bf16 columns x R rows with 128-byte swizzle
// leaves behind: row r at byte r * 128, its 16-byte chunks permuted by (r & 7); 8 rows = one
// 1024-byte swizzle atom.  The tile base must be 1024-byte aligned.

constexpr uint32_t kSwizzleAtomBytes = 1024;
// A 64-bit shared-memory descriptor is {low word, high word}.  The high word is the same for every
// operand used here: stride between 8-row groups (1024 B >> 4) in bits 0-13, descriptor version 1
// in bit 14 (bit 46 of the descriptor), 128-byte swizzle (code 2) in bits 29-31 (bits 61-63).
// The low word carries the start address (>> 4, bits 0-13) and the leading-dimension offset
// (>> 4, bits 16-29), so stepping through a tile is a 32-bit add on the low word: the MMA-issuing
// thread is a single instruction stream and every instruction it spends on address arithmetic
// delays the tensor pipe.
constexpr uint32_t kDescHi = (kSwizzleAtomBytes >> 4) | (1u << 14) | (2u << 29);

// Operand whose contraction (K) index runs along the 128-byte rows ("K-major"): rows are the M or N
// index.  Add desc_step_k_major(kk, box_bytes) to reach the kk-th group of 16 K values.
__device__ __forceinline__ uint32_t desc_lo_k_major(uint32_t saddr) {
    return ((saddr & 0x3FFFFu) >> 4) | (1u << 16);  // leading offset unused for this layout
}
__host__ __device__ constexpr uint32_t desc_step_k_major(int kk, uint32_t box_bytes) {
    return ((kk >> 2) * box_bytes + (kk & 3) * 32u) >> 4;  // 4 groups of 16 per 64-column box
}
// Operand whose M or N index runs along the 128-byte rows ("MN-major"): rows are the K index.
// `block_stride_bytes` is the distance between consecutive 64-wide blocks of the M/N index (the
// size of one TMA box); groups of 8 K rows are 1024 bytes apart.  16 K rows further: + kDescStepMn.
__device__ __forceinline__ uint32_t desc_lo_mn_major(uint32_t saddr, uint32_t block_stride_bytes) {
    return ((saddr & 0x3FFFFu) >> 4) | (((block_stride_bytes >> 4) & 0x3FFFu) << 16);
}
constexpr uint32_t kDescStepMn = 2048u >> 4;
// MN-major operand WITHOUT swizzle: 8 K rows of one 16-byte chunk (8 values of the M/N index) are 128
// contiguous bytes; `k_group_bytes` separates consecutive groups of 8 K rows (low word, leading
// offset), `mn_chunk_bytes` consecutive chunks along M/N (high word, stride offset).
__device__ __forceinline__ uint32_t desc_lo_mn_major_plain(uint32_t saddr, uint32_t k_group_bytes) {
    return ((saddr & 0x3FFFFu) >> 4) | (((k_group_bytes >> 4) & 0x3FFFu) << 16);
}
__host__ __device__ constexpr uint32_t desc_hi_plain(uint32_t mn_chunk_bytes) {
    return ((mn_chunk_bytes >> 4) & 0x3FFFu) | (1u << 14);  // descriptor version 1, swizzle code 0
}

// Instruction descriptor for kind::f16 with bf16 A and B, fp32 D, M x N tile.
// a_mn / b_mn: operand is MN-major (1) or K-major (0).
__host__ __device__ constexpr uint32_t idesc_bf16(int M, int N, int a_mn, int b_mn) {
    return (1u << 4)                      // D format: fp32
           | (1u << 7)                    // A format: bf16
           | (1u << 10)                   // B format: bf16
           | ((uint32_t)a_mn << 15)       // A major-ness
           | ((uint32_t)b_mn << 16)       // B major-ness
           | ((uint32_t)(N >> 3) << 17)   // N / 8
           | ((uint32_t)(M >> 4) << 24);  // M / 16
}

// D[tmem] (+)= A[smem] * B[smem]; issued by ONE thread.  a_lo / b_lo: descriptor low words.
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc,
                                       uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        ".reg .b64 da, db;\n"
        "mov.b64 da, {%1, %5};\n"
        "mov.b64 db, {%2, %5};\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n"
        "}\n" ::"r"(d_tmem),
        "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHi)
        : "memory");
}
// The same with a separate high word for each operand (operands of different layouts).
__device__ __forceinline__ void mma_ss_hi(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                          uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        ".reg .b64 da, db;\n"
        "mov.b64 da, {%1, %2};\n"
        "mov.b64 db, {%3, %4};\n"
        "setp.ne.b32 p, %6, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n"
        "}\n" ::"r"(d_tmem),
        "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
        : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]; A holds bf16 pairs, one M row per lane, 16 K values per 8 columns.
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t idesc,
                                       uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        ".reg .b64 db;\n"
        "mov.b64 db, {%2, %5};\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %3, p;\n"
        "}\n" ::"r"(d_tmem),
        "r"(a_tmem), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHi)
        : "memory");
}
// Arrive once on `bar` when every MMA this thread issued so far has completed.
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

// ---------------------------------------------------------------------------------------------
// small helpers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Packed fp32 pairs (one 64-bit register pair, one instruction for two lanes of arithmetic):
// halves the number of issue slots the elementwise warps spend on multiplies and adds.
__device__ __forceinline__ uint64_t f2_pack(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void f2_unpack(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t f2_mul(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t f2_sub(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t f2_add(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// 2^x for a pair of fp32 values on the FMA and integer pipes instead of the special-function unit,
// whose 16 results per clock per SM bound the elementwise warps (a loop of tensor-memory load, exp2,
// multiply, pack and store alone runs at 1093 clocks per 128x128 tile, 358 without the exp2): split
// x = n + r with n = round(x), |r| <= 1/2 (adding 1.5 * 2^23 leaves n in the low mantissa bits), a
// cubic for 2^r (relative error 7.5e-5, far below the bf16 rounding that follows) and n added into
// the exponent field.  x is clamped at -126; meant for x <= 0 (probabilities).  It costs about as much
// issue time as the special-function unit saves, so only a fraction of the values should take it
// (5 of 16: 898 clocks for the same loop).
__device__ __forceinline__ uint64_t poly_exp2_x2(uint64_t x2) {
    float x0, x1;
    f2_unpack(x2, x0, x1);
    x0 = fmaxf(x0, -126.f);
    x1 = fmaxf(x1, -126.f);
    const uint64_t xc = f2_pack(x0, x1);
    const uint64_t magic = f2_pack(12582912.f, 12582912.f);
    const uint64_t t = f2_add(xc, magic);
    const uint64_t r = f2_sub(xc, f2_sub(t, magic));
    const uint64_t c3 = f2_pack(0.05517132207751274f, 0.05517132207751274f);
    const uint64_t c2 = f2_pack(0.24261054396629333f, 0.24261054396629333f);
    const uint64_t c1 = f2_pack(0.6932609677314758f, 0.6932609677314758f);
    const uint64_t c0 = f2_pack(0.9999281167984009f, 0.9999281167984009f);
    const uint64_t p = f2_fma(f2_fma(f2_fma(c3, r, c2), r, c1), r, c0);
    float p0, p1, t0, t1;
    f2_unpack(p, p0, p1);
    f2_unpack(t, t0, t1);
    p0 = __int_as_float(__float_as_int(p0) + (__float_as_int(t0) << 23));
    p1 = __int_as_float(__float_as_int(p1) + (__float_as_int(t1) << 23));
    return f2_pack(p0, p1);
}
// Which of the 16 column pairs of a 32-column chunk take poly_exp2_x2 (bit e = pair e): 5 of 16.
constexpr uint32_t kPolyExpMask = 0x4924u;
// two fp32 -> packed bf16x2 (lo in the low half), round-to-nearest-even
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

}  // namespace s2a
