// Host side of the C-ABI declared in include/s2a.h: argument validation, TMA tensor maps,
// kernel launches.  Nothing here allocates device memory.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <mutex>

#include "../../include/s2a.h"
#include "s2a_params.h"
#include "sm100_ptx.cuh"

namespace s2a {
namespace {

// Device-wide status word written by kernels whose bounded wait expired (one copy per device
// that loads this library).
__device__ int g_status_word;

// Host-visible mirrors of the status words, one per device (64 bytes apart): page-locked and mapped
// into the device address space, so that a kernel can store the code of an expired wait where the
// next entry point sees it without synchronising.  This is ordinary static memory, pinned in place
// once per process; nothing is allocated.
constexpr int kMirrorStride = 16;  // ints
constexpr int kMaxDevicesMirror = 64;
alignas(4096) int g_host_status[kMaxDevicesMirror * kMirrorStride];
bool g_host_status_registered = false;

thread_local int tl_last_cuda_error = 0;

constexpr int kMaxDevices = 64;
constexpr int kMaxHostChunks = 16;
struct DeviceState {
    bool ready = false;
    int* status_ptr = nullptr;        // device address of g_status_word
    volatile int* host_word = nullptr;  // this device's mirror, host address
    int* host_word_dev = nullptr;     // the same word as the device sees it
    int n_sm = 0;                     // multiprocessors (grid of the persistent kernel)
    // s2a_fwd_bwd_host only: copy streams and the events that order them against the caller's stream
    bool host_path_ready = false;
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    cudaEvent_t ev_start = nullptr, ev_done = nullptr, ev_in_done = nullptr;
    cudaEvent_t ev_in[kMaxHostChunks] = {}, ev_compute[kMaxHostChunks] = {};
};
DeviceState g_dev[kMaxDevices];
static_assert(kMaxDevices == kMaxDevicesMirror, "one mirror word per device");
std::mutex g_dev_mutex;  // guards the one-time set-up of a DeviceState (calls may come from several host threads)

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

int cuda_fail(cudaError_t e) {
    tl_last_cuda_error = static_cast<int>(e);
    return S2A_ERR_CUDA;
}

// Per-device set-up: architecture check, shared-memory attributes, address of the status word.
int prepare_device(DeviceState** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= kMaxDevices) return S2A_ERR_UNSUPPORTED;
    DeviceState& ds = g_dev[dev];
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (!ds.ready) {
        int major = 0;
        e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e != cudaSuccess) return cuda_fail(e);
        if (major != 10) return S2A_ERR_UNSUPPORTED;
        e = cudaDeviceGetAttribute(&ds.n_sm, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return cuda_fail(e);
        if (!g_encode) {
            void* fn = nullptr;
            cudaDriverEntryPointQueryResult qres;
            e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
            if (e != cudaSuccess) return cuda_fail(e);
            if (qres != cudaDriverEntryPointSuccess || !fn) return cuda_fail(cudaErrorNotSupported);
            g_encode = reinterpret_cast<EncodeTiledFn>(fn);
        }
        e = configure_fwd();
        if (e != cudaSuccess) return cuda_fail(e);
        e = configure_bwd();
        if (e != cudaSuccess) return cuda_fail(e);
        e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ds.status_ptr), g_status_word);
        if (e != cudaSuccess) return cuda_fail(e);
        if (!g_host_status_registered) {
            e = cudaHostRegister(g_host_status, sizeof g_host_status, cudaHostRegisterPortable | cudaHostRegisterMapped);
            if (e != cudaSuccess) return cuda_fail(e);
            g_host_status_registered = true;
        }
        ds.host_word = &g_host_status[dev * kMirrorStride];
        e = cudaHostGetDevicePointer(reinterpret_cast<void**>(&ds.host_word_dev), const_cast<int*>(ds.host_word), 0);
        if (e != cudaSuccess) return cuda_fail(e);
        ds.ready = true;
    }
    *out = &ds;
    return S2A_OK;
}

// bf16 tensor [B, N, heads, d] viewed as (d, heads, N, B); box = 64 columns x `box_rows` tokens of
// one head, written to shared memory with the 128-byte swizzle the MMA descriptors expect.
// `tok_stride` = elements between consecutive tokens (heads * d when the tensor is dense; 3 * H * d for
// the slices of a packed [B, N, 3, H, d] tensor).
int make_tmap(CUtensorMap* tm, const void* base, int d, int heads, int N, int B, int box_rows, long long tok_stride = 0) {
    if (tok_stride == 0) tok_stride = static_cast<long long>(heads) * d;
    const cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)heads, (cuuint64_t)N, (cuuint64_t)B};
    const cuuint64_t strides[3] = {(cuuint64_t)d * 2, (cuuint64_t)tok_stride * 2, (cuuint64_t)N * tok_stride * 2};
    const cuuint32_t box[4] = {64, 1, (cuuint32_t)box_rows, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        tl_last_cuda_error = static_cast<int>(cudaErrorInvalidValue);
        return S2A_ERR_CUDA;
    }
    return S2A_OK;
}

// variants 2 and 3 of Appendix B exclude each other; no other bits are defined
bool flags_ok(unsigned flags) {
    return (flags & ~static_cast<unsigned>(S2A_FLAG_LEAK_FREE | S2A_FLAG_SWAP_WRAPPED)) == 0 &&
           flags != (S2A_FLAG_LEAK_FREE | S2A_FLAG_SWAP_WRAPPED);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_shape(int B, int N, int H, int Hkv, int d, int G, float scale, int n_unshifted, int shift) {
    if (B <= 0 || N <= 0 || H <= 0 || Hkv <= 0 || d <= 0 || G <= 0) return S2A_ERR_INVALID_ARG;
    if (N % G != 0 || H % Hkv != 0) return S2A_ERR_INVALID_ARG;
    if (n_unshifted < 0 || n_unshifted > H) return S2A_ERR_INVALID_ARG;
    if (!(scale > 0.f) || !isfinite(scale)) return S2A_ERR_INVALID_ARG;
    if (shift <= -N || shift >= N) return S2A_ERR_INVALID_ARG;
    if (d != 64 && d != 128) return S2A_ERR_UNSUPPORTED;
    // Every run of tokens of a group must start and end on a multiple of 4 tokens (16 bytes of the
    // fp32 row statistics, which travel by bulk copies); a tensor map wants at least one whole box.
    if (G % 4 != 0 || shift % 4 != 0 || N < kTile) return S2A_ERR_UNSUPPORTED;
    // Ragged tiles (G or shift not a multiple of 128): the key tiles of a KV head follow the partition
    // of its query heads, which must then all have the same shift.
    if ((G % kTile != 0 || shift % kTile != 0) && n_unshifted % (H / Hkv) != 0) return S2A_ERR_UNSUPPORTED;
    // grid sizes and 32-bit token arithmetic
    const long long tiles = (long long)B * H * (N / G) * (G / kTile + 2);
    if (tiles > 0x7fffffffLL || (long long)N + G >= 0x40000000LL) return S2A_ERR_UNSUPPORTED;
    return S2A_OK;
}

// Shape rules of the default entry points (shift G/2 on the second half of the heads).
int check_default_shape(int N, int H, int d, int G) {
    if (d <= 0 || H <= 0 || (H & 1) || (G & 1)) return S2A_ERR_INVALID_ARG;
    if (G % 8 != 0) return (G > 0 && N > 0 && N % G == 0) ? S2A_ERR_UNSUPPORTED : S2A_ERR_INVALID_ARG;
    return S2A_OK;
}

Geometry make_geometry(int B, int N, int H, int Hkv, int G, int n_unshifted, int shift, unsigned flags = 0u) {
    Geometry g;
    g.B = B, g.N = N, g.H = H, g.Hkv = Hkv, g.G = G;
    g.n_unshifted = n_unshifted;
    g.shift = shift;
    g.groups = N / G;
    g.leak_free = (flags & S2A_FLAG_LEAK_FREE) ? 1 : 0;
    g.swap_wrapped = (flags & S2A_FLAG_SWAP_WRAPPED) ? 1 : 0;
    // the grid has one slot per (unit, tile rank); groups with fewer tiles leave their last slots idle
    g.tiles_per_group = 0;
    const int shifts[2] = {0, shift};
    for (int which = 0; which < 2; ++which) {
        if ((which == 0 && n_unshifted == 0) || (which == 1 && n_unshifted == H)) continue;
        for (int grp = 0; grp < g.groups; ++grp) {
            const int n = group_layout(g, shifts[which], grp).nTiles;
            if (n > g.tiles_per_group) g.tiles_per_group = n;
        }
    }
    return g;
}

constexpr float kLog2eHost = 1.4426950408889634f;

// Diagnostic kernel behind s2a_selftest_wait_expiry: one warp waits, with the library's own bounded
// wait and the given limit, on a barrier nothing ever arrives on.  The wait runs out, the expiry is
// reported exactly as a production kernel reports one, and the kernel returns.
constexpr int kWaitSelfTest = 900;
__global__ void __launch_bounds__(32) s2a_wait_selftest_kernel(int* status, int* host_status, long long limit) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();
    if (*reinterpret_cast<volatile int*>(status) != 0) return;  // like every kernel here: a set status word means "do nothing"
    const WaitCtx ctx{&abort_flag, status, host_status};
    mbar_wait_limit(&bar, 0, ctx, kWaitSelfTest + 1, limit);
}

}  // namespace
}  // namespace s2a

using namespace s2a;

#pragma GCC visibility push(default)
extern "C" {

int s2a_version(void) { return 200; }

int s2a_last_cuda_error(void) { return tl_last_cuda_error; }

const char* s2a_status_string(int status) {
    switch (status) {
        case S2A_OK: return "ok";
        case S2A_ERR_INVALID_ARG: return "invalid argument (null or misaligned pointer, bad size, or workspace too small)";
        case S2A_ERR_UNSUPPORTED: return "unsupported shape or device (need d in {64,128}, G and shift multiples of 4 tokens, N >= 128, sm_100)";
        case S2A_ERR_CUDA: return "a CUDA call failed; see s2a_last_cuda_error()";
        case S2A_ERR_TIMEOUT: return "a bounded device-side wait expired";
        case S2A_ERR_TOO_LARGE: return "B*H*N exceeds the built-in scratch of s2a_bwd_noalloc (see s2a_bwd_noalloc_max_rows)";
        default: return "unknown status";
    }
}

namespace {
// Token strides in elements; 0 means dense ([B, N, heads, d]).
struct TokStrides {
    long long q = 0, kv = 0, dq = 0, dkv = 0;
};

int fwd_impl(const void* q, const void* k, const void* v, void* o, float* lse, int B, int N, int H, int Hkv, int d,
             int G, float scale, int n_unshifted, int shift, unsigned flags, void* stream, const TokStrides& ts) {
    if (!flags_ok(flags)) return S2A_ERR_INVALID_ARG;
    if (!q || !k || !v || !o || !lse) return S2A_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(lse)) return S2A_ERR_INVALID_ARG;
    int rc = check_shape(B, N, H, Hkv, d, G, scale, n_unshifted, shift);
    if (rc != S2A_OK) return rc;
    DeviceState* ds = nullptr;
    rc = prepare_device(&ds);
    if (rc != S2A_OK) return rc;
    if (*ds->host_word != 0) return S2A_ERR_TIMEOUT;  // an earlier launch gave up: see s2a_device_status()

    FwdParams p;
    memset(&p, 0, sizeof p);
    if ((rc = make_tmap(&p.tm_q, q, d, H, N, B, kTile, ts.q)) != S2A_OK) return rc;
    if ((rc = make_tmap(&p.tm_k, k, d, Hkv, N, B, kTile, ts.kv)) != S2A_OK) return rc;
    if ((rc = make_tmap(&p.tm_v, v, d, Hkv, N, B, kTile, ts.kv)) != S2A_OK) return rc;
    p.o = static_cast<__nv_bfloat16*>(o);
    p.lse = lse;
    p.status = ds->status_ptr;
    p.host_status = ds->host_word_dev;
    p.geo = make_geometry(B, N, H, Hkv, G, n_unshifted, shift, flags);
    p.scale_log2 = scale * kLog2eHost;
    cudaError_t e = launch_fwd(p, d, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? S2A_OK : cuda_fail(e);
}
}  // namespace

int s2a_fwd_ex(const void* q, const void* k, const void* v, void* o, float* lse, int B, int N, int H, int Hkv, int d,
               int G, float scale, int n_unshifted, int shift, unsigned flags, void* stream) {
    return fwd_impl(q, k, v, o, lse, B, N, H, Hkv, d, G, scale, n_unshifted, shift, flags, stream, TokStrides());
}

int s2a_fwd_packed(const void* qkv, void* o, float* lse, int B, int N, int H, int d, int G, void* stream) {
    if (!qkv) return S2A_ERR_INVALID_ARG;
    if (const int bad = check_default_shape(N, H, d, G)) return bad;
    const __nv_bfloat16* base = static_cast<const __nv_bfloat16*>(qkv);
    const long long hd = static_cast<long long>(H) * d;
    TokStrides ts;
    ts.q = ts.kv = 3 * hd;
    return fwd_impl(base, base + hd, base + 2 * hd, o, lse, B, N, H, H, d, G, 1.0f / sqrtf(static_cast<float>(d)), H / 2,
                    G / 2, 0u, stream, ts);
}

int s2a_fwd(const void* q, const void* k, const void* v, void* o, float* lse, int B, int N, int H, int Hkv, int d,
            int G, void* stream) {
    if (const int bad = check_default_shape(N, H, d, G)) return bad;
    return s2a_fwd_ex(q, k, v, o, lse, B, N, H, Hkv, d, G, 1.0f / sqrtf(static_cast<float>(d)), H / 2, G / 2, 0u, stream);
}

namespace {
// Workspace layout: D [B, H, N] fp32 padded to 256 bytes, 256 bytes of work counters for the persistent
// kernels (together the minimum), then the spill area.
constexpr size_t kCounterBytes = 256;
size_t d_bytes(int B, int N, int H) {
    return (static_cast<size_t>(B) * H * N * sizeof(float) + 255) & ~static_cast<size_t>(255);
}
}  // namespace

size_t s2a_bwd_workspace_bytes(int B, int N, int H, int Hkv, int d, int G) {
    if (B <= 0 || N <= 0 || H <= 0 || Hkv <= 0 || d <= 0 || G <= 0) return 0;
    if (N % G != 0 || H % Hkv != 0) return 0;
    return d_bytes(B, N, H) + kCounterBytes;
}

namespace {
constexpr size_t kSpillBlockBytes = static_cast<size_t>(kSpillBlockElems) * 2;
// spill blocks of one KV head with its query heads, for groups of at most T tiles
size_t spill_blocks_per_kv_head(int B, int N, int H, int Hkv, int G, int T) {
    return static_cast<size_t>(B) * (H / Hkv) * (N / G) * static_cast<size_t>(spill_blocks_per_unit(T));
}
}  // namespace

size_t s2a_bwd_workspace_bytes_fast(int B, int N, int H, int Hkv, int d, int G, size_t budget) {
    const size_t min_bytes = s2a_bwd_workspace_bytes(B, N, H, Hkv, d, G);
    if (min_bytes == 0) return 0;
    // tiles of the largest group: G / 128 when G and the default shift G / 2 are multiples of the tile,
    // otherwise one partial tile per run of the group that wraps
    const int T = (G % (2 * kTile) == 0) ? G / kTile : (G + kTile - 1) / kTile + 1;
    const size_t per_kv = spill_blocks_per_kv_head(B, N, H, Hkv, G, T) * kSpillBlockBytes;
    if (budget <= min_bytes) return min_bytes;
    size_t nk = (budget - min_bytes) / per_kv;
    if (nk > static_cast<size_t>(Hkv)) nk = Hkv;
    return nk == 0 ? min_bytes : min_bytes + nk * per_kv;
}

namespace {
enum : unsigned { kStagePre = 1u, kStageDkDv = 2u, kStageDq = 4u, kStageAll = 7u };

int bwd_impl(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* dO, void* dq,
             void* dk, void* dv, int B, int N, int H, int Hkv, int d, int G, float scale, int n_unshifted, int shift,
             void* workspace, size_t workspace_bytes, void* stream, unsigned stages, unsigned flags = 0u,
             const TokStrides& ts = TokStrides(), bool may_spill = true) {
    if (!q || !k || !v || !o || !lse || !dO || !dq || !dk || !dv || !workspace) return S2A_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(lse) || !aligned16(dO) ||
        !aligned16(dq) || !aligned16(dk) || !aligned16(dv))
        return S2A_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return S2A_ERR_INVALID_ARG;
    int rc = check_shape(B, N, H, Hkv, d, G, scale, n_unshifted, shift);
    if (rc != S2A_OK) return rc;
    if (workspace_bytes < s2a_bwd_workspace_bytes(B, N, H, Hkv, d, G)) return S2A_ERR_INVALID_ARG;
    DeviceState* ds = nullptr;
    rc = prepare_device(&ds);
    if (rc != S2A_OK) return rc;
    if (*ds->host_word != 0) return S2A_ERR_TIMEOUT;  // an earlier launch gave up: see s2a_device_status()
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!flags_ok(flags)) return S2A_ERR_INVALID_ARG;
    const Geometry geo = make_geometry(B, N, H, Hkv, G, n_unshifted, shift, flags);
    float* Dsum = static_cast<float*>(workspace);

    BwdDqParams pq;
    memset(&pq, 0, sizeof pq);
    if ((rc = make_tmap(&pq.tm_q, q, d, H, N, B, kTile, ts.q)) != S2A_OK) return rc;
    if ((rc = make_tmap(&pq.tm_do, dO, d, H, N, B, kTile)) != S2A_OK) return rc;
    if ((rc = make_tmap(&pq.tm_k, k, d, Hkv, N, B, kTile, ts.kv)) != S2A_OK) return rc;
    if ((rc = make_tmap(&pq.tm_v, v, d, Hkv, N, B, kTile, ts.kv)) != S2A_OK) return rc;
    pq.dq_tok_stride = ts.dq ? ts.dq : static_cast<long long>(H) * d;
    pq.lse = lse, pq.Dsum = Dsum, pq.dq = static_cast<__nv_bfloat16*>(dq);
    pq.status = ds->status_ptr, pq.host_status = ds->host_word_dev, pq.geo = geo, pq.scale = scale, pq.scale_log2 = scale * kLog2eHost;

    BwdDkDvParams pk;
    memset(&pk, 0, sizeof pk);
    if ((rc = make_tmap(&pk.tm_k, k, d, Hkv, N, B, kTile, ts.kv)) != S2A_OK) return rc;
    if ((rc = make_tmap(&pk.tm_v, v, d, Hkv, N, B, kTile, ts.kv)) != S2A_OK) return rc;
    if ((rc = make_tmap(&pk.tm_q, q, d, H, N, B, kSubTile, ts.q)) != S2A_OK) return rc;
    if ((rc = make_tmap(&pk.tm_do, dO, d, H, N, B, kSubTile)) != S2A_OK) return rc;
    pk.dkv_tok_stride = ts.dkv ? ts.dkv : static_cast<long long>(Hkv) * d;
    pk.lse = lse, pk.Dsum = Dsum;
    pk.dk = static_cast<__nv_bfloat16*>(dk), pk.dv = static_cast<__nv_bfloat16*>(dv);
    pk.status = ds->status_ptr, pk.host_status = ds->host_word_dev, pk.geo = geo, pk.scale = scale, pk.scale_log2 = scale * kLog2eHost;
    pk.spill = nullptr;
    pk.pass.hk0 = 0, pk.pass.nk = Hkv;

    PreParams pp;
    pp.o = static_cast<const __nv_bfloat16*>(o), pp.dO = static_cast<const __nv_bfloat16*>(dO), pp.Dsum = Dsum;
    pp.B = B, pp.N = N, pp.H = H;

    // How many KV heads' worth of dS^T the workspace can hold beyond D: with room for at least one, the
    // dK,dV kernel spills dS^T and dQ is a plain product (several passes over the KV heads if they do
    // not all fit); otherwise dQ recomputes S and dP.  A single-stage call spills only in one pass, so
    // that stages 0, 1, 2 in order stay equal to the whole backward.
    const size_t min_bytes = s2a_bwd_workspace_bytes(B, N, H, Hkv, d, G);
    const size_t per_kv = spill_blocks_per_kv_head(B, N, H, Hkv, G, geo.tiles_per_group);
    size_t nk_fit = 0;
    if (may_spill && workspace_bytes > min_bytes)
        nk_fit = (workspace_bytes - min_bytes) / (per_kv * kSpillBlockBytes);
    if (nk_fit > static_cast<size_t>(Hkv)) nk_fit = Hkv;
    if (stages != kStageAll && nk_fit < static_cast<size_t>(Hkv)) nk_fit = 0;

    char* base = static_cast<char*>(workspace);
    int* counters = reinterpret_cast<int*>(base + d_bytes(B, N, H));  // [0] dK,dV kernel, [1] dQ-from-spill kernel
    pk.counter = counters;
    cudaError_t e;
    if (stages & kStagePre) {
        e = launch_bwd_preprocess(pp, d, st);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    if (nk_fit == 0) {
        if (stages & kStageDkDv) {
            e = cudaMemsetAsync(counters, 0, sizeof(int), st);
            if (e != cudaSuccess) return cuda_fail(e);
            e = launch_bwd_dkdv(pk, d, ds->n_sm, st);
            if (e != cudaSuccess) return cuda_fail(e);
        }
        if (stages & kStageDq) {
            e = launch_bwd_dq(pq, d, st);
            if (e != cudaSuccess) return cuda_fail(e);
        }
        return S2A_OK;
    }

    pk.spill = reinterpret_cast<__nv_bfloat16*>(base + min_bytes);
    BwdDqSpillParams ps;
    memset(&ps, 0, sizeof ps);
    ps.tm_k = pq.tm_k;
    ps.spill = pk.spill;
    ps.dq = pq.dq, ps.dq_tok_stride = pq.dq_tok_stride, ps.counter = counters + 1;
    ps.status = ds->status_ptr, ps.host_status = ds->host_word_dev, ps.geo = geo, ps.scale = scale;
    for (int hk0 = 0; hk0 < Hkv; hk0 += static_cast<int>(nk_fit)) {
        const int nk = Hkv - hk0 < static_cast<int>(nk_fit) ? Hkv - hk0 : static_cast<int>(nk_fit);
        pk.pass.hk0 = hk0, pk.pass.nk = nk;
        ps.pass = pk.pass;
        if (stages & kStageDkDv) {
            e = cudaMemsetAsync(counters, 0, sizeof(int), st);
            if (e != cudaSuccess) return cuda_fail(e);
            e = launch_bwd_dkdv(pk, d, ds->n_sm, st);
            if (e != cudaSuccess) return cuda_fail(e);
        }
        if (stages & kStageDq) {
            e = cudaMemsetAsync(counters + 1, 0, sizeof(int), st);
            if (e != cudaSuccess) return cuda_fail(e);
            e = launch_bwd_dq_spill(ps, d, ds->n_sm, st);
            if (e != cudaSuccess) return cuda_fail(e);
        }
    }
    return S2A_OK;
}
}  // namespace

int s2a_bwd_ex(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* dO, void* dq,
               void* dk, void* dv, int B, int N, int H, int Hkv, int d, int G, float scale, int n_unshifted,
               int shift, unsigned flags, void* workspace, size_t workspace_bytes, void* stream) {
    return bwd_impl(q, k, v, o, lse, dO, dq, dk, dv, B, N, H, Hkv, d, G, scale, n_unshifted, shift, workspace,
                    workspace_bytes, stream, kStageAll, flags);
}

int s2a_bwd_packed(const void* qkv, const void* o, const float* lse, const void* dO, void* dqkv, int B, int N, int H,
                   int d, int G, void* workspace, size_t workspace_bytes, void* stream) {
    if (!qkv || !dqkv) return S2A_ERR_INVALID_ARG;
    if (const int bad = check_default_shape(N, H, d, G)) return bad;
    const __nv_bfloat16* in = static_cast<const __nv_bfloat16*>(qkv);
    __nv_bfloat16* out = static_cast<__nv_bfloat16*>(dqkv);
    const long long hd = static_cast<long long>(H) * d;
    TokStrides ts;
    ts.q = ts.kv = ts.dq = ts.dkv = 3 * hd;
    return bwd_impl(in, in + hd, in + 2 * hd, o, lse, dO, out, out + hd, out + 2 * hd, B, N, H, H, d, G,
                    1.0f / sqrtf(static_cast<float>(d)), H / 2, G / 2, workspace, workspace_bytes, stream, kStageAll, 0u, ts);
}

int s2a_bwd_stage(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* dO,
                  void* dq, void* dk, void* dv, int B, int N, int H, int Hkv, int d, int G, void* workspace,
                  size_t workspace_bytes, int stage, void* stream) {
    if (stage < 0 || stage > 2) return S2A_ERR_INVALID_ARG;
    if (const int bad = check_default_shape(N, H, d, G)) return bad;
    return bwd_impl(q, k, v, o, lse, dO, dq, dk, dv, B, N, H, Hkv, d, G, 1.0f / sqrtf(static_cast<float>(d)), H / 2,
                    G / 2, workspace, workspace_bytes, stream, 1u << stage);
}

int s2a_bwd(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* dO, void* dq,
            void* dk, void* dv, int B, int N, int H, int Hkv, int d, int G, void* workspace, size_t workspace_bytes,
            void* stream) {
    if (const int bad = check_default_shape(N, H, d, G)) return bad;
    return s2a_bwd_ex(q, k, v, o, lse, dO, dq, dk, dv, B, N, H, Hkv, d, G, 1.0f / sqrtf(static_cast<float>(d)), H / 2,
                      G / 2, 0u, workspace, workspace_bytes, stream);
}

int s2a_fwd_bwd_host(const void* h_q, const void* h_k, const void* h_v, const void* h_dO, void* h_o, float* h_lse,
                     void* h_dq, void* h_dk, void* h_dv, void* d_q, void* d_k, void* d_v, void* d_dO, void* d_o,
                     float* d_lse, void* d_dq, void* d_dk, void* d_dv, int B, int N, int H, int Hkv, int d, int G,
                     void* workspace, size_t workspace_bytes, void* stream) {
    if (!h_q || !h_k || !h_v || !h_dO || !h_o || !h_lse || !h_dq || !h_dk || !h_dv) return S2A_ERR_INVALID_ARG;
    if (!d_q || !d_k || !d_v || !d_dO || !d_o || !d_lse || !d_dq || !d_dk || !d_dv) return S2A_ERR_INVALID_ARG;
    if (const int bad = check_default_shape(N, H, d, G)) return bad;
    int rc = check_shape(B, N, H, Hkv, d, G, 1.0f, H / 2, G / 2);
    if (rc != S2A_OK) return rc;
    if (!workspace || workspace_bytes < s2a_bwd_workspace_bytes(B, N, H, Hkv, d, G)) return S2A_ERR_INVALID_ARG;
    DeviceState* ds = nullptr;
    if ((rc = prepare_device(&ds)) != S2A_OK) return rc;
    cudaError_t e;
    std::unique_lock<std::mutex> lock(g_dev_mutex);
    if (!ds->host_path_ready) {
        if ((e = cudaStreamCreateWithFlags(&ds->copy_in, cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaStreamCreateWithFlags(&ds->copy_out, cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaEventCreateWithFlags(&ds->ev_start, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaEventCreateWithFlags(&ds->ev_done, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaEventCreateWithFlags(&ds->ev_in_done, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
        for (int c = 0; c < kMaxHostChunks; ++c) {
            if ((e = cudaEventCreateWithFlags(&ds->ev_in[c], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaEventCreateWithFlags(&ds->ev_compute[c], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
        }
        ds->host_path_ready = true;
    }
    lock.unlock();
    // Heads are independent, so the job is cut into chunks of whole KV heads (with their query heads):
    // while chunk c is computed, chunk c+1 travels to the device and the results of chunk c-1 travel
    // back.  Only the first chunk's upload and the last chunk's download cannot be hidden, so the
    // chunks at both ends are small and grow towards the middle, where wide rows keep the strided
    // copies efficient: 2,2,4,8,8,4,2,2 KV heads for Hkv = 32 (a chunk of a single 256-byte head row per
    // token copies at well under the link's rate, which costs more than its shorter exposure saves).
    // Chunk c holds the KV
    // heads [kv0[c], kv0[c] + kvn[c]) and sits densely ([B, N, heads of the chunk, d]) at the matching
    // offset of the caller's device buffers.
    const int rep = H / Hkv;
    int kv0[kMaxHostChunks], kvn[kMaxHostChunks];
    int chunks = 0;
    {
        int left[kMaxHostChunks / 2], right[kMaxHostChunks / 2], nl = 0, nr = 0;
        const int first = Hkv >= 32 ? Hkv / 16 : 1;
        int remaining = Hkv, size = first, uses = 0;
        const int cap = Hkv >= 8 ? Hkv / 4 : 1;
        while (remaining > 0) {
            const int a = size < remaining ? size : remaining;
            if (nl <= nr) left[nl++] = a; else right[nr++] = a;
            remaining -= a;
            if (++uses == (size == first ? 4 : 2)) {   // the smallest size twice at each end, then every size once per end
                uses = 0;
                if (size * 2 <= cap) size *= 2;
            }
            if (nl + nr == kMaxHostChunks - 1 && remaining > 0) {   // out of slots: the rest in one chunk
                if (nl <= nr) left[nl++] = remaining; else right[nr++] = remaining;
                remaining = 0;
            }
        }
        int at_kv = 0;
        for (int x = 0; x < nl; ++x) kv0[chunks] = at_kv, kvn[chunks] = left[x], at_kv += left[x], ++chunks;
        for (int x = nr - 1; x >= 0; --x) kv0[chunks] = at_kv, kvn[chunks] = right[x], at_kv += right[x], ++chunks;
    }
    const size_t rows = static_cast<size_t>(B) * N;
    const size_t hb = static_cast<size_t>(d) * 2;                                              // bytes of one head of one token
    const size_t pq = static_cast<size_t>(H) * d * 2, pk = static_cast<size_t>(Hkv) * d * 2;   // host pitches
    const size_t pl = static_cast<size_t>(H) * N * sizeof(float);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    auto at = [](const void* base, size_t bytes) { return const_cast<char*>(static_cast<const char*>(base)) + bytes; };

    if ((e = cudaEventRecord(ds->ev_start, st)) != cudaSuccess) return cuda_fail(e);
    // From here on work may sit in the two copy streams: whatever happens, `stream` is made to wait
    // for both before this function returns, so that the caller's synchronisation covers it all.
    auto join = [&]() -> cudaError_t {
        cudaError_t e1 = cudaEventRecord(ds->ev_done, ds->copy_out);
        if (e1 == cudaSuccess) e1 = cudaStreamWaitEvent(st, ds->ev_done, 0);
        cudaError_t e2 = cudaEventRecord(ds->ev_in_done, ds->copy_in);
        if (e2 == cudaSuccess) e2 = cudaStreamWaitEvent(st, ds->ev_in_done, 0);
        return e1 != cudaSuccess ? e1 : e2;
    };
    auto enqueue_all = [&]() -> int {
        if ((e = cudaStreamWaitEvent(ds->copy_in, ds->ev_start, 0)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaStreamWaitEvent(ds->copy_out, ds->ev_start, 0)) != cudaSuccess) return cuda_fail(e);
        for (int c = 0; c < chunks; ++c) {
            const int kvc = kvn[c], hc = kvc * rep, h0 = kv0[c] * rep;   // KV heads, query heads, first query head of the chunk
            const size_t wq = hc * hb, wk = kvc * hb;                    // bytes per token of the chunk
            const size_t wl = static_cast<size_t>(hc) * N * sizeof(float);
            const size_t oq = rows * h0 * hb, ok_ = rows * kv0[c] * hb, ol = static_cast<size_t>(B) * h0 * N * sizeof(float);
            void *cq = at(d_q, oq), *ck = at(d_k, ok_), *cv = at(d_v, ok_), *cdo = at(d_dO, oq), *co = at(d_o, oq);
            void *cdq = at(d_dq, oq), *cdk = at(d_dk, ok_), *cdv = at(d_dv, ok_);
            float* cl = reinterpret_cast<float*>(at(d_lse, ol));
            // host -> device: the chunk's heads of every token
            if ((e = cudaMemcpy2DAsync(cq, wq, at(h_q, h0 * hb), pq, wq, rows, cudaMemcpyHostToDevice, ds->copy_in)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaMemcpy2DAsync(ck, wk, at(h_k, kv0[c] * hb), pk, wk, rows, cudaMemcpyHostToDevice, ds->copy_in)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaMemcpy2DAsync(cv, wk, at(h_v, kv0[c] * hb), pk, wk, rows, cudaMemcpyHostToDevice, ds->copy_in)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaMemcpy2DAsync(cdo, wq, at(h_dO, h0 * hb), pq, wq, rows, cudaMemcpyHostToDevice, ds->copy_in)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaEventRecord(ds->ev_in[c], ds->copy_in)) != cudaSuccess) return cuda_fail(e);
            // compute on the caller's stream; the second half of ALL heads is shifted
            if ((e = cudaStreamWaitEvent(st, ds->ev_in[c], 0)) != cudaSuccess) return cuda_fail(e);
            int n_unshifted = H / 2 - h0;
            n_unshifted = n_unshifted < 0 ? 0 : (n_unshifted > hc ? hc : n_unshifted);
            const float scale = 1.0f / sqrtf(static_cast<float>(d));
            int rc2 = fwd_impl(cq, ck, cv, co, cl, B, N, hc, kvc, d, G, scale, n_unshifted, G / 2, 0u, stream, TokStrides());
            if (rc2 != S2A_OK) return rc2;
            rc2 = bwd_impl(cq, ck, cv, co, cl, cdo, cdq, cdk, cdv, B, N, hc, kvc, d, G, scale, n_unshifted, G / 2, workspace,
                           workspace_bytes, stream, kStageAll);
            if (rc2 != S2A_OK) return rc2;
            if ((e = cudaEventRecord(ds->ev_compute[c], st)) != cudaSuccess) return cuda_fail(e);
            // device -> host
            if ((e = cudaStreamWaitEvent(ds->copy_out, ds->ev_compute[c], 0)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaMemcpy2DAsync(at(h_o, h0 * hb), pq, co, wq, wq, rows, cudaMemcpyDeviceToHost, ds->copy_out)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaMemcpy2DAsync(at(h_lse, static_cast<size_t>(h0) * N * sizeof(float)), pl, cl, wl, wl, B, cudaMemcpyDeviceToHost, ds->copy_out)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaMemcpy2DAsync(at(h_dq, h0 * hb), pq, cdq, wq, wq, rows, cudaMemcpyDeviceToHost, ds->copy_out)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaMemcpy2DAsync(at(h_dk, kv0[c] * hb), pk, cdk, wk, wk, rows, cudaMemcpyDeviceToHost, ds->copy_out)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaMemcpy2DAsync(at(h_dv, kv0[c] * hb), pk, cdv, wk, wk, rows, cudaMemcpyDeviceToHost, ds->copy_out)) != cudaSuccess) return cuda_fail(e);
        }
        return S2A_OK;
    };
    rc = enqueue_all();
    // the caller's stream is done when the last copy back is (also after a failure part-way)
    const int saved_cuda_error = tl_last_cuda_error;
    const cudaError_t ej = join();
    if (rc != S2A_OK) {
        tl_last_cuda_error = saved_cuda_error;
        return rc;
    }
    return ej == cudaSuccess ? S2A_OK : cuda_fail(ej);
}

// ---------------------------------------------------------------------------------------------
// Backward without caller-provided scratch
// ---------------------------------------------------------------------------------------------
namespace {

// Built-in home for D = rowsum(dO * o) and the work counters when the caller cannot provide a
// workspace: 2^20 fp32 rows and 256 bytes (4 MiB in all), which every GPU that loads this library keeps
// resident until the process exits.
constexpr size_t kBuiltinScratchRows = size_t(1) << 20;
static __device__ __align__(256) float g_builtin_scratch[kBuiltinScratchRows + kCounterBytes / sizeof(float)];

// In host code `g_builtin_scratch` is only a handle for the runtime, not an address a kernel may
// use; the device address is looked up once per device, with that device current.
float* g_builtin_scratch_ptr[kMaxDevices] = {};

int builtin_scratch(float** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= kMaxDevices) return S2A_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (!g_builtin_scratch_ptr[dev]) {
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_builtin_scratch);
        if (e != cudaSuccess) return cuda_fail(e);
        g_builtin_scratch_ptr[dev] = static_cast<float*>(ptr);
    }
    *out = g_builtin_scratch_ptr[dev];
    return S2A_OK;
}

}  // namespace

int s2a_bwd_noalloc(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* dO,
                    void* dq, void* dk, void* dv, int B, int N, int H, int Hkv, int d, int G, void* stream) {
    if (B <= 0 || N <= 0 || H <= 0) return S2A_ERR_INVALID_ARG;
    if (static_cast<unsigned long long>(B) * static_cast<unsigned long long>(H) * static_cast<unsigned long long>(N) >
        kBuiltinScratchRows)
        return S2A_ERR_TOO_LARGE;
    if (const int bad = check_default_shape(N, H, d, G)) return bad;
    float* scratch = nullptr;
    const int rc = builtin_scratch(&scratch);
    if (rc != S2A_OK) return rc;
    // Every row of D that the two gradient kernels read is rewritten by the first kernel of this
    // call and the work counter is cleared by a memset ahead of its kernel, so nothing left in the
    // array by an earlier call matters.
    return bwd_impl(q, k, v, o, lse, dO, dq, dk, dv, B, N, H, Hkv, d, G, 1.0f / sqrtf(static_cast<float>(d)), H / 2,
                    G / 2, scratch, kBuiltinScratchRows * sizeof(float) + kCounterBytes, stream, kStageAll, 0u, TokStrides(), false);
}

size_t s2a_bwd_noalloc_max_rows(void) { return kBuiltinScratchRows; }

int s2a_selftest_wait_expiry(long long limit_cycles, void* stream) {
    if (limit_cycles < 1 || limit_cycles > kWaitLimitCycles) return S2A_ERR_INVALID_ARG;
    DeviceState* ds = nullptr;
    const int rc = prepare_device(&ds);
    if (rc != S2A_OK) return rc;
    s2a_wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(ds->status_ptr, ds->host_word_dev, limit_cycles);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? S2A_OK : cuda_fail(e);
}

int s2a_device_status(int* where) {
    DeviceState* ds = nullptr;
    int rc = prepare_device(&ds);
    if (rc != S2A_OK) return rc;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return cuda_fail(e);
    int word = 0;
    e = cudaMemcpy(&word, ds->status_ptr, sizeof word, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e);
    if (word != 0) {
        const int zero = 0;
        e = cudaMemcpy(ds->status_ptr, &zero, sizeof zero, cudaMemcpyHostToDevice);
        if (e != cudaSuccess) return cuda_fail(e);
        *ds->host_word = 0;
        if (where) *where = word;
        return S2A_ERR_TIMEOUT;
    }
    if (where) *where = 0;
    return S2A_OK;
}

}  // extern "C"
#pragma GCC visibility pop
