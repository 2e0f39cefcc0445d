// Kernel parameter blocks and launcher declarations shared by the host entry points and the kernels.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace s2a {

constexpr int kTile = 128;     // tokens per resident tile (query rows in forward / dQ, key rows in dK,dV)
constexpr int kSubTile = 64;   // tokens per streamed tile in the backward kernels

// Codes recorded when a bounded device-side wait expires: kernel id * 100 + wait id.
enum WaitCode : int {
    kWaitFwd = 100,
    kWaitBwdDq = 200,
    kWaitBwdDkDv = 300,
    kWaitBwdDqSpill = 400,
};

// Block order shared by the tensor-core kernels.  A "unit" is one (batch, head, group); it has
// `tiles` tiles whose cost falls with their rank (rank 0 = most work).  Units are taken in chunks of
// kUnitChunk: inside a chunk all rank-0 tiles come first, then all rank-1 tiles, and so on.  So the
// blocks that run together belong to a few units (their streamed operands stay in L2), heavy tiles
// start first, and the tail of the grid consists of the lightest tiles only.
constexpr int kUnitChunk = 8;
__host__ __device__ inline void decode_block(long long idx, int units, int tiles, int* unit, int* rank) {
    const long long per_chunk = static_cast<long long>(kUnitChunk) * tiles;
    const int chunk = static_cast<int>(idx / per_chunk);
    const int within = static_cast<int>(idx % per_chunk);
    const int first = chunk * kUnitChunk;
    const int in_chunk = (units - first) < kUnitChunk ? (units - first) : kUnitChunk;
    *rank = within / in_chunk;
    *unit = first + within % in_chunk;
}

// Geometry of the shifted grouping (Algorithm 1): common to every kernel.
struct Geometry {
    int B, N, H, Hkv, G;
    int n_unshifted;      // heads [0, n_unshifted) use the unshifted partition
    int shift;            // tokens; the rest of the heads are rolled by -shift (G/2 in Algorithm 1)
    int tiles_per_group;  // largest number of 128-token tiles any group has (G / 128 when G and shift are multiples of 128)
    int groups;           // N / G
    int leak_free;        // variant 2 of Appendix B: cut the wrapped group of a shifted head at the wrap
    int swap_wrapped;     // variant 3 of Appendix B: the two runs of the wrapped group change places
};

// Where the tokens of one group live.  Group g of a head with shift s holds rolled positions
// [g G, (g+1) G), i.e. original tokens (x + s) mod N: one run [a0, a0 + lenA) and, only in the group
// that wraps past token N-1, a second run [0, lenB).  Each run is cut into 128-token tiles from its own
// start, so a tile is always a contiguous range of original tokens (one TMA box, no wrap inside a
// tile) and only the last tile of a run can have fewer than 128 valid rows.  Tiles are numbered in
// causal order: the nA tiles of the first run, then those of the second (the other way round in
// variant 3 of Appendix B).
struct GroupLayout {
    int a0, lenA, lenB;
    int nA, nTiles;
    int cut;      // variant 2: tile index at which the wrapped group is cut in two (0 = no cut)
    int swapped;  // variant 3: the tiles of the second run ([0, lenB), the front of the sequence) come first
};
__host__ __device__ inline GroupLayout group_layout(const Geometry& geo, int s, int g) {
    GroupLayout L;
    long long a = (static_cast<long long>(g) * geo.G + s) % geo.N;
    if (a < 0) a += geo.N;
    L.a0 = static_cast<int>(a);
    L.lenA = (geo.N - L.a0 < geo.G) ? geo.N - L.a0 : geo.G;
    L.lenB = geo.G - L.lenA;
    L.nA = (L.lenA + kTile - 1) / kTile;
    L.nTiles = L.nA + (L.lenB + kTile - 1) / kTile;
    // Variant 2: the second run starts at original token 0; queries there attend keys from the cut
    // on, keys before the cut are attended by queries before the cut only.
    L.cut = (geo.leak_free && L.lenB > 0) ? L.nA : 0;
    // Variant 3: the wrapped group is attended in original token order, front tokens first.
    L.swapped = (geo.swap_wrapped && L.lenB > 0) ? 1 : 0;
    return L;
}
struct TileRef {
    int tok0;   // original token of row 0
    int valid;  // rows that belong to the group (the rest of the box is other tokens or zero fill)
};
__host__ __device__ inline TileRef tile_ref(const GroupLayout& L, int i) {
    TileRef t;
    const int nFirst = L.swapped ? L.nTiles - L.nA : L.nA;  // tiles of the run that comes first
    const bool in_run_a = L.swapped ? (i >= nFirst) : (i < nFirst);
    const int k = (i < nFirst) ? i : i - nFirst;             // tile within its run
    if (in_run_a) {
        t.tok0 = L.a0 + k * kTile;
        t.valid = L.lenA - k * kTile;
    } else {
        t.tok0 = k * kTile;
        t.valid = L.lenB - k * kTile;
    }
    if (t.valid > kTile) t.valid = kTile;
    return t;
}
// 64-row halves of the tiles, numbered 2 i and 2 i + 1; a half can be empty (valid = 0).
__host__ __device__ inline TileRef subtile_ref(const GroupLayout& L, int n) {
    TileRef t = tile_ref(L, n >> 1);
    const int off = (n & 1) * kSubTile;
    t.tok0 += off;
    t.valid -= off;
    if (t.valid > kSubTile) t.valid = kSubTile;
    if (t.valid < 0) t.valid = 0;
    return t;
}
// Causal range in tiles: query tile i attends key tiles [first_key_tile, i]; key tile j is attended
// by query tiles [j, end_query_tile).
__host__ __device__ inline int first_key_tile(const GroupLayout& L, int i) { return (L.cut > 0 && i >= L.cut) ? L.cut : 0; }
__host__ __device__ inline int end_query_tile(const GroupLayout& L, int j) { return (L.cut > 0 && j < L.cut) ? L.cut : L.nTiles; }

struct alignas(64) FwdParams {
    CUtensorMap tm_q;  // bf16 (d, H,   N, B), box (64, 1, 128, 1), 128-byte swizzle
    CUtensorMap tm_k;  // bf16 (d, Hkv, N, B), same box
    CUtensorMap tm_v;
    __nv_bfloat16* o;
    float* lse;
    int* status;       // device status word (see WaitCtx)
    int* host_status;  // its mirror in mapped host memory
    Geometry geo;
    float scale_log2;  // softmax scale * log2(e)
};

struct PreParams {
    const __nv_bfloat16* o;
    const __nv_bfloat16* dO;
    float* Dsum;  // [B, H, N]
    int B, N, H;
};

struct alignas(64) BwdDqParams {
    CUtensorMap tm_q, tm_do;  // box (64, 1, 128, 1): the resident query tile
    CUtensorMap tm_k, tm_v;   // box (64, 1, 128, 1): streamed key tiles
    const float* lse;         // [B, H, N]
    const float* Dsum;        // [B, H, N]
    __nv_bfloat16* dq;
    long long dq_tok_stride;  // elements between consecutive tokens of dq (H * d when dense)
    int* status;       // device status word (see WaitCtx)
    int* host_status;  // its mirror in mapped host memory
    Geometry geo;
    float scale, scale_log2;
};

// The dK,dV kernel can leave its dS^T values (bf16) in global memory for a dQ kernel that then only
// has to multiply them with K instead of recomputing S and dP.  One pass covers the KV heads
// [hk0, hk0 + nk) with their query heads; a "spill unit" is one (batch, query head of the pass, group),
// numbered (b * nk * rep + (hq - hk0 * rep)) * groups + g.  A unit owns T (T + 1) blocks, T =
// tiles_per_group: block (j, n) holds dS^T of key tile j and 64-query sub-tile n >= 2 j, 128 key rows of
// 64 bf16 (16 KB), stored chunk-major: the 16-byte chunk c (queries 8 c .. 8 c + 7) of key row r sits at
// byte (c * 128 + r) * 16 of the block, which is both what a warp of the dK,dV kernel writes in one
// coalesced store and an operand layout the tensor core reads directly.  Masked entries and rows that
// are not part of the group are zero.
struct SpillPass {
    int hk0, nk;  // KV heads of this pass
};
__host__ __device__ inline long long spill_blocks_per_unit(int T) { return static_cast<long long>(T) * (T + 1); }
__host__ __device__ inline long long spill_block(long long unit, int T, int j, int n) {
    return unit * spill_blocks_per_unit(T) + static_cast<long long>(j) * (2 * T - j + 1) + (n - 2 * j);
}
constexpr int kSpillBlockElems = kTile * kSubTile;  // bf16 values per block

struct alignas(64) BwdDkDvParams {
    CUtensorMap tm_k, tm_v;   // box (64, 1, 128, 1): the resident key tile
    CUtensorMap tm_q, tm_do;  // box (64, 1,  64, 1): streamed query sub-tiles
    const float* lse;
    const float* Dsum;
    __nv_bfloat16* dk;
    __nv_bfloat16* dv;
    long long dkv_tok_stride;  // elements between consecutive tokens of dk and dv (Hkv * d when dense)
    __nv_bfloat16* spill;      // dS^T blocks of this pass (spilling variant only)
    SpillPass pass;            // KV heads this launch covers (all of them when nothing is spilled)
    int* counter;              // next work item; zero when the kernel starts
    int* status;       // device status word (see WaitCtx)
    int* host_status;  // its mirror in mapped host memory
    Geometry geo;
    float scale, scale_log2;
};

// dQ from spilled dS^T: dQ_i = scale * sum_j dS_ij K_j, one CTA per 128-query tile.
struct alignas(64) BwdDqSpillParams {
    CUtensorMap tm_k;   // box (64, 1, 128, 1): streamed key tiles
    const __nv_bfloat16* spill;  // the blocks the dK,dV kernel of this pass wrote
    __nv_bfloat16* dq;
    long long dq_tok_stride;
    int* counter;  // next work item; zero when the kernel starts
    SpillPass pass;
    int* status;
    int* host_status;
    Geometry geo;
    float scale;
};

// Enqueue one kernel each on `stream`; return the launch error, if any.
cudaError_t launch_fwd(const FwdParams& p, int d, cudaStream_t stream);
cudaError_t launch_bwd_preprocess(const PreParams& p, int d, cudaStream_t stream);
cudaError_t launch_bwd_dq(const BwdDqParams& p, int d, cudaStream_t stream);
cudaError_t launch_bwd_dkdv(const BwdDkDvParams& p, int d, int n_sm, cudaStream_t stream);  // persistent; p.spill != nullptr: spilling variant
cudaError_t launch_bwd_dq_spill(const BwdDqSpillParams& p, int d, int n_sm, cudaStream_t stream);  // persistent: one CTA per SM

// Per-device kernel attribute set-up (dynamic shared memory sizes).
cudaError_t configure_fwd();
cudaError_t configure_bwd();

}  // namespace s2a
