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
};

// Geometry of the shifted grouping (Algorithm 1): common to every kernel.
struct Geometry {
    int B, N, H, Hkv, G;
    int n_unshifted;      // heads [0, n_unshifted) use the unshifted partition
    int shift;            // tokens; the rest of the heads are rolled by -shift (G/2 in Algorithm 1)
    int tiles_per_group;  // G / 128
    int groups;           // N / G
};

struct alignas(64) FwdParams {
    CUtensorMap tm_q;  // bf16 (d, H,   N, B), box (64, 1, 128, 1), 128-byte swizzle
    CUtensorMap tm_k;  // bf16 (d, Hkv, N, B), same box
    CUtensorMap tm_v;
    __nv_bfloat16* o;
    float* lse;
    int* status;
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
    CUtensorMap tm_k, tm_v;   // box (64, 1,  64, 1): streamed key sub-tiles
    const float* lse;         // [B, H, N]
    const float* Dsum;        // [B, H, N]
    __nv_bfloat16* dq;
    int* status;
    Geometry geo;
    float scale, scale_log2;
};

struct alignas(64) BwdDkDvParams {
    CUtensorMap tm_k, tm_v;   // box (64, 1, 128, 1): the resident key tile
    CUtensorMap tm_q, tm_do;  // box (64, 1,  64, 1): streamed query sub-tiles
    const float* lse;
    const float* Dsum;
    __nv_bfloat16* dk;
    __nv_bfloat16* dv;
    int* status;
    Geometry geo;
    float scale, scale_log2;
};

// Enqueue one kernel each on `stream`; return the launch error, if any.
cudaError_t launch_fwd(const FwdParams& p, int d, cudaStream_t stream);
cudaError_t launch_bwd_preprocess(const PreParams& p, int d, cudaStream_t stream);
cudaError_t launch_bwd_dq(const BwdDqParams& p, int d, cudaStream_t stream);
cudaError_t launch_bwd_dkdv(const BwdDkDvParams& p, int d, cudaStream_t stream);

// Per-device kernel attribute set-up (dynamic shared memory sizes).
cudaError_t configure_fwd();
cudaError_t configure_bwd();

}  // namespace s2a
