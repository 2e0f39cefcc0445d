// Kernel parameter blocks and launcher declarations shared by the host entry points and the kernels.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace s2a {

constexpr int kTile = 128;  // tokens per tile, both for queries and for keys

// Codes recorded when a bounded device-side wait expires: kernel id * 100 + wait id.
enum WaitCode : int {
    kWaitFwd = 100,
    kWaitBwdDq = 200,
    kWaitBwdDkDv = 300,
};

struct alignas(64) FwdParams {
    CUtensorMap tm_q;  // bf16 (d, H,   N, B), box (64, 1, 128, 1), 128-byte swizzle
    CUtensorMap tm_k;  // bf16 (d, Hkv, N, B)
    CUtensorMap tm_v;
    __nv_bfloat16* o;
    float* lse;
    int* status;
    int B, N, H, Hkv, G;
    int n_unshifted;      // heads [0, n_unshifted) use the unshifted partition
    int shift;            // tokens; the rest of the heads are rolled by -shift (G/2 in Algorithm 1)
    int tiles_per_group;  // G / 128
    int groups;           // N / G
    float scale_log2;     // softmax scale * log2(e)
};

struct alignas(64) BwdParams {
    CUtensorMap tm_q, tm_k, tm_v, tm_do;
    const __nv_bfloat16* o;
    const __nv_bfloat16* dO;
    const float* lse;
    float* Dsum;  // [B, H, N] fp32 scratch: dO . o per query row
    __nv_bfloat16* dq;
    __nv_bfloat16* dk;
    __nv_bfloat16* dv;
    int* status;
    int B, N, H, Hkv, G;
    int n_unshifted, shift, tiles_per_group, groups;
    float scale;       // softmax scale
    float scale_log2;  // scale * log2(e)
};

// Enqueue one kernel each on `stream`; return the launch error, if any.
cudaError_t launch_fwd(const FwdParams& p, int d, cudaStream_t stream);
cudaError_t launch_bwd_preprocess(const BwdParams& p, int d, cudaStream_t stream);
cudaError_t launch_bwd_dq(const BwdParams& p, int d, cudaStream_t stream);
cudaError_t launch_bwd_dkdv(const BwdParams& p, int d, cudaStream_t stream);

// One-time per-device kernel attribute set-up (dynamic shared memory sizes).
cudaError_t configure_fwd();
cudaError_t configure_bwd();

}  // namespace s2a
