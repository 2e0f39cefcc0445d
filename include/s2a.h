/*
 * s2a -- shifted sparse attention (S2-Attn) for NVIDIA B200 (sm_100a), forward and backward.
 *
 * The operation is the one LongLoRA states in Algorithm 1 and Section 3.2, with the attention of
 * Eq. 1 inside each group:
 *   - the N tokens of a sequence are cut into N/G groups of G consecutive tokens;
 *   - in the second half of the heads (h >= H/2) the tokens are rolled by -G/2 first, so that the
 *     group boundaries sit half a group later and the last group wraps around the sequence end
 *     (Algorithm 1, its shift step; Section 3.2: with N=8192, G=2048 the first shifted group holds
 *     tokens 1025..3072 and the first and last 1024 tokens share a group);
 *   - causal softmax attention, scores scaled by 1/sqrt(d), runs inside each group in rolled order;
 *   - the second half of the heads is rolled back by +G/2 (Algorithm 1, its roll-back step), so every output is indexed
 *     by ORIGINAL token position.
 * Grouped-query attention: query head h reads KV head floor(h / (H/Hkv)) at the same (rolled)
 * coordinates as itself.  The wrapped group of a shifted head is kept as the paper's default
 * method has it: its first-half tokens attend the sequence's last G/2 tokens.
 *
 * Conventions shared by all entry points
 *   - Every tensor pointer is a DEVICE pointer owned by the caller unless a function says "host".
 *     The library never allocates, frees or keeps them.  All tensors are dense, last index fastest.
 *   - q, o, dO, dq : bf16 [B, N, H,   d]
 *     k, v, dk, dv : bf16 [B, N, Hkv, d]
 *     lse          : fp32 [B, H, N]   natural-log sum-exp of the scaled scores, original token order
 *   - `stream` is a cudaStream_t passed as void* (NULL = legacy default stream).  Calls only enqueue
 *     work and return without synchronising.
 *   - Return value: S2A_OK (0) or a negative s2a_status.  Arguments are checked before anything is
 *     enqueued, so S2A_ERR_INVALID_ARG, S2A_ERR_UNSUPPORTED, S2A_ERR_TOO_LARGE and S2A_ERR_TIMEOUT mean
 *     that nothing was enqueued.  S2A_ERR_CUDA means a CUDA call failed while enqueuing: an entry
 *     point that makes several launches or copies (s2a_bwd and its variants, s2a_fwd_bwd_host) may by
 *     then have enqueued the earlier ones, so the outputs are unspecified; `stream` still covers
 *     everything that was enqueued (s2a_fwd_bwd_host joins its copy streams into it on every path).
 *   - Supported shapes: d in {64, 128}; N a multiple of G, N >= 128; G a multiple of 8 (so that every
 *     run of tokens of a group, shifted by G/2 or not, starts and ends on a multiple of 4 tokens);
 *     H even; H a multiple of Hkv; pointers 16-byte aligned; a device of compute capability 10.x.
 *     G need not be a multiple of the kernels' 128-token tile (the paper's G = N/4 of N = 100,000 is
 *     25,000): a group is then covered by tiles whose last one is partly masked, and the group that
 *     wraps around the end of the sequence by two such runs of tiles.  Anything else is rejected,
 *     never approximated.
 *   - Rows of a partly masked tile that belong to a neighbouring group are read and masked by
 *     multiplying with zero weights, so inputs are assumed finite: where G or G/2 is not a multiple of
 *     128, a NaN or infinity in one token's q, k, v or dO can reach o, dq, dk or dv of the adjacent
 *     group's tokens.
 *   - Host threads: entry points may be called from several host threads (the one-time set-up of a
 *     device is serialised); s2a_fwd_bwd_host and s2a_bwd_noalloc keep per-device state (copy streams,
 *     built-in scratch), so calls of either on one device must not overlap.
 *   - Device-side waits are bounded (about a second of SM clock cycles, so heavy time-slicing of the
 *     GPU can in principle trip one).  If a wait expires the kernel records where, in a status word on
 *     the device and in a host-visible copy of it, and stops cleanly; the outputs of that launch are
 *     undefined.  The status is STICKY: until s2a_device_status() has read and cleared it, every
 *     kernel of this library that is already enqueued or gets launched on that device returns at once
 *     without writing its outputs, and every entry point that would enqueue work returns
 *     S2A_ERR_TIMEOUT instead (a host-side check of the copy; no synchronisation).  So a caller that
 *     sees S2A_ERR_TIMEOUT calls s2a_device_status(), discards the results since the last clean
 *     check, and goes on.
 *   - The first call on a device sets the library up for it (kernel attributes, the address of the
 *     status word, page-locking of a 4 KiB static status area); it allocates nothing, and should be
 *     made outside any stream capture.
 */
#ifndef S2A_H_
#define S2A_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum s2a_status {
    S2A_OK = 0,
    S2A_ERR_INVALID_ARG = -1, /* null pointer, non-positive size, N % G, odd G or H, H % Hkv, misaligned pointer, small workspace */
    S2A_ERR_UNSUPPORTED = -2, /* d not in {64,128}, G or shift not a multiple of 4 tokens (G/2 for the default shift), N < 128,
                                 ragged tiles with mixed shifts on one KV head, device is not sm_100 */
    S2A_ERR_CUDA = -3,        /* a CUDA call failed while enqueuing; see s2a_last_cuda_error() */
    S2A_ERR_TIMEOUT = -4,     /* reported by s2a_device_status(): a bounded device-side wait expired */
    S2A_ERR_TOO_LARGE = -5    /* s2a_bwd_noalloc only: B*H*N is more than its built-in scratch holds */
} s2a_status;

/*
 * Forward (Algorithm 1 with Eq. 1 inside each group).
 *   in : q, k, v                     out: o (bf16, rounded once from fp32), lse (fp32)
 * Scores and the P.V product accumulate in fp32 on the tensor cores; P is rounded to bf16 before
 * the second product.  One kernel launch on `stream`.
 */
int s2a_fwd(const void* q, const void* k, const void* v, void* o, float* lse,
            int B, int N, int H, int Hkv, int d, int G, void* stream);

/*
 * Backward: gradients of sum(o * dO) with respect to q, k, v (the paper trains through
 * Algorithm 1 by automatic differentiation; this is that derivative written out).
 *   in : q, k, v, o, lse (o and lse exactly as s2a_fwd produced them), dO
 *   out: dq, dk, dv (overwritten, not accumulated into)
 *   workspace: caller-owned device scratch of at least s2a_bwd_workspace_bytes(...) bytes,
 *              256-byte aligned; holds D[b,h,t] = dO[b,t,h,:] . o[b,t,h,:] in fp32, the work counters of
 *              the persistent kernels and, if it is large enough, the spilled dS (below).  Its contents
 *              before the call do not matter; calls that can overlap on the GPU need a workspace each.
 * dk and dv sum over the H/Hkv query heads that share a KV head inside one thread block, and every dq
 * row is summed by one thread block in a fixed order, so the results are deterministic (no atomics).
 *
 * Two ways to dq, chosen by the size of the workspace alone:
 *   - minimum workspace: the dq kernel recomputes the scores and dP that the dk/dv kernel also
 *     computes (14 d multiply-adds per attended pair are executed for the 10 d the derivative needs).
 *     Three kernel launches on `stream`.
 *   - a workspace of s2a_bwd_workspace_bytes_fast(...) bytes: the dk/dv kernel also leaves dS (bf16,
 *     the very values it multiplies with q) in the workspace and dq = scale * dS k is a plain product
 *     that reads them back: nothing is computed twice, at the price of 2 bytes of scratch per attended
 *     pair, written once and read once.  If the workspace holds the dS of only some of the KV heads,
 *     the KV heads are worked off in several passes (two launches and one 4-byte memset per pass).
 *   dk and dv are bit-identical either way; dq agrees to rounding (the fp32 sums inside the score
 *   products run in a different order).
 */
int s2a_bwd(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* dO,
            void* dq, void* dk, void* dv,
            int B, int N, int H, int Hkv, int d, int G,
            void* workspace, size_t workspace_bytes, void* stream);

/* Least bytes of scratch s2a_bwd needs for these sizes (0 if the sizes are invalid). */
size_t s2a_bwd_workspace_bytes(int B, int N, int H, int Hkv, int d, int G);

/*
 * The workspace size, not above `budget` bytes, with which s2a_bwd and its variants are fastest: the
 * minimum plus room for the dS of as many whole KV heads (with their H/Hkv query heads) as the budget
 * allows, all of them if it can: B * H * (N/G) * T * (T+1) * 16 KiB with T = G/128 tiles per group
 * (one more per run of a group where G/2 is not a multiple of 128).  Returns the minimum size when not
 * even one KV head fits, 0 if the sizes are invalid.  Any workspace between the two sizes is valid;
 * what counts is how many KV heads fit.  (The paper has no counterpart: it trains through a library
 * attention kernel.)
 */
size_t s2a_bwd_workspace_bytes_fast(int B, int N, int H, int Hkv, int d, int G, size_t budget);

/*
 * Generalised forms (Section 3.2 pilot study, Table 6 and Appendix B variants 1 and 2): the first
 * `n_unshifted` heads use the unshifted partition, the remaining heads are rolled by -shift
 * tokens (G and shift multiples of 4, |shift| < N; the paper's method is n_unshifted = H/2,
 * shift = G/2).  When G or shift is not a multiple of 128 the query heads of one KV head must all be
 * on the same side of n_unshifted (n_unshifted a multiple of H/Hkv).  n_unshifted = H gives "pattern 1 only"; with G = N as well it is ordinary full
 * causal attention, which the fine-tuned model uses at inference.  `scale` multiplies the scores
 * (pass 1/sqrt(d) for the standard choice).  H may be odd here.
 * flags: S2A_FLAG_LEAK_FREE selects variant 2 of Appendix B / Table 8: in a shifted head the group
 * that wraps around the sequence end is cut in two at the wrap, so the sequence's first tokens no
 * longer attend its last tokens.
 * S2A_FLAG_SWAP_WRAPPED selects variant 3 of Appendix B / Table 8 (its figure is not in the paper's
 * text, so this is a reading): in that same group the two parts change places, i.e. the group is
 * attended in original token order - the first tokens of the sequence, then its last ones - so that
 * no token attends a later one.  The two flags exclude each other; other bits must be 0.
 */
#define S2A_FLAG_LEAK_FREE 1u
#define S2A_FLAG_SWAP_WRAPPED 2u
int s2a_fwd_ex(const void* q, const void* k, const void* v, void* o, float* lse,
               int B, int N, int H, int Hkv, int d, int G,
               float scale, int n_unshifted, int shift, unsigned flags, void* stream);
int s2a_bwd_ex(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* dO,
               void* dq, void* dk, void* dv,
               int B, int N, int H, int Hkv, int d, int G,
               float scale, int n_unshifted, int shift, unsigned flags,
               void* workspace, size_t workspace_bytes, void* stream);

/*
 * The calling convention of Algorithm 1 itself: queries, keys and values packed in one tensor
 *   qkv  : bf16 [B, N, 3, H, d]   (index 0 = q, 1 = k, 2 = v; H query heads = H KV heads)
 *   dqkv : bf16 [B, N, 3, H, d]   gradients in the same packing (overwritten)
 * o, dO [B, N, H, d] and lse [B, H, N] stay dense.  Nothing is unpacked or copied: the packed layout
 * only changes the strides of the TMA tensor maps and of the gradient stores.  Semantics, shape
 * limits, workspace and errors are those of s2a_fwd / s2a_bwd with Hkv = H.
 */
int s2a_fwd_packed(const void* qkv, void* o, float* lse, int B, int N, int H, int d, int G, void* stream);
int s2a_bwd_packed(const void* qkv, const void* o, const float* lse, const void* dO, void* dqkv,
                   int B, int N, int H, int d, int G,
                   void* workspace, size_t workspace_bytes, void* stream);

/*
 * s2a_bwd for callers that have no scratch to give.  (The paper has no counterpart to this entry
 * point; it exists for integration reasons only.)
 *
 * Who needs it: code that is not allowed, or not able, to obtain device memory at the moment it
 * wants gradients -- a plug-in running inside a host application that owns all device memory and
 * exposes no allocator; a service whose memory budget was handed out in full at start-up; a
 * latency-critical loop that must not meet the implicit device-wide synchronisation and the
 * unpredictable cost of cudaMalloc / cudaFree; a component whose rules forbid allocation after
 * initialisation.  s2a_bwd wants a workspace from such a caller; this variant does not.
 *
 * It computes exactly what s2a_bwd computes with a minimum workspace (same kernels, same results), but keeps
 * D = rowsum(dO * o) and the work counter of its persistent kernel in an array that is part of the
 * library image: 2^20 fp32 values and 256 bytes (4 MiB in all) on every GPU that loads the library,
 * held until the process exits.  It calls no allocation routine of any kind.
 *
 *   Limit     : B * H * N <= s2a_bwd_noalloc_max_rows() (= 1,048,576; e.g. B=1, H=32, N=32768).
 *               Larger problems return S2A_ERR_TOO_LARGE and enqueue nothing; use s2a_bwd.
 *   Set-up    : the first call on each device looks up the array's device address (with that
 *               device current).  Make that first call outside any stream capture.
 *   Sharing   : all calls on a device use the same array.  Calls issued to one stream are ordered
 *               and safe.  Two calls that can run on the GPU at the same time (different streams,
 *               or different host threads on different streams) overwrite each other's D and
 *               give wrong gradients: serialise them, or use s2a_bwd with separate workspaces.
 *   Contents  : the array keeps whatever the previous call left; every value of D a call reads is
 *               first rewritten by that same call, and the work counter is set to zero by a 4-byte
 *               memset on `stream` ahead of the kernel that counts with it, so the caller clears nothing.
 * Other arguments, shapes, errors and the meaning of `stream` are those of s2a_bwd.
 */
int s2a_bwd_noalloc(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* dO,
                    void* dq, void* dk, void* dv,
                    int B, int N, int H, int Hkv, int d, int G, void* stream);

/* Largest B * H * N that s2a_bwd_noalloc accepts. */
size_t s2a_bwd_noalloc_max_rows(void);

/*
 * One kernel of s2a_bwd at a time, for profiling and per-kernel timing: same arguments and
 * semantics as s2a_bwd, but only kernel `stage` is enqueued:
 *   0 = D = rowsum(dO * o) into the workspace, 1 = dk and dv, 2 = dq.
 * Stages 1 and 2 read the workspace stage 0 wrote (stage 2 also what stage 1 left there, when the
 * workspace is large enough to hold the dS of ALL KV heads; a smaller one selects the recomputing dq
 * kernel here).  Calling stages 0, 1, 2 in order on one stream is exactly s2a_bwd with that choice.
 */
int s2a_bwd_stage(const void* q, const void* k, const void* v, const void* o, const float* lse, const void* dO,
                  void* dq, void* dk, void* dv,
                  int B, int N, int H, int Hkv, int d, int G,
                  void* workspace, size_t workspace_bytes, int stage, void* stream);

/*
 * Forward + backward from HOST buffers (pinned memory, or the copies are not asynchronous): q, k, v,
 * dO go to the caller's device buffers, s2a_fwd and s2a_bwd run there, and o, lse, dq, dk, dv come
 * back.  Heads are independent, so the work is cut into up to 16 chunks of whole KV heads - small ones
 * at either end, growing towards the middle - and the copy of one chunk, the kernels of the previous
 * one and the copy back of the one before that overlap (two copy streams owned by the library,
 * created by the first call on a device, ordered
 * against `stream` by events).  Everything is ordered after the work already in `stream` and
 * `stream` is complete only when the last result has landed: the caller synchronises `stream`
 * before reading the host outputs.  Results are bit-identical to s2a_fwd + s2a_bwd given the same
 * workspace size (which selects how dq is computed, see s2a_bwd; what counts here is how many KV heads
 * of the largest chunk the workspace has dS room for).
 *   h_*  : host pointers, same layouts and types as the device tensors
 *   d_*  : device buffers of the same sizes, owned by the caller (the library allocates no memory);
 *          used as staging space: their contents after the call are unspecified
 */
int s2a_fwd_bwd_host(const void* h_q, const void* h_k, const void* h_v, const void* h_dO,
                     void* h_o, float* h_lse, void* h_dq, void* h_dk, void* h_dv,
                     void* d_q, void* d_k, void* d_v, void* d_dO, void* d_o, float* d_lse,
                     void* d_dq, void* d_dk, void* d_dv,
                     int B, int N, int H, int Hkv, int d, int G,
                     void* workspace, size_t workspace_bytes, void* stream);

/*
 * Diagnostic (the paper has no counterpart): enqueues one tiny kernel on `stream` in which a single
 * warp waits, with the library's own bounded wait and a limit of `limit_cycles` SM clock cycles
 * (1 .. 2,000,000,000; a million is well under a millisecond), on a barrier that nothing ever arrives
 * on.  The wait runs out, the kernel reports it exactly as a production kernel would (wait code 901)
 * and returns; nothing hangs and nothing faults.  It lets a caller, or a test, see the whole
 * time-out path: the sticky status, S2A_ERR_TIMEOUT from the entry points, s2a_device_status().
 */
int s2a_selftest_wait_expiry(long long limit_cycles, void* stream);

/*
 * Reads (and clears) the device-side status word of the current device.  Synchronises the device.
 * Returns S2A_OK, S2A_ERR_TIMEOUT (a bounded wait expired in some kernel since the last call; if
 * `where` is non-NULL it receives a code naming the kernel and the wait), or S2A_ERR_CUDA.
 */
int s2a_device_status(int* where);

/* Static, human-readable text for a status code. */
const char* s2a_status_string(int status);

/* cudaError_t value of the most recent failing CUDA call made by this library on this thread. */
int s2a_last_cuda_error(void);

/* Library version: major * 10000 + minor * 100 + patch. */
int s2a_version(void);

#ifdef __cplusplus
}
#endif
#endif /* S2A_H_ */
