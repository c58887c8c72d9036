/*
 * blockffn.h - C ABI of the BlockFFN chunk-verify FFN forward for NVIDIA B200 (sm_100a).
 *
 * One call evaluates one BlockFFN layer for a chunk of L draft tokens that a
 * speculative-decoding step verifies in parallel (Sec. 3.3 of the BlockFFN paper):
 *   1. router       A(x) = RMSNorm(ReLU(W_router^T x))                       (Eq. 3)
 *   2. chunk union  Union(x) = experts activated by any of the L tokens      (Sec. 3.3)
 *   3. expert FFN   FFN(x_t) = sum_{i in Union} A_i(x_t) W_down^(i)T Swish(W_up^(i)T x_t)
 *                                                                            (Eq. 1, Eq. 2)
 * Only the union experts' weights are read from device memory.
 *
 * Conventions (all entry points)
 *   - Every data pointer is a DEVICE pointer owned by the caller, 16-byte aligned,
 *     valid until the work enqueued by the call has finished. The library owns only
 *     the workspace inside its handle.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Calls only enqueue work: no allocation, no host synchronisation, no copy to
 *     the host. Two calls on one handle must not run concurrently on the device
 *     (they share the handle's workspace); use one handle per stream.
 *   - Row-major layouts. bf16 = the upper 16 bits of an IEEE float32.
 *       x       bf16 [L][d]           hidden states of the chunk
 *       scores  f32  [L][E]           A(x); expert i is active for token t iff
 *                                     scores[t][i] != 0.0f by value (-0.0f is zero,
 *                                     NaN counts as active and propagates)
 *       out     f32  [L][d]
 *   - The return value reports what the host can detect (bad arguments, launch
 *     failures). Problems found on the device (a union id out of range, a count
 *     larger than E) set bits in a sticky status word, skip the offending work and
 *     never fault; read it with blockffn_last_status().
 *   - Limits: 1 <= L <= L_max <= 32 per call; d % 8 == 0; d_e % 8 == 0;
 *     1 <= E <= 1024.
 */
#ifndef BLOCKFFN_H_
#define BLOCKFFN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(_WIN32)
#define BLOCKFFN_API
#else
#define BLOCKFFN_API __attribute__((visibility("default")))
#endif

typedef enum {
  BLOCKFFN_OK = 0,
  BLOCKFFN_ERR_INVALID_ARG = 1, /* NULL / misaligned pointer, size out of range   */
  BLOCKFFN_ERR_UNSUPPORTED = 2, /* shape outside the limits above                 */
  BLOCKFFN_ERR_WORKSPACE = 3,   /* workspace allocation failed in blockffn_create */
  BLOCKFFN_ERR_CUDA = 4,        /* a CUDA runtime call or launch failed           */
  BLOCKFFN_ERR_DEVICE = 5       /* the device status word is nonzero              */
} blockffn_status;

/* Bits of the device status word (blockffn_last_status). */
#define BLOCKFFN_DEV_BAD_UNION_ID 1u    /* a union id was < 0 or >= E: that entry was skipped   */
#define BLOCKFFN_DEV_BAD_UNION_COUNT 2u /* n_union was < 0 or > E: it was clamped               */
#define BLOCKFFN_DEV_WAIT_EXPIRED 4u    /* a bounded wait inside a kernel ran out: the call's out is invalid */

/* Kernel family used by the expert stage. AUTO picks by L and shape. */
#define BLOCKFFN_VARIANT_AUTO 0
#define BLOCKFFN_VARIANT_SIMT 1   /* CUDA-core dot products, fp32 intermediate             */
#define BLOCKFFN_VARIANT_MMA 2    /* asynchronously staged, tensor-core tiles, bf16 intermediate;
                                     blockffn_create returns UNSUPPORTED for a shape or ring
                                     depth these kernels do not take (d % 64, d_e a power of
                                     two >= 64, ring depths >= 3 / 2)                        */

typedef struct {
  int32_t d;       /* hidden size d_h                                          */
  int32_t E;       /* number of experts N_e                                    */
  int32_t d_e;     /* expert width                                             */
  int32_t L_max;   /* largest chunk length a call may pass (<= 32)             */
  float rms_eps;   /* RMSNorm epsilon, added to the mean square (Eq. 3); 1e-6;
                      BLOCKFFN_NO_RMSNORM: the router of the Sec. 4.2.3 ablation  */
  int32_t variant; /* BLOCKFFN_VARIANT_*                                       */
  int32_t flags;   /* tuning, 0 = defaults: bits 0-7 ring depth of the up-projection
                      kernel, bits 8-15 of the down-projection kernel (stages of shared
                      memory, 0 = chosen from the shape), BLOCKFFN_CFG_* bits        */
} blockffn_config;

/* rms_eps value that takes RMSNorm out of the router (the ablation of Sec. 4.2.3, the
 * ReMoE-style router of Table 1): scores = ReLU(W_router^T x + bias), no normalisation and no
 * gain (blockffn_weights.gain is not read and may be NULL). Every other rms_eps must be >= 0. */
#define BLOCKFFN_NO_RMSNORM (-1.0f)

/* The tensor-core kernels are normally launched so that a kernel may start fetching its
 * weights while the kernel enqueued before it on the stream is still finishing
 * (programmatic dependent launch); this bit launches them fully serialised instead. */
#define BLOCKFFN_CFG_NO_CHAINING 0x10000
/* A call whose x is stable normally runs as one kernel, several calls in flight per SM; this
 * bit selects the two-kernel form (up projection, down projection), the form every other call
 * takes, for those calls too. Same results within the tolerance; kept for comparison.        */
#define BLOCKFFN_CFG_TWO_KERNELS 0x20000000
/* The one-kernel form runs a call whose x is promised stable (BLOCKFFN_CALL_INDEPENDENT_X) on
 * about a third of the SMs, so that about three times as many such calls are in flight: every CTA reads all
 * of x and of the intermediate from L2, and fewer, larger CTAs per call keep that broadcast
 * small next to the weight stream. This bit gives those calls the whole device each, like the
 * calls of a dependent chain.                                                              */
#define BLOCKFFN_CFG_NO_SPLIT 0x40000000
/* Test aid: the one-kernel form's hand-over waits for an arrival that never comes, gives up
 * after two milliseconds, sets BLOCKFFN_DEV_WAIT_EXPIRED and leaves out untouched. Exercises
 * the bounded wait without any fault.                                                      */
#define BLOCKFFN_CFG_TEST_EXPIRE_WAIT 0x10000000
/* How many experts the caller expects in a chunk's union (1 .. E), bits 17-27 of flags. The
 * tensor-core kernels size their shared memory before the union is known: when the expected
 * union's share fits half an SM, two kernels share an SM and consecutive launches overlap
 * (best for the paper's operating points); a larger expected union gives each kernel a whole
 * SM and fewer, larger stages instead. 0 = assume the paper's sparsity: 30 % of the experts
 * for a chunk (CLS of Table "moe-ppl"), 12.5 % for a single token (Sec. 4.4). The hint only
 * changes speed; any union size gives the same results under any hint.                     */
#define BLOCKFFN_CFG_EXPECTED_UNION(u) (((u) & 0x7ff) << 17)

/* Layer parameters: device pointers, caller-owned, read-only to the library. */
typedef struct {
  const void* W_r;   /* bf16 [E][d]: row i = column i of W_router (Eq. 3). May be NULL for
                        scores-in calls.                                                   */
  const float* gain; /* f32 [E]: RMSNorm gain (Eq. 3). May be NULL for scores-in calls.    */
  const float* bias; /* f32 [E] added to the router logits, or NULL (NULL = Eq. 3 as
                        printed; a synthetic router uses it to set its sparsity).          */
  const void* U;     /* bf16 [E][d_e][d]: U[i][j][k] = W_up^(i)[k][j]   (Eq. 2)            */
  const void* D;     /* bf16 [E][d][d_e]: D[i][c][j] = W_down^(i)[j][c] (Eq. 2)            */
} blockffn_weights;

/* Counters behind TLS and CLS_L (Sec. 2.1), accumulated on the device, one chunk per call. */
typedef struct {
  uint64_t n_tokens; /* tokens seen                                  */
  uint64_t n_active; /* sum over tokens of |experts active for it|   */
  uint64_t n_chunks; /* chunks seen                                  */
  uint64_t n_union;  /* sum over chunks of |Union|                   */
} blockffn_stats;

/* Per-call flags. */
#define BLOCKFFN_CALL_ACCUMULATE 1 /* out += FFN(x) (residual, fp32) instead of out = FFN(x)     */
/* The tensor-core kernels of a call may start while the kernels enqueued before it on `stream`
 * are still running (programmatic dependent launch). What they read before they have waited for
 * that earlier work to finish is governed by two promises of the caller:                      */
#define BLOCKFFN_CALL_INDEPENDENT 2 /* scores, union_ids, n_union and the weights of this call are
                                       stable: nothing enqueued on `stream` since the last call made
                                       without this flag (or since the last host synchronisation)
                                       writes them. x and out may still come from the work just
                                       before. The weight fetch then overlaps the previous kernel
                                       (a chunk of more than 8 tokens then runs as one kernel that
                                       waits for that work before it reads x).                      */
#define BLOCKFFN_CALL_INDEPENDENT_X 4 /* in addition x is stable in the same sense (the chunk does
                                       not consume the previous call's output); implies
                                       BLOCKFFN_CALL_INDEPENDENT. The up projection then runs in full
                                       under the previous call and only its store waits. In
                                       blockffn_layer_forward the router then runs inside the expert
                                       kernel (one launch per call) where the shape allows it, else
                                       ahead of it on a stream of the handle.                       */

typedef struct blockffn_ctx* blockffn_handle;

/* Creates a handle on the current CUDA device and allocates its workspace there
 * (the only allocation the library ever makes), plus one non-blocking stream and a few events
 * of its own for the router of blockffn_layer_forward (the handle works without them if they
 * cannot be created). Returns WORKSPACE if the allocation fails.                          */
BLOCKFFN_API blockffn_status blockffn_create(const blockffn_config* cfg, blockffn_handle* out);
/* Frees the workspace. The caller synchronises outstanding work first. */
BLOCKFFN_API blockffn_status blockffn_destroy(blockffn_handle h);

/* Eq. 3. scores[t][i] = gain[i] * a1 / sqrt(mean_i(a1^2) + rms_eps), a1 = max(0, x_t . W_r[i] + bias[i]);
 * tok_mask[t][w] bit b = (scores[t][32 w + b] != 0), bits at and beyond E zero
 * (tok_mask: u32 [L][ceil(E/32)], may be NULL). The mean runs over all E entries.      */
BLOCKFFN_API blockffn_status blockffn_router(blockffn_handle h, const blockffn_weights* w,
                                             const void* x, int32_t L, float* scores,
                                             uint32_t* tok_mask, void* stream);

/* Sec. 3.3 Union(x) from a score matrix: union_mask u32 [ceil(E/32)] (may be NULL);
 * union_ids i32 [E], ascending expert ids, entries from n_union on are -1; n_union i32 [1]
 * (device). stats (device, may be NULL) is advanced by this chunk (Sec. 2.1 counters). */
BLOCKFFN_API blockffn_status blockffn_chunk_union(blockffn_handle h, const float* scores, int32_t L,
                                                  uint32_t* union_mask, int32_t* union_ids,
                                                  int32_t* n_union, blockffn_stats* stats,
                                                  void* stream);

/* Eq. 1 + Eq. 2 restricted to the listed experts: reads U_i, D_i only for
 * i in union_ids[0 .. *n_union). out = (out +) sum_i scores[t][i] * D_i Swish(U_i x_t).
 * union_ids must be a readable i32 [E] array (what blockffn_chunk_union writes); only its
 * first *n_union entries count, the rest may hold anything and are ignored.
 * x_next (bf16 [L][d], may be NULL, must not alias x) receives the bf16 rounding of the
 * final out: the next layer's input when out is a running fp32 residual.
 * An expert missing from the list contributes nothing, whatever its score.              */
BLOCKFFN_API blockffn_status blockffn_expert_ffn(blockffn_handle h, const blockffn_weights* w,
                                                 const void* x, const float* scores, int32_t L,
                                                 const int32_t* union_ids, const int32_t* n_union,
                                                 float* out, void* x_next, int32_t call_flags,
                                                 void* stream);

/* Whole layer, router on: Eq. 3 -> Union(x) -> Eq. 1/2, everything device side.
 * The scores, masks, ids and count land in the handle's workspace
 * (blockffn_read_routing). stats may be NULL.
 * call_flags: ACCUMULATE as above. With INDEPENDENT_X (x and the weights are stable, see the
 * flag) the router is launched on the handle's own stream, ordered behind layer calls made a
 * few calls earlier on `stream` and in front of this call's expert kernels (event record /
 * wait, also inside a stream capture), so that it runs under the calls before it; the expert
 * kernels then fetch their weights under the previous call as a scores-in call does. The
 * first such calls on a stream, or after the stream or its capture changed, keep the router
 * on `stream`. All work of the call is complete when `stream` has reached its end.        */
BLOCKFFN_API blockffn_status blockffn_layer_forward(blockffn_handle h, const blockffn_weights* w,
                                                    const void* x, int32_t L, float* out,
                                                    void* x_next, blockffn_stats* stats,
                                                    int32_t call_flags, void* stream);

/* Whole layer from precomputed router scores (the scores-in entry): Union(x) -> Eq. 1/2. */
BLOCKFFN_API blockffn_status blockffn_layer_forward_scores(blockffn_handle h,
                                                           const blockffn_weights* w, const void* x,
                                                           const float* scores, int32_t L,
                                                           float* out, void* x_next,
                                                           blockffn_stats* stats,
                                                           int32_t call_flags, void* stream);

/* Enqueues device-to-device copies of what the last layer call on this handle derived
 * (kept in the handle's workspace until the next call overwrites it) into caller buffers:
 * scores f32 [L][E] and tok_mask u32 [L][ceil(E/32)] (router-on calls only),
 * union_mask u32 [ceil(E/32)], union_ids i32 [E], n_union i32 [1]. Any may be NULL. */
BLOCKFFN_API blockffn_status blockffn_read_routing(blockffn_handle h, int32_t L, float* scores,
                                                   uint32_t* tok_mask, uint32_t* union_mask,
                                                   int32_t* union_ids, int32_t* n_union,
                                                   void* stream);

/* Synchronises `stream`, then returns OK if the device status word is zero, DEVICE otherwise;
 * *bits (may be NULL) receives the BLOCKFFN_DEV_* bits; clear != 0 resets the word.      */
BLOCKFFN_API blockffn_status blockffn_last_status(blockffn_handle h, uint32_t* bits, int32_t clear,
                                                  void* stream);

/* Sec. 2.1, from a HOST copy of the counters: TLS = 1 - n_active / (n_tokens E),
 * CLS_L = 1 - n_union / (n_chunks E) with L the chunk length of the calls counted.      */
BLOCKFFN_API double blockffn_tls(const blockffn_stats* host_stats, int32_t E);
BLOCKFFN_API double blockffn_cls(const blockffn_stats* host_stats, int32_t E);

/* Reuse ratio between successive tokens (Sec. 4.1.2). With S_i the experts token i of a
 * sequence activates (nonzero score, by value), adds to reuse[0] the ratios
 * |S_i n S_{i+1}| / |S_i| of the sequence's L - 1 successive pairs, one after the other in
 * token order, and to reuse[1] the number of pairs counted; a pair whose first token activates
 * no expert has no ratio and is left out of both. The sequence's (or, over many calls, the
 * average) reuse ratio is reuse[0] / reuse[1].
 * scores: f32 [L][E], device; NULL = the scores the last router-on layer call on this handle
 * left in its workspace (then L <= L_max). L >= 1 is otherwise not limited by L_max: a
 * sequence is not a chunk. reuse: f64 [2], device, 8-byte aligned, caller-owned and zeroed
 * by the caller; calls that share it must be ordered (one stream).
 * Errors: INVALID_ARG (NULL or misaligned pointer, L < 1, scores NULL with L > L_max).      */
BLOCKFFN_API blockffn_status blockffn_reuse_ratio(blockffn_handle h, const float* scores,
                                                  int32_t L, double* reuse, void* stream);

/* Number of kernels the library has launched through this handle (host counter). */
BLOCKFFN_API uint64_t blockffn_launch_count(blockffn_handle h);

/* Largest fp32 intermediate blockffn_expert_ffn_noalloc can hold: E * L * d_e * 4 bytes of a
 * call must not exceed it (1 MiB: E = 64, d_e = 128 up to L = 32). */
#define BLOCKFFN_NOALLOC_SCRATCH_BYTES (1 << 20)

/* The paper has no counterpart of this entry point; it exists for deployment reasons only.
 * It is blockffn_expert_ffn (Eq. 1 + Eq. 2 over the listed experts, same arguments, same
 * result as the CUDA-core variant) for callers that are not allowed to allocate device
 * memory and therefore cannot call blockffn_create, whose workspace comes from cudaMalloc:
 * for instance a plug-in that runs inside a host application which has handed all device
 * memory to its own pool (an allocation would fail, or would stall every stream of the
 * process while the driver maps it), or code on a latency-critical path where an
 * allocator call is forbidden by policy. It takes the shape in a blockffn_config
 * (d, E, d_e, rms_eps unused; L_max, variant and flags are ignored) instead of a handle and
 * makes no call that allocates or frees memory.
 *   - Its intermediate lives in a fixed array inside the library image, which every GPU that
 *     loads the library keeps until the process exits: BLOCKFFN_NOALLOC_SCRATCH_BYTES plus a
 *     256-byte header. A call whose E * L * d_e * 4 exceeds that size returns
 *     BLOCKFFN_ERR_WORKSPACE and enqueues nothing.
 *   - The first call on a device looks up the array's device address (with that device
 *     current) and caches it; make that first call at start-up, outside any stream capture.
 *     That first call is also where the driver may load the library's image onto the device,
 *     array included. Later calls find the address under a lock and may come from any host
 *     thread.
 *   - All calls on a device share the one array. Calls enqueued on the same stream are safe;
 *     two calls that may run on the GPU at the same time (different streams, or graph
 *     branches) race on it and give wrong results. Nothing in the array carries over from
 *     one call to the next: the part a call reads is rewritten by that call first.
 *   - Out-of-range union entries are skipped as in blockffn_expert_ffn but are not reported:
 *     there is no handle whose status word could be read.                                  */
BLOCKFFN_API blockffn_status blockffn_expert_ffn_noalloc(
    const blockffn_config* cfg, const blockffn_weights* w, const void* x, const float* scores,
    int32_t L, const int32_t* union_ids, const int32_t* n_union, float* out, void* x_next,
    int32_t call_flags, void* stream);

/* Human-readable name of a status code (static storage). */
BLOCKFFN_API const char* blockffn_status_string(blockffn_status s);

#ifdef __cplusplus
}
#endif
#endif /* BLOCKFFN_H_ */
