// Shared declarations of the BlockFFN CUDA library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "blockffn.h"

// Logit buffers a handle cycles through: the router of a layer call may start as soon as the
// call kLogitRing - 1 calls earlier has started, i.e. once the readers of its buffer are done.
// (Eight: a router-on call whose x is stable runs on about a third of the SMs, three CTAs per
// SM, so about seven of them are in flight and as many routers must be able to run ahead. One
// stream for those routers: spread over two or three streams they measured slower, 14.2 and 14.7
// against 12.6 us per call with unions of 54 experts.)
constexpr int kLogitRing = 8;

struct blockffn_ctx {
  blockffn_config cfg;
  int device;
  int num_sms;
  int words;            // ceil(E / 32)
  uint64_t launches;    // host-side count of kernels launched through this handle
  // ---- workspace (device) ----
  void* ws_base;
  float* a0;            // [L_max][E] router logits
  float* a0_ring[kLogitRing];   // the logit buffers blockffn_layer_forward cycles through
  int a0_phase;         // which of them its next call writes
  // ---- router on a stream of its own (blockffn_layer_forward with x stable) ----
  cudaStream_t side;          // non-blocking; NULL when it could not be created
  cudaEvent_t ev_call[kLogitRing];     // recorded on the caller's stream at the start of a layer call
  cudaEvent_t ev_router[kLogitRing];   // recorded on `side` behind the router of a layer call
  struct {
    bool set;                 // ev_call[i] holds a record that may be waited for
    cudaStream_t stream;      // ... made on this stream
    bool capturing;           // ... inside a stream capture
    unsigned long long id;    // ... with this capture id
  } call_mark[kLogitRing];
  bool last_layer_waited_first;   // the previous layer call's up kernel waited before anything
  float* scores;        // [L_max][E]
  uint32_t* tok_mask;   // [L_max][words]
  uint32_t* union_mask; // [words]
  int32_t* union_ids;   // [E]
  int32_t* n_union;     // [1]
  float* h32;           // [E][L_max][d_e] fp32 intermediate (SIMT variant)
  void* h16;            // bf16 intermediate (MMA variant), slot-major padded rows
  void* lean_ring;      // rings of bf16 intermediates of the one-kernel form, then its rings of
                        // router logits (NULL: not used)
  unsigned long long* lean_seq;   // per ring (four of them, 64 words apart): [0] call tickets,
                                  // [1 .. 16] arrival counters of the ring slots, [17 .. 32] those
                                  // of the logit hand-over when the router runs inside the kernel
  float* ones;          // [E] of 1.0f: the gain of the router without RMSNorm
  unsigned int* ticket; // last-block-done counters [8]
  uint32_t* status;     // sticky device status word
};

// ---- device helpers -------------------------------------------------------
__device__ __forceinline__ float bf16_lo(uint32_t packed) { return __uint_as_float(packed << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t packed) {
  return __uint_as_float(packed & 0xffff0000u);
}
// float -> bf16 bits, round to nearest even, NaN kept quiet
__device__ __forceinline__ uint32_t f32_to_bf16_bits(float f) {
  uint32_t w = __float_as_uint(f);
  if ((w & 0x7fffffffu) > 0x7f800000u) return (w >> 16) | 0x40u;
  return (w + 0x7fffu + ((w >> 16) & 1u)) >> 16;
}
__device__ __forceinline__ float swish(float z) { return z / (1.0f + __expf(-z)); }

// The router without RMSNorm (rms_eps == BLOCKFFN_NO_RMSNORM) has no gain: the kernels multiply
// by a vector of ones and skip the normalisation where they see a negative eps.
inline bool no_rmsnorm(const blockffn_ctx* c) { return c->cfg.rms_eps < 0.0f; }
inline const float* router_gain(const blockffn_ctx* c, const blockffn_weights* w) {
  return no_rmsnorm(c) ? c->ones : w->gain;
}

// ---- launchers (each returns the cudaError_t of its launch) ----------------
cudaError_t launch_router(blockffn_ctx* c, const blockffn_weights* w, const void* x, int L,
                          float* scores, uint32_t* tok_mask, bool fuse_union,
                          blockffn_stats* stats, bool raw, float* logits, int mode,
                          cudaStream_t st);
// mode: 0 the kernel waits for the work before it first; 1 (raw only) it computes under that
// work and waits at its end; 2 (raw only) it is launched without programmatic chaining on a
// stream of its own and lets its dependents go only by exiting, behind a fence.
cudaError_t launch_chunk_union(blockffn_ctx* c, const float* scores, int L, uint32_t* union_mask,
                               int32_t* union_ids, int32_t* n_union, blockffn_stats* stats,
                               cudaStream_t st);
cudaError_t launch_reuse_ratio(blockffn_ctx* c, const float* scores, int L, double* reuse,
                               cudaStream_t st);
cudaError_t launch_expert_simt(blockffn_ctx* c, const blockffn_weights* w, const void* x,
                               const float* scores, int L, const int32_t* union_ids,
                               const int32_t* n_union, float* out, void* x_next, int call_flags,
                               cudaStream_t st);

// Where a kernel that derives Union(x) itself publishes it (each pointer may be NULL).
struct RoutingOut {
  uint32_t* union_mask;
  int32_t* union_ids;
  int32_t* n_union;
  blockffn_stats* stats;
  float* scores;        // [L][E], written only when the kernel normalises router logits itself
  uint32_t* tok_mask;   // [L][words], likewise
};
// Raw router logits (Eq. 3 before ReLU) for kernels that finish the router themselves.
struct RouterLogits {
  const float* a0;      // [L][E]
  const float* gain;    // [E]
  float eps;
};

// One-kernel form of the tensor-core expert stage for chunks of at most 8 tokens (same
// arguments as launch_expert_mma below).
bool expert_lean_supported(const blockffn_ctx* c, int L, bool with_logits, bool shared,
                           bool inside = false);
size_t expert_lean_ws_bytes(const blockffn_config* cfg, int grid);
cudaError_t expert_lean_setup(blockffn_ctx* c);
cudaError_t launch_expert_lean(blockffn_ctx* c, const blockffn_weights* w, const void* x,
                               const float* scores, int L, const int32_t* union_ids,
                               const int32_t* n_union, float* out, void* x_next, int call_flags,
                               const RoutingOut* pub, const RouterLogits* logits, bool logits_final,
                               cudaStream_t st);

// Tensor-core / bulk-copy variant of the expert stage. union_ids == NULL: the kernels derive
// the union from the nonzero pattern of scores and publish it through pub; with logits != NULL
// they first turn the raw router logits into scores (ReLU, RMSNorm, gain) and scores is unused.
bool expert_mma_supported(const blockffn_ctx* c, int L);
size_t expert_mma_h_bytes(const blockffn_config* cfg);
cudaError_t expert_mma_setup(blockffn_ctx* c);
cudaError_t launch_expert_mma(blockffn_ctx* c, const blockffn_weights* w, const void* x,
                              const float* scores, int L, const int32_t* union_ids,
                              const int32_t* n_union, float* out, void* x_next, int call_flags,
                              const RoutingOut* pub, const RouterLogits* logits, bool logits_final,
                              cudaStream_t st);
