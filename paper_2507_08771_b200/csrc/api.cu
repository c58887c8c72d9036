// C ABI of the BlockFFN library: argument checks, workspace, dispatch.
#include <new>
#include <vector>

#include "common.cuh"

namespace {

constexpr int kCallFlags =
    BLOCKFFN_CALL_ACCUMULATE | BLOCKFFN_CALL_INDEPENDENT | BLOCKFFN_CALL_INDEPENDENT_X;

inline bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

blockffn_status check_call(blockffn_ctx* c, int L) {
  if (!c) return BLOCKFFN_ERR_INVALID_ARG;
  if (L < 1 || L > c->cfg.L_max) return BLOCKFFN_ERR_INVALID_ARG;
  return BLOCKFFN_OK;
}

bool use_mma(const blockffn_ctx* c, int L) {
  return c->cfg.variant != BLOCKFFN_VARIANT_SIMT && expert_mma_supported(c, L);
}

// Tensor-core expert stage: one kernel per call or the up/down pair.
cudaError_t launch_tensor_core(blockffn_ctx* c, const blockffn_weights* w, const void* x,
                               const float* scores, int L, const int32_t* union_ids,
                               const int32_t* n_union, float* out, void* x_next, int call_flags,
                               const RoutingOut* pub, const RouterLogits* logits, bool logits_final,
                               cudaStream_t st) {
  // The one-kernel form pays off where calls overlap freely, i.e. where x is stable (for a
  // router-on call: the router has finished before the expert stage starts). A call of up to 8
  // tokens in a dependent chain (x comes from the call before) runs as the pair, whose two
  // hand-overs are shorter than a grid-wide exchange inside one kernel; a longer chunk in such a
  // chain (weights and scores promised stable) takes the one-kernel form on the whole device,
  // which keeps its weights in shared memory for all tokens at once.
  const bool x_stable = logits ? logits_final : (call_flags & BLOCKFFN_CALL_INDEPENDENT_X) != 0;
  const bool dep_long = !x_stable && !logits && (call_flags & BLOCKFFN_CALL_INDEPENDENT) && L > 8;
  const bool dep_inside = !x_stable && logits && logits->a0 == nullptr;   // router inside the kernel
  if ((x_stable || dep_long || dep_inside) &&
      expert_lean_supported(c, L, logits != nullptr, x_stable, logits && logits->a0 == nullptr))
    return launch_expert_lean(c, w, x, scores, L, union_ids, n_union, out, x_next, call_flags, pub,
                              logits, logits_final, st);
  return launch_expert_mma(c, w, x, scores, L, union_ids, n_union, out, x_next, call_flags, pub,
                           logits, logits_final, st);
}

// Expert stage from a given union list.
blockffn_status expert_dispatch(blockffn_ctx* c, const blockffn_weights* w, const void* x,
                                const float* scores, int L, const int32_t* union_ids,
                                const int32_t* n_union, float* out, void* x_next, int call_flags,
                                cudaStream_t st) {
  cudaError_t e;
  if (use_mma(c, L))
    e = launch_tensor_core(c, w, x, scores, L, union_ids, n_union, out, x_next, call_flags, nullptr,
                           nullptr, false, st);
  else
    e = launch_expert_simt(c, w, x, scores, L, union_ids, n_union, out, x_next, call_flags, st);
  return e == cudaSuccess ? BLOCKFFN_OK : BLOCKFFN_ERR_CUDA;
}

}  // namespace

extern "C" {

// Frees the side stream and its events (those that exist).
static void release_side(blockffn_ctx* c) {
  for (int i = 0; i < kLogitRing; ++i) {
    if (c->ev_call[i]) cudaEventDestroy(c->ev_call[i]);
    if (c->ev_router[i]) cudaEventDestroy(c->ev_router[i]);
    c->ev_call[i] = c->ev_router[i] = nullptr;
  }
  if (c->side) cudaStreamDestroy(c->side);
  c->side = nullptr;
}

// Whether `st` is being captured, and under which capture id. False when that cannot be told.
static bool capture_state(cudaStream_t st, bool* capturing, unsigned long long* id) {
  cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
  unsigned long long cid = 0;
  if (cudaStreamGetCaptureInfo(st, &cs, &cid) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  if (cs == cudaStreamCaptureStatusInvalidated) return false;
  *capturing = cs == cudaStreamCaptureStatusActive;
  *id = *capturing ? cid : 0;
  return true;
}

blockffn_status blockffn_create(const blockffn_config* cfg, blockffn_handle* out) {
  if (!cfg || !out) return BLOCKFFN_ERR_INVALID_ARG;
  *out = nullptr;
  if (cfg->d < 8 || cfg->d_e < 8 || cfg->E < 1 || cfg->L_max < 1) return BLOCKFFN_ERR_INVALID_ARG;
  if (cfg->d % 8 || cfg->d_e % 8 || cfg->E > 1024 || cfg->L_max > 32 || cfg->d > (1 << 20) ||
      cfg->d_e > (1 << 16))
    return BLOCKFFN_ERR_UNSUPPORTED;
  if (!(cfg->rms_eps >= 0.0f) && cfg->rms_eps != BLOCKFFN_NO_RMSNORM) return BLOCKFFN_ERR_INVALID_ARG;
  if (cfg->variant < BLOCKFFN_VARIANT_AUTO || cfg->variant > BLOCKFFN_VARIANT_MMA)
    return BLOCKFFN_ERR_INVALID_ARG;
  if (cfg->flags & ~0x7fffffff) return BLOCKFFN_ERR_INVALID_ARG;
  if (((cfg->flags >> 17) & 0x7ff) > cfg->E) return BLOCKFFN_ERR_INVALID_ARG;
  blockffn_ctx* c = new (std::nothrow) blockffn_ctx();
  if (!c) return BLOCKFFN_ERR_WORKSPACE;
  c->cfg = *cfg;
  c->words = (cfg->E + 31) / 32;
  c->launches = 0;
  if (cudaGetDevice(&c->device) != cudaSuccess ||
      cudaDeviceGetAttribute(&c->num_sms, cudaDevAttrMultiProcessorCount, c->device) !=
          cudaSuccess) {
    delete c;
    return BLOCKFFN_ERR_CUDA;
  }
  const size_t E = cfg->E, L = cfg->L_max, d_e = cfg->d_e, W = c->words;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes, 256);
    return o;
  };
  const size_t o_a0 = take(sizeof(float) * L * E);
  size_t o_ring[kLogitRing];
  for (int i = 0; i < kLogitRing; ++i) o_ring[i] = take(sizeof(float) * L * E);
  const size_t o_sc = take(sizeof(float) * L * E);
  const size_t o_tm = take(sizeof(uint32_t) * L * W);
  const size_t o_um = take(sizeof(uint32_t) * W);
  const size_t o_id = take(sizeof(int32_t) * E);
  const size_t o_nu = take(sizeof(int32_t));
  const size_t o_h32 = take(sizeof(float) * E * L * d_e);
  const size_t o_h16 = take(expert_mma_h_bytes(cfg));
  const size_t lean_bytes = expert_lean_ws_bytes(cfg, c->num_sms);
  const size_t o_lean = take(lean_bytes);
  const size_t o_seq = take(sizeof(unsigned long long) * 256);   // four rings, 64 words each
  const size_t o_one = take(sizeof(float) * E);
  const size_t o_tk = take(sizeof(unsigned int) * 8);
  const size_t o_st = take(sizeof(uint32_t));
  void* base = nullptr;
  if (cudaMalloc(&base, off) != cudaSuccess) {
    cudaGetLastError();
    delete c;
    return BLOCKFFN_ERR_WORKSPACE;
  }
  if (cudaMemset(base, 0, off) != cudaSuccess) {
    cudaFree(base);
    delete c;
    return BLOCKFFN_ERR_CUDA;
  }
  char* b = static_cast<char*>(base);
  c->ws_base = base;
  c->a0 = reinterpret_cast<float*>(b + o_a0);
  for (int i = 0; i < kLogitRing; ++i) c->a0_ring[i] = reinterpret_cast<float*>(b + o_ring[i]);
  c->a0_phase = 0;
  c->scores = reinterpret_cast<float*>(b + o_sc);
  c->tok_mask = reinterpret_cast<uint32_t*>(b + o_tm);
  c->union_mask = reinterpret_cast<uint32_t*>(b + o_um);
  c->union_ids = reinterpret_cast<int32_t*>(b + o_id);
  c->n_union = reinterpret_cast<int32_t*>(b + o_nu);
  c->h32 = reinterpret_cast<float*>(b + o_h32);
  c->h16 = b + o_h16;
  c->lean_ring = lean_bytes ? b + o_lean : nullptr;
  c->lean_seq = reinterpret_cast<unsigned long long*>(b + o_seq);
  c->ones = reinterpret_cast<float*>(b + o_one);
  c->ticket = reinterpret_cast<unsigned int*>(b + o_tk);
  c->status = reinterpret_cast<uint32_t*>(b + o_st);
  {
    const std::vector<float> ones(E, 1.0f);
    if (cudaMemcpy(c->ones, ones.data(), sizeof(float) * E, cudaMemcpyHostToDevice) != cudaSuccess) {
      cudaFree(base);
      delete c;
      return BLOCKFFN_ERR_CUDA;
    }
  }
  if (expert_mma_setup(c) != cudaSuccess || expert_lean_setup(c) != cudaSuccess) {
    cudaFree(base);
    delete c;
    return BLOCKFFN_ERR_CUDA;
  }
  // A caller that names the tensor-core kernels gets them or an error, never a silent switch
  // to the other family (AUTO keeps choosing per call).
  if (cfg->variant == BLOCKFFN_VARIANT_MMA &&
      !(expert_mma_supported(c, 1) && expert_mma_supported(c, cfg->L_max))) {
    cudaFree(base);
    delete c;
    return BLOCKFFN_ERR_UNSUPPORTED;
  }
  // The stream and events the router of blockffn_layer_forward may run on; without them that
  // call keeps its router on the caller's stream.
  c->side = nullptr;
  c->last_layer_waited_first = false;
  for (int i = 0; i < kLogitRing; ++i) {
    c->ev_call[i] = c->ev_router[i] = nullptr;
    c->call_mark[i].set = false;
  }
  bool side_ok = cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) == cudaSuccess;
  for (int i = 0; i < kLogitRing && side_ok; ++i)
    side_ok = cudaEventCreateWithFlags(&c->ev_call[i], cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&c->ev_router[i], cudaEventDisableTiming) == cudaSuccess;
  if (!side_ok) {
    cudaGetLastError();
    release_side(c);
  }
  *out = c;
  return BLOCKFFN_OK;
}

blockffn_status blockffn_destroy(blockffn_handle h) {
  if (!h) return BLOCKFFN_ERR_INVALID_ARG;
  release_side(h);
  cudaError_t e = cudaFree(h->ws_base);
  delete h;
  return e == cudaSuccess ? BLOCKFFN_OK : BLOCKFFN_ERR_CUDA;
}

blockffn_status blockffn_router(blockffn_handle h, const blockffn_weights* w, const void* x,
                                int32_t L, float* scores, uint32_t* tok_mask, void* stream) {
  blockffn_status s = check_call(h, L);
  if (s != BLOCKFFN_OK) return s;
  if (!w || !w->W_r || (!w->gain && !no_rmsnorm(h)) || !x || !scores) return BLOCKFFN_ERR_INVALID_ARG;
  if (misaligned(w->W_r) || misaligned(x) || misaligned(scores) ||
      (reinterpret_cast<uintptr_t>(w->gain) & 3u) || (reinterpret_cast<uintptr_t>(w->bias) & 3u) ||
      (reinterpret_cast<uintptr_t>(tok_mask) & 3u))
    return BLOCKFFN_ERR_INVALID_ARG;
  cudaError_t e =
      launch_router(h, w, x, L, scores, tok_mask, false, nullptr, false, h->a0, 0,
                    static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? BLOCKFFN_OK : BLOCKFFN_ERR_CUDA;
}

blockffn_status blockffn_chunk_union(blockffn_handle h, const float* scores, int32_t L,
                                     uint32_t* union_mask, int32_t* union_ids, int32_t* n_union,
                                     blockffn_stats* stats, void* stream) {
  blockffn_status s = check_call(h, L);
  if (s != BLOCKFFN_OK) return s;
  if (!scores || !union_ids || !n_union) return BLOCKFFN_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(scores) & 3u) || (reinterpret_cast<uintptr_t>(union_mask) & 3u) ||
      (reinterpret_cast<uintptr_t>(union_ids) & 3u) || (reinterpret_cast<uintptr_t>(n_union) & 3u) ||
      (reinterpret_cast<uintptr_t>(stats) & 7u))
    return BLOCKFFN_ERR_INVALID_ARG;
  cudaError_t e = launch_chunk_union(h, scores, L, union_mask, union_ids, n_union, stats,
                                     static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? BLOCKFFN_OK : BLOCKFFN_ERR_CUDA;
}

blockffn_status blockffn_expert_ffn(blockffn_handle h, const blockffn_weights* w, const void* x,
                                    const float* scores, int32_t L, const int32_t* union_ids,
                                    const int32_t* n_union, float* out, void* x_next,
                                    int32_t call_flags, void* stream) {
  blockffn_status s = check_call(h, L);
  if (s != BLOCKFFN_OK) return s;
  if (!w || !w->U || !w->D || !x || !scores || !union_ids || !n_union || !out)
    return BLOCKFFN_ERR_INVALID_ARG;
  if (misaligned(w->U) || misaligned(w->D) || misaligned(x) || misaligned(out) ||
      misaligned(x_next) || (reinterpret_cast<uintptr_t>(scores) & 3u) ||
      (reinterpret_cast<uintptr_t>(union_ids) & 3u) || (reinterpret_cast<uintptr_t>(n_union) & 3u))
    return BLOCKFFN_ERR_INVALID_ARG;
  if (x_next == x) return BLOCKFFN_ERR_INVALID_ARG;
  if (call_flags & ~kCallFlags)
    return BLOCKFFN_ERR_INVALID_ARG;
  return expert_dispatch(h, w, x, scores, L, union_ids, n_union, out, x_next, call_flags,
                         static_cast<cudaStream_t>(stream));
}

blockffn_status blockffn_layer_forward(blockffn_handle h, const blockffn_weights* w, const void* x,
                                       int32_t L, float* out, void* x_next, blockffn_stats* stats,
                                       int32_t call_flags, void* stream) {
  blockffn_status s = check_call(h, L);
  if (s != BLOCKFFN_OK) return s;
  if (!w || !w->W_r || (!w->gain && !no_rmsnorm(h)) || !w->U || !w->D || !x || !out)
    return BLOCKFFN_ERR_INVALID_ARG;
  if (misaligned(w->W_r) || misaligned(w->U) || misaligned(w->D) || misaligned(x) ||
      misaligned(out) || misaligned(x_next) || (reinterpret_cast<uintptr_t>(w->gain) & 3u) ||
      (reinterpret_cast<uintptr_t>(w->bias) & 3u) || (reinterpret_cast<uintptr_t>(stats) & 7u))
    return BLOCKFFN_ERR_INVALID_ARG;
  if (x_next == x) return BLOCKFFN_ERR_INVALID_ARG;
  if (call_flags & ~kCallFlags)
    return BLOCKFFN_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The router writes the scores this very call consumes: the expert kernels are never
  // "independent". The router itself may run ahead when x is stable.
  const int flags = call_flags & ~(BLOCKFFN_CALL_INDEPENDENT | BLOCKFFN_CALL_INDEPENDENT_X);
  if (use_mma(h, L)) {
    // The router kernel leaves the raw logits; the expert kernels (every CTA needs the union
    // before it can fetch a weight byte) apply ReLU, RMSNorm and gain themselves and CTA 0
    // publishes scores, masks, union and counters.
    // Successive calls cycle through kLogitRing logit buffers: a router that runs under earlier
    // calls never writes what their kernels still read.
    const bool x_stable_call = (call_flags & BLOCKFFN_CALL_INDEPENDENT_X) != 0;
    if (expert_lean_supported(h, L, true, x_stable_call, true)) {
      // The shape takes the one-kernel form: the router runs inside that kernel (its CTAs share
      // the experts' logits out between them and exchange them through L2), so the call is one
      // launch. With x stable it overlaps its neighbours like a scores-in call; otherwise it
      // owns the device and waits for the work before it ahead of its first read.
      const RoutingOut pub_in{h->union_mask, h->union_ids, h->n_union, stats, h->scores, h->tok_mask};
      const RouterLogits lg_in{nullptr, router_gain(h, w), h->cfg.rms_eps};
      h->last_layer_waited_first = false;
      return launch_tensor_core(h, w, x, h->scores, L, nullptr, nullptr, out, x_next, flags, &pub_in,
                                &lg_in, x_stable_call, st) == cudaSuccess
                 ? BLOCKFFN_OK
                 : BLOCKFFN_ERR_CUDA;
    }
    const int b = h->a0_phase;
    const int oldest = (b + 1) % kLogitRing;   // the call kLogitRing - 1 calls back
    h->a0_phase = oldest;
    float* logits = h->a0_ring[b];
    const bool x_stable = (call_flags & BLOCKFFN_CALL_INDEPENDENT_X) != 0;
    const bool chained = !(h->cfg.flags & BLOCKFFN_CFG_NO_CHAINING);
    const RoutingOut pub{h->union_mask, h->union_ids, h->n_union, stats, h->scores, h->tok_mask};
    const RouterLogits lg{logits, router_gain(h, w), h->cfg.rms_eps};
    // With x stable the router needs nothing from the caller's stream except that the readers
    // of its logit buffer (the layer call kLogitRing calls back) are done. It then runs on the
    // handle's own stream behind the mark that the call kLogitRing - 1 calls back left at its
    // start, and the expert kernels, which start behind the finished router, fetch their
    // weights under the previous call like a scores-in call does. The mark must come from the
    // same stream and the same capture (or both from none); otherwise the router stays on the
    // caller's stream.
    bool capturing = false;
    unsigned long long cap_id = 0;
    const bool marks = x_stable && chained && h->side && capture_state(st, &capturing, &cap_id);
    cudaStream_t side = h->side;
    const auto& prev = h->call_mark[oldest];
    const bool aside = marks && prev.set && prev.stream == st && prev.capturing == capturing &&
                       prev.id == cap_id;
    h->call_mark[b].set = false;
    if (marks && cudaEventRecord(h->ev_call[b], st) == cudaSuccess) {
      h->call_mark[b].set = true;
      h->call_mark[b].stream = st;
      h->call_mark[b].capturing = capturing;
      h->call_mark[b].id = cap_id;
    }
    if (aside) {
      if (cudaStreamWaitEvent(side, h->ev_call[oldest], 0) != cudaSuccess ||
          launch_router(h, w, x, L, h->scores, h->tok_mask, false, nullptr, true, logits, 2,
                        side) != cudaSuccess ||
          cudaEventRecord(h->ev_router[b], side) != cudaSuccess ||
          cudaStreamWaitEvent(st, h->ev_router[b], 0) != cudaSuccess)
        return BLOCKFFN_ERR_CUDA;
      h->last_layer_waited_first = false;
      return launch_tensor_core(h, w, x, h->scores, L, nullptr, nullptr, out, x_next, flags, &pub,
                                &lg, true, st) == cudaSuccess
                 ? BLOCKFFN_OK
                 : BLOCKFFN_ERR_CUDA;
    }
    // Router on the caller's stream. It may still compute under the previous call when x is
    // stable, as long as that call's up kernel waited first: what read this logit buffer then
    // finished before anything behind that kernel could start (the router before it waited
    // before it ended, and so does every kernel).
    const bool ahead = x_stable && h->last_layer_waited_first;
    h->last_layer_waited_first = true;
    if (launch_router(h, w, x, L, h->scores, h->tok_mask, false, nullptr, true, logits,
                      ahead ? 1 : 0, st) != cudaSuccess)
      return BLOCKFFN_ERR_CUDA;
    return launch_tensor_core(h, w, x, h->scores, L, nullptr, nullptr, out, x_next, flags, &pub, &lg,
                              false, st) == cudaSuccess
               ? BLOCKFFN_OK
               : BLOCKFFN_ERR_CUDA;
  }
  h->last_layer_waited_first = false;
  if (launch_router(h, w, x, L, h->scores, h->tok_mask, true, stats, false, h->a0, 0, st) != cudaSuccess)
    return BLOCKFFN_ERR_CUDA;
  return expert_dispatch(h, w, x, h->scores, L, h->union_ids, h->n_union, out, x_next, flags, st);
}

blockffn_status blockffn_layer_forward_scores(blockffn_handle h, const blockffn_weights* w,
                                              const void* x, const float* scores, int32_t L,
                                              float* out, void* x_next, blockffn_stats* stats,
                                              int32_t call_flags, void* stream) {
  blockffn_status s = check_call(h, L);
  if (s != BLOCKFFN_OK) return s;
  if (!w || !w->U || !w->D || !x || !scores || !out) return BLOCKFFN_ERR_INVALID_ARG;
  if (misaligned(w->U) || misaligned(w->D) || misaligned(x) || misaligned(out) ||
      misaligned(x_next) || misaligned(scores) || (reinterpret_cast<uintptr_t>(stats) & 7u))
    return BLOCKFFN_ERR_INVALID_ARG;
  if (x_next == x) return BLOCKFFN_ERR_INVALID_ARG;
  if (call_flags & ~kCallFlags)
    return BLOCKFFN_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (use_mma(h, L)) {
    // The expert kernels derive Union(x) from the scores themselves (every CTA needs the
    // list before it can fetch a weight byte) and CTA 0 publishes it: no separate launch.
    const RoutingOut pub{h->union_mask, h->union_ids, h->n_union, stats, nullptr, nullptr};
    return launch_tensor_core(h, w, x, scores, L, nullptr, nullptr, out, x_next, call_flags, &pub,
                              nullptr, false, st) == cudaSuccess
               ? BLOCKFFN_OK
               : BLOCKFFN_ERR_CUDA;
  }
  if (launch_chunk_union(h, scores, L, h->union_mask, h->union_ids, h->n_union, stats, st) !=
      cudaSuccess)
    return BLOCKFFN_ERR_CUDA;
  // The union list is produced inside this call: the expert stage must wait for it.
  const int flags = call_flags & ~(BLOCKFFN_CALL_INDEPENDENT | BLOCKFFN_CALL_INDEPENDENT_X);
  return expert_dispatch(h, w, x, scores, L, h->union_ids, h->n_union, out, x_next, flags, st);
}

blockffn_status blockffn_read_routing(blockffn_handle h, int32_t L, float* scores,
                                      uint32_t* tok_mask, uint32_t* union_mask,
                                      int32_t* union_ids, int32_t* n_union, void* stream) {
  blockffn_status s = check_call(h, L);
  if (s != BLOCKFFN_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t E = h->cfg.E, W = h->words;
  cudaError_t e = cudaSuccess;
  auto copy = [&](void* dst, const void* src, size_t n) {
    if (dst && e == cudaSuccess) e = cudaMemcpyAsync(dst, src, n, cudaMemcpyDeviceToDevice, st);
  };
  copy(scores, h->scores, sizeof(float) * L * E);
  copy(tok_mask, h->tok_mask, sizeof(uint32_t) * L * W);
  copy(union_mask, h->union_mask, sizeof(uint32_t) * W);
  copy(union_ids, h->union_ids, sizeof(int32_t) * E);
  copy(n_union, h->n_union, sizeof(int32_t));
  return e == cudaSuccess ? BLOCKFFN_OK : BLOCKFFN_ERR_CUDA;
}

blockffn_status blockffn_reuse_ratio(blockffn_handle h, const float* scores, int32_t L,
                                     double* reuse, void* stream) {
  if (!h || !reuse || L < 1) return BLOCKFFN_ERR_INVALID_ARG;
  if (!scores && L > h->cfg.L_max) return BLOCKFFN_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(scores) & 3u) || (reinterpret_cast<uintptr_t>(reuse) & 7u))
    return BLOCKFFN_ERR_INVALID_ARG;
  const cudaError_t e = launch_reuse_ratio(h, scores ? scores : h->scores, L, reuse,
                                           static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? BLOCKFFN_OK : BLOCKFFN_ERR_CUDA;
}

blockffn_status blockffn_last_status(blockffn_handle h, uint32_t* bits, int32_t clear,
                                     void* stream) {
  if (!h) return BLOCKFFN_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t v = 0;
  if (cudaMemcpyAsync(&v, h->status, sizeof v, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess)
    return BLOCKFFN_ERR_CUDA;
  if (clear && v) {
    if (cudaMemsetAsync(h->status, 0, sizeof v, st) != cudaSuccess) return BLOCKFFN_ERR_CUDA;
  }
  if (bits) *bits = v;
  return v ? BLOCKFFN_ERR_DEVICE : BLOCKFFN_OK;
}

double blockffn_tls(const blockffn_stats* s, int32_t E) {
  if (!s || E < 1 || s->n_tokens == 0) return 0.0;
  return 1.0 - (double)s->n_active / ((double)s->n_tokens * (double)E);
}

double blockffn_cls(const blockffn_stats* s, int32_t E) {
  if (!s || E < 1 || s->n_chunks == 0) return 0.0;
  return 1.0 - (double)s->n_union / ((double)s->n_chunks * (double)E);
}

uint64_t blockffn_launch_count(blockffn_handle h) { return h ? h->launches : 0; }

const char* blockffn_status_string(blockffn_status s) {
  switch (s) {
    case BLOCKFFN_OK: return "ok";
    case BLOCKFFN_ERR_INVALID_ARG: return "invalid argument";
    case BLOCKFFN_ERR_UNSUPPORTED: return "unsupported shape";
    case BLOCKFFN_ERR_WORKSPACE: return "workspace allocation failed";
    case BLOCKFFN_ERR_CUDA: return "CUDA error";
    case BLOCKFFN_ERR_DEVICE: return "device status word set";
  }
  return "unknown";
}

}  // extern "C"
