// Router (Eq. 3) and chunk union (Sec. 3.3) kernels.
//
// router_kernel: one block per expert computes that expert's logit for every
// token of the chunk (x . W_r[i] + bias[i]) with 128-bit loads and fp32 FMAs; the
// block that finishes last (a ticket counter, no waiting) applies ReLU and RMSNorm
// with the per-expert gain, writes the scores and the per-token nonzero masks
// (warp ballot), and, for the fused layer call, derives the chunk union right away.
//
// union_kernel: one block ORs the per-token nonzero patterns of a score matrix,
// compacts the union's expert ids in ascending order with a warp prefix count, and
// advances the TLS / CLS counters (Sec. 2.1).
#include "common.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxWords = 32;  // E <= 1024

// All 256 threads of the block take part. sm: >= 3 * kMaxWords ints.
__device__ void chunk_union_block(const float* scores, int L, int E, uint32_t* union_mask,
                                  int32_t* union_ids, int32_t* n_union, blockffn_stats* stats,
                                  int* sm) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int words = (E + 31) >> 5;
  int* cnt = sm;                                   // popcount of each union word
  int* act = sm + kMaxWords;                       // active (token, expert) pairs per word
  uint32_t* um = reinterpret_cast<uint32_t*>(sm + 2 * kMaxWords);
  for (int w = warp; w < words; w += kWarps) {
    const int e = 32 * w + lane;
    uint32_t un = 0;
    int nact = 0;
    for (int t = 0; t < L; ++t) {
      float v = (e < E) ? scores[(size_t)t * E + e] : 0.0f;
      uint32_t m = __ballot_sync(0xffffffffu, v != 0.0f);
      un |= m;
      nact += __popc(m);
    }
    if (lane == 0) {
      cnt[w] = __popc(un);
      act[w] = nact;
      um[w] = un;
      if (union_mask) union_mask[w] = un;
    }
  }
  __syncthreads();
  int total = 0, total_act = 0;
  for (int w = 0; w < words; ++w) {
    total += cnt[w];
    total_act += act[w];
  }
  for (int w = warp; w < words; w += kWarps) {
    int off = 0;
    for (int v = 0; v < w; ++v) off += cnt[v];
    const uint32_t un = um[w];
    if ((un >> lane) & 1u) union_ids[off + __popc(un & ((1u << lane) - 1u))] = 32 * w + lane;
  }
  for (int idx = total + threadIdx.x; idx < E; idx += kThreads) union_ids[idx] = -1;
  if (threadIdx.x == 0) {
    *n_union = total;
    if (stats) {
      atomicAdd(reinterpret_cast<unsigned long long*>(&stats->n_tokens), (unsigned long long)L);
      atomicAdd(reinterpret_cast<unsigned long long*>(&stats->n_active),
                (unsigned long long)total_act);
      atomicAdd(reinterpret_cast<unsigned long long*>(&stats->n_chunks), 1ull);
      atomicAdd(reinterpret_cast<unsigned long long*>(&stats->n_union), (unsigned long long)total);
    }
  }
}

__global__ void __launch_bounds__(kThreads)
union_kernel(const float* __restrict__ scores, int L, int E, uint32_t* union_mask,
             int32_t* union_ids, int32_t* n_union, blockffn_stats* stats) {
  __shared__ int sm[3 * kMaxWords];
  chunk_union_block(scores, L, E, union_mask, union_ids, n_union, stats, sm);
}

__global__ void __launch_bounds__(kThreads)
router_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ W_r,
              const float* __restrict__ gain, const float* __restrict__ bias, float* a0,
              float* scores, uint32_t* tok_mask, int L, int d, int E, float eps,
              unsigned int* ticket, int fuse_union, uint32_t* union_mask, int32_t* union_ids,
              int32_t* n_union, blockffn_stats* stats, int raw, int mode) {
  __shared__ float red[kWarps][8];
  __shared__ int sm[3 * kMaxWords];
  __shared__ int is_last;
  const int i = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int chunks = d >> 3;
  const uint4* wrow = reinterpret_cast<const uint4*>(W_r + (size_t)i * d);
  const float b = bias ? bias[i] : 0.0f;
  // The kernel may have been started while the work before it on the stream still runs
  // (programmatic dependent launch): the router weights are stable and are requested now,
  // x and everything this kernel writes are touched only after the wait.
  // mode 2 (raw, launched on a stream of its own): dependents are let go only by the exit of
  // the blocks, behind a fence, because they read the logits without waiting (see the end).
  if (mode != 2) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  uint4 w_first = make_uint4(0u, 0u, 0u, 0u);
  if ((int)threadIdx.x < chunks) w_first = __ldg(wrow + threadIdx.x);
  {  // x may still change until the wait is over, but asking L2 for its lines now is harmless
    // (L2 is where writes land too); the blocks share the lines out between them
    const int lines = (L * d * 2 + 127) >> 7;
    for (int ln = i + (int)gridDim.x * (int)threadIdx.x; ln < lines; ln += gridDim.x * kThreads)
      asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(x) + (size_t)ln * 128));
  }
  // mode 1 (raw only): x does not come from the work before and a0 is a buffer that work
  // does not read, so the logits are computed under it; the wait moves to the end.
  if (mode == 0) asm volatile("griddepcontrol.wait;" ::: "memory");

  for (int t0 = 0; t0 < L; t0 += 8) {
    float acc[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) acc[t] = 0.0f;
    for (int c = threadIdx.x; c < chunks; c += kThreads) {
      const uint4 wv = c == (int)threadIdx.x ? w_first : __ldg(wrow + c);
      const uint32_t wp[4] = {wv.x, wv.y, wv.z, wv.w};
      // all eight token vectors are requested before the first is used: one memory latency
      uint4 xv[8];
#pragma unroll
      for (int t = 0; t < 8; ++t)
        xv[t] = t0 + t < L ? __ldcg(reinterpret_cast<const uint4*>(x + (size_t)(t0 + t) * d) + c)
                           : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        const uint32_t xp[4] = {xv[t].x, xv[t].y, xv[t].z, xv[t].w};
#pragma unroll
        for (int p = 0; p < 4; ++p) {
          acc[t] = fmaf(bf16_lo(wp[p]), bf16_lo(xp[p]), acc[t]);
          acc[t] = fmaf(bf16_hi(wp[p]), bf16_hi(xp[p]), acc[t]);
        }
      }
    }
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      float v = acc[t];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0) red[warp][t] = v;
    }
    __syncthreads();
    if (threadIdx.x < 8 && t0 + threadIdx.x < L) {
      float v = b;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) v += red[w][threadIdx.x];
      a0[(size_t)(t0 + threadIdx.x) * E + i] = v;
    }
    __syncthreads();
  }

  // raw: the logits are all the caller wants (the tensor-core expert kernels normalise them
  // themselves, which saves this kernel's serial tail)
  if (raw) {
    // every kernel of a chain waits before it ends: completion of one implies all before it
    if (mode == 1) asm volatile("griddepcontrol.wait;" ::: "memory");
    // mode 2: a kernel launched with the programmatic attribute treats every kernel it depends
    // on as a programmatic prerequisite, event edges from other streams included, so the expert
    // kernels may start as soon as this grid's blocks have exited. The fence makes each block's
    // logits visible device-wide before that exit.
    if (mode == 2) __threadfence();
    return;
  }
  // last block done: normalise. The ticket is reset for the next call.
  __threadfence();
  if (threadIdx.x == 0) {
    unsigned int tk = atomicAdd(ticket, 1u);
    is_last = (tk == gridDim.x - 1);
    if (is_last) *ticket = 0u;
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();

  const int words = (E + 31) >> 5;
  for (int t = warp; t < L; t += kWarps) {
    float ss = 0.0f;
    for (int e = lane; e < E; e += 32) {
      float v = __ldcg(a0 + (size_t)t * E + e);
      v = v > 0.0f ? v : 0.0f;
      ss = fmaf(v, v, ss);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    // eps < 0 marks the router without RMSNorm (Sec. 4.2.3): the ReLU values are the scores
    // (the host passes a gain of ones)
    const float r = eps < 0.0f ? 1.0f : 1.0f / sqrtf(ss / (float)E + eps);
    for (int w = 0; w < words; ++w) {
      const int e = 32 * w + lane;
      float s = 0.0f;
      if (e < E) {
        float v = __ldcg(a0 + (size_t)t * E + e);
        v = v > 0.0f ? v : 0.0f;
        s = gain[e] * v * r;
        scores[(size_t)t * E + e] = s;
      }
      const uint32_t m = __ballot_sync(0xffffffffu, s != 0.0f);
      if (tok_mask && lane == 0) tok_mask[(size_t)t * words + w] = m;
    }
  }
  if (fuse_union) {
    __syncthreads();
    chunk_union_block(scores, L, E, union_mask, union_ids, n_union, stats, sm);
  }
}

}  // namespace

cudaError_t launch_router(blockffn_ctx* c, const blockffn_weights* w, const void* x, int L,
                          float* scores, uint32_t* tok_mask, bool fuse_union,
                          blockffn_stats* stats, bool raw, float* logits, int mode,
                          cudaStream_t st) {
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t lc{};
  lc.gridDim = dim3(c->cfg.E);
  lc.blockDim = dim3(kThreads);
  lc.stream = st;
  lc.attrs = attr;
  lc.numAttrs = (mode == 2 || (c->cfg.flags & BLOCKFFN_CFG_NO_CHAINING)) ? 0 : 1;
  const cudaError_t e = cudaLaunchKernelEx(
      &lc, router_kernel, static_cast<const uint16_t*>(x), static_cast<const uint16_t*>(w->W_r),
      router_gain(c, w), w->bias, logits, scores, tok_mask, L, c->cfg.d, c->cfg.E, c->cfg.rms_eps,
      c->ticket,
      fuse_union ? 1 : 0, c->union_mask, c->union_ids, c->n_union, stats, raw ? 1 : 0,
      raw ? mode : 0);
  if (e == cudaSuccess) c->launches += 1;
  return e;
}

namespace {

// Reuse ratio (Sec. 4.1.2). One block. Warp w takes the pairs w, w + 8, ... of a round of eight; thread 0 then adds the
// round's ratios to the running sum in token order, so the sum has one summation order.
__global__ void __launch_bounds__(kThreads)
reuse_ratio_kernel(const float* __restrict__ scores, int L, int E, double* reuse) {
  __shared__ int n_first[kWarps], n_both[kWarps];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  double sum = 0.0, pairs = 0.0;
  if (threadIdx.x == 0) {
    sum = reuse[0];
    pairs = reuse[1];
  }
  for (int i0 = 0; i0 + 1 < L; i0 += kWarps) {
    const int i = i0 + warp;
    int a = 0, b = 0;
    if (i + 1 < L) {
      for (int e = lane; e < E; e += 32) {
        const bool now = scores[(size_t)i * E + e] != 0.0f;
        const bool next = scores[(size_t)(i + 1) * E + e] != 0.0f;
        a += now;
        b += now && next;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      a += __shfl_xor_sync(0xffffffffu, a, o);
      b += __shfl_xor_sync(0xffffffffu, b, o);
    }
    if (lane == 0) {
      n_first[warp] = a;
      n_both[warp] = b;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int w = 0; w < kWarps && i0 + w + 1 < L; ++w) {
        if (n_first[w] == 0) continue;
        sum += (double)n_both[w] / (double)n_first[w];
        pairs += 1.0;
      }
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    reuse[0] = sum;
    reuse[1] = pairs;
  }
}

}  // namespace

cudaError_t launch_reuse_ratio(blockffn_ctx* c, const float* scores, int L, double* reuse,
                               cudaStream_t st) {
  reuse_ratio_kernel<<<1, kThreads, 0, st>>>(scores, L, c->cfg.E, reuse);
  c->launches += 1;
  return cudaGetLastError();
}

cudaError_t launch_chunk_union(blockffn_ctx* c, const float* scores, int L, uint32_t* union_mask,
                               int32_t* union_ids, int32_t* n_union, blockffn_stats* stats,
                               cudaStream_t st) {
  union_kernel<<<1, kThreads, 0, st>>>(scores, L, c->cfg.E, union_mask, union_ids, n_union, stats);
  c->launches += 1;
  return cudaGetLastError();
}
