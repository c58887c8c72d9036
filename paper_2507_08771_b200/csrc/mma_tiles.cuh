// Building blocks shared by the tensor-core kernels of the expert stage (Eq. 1, Eq. 2 over
// Union(x), Sec. 3.3): shared-memory layouts, asynchronous-copy and mma wrappers, the 64-wide
// operand fragments, and the derivation of Union(x) inside a CTA.
#pragma once

#include "common.cuh"

namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kMaxStages = 32;                   // slots of the down kernel's ring
constexpr int kUpStages = 3;                     // slots of the up kernel's ring
constexpr int kSmemMax = 232448;                 // 227 KB per CTA
constexpr int kSmemHalf = 113 * 1024;            // lets an up and a down CTA share one SM
// (registers too: for L <= 16 the kernels are compiled for two CTAs per SM, 128 per thread)

// ---- shared-memory layout ----------------------------------------------------
__host__ __device__ inline int align128(int v) { return (v + 127) & ~127; }

constexpr int kCtlBytes = 640;  // ints: [0] nu, [2] n_active, [3] bad bits; [8..40) union mask
                                // words; [40..72), [72..104) scratch; [104..136) 1/rms per token
constexpr int kOffCtl = 0;
constexpr int kOffIds = kOffCtl + kCtlBytes;

struct UpLayout {
  int off_red, off_x, off_ring, total;
};
// red: per warp a 32 x 8 tile; x: one tile of 8 tokens (2d bytes each); ring: ring_rows rows
__host__ __device__ inline UpLayout up_layout(int d, int E, int ring_rows) {
  UpLayout s;
  s.off_red = kOffIds + align128(E * 4);
  s.off_x = s.off_red + kWarps * 32 * 8 * 4;
  s.off_ring = s.off_x + align128(8 * 2 * d);
  s.total = s.off_ring + ring_rows * 2 * d;
  return s;
}

struct DownLayout {
  int off_red, off_h, off_d, slot_h, slot_d, total;
};
// h ring: ns slots of 8 token rows of 2 d_e bytes; D ring: ns slots of max_cols rows of 2 d_e bytes
__host__ __device__ inline DownLayout down_layout(int d_e, int E, int ns, int max_cols) {
  DownLayout s;
  s.off_red = kOffIds + align128(E * 4);
  s.off_h = s.off_red + kWarps * 16 * 8 * 4;
  s.slot_h = 8 * 2 * d_e;
  s.slot_d = max_cols * 2 * d_e;
  s.off_d = s.off_h + align128(ns * s.slot_h);
  s.total = s.off_d + ns * s.slot_d;
  return s;
}

// ---- PTX wrappers --------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
// 16-byte asynchronous copy global -> shared, cached in L2 only.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() {
  asm volatile("cp.async.commit_group;" ::: "memory");
}
// Waits until at most N of this thread's most recent commit groups are still in flight.
template <int N>
__device__ __forceinline__ void cp_async_wait_group() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.wait_all;" ::: "memory");
}
// Contiguous run of bytes (a multiple of 16), spread over the CTA's threads. Runs should be
// long: consecutive cp.async of one thread only overlap when the loop is unrolled (distinct
// address registers), so many short runs issue several times slower than one long one.
__device__ __forceinline__ void copy_run(uint32_t dst, const void* src, int bytes) {
  const char* s = static_cast<const char*>(src);
#pragma unroll 4
  for (int o = threadIdx.x * 16; o < bytes; o += kThreads * 16) cp_async16(dst + o, s + o);
}
// n_pieces pieces of piece_bytes each (a multiple of 16), piece i from src(i) to
// dst0 + i * dst_stride. The loop over the pieces is the unrolled one (a loop nested inside
// it would stop the unrolling and with it the overlap of the copies).
template <class SrcOf>
__device__ __forceinline__ void copy_pieces(uint32_t dst0, int dst_stride, int n_pieces,
                                            int piece_bytes, SrcOf src) {
  for (int o = threadIdx.x * 16; o < piece_bytes; o += kThreads * 16) {
#pragma unroll 4
    for (int i = 0; i < n_pieces; ++i) cp_async16(dst0 + i * dst_stride + o, src(i) + o);
  }
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
// D(16x8, f32) += A(16x16, bf16, row) * B(16x8, bf16, col). Not volatile: the compiler is
// free to interleave independent mma chains and the shared-memory loads that feed them.
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                         uint32_t a3, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
      "{%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float swish_fast(float z) { return __fdividef(z, 1.0f + __expf(-z)); }

// ---- Union(x) inside the CTA -----------------------------------------------------
// Fills ids_sm[0 .. nu) with the ascending valid expert ids and returns nu. All global
// loads of one call are independent of each other, so the routine costs one memory latency.
// ids_in == NULL: derived from the nonzero pattern of scores (Sec. 3.3); ctl[2] then holds
// the number of active (token, expert) pairs and ctl[8 ..] the union mask words.
// ids_in != NULL: taken from the caller's list (E entries are readable); entries out of
// range are dropped and reported, a count out of range is clamped and reported.
// tm: scratch of at least 32 * ceil(E/32) words of shared memory (word-major, 32 tokens per word).
// MODE: 0 from scores, 1 from the caller's list, 2 from raw router logits
// hook: called by thread 0 once, after its first routing loads have been issued and before it
// needs them (a place for work whose own latency should run under that of the loads).
struct NoHook {
  __device__ __forceinline__ void operator()() const {}
};
template <int MODE, class Hook = NoHook>
__device__ int derive_union(const float* scores, const RouterLogits& lg, const int32_t* ids_in,
                            const int32_t* n_in, int L, int E, int* ids_sm, int* ctl,
                            uint32_t* tm, Hook hook = Hook()) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nwarps = blockDim.x >> 5;
  const int words = (E + 31) >> 5;
  int* cnt = ctl + 40;
  int* act = ctl + 72;
  uint32_t* um = reinterpret_cast<uint32_t*>(ctl + 8);
  float* rinv = reinterpret_cast<float*>(ctl + 104);
  if constexpr (MODE == 2) {
    // Raw router logits: finish Eq. 3 here (ReLU, RMSNorm over all E entries, gain), with the
    // arithmetic of the router kernel's own normalisation, and take the nonzero pattern.
    // (up to 128 experts a lane keeps its logits and gains in registers: one round trip)
    const bool few = words <= 4;
    for (int t = warp; t < L; t += nwarps) {
      float ss = 0.0f, v4[4], g4[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int e = 32 * u + lane;
        const bool in = few && e < E;
        v4[u] = in ? __ldcg(lg.a0 + (size_t)t * E + e) : 0.0f;
        g4[u] = in ? __ldg(lg.gain + e) : 0.0f;
      }
      if (threadIdx.x == 0) hook();
      if (few) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          v4[u] = v4[u] > 0.0f ? v4[u] : 0.0f;
          ss = fmaf(v4[u], v4[u], ss);
        }
      } else {
        for (int e = lane; e < E; e += 32) {
          float v = __ldcg(lg.a0 + (size_t)t * E + e);
          v = v > 0.0f ? v : 0.0f;
          ss = fmaf(v, v, ss);
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
      // a negative eps marks the router without RMSNorm (Sec. 4.2.3; lg.gain is then all ones)
      const float r = lg.eps < 0.0f ? 1.0f : 1.0f / sqrtf(ss / (float)E + lg.eps);
      if (lane == 0) rinv[t] = r;
      if (few) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const uint32_t m = __ballot_sync(0xffffffffu, g4[u] * v4[u] * r != 0.0f);
          if (lane == 0 && u < words) tm[u * 32 + t] = m;
        }
      } else {
        for (int w = 0; w < words; ++w) {
          const int e = 32 * w + lane;
          float s = 0.0f;
          if (e < E) {
            float v = __ldcg(lg.a0 + (size_t)t * E + e);
            v = v > 0.0f ? v : 0.0f;
            s = __ldg(lg.gain + e) * v * r;
          }
          const uint32_t m = __ballot_sync(0xffffffffu, s != 0.0f);
          if (lane == 0) tm[w * 32 + t] = m;
        }
      }
    }
  } else if constexpr (MODE == 0) {
    // warp -> tokens warp, warp + nwarps, ...; four mask words in flight per step
    for (int t = warp; t < L; t += nwarps) {
      for (int w0 = 0; w0 < words; w0 += 4) {
        float v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int e = 32 * (w0 + u) + lane;
          v[u] = e < E ? __ldcg(scores + (size_t)t * E + e) : 0.0f;
        }
        if (threadIdx.x == 0 && w0 == 0) hook();
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const uint32_t m = __ballot_sync(0xffffffffu, v[u] != 0.0f);
          if (lane == 0 && w0 + u < words) tm[(w0 + u) * 32 + t] = m;
        }
      }
    }
  }
  if constexpr (MODE != 1) {
    __syncthreads();
    if (words <= 4) {
      // Up to 128 experts every warp folds the token masks itself (lane t holds token t's
      // mask of a word; one warp-wide OR per word), so offsets and the union size need no
      // second exchange through shared memory.
      uint32_t un[4];
      int nact = 0;
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const uint32_t m = (w < words && lane < L) ? tm[w * 32 + lane] : 0u;
        un[w] = __reduce_or_sync(0xffffffffu, m);
        nact += __popc(m);
      }
      int off = 0, total = 0;
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        if (w < warp) off += __popc(un[w]);
        total += __popc(un[w]);
      }
      if (warp < words) {
        uint32_t mine = un[0];
#pragma unroll
        for (int w = 1; w < 4; ++w) mine = warp == w ? un[w] : mine;
        if ((mine >> lane) & 1u) ids_sm[off + __popc(mine & ((1u << lane) - 1u))] = 32 * warp + lane;
      }
      if (warp == 4) {    // a warp without a word of its own leaves the summary
        nact = __reduce_add_sync(0xffffffffu, nact);
        if (lane < 4) um[lane] = lane == 0 ? un[0] : lane == 1 ? un[1] : lane == 2 ? un[2] : un[3];
        if (lane == 0) {
          ctl[0] = total;
          ctl[2] = nact;
        }
      }
      __syncthreads();
      return total;
    }
    if (threadIdx.x < words) {
      uint32_t un = 0;
      int nact = 0;
      for (int t = 0; t < L; ++t) {
        const uint32_t m = tm[threadIdx.x * 32 + t];
        un |= m;
        nact += __popc(m);
      }
      cnt[threadIdx.x] = __popc(un);
      act[threadIdx.x] = nact;
      um[threadIdx.x] = un;
    }
    __syncthreads();
    for (int w = warp; w < words; w += nwarps) {
      int off = 0;
      for (int v = 0; v < w; ++v) off += cnt[v];
      const uint32_t un = um[w];
      if ((un >> lane) & 1u) ids_sm[off + __popc(un & ((1u << lane) - 1u))] = 32 * w + lane;
    }
    if (threadIdx.x == 0) {
      int total = 0, total_act = 0;
      for (int w = 0; w < words; ++w) {
        total += cnt[w];
        total_act += act[w];
      }
      ctl[0] = total;
      ctl[2] = total_act;
    }
  } else {
    int n = __ldcg(n_in);
    {
      const int q0 = threadIdx.x;
      const int id0 = q0 < E ? __ldcg(ids_in + q0) : 0;
      if (threadIdx.x == 0) hook();
      if (q0 < E) ids_sm[q0] = id0;
      for (int q = q0 + blockDim.x; q < E; q += blockDim.x) ids_sm[q] = __ldcg(ids_in + q);
    }
    int bad = 0;
    if (n < 0 || n > E) {
      bad = BLOCKFFN_DEV_BAD_UNION_COUNT;
      n = n < 0 ? 0 : E;
    }
    __syncthreads();
    if (warp == 0) {   // in-place ordered compaction of the valid entries
      int k = 0;
      for (int base = 0; base < n; base += 32) {
        const int q = base + lane;
        const int id = q < n ? ids_sm[q] : 0;
        const bool in = q < n, ok = in && id >= 0 && id < E;
        const uint32_t m = __ballot_sync(0xffffffffu, ok);
        if (__ballot_sync(0xffffffffu, in && !ok)) bad |= BLOCKFFN_DEV_BAD_UNION_ID;
        if (ok) ids_sm[k + __popc(m & ((1u << lane) - 1u))] = id;
        k += __popc(m);
      }
      if (lane == 0) {
        ctl[0] = k;
        ctl[3] = bad;
      }
    }
  }
  __syncthreads();
  return ctl[0];
}

// One 64-wide k block of a 16-row operand tile: rows row_a / row_b (byte addresses of the
// block within the row), this lane's 16 bytes of each 32-wide half. Lanes of odd rows
// read the halves in the opposite order (bank spread) and swap them back.
struct Frag64 {
  uint4 lo, hi;   // first / second 32-wide half
};
// row: shared-memory address of the 64-wide block inside the operand row (128-byte aligned)
__device__ __forceinline__ Frag64 load_frag64(const unsigned char* row, int par, int tg) {
  const uint4 first = *reinterpret_cast<const uint4*>(row + 64 * par + 16 * tg);
  const uint4 second = *reinterpret_cast<const uint4*>(row + 64 * (par ^ 1) + 16 * tg);
  Frag64 f;
  f.lo = par ? second : first;
  f.hi = par ? first : second;
  return f;
}
// acc0 takes the first 32-wide half, acc1 the second: two independent dependency chains.
template <int NT>
__device__ __forceinline__ void mma_block64(float (&acc0)[NT][4], float (&acc1)[NT][4],
                                            const Frag64& ra, const Frag64& rb,
                                            const Frag64 (&xb)[NT]) {
#pragma unroll
  for (int n = 0; n < NT; ++n) {
    mma_bf16(acc0[n], ra.lo.x, rb.lo.x, ra.lo.y, rb.lo.y, xb[n].lo.x, xb[n].lo.y);
    mma_bf16(acc1[n], ra.hi.x, rb.hi.x, ra.hi.y, rb.hi.y, xb[n].hi.x, xb[n].hi.y);
    mma_bf16(acc0[n], ra.lo.z, rb.lo.z, ra.lo.w, rb.lo.w, xb[n].lo.z, xb[n].lo.w);
    mma_bf16(acc1[n], ra.hi.z, rb.hi.z, ra.hi.w, rb.hi.w, xb[n].hi.z, xb[n].hi.w);
  }
}
// The 16 x (8 NT) accumulator tile of one warp (both chains summed) -> mine[t * ld + m0 + .]
template <int NT>
__device__ __forceinline__ void store_partial(float* mine, int ld, int m0, const float (&a0)[NT][4],
                                              const float (&a1)[NT][4], int g, int tg) {
#pragma unroll
  for (int n = 0; n < NT; ++n) {
    const int t = 8 * n + 2 * tg;
    mine[t * ld + m0 + g] = a0[n][0] + a1[n][0];
    mine[(t + 1) * ld + m0 + g] = a0[n][1] + a1[n][1];
    mine[t * ld + m0 + g + 8] = a0[n][2] + a1[n][2];
    mine[(t + 1) * ld + m0 + g + 8] = a0[n][3] + a1[n][3];
  }
}
template <int NT>
__device__ __forceinline__ void zero_acc(float (&a)[NT][4]) {
#pragma unroll
  for (int n = 0; n < NT; ++n)
#pragma unroll
    for (int v = 0; v < 4; ++v) a[n][v] = 0.0f;
}

}  // namespace
