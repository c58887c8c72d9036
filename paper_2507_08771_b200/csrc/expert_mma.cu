// Expert stage (Eq. 1, Eq. 2 restricted to Union(x), Sec. 3.3): bulk-copy staged,
// tensor-core variant.
//
// Two kernels per call, one CTA per SM each, chained by programmatic dependent
// launch so that the weight fetch of a kernel overlaps the tail of the one before:
//
//   expert_up_mma    CTA b owns an equal share of the union's neuron rows (u * d_e
//                    rows of U, d contiguous bf16 each). One producer lane gathers the
//                    rows into a shared-memory ring with 1-D bulk async copies that
//                    complete on mbarriers; eight consumer warps split K, multiply the
//                    16-row tile with all L tokens on mma.sync m16n8k16 (weights are
//                    the M operand, tokens the N operand), reduce across warps, apply
//                    Swish and the token's router score and store the bf16 intermediate
//                    h[q][t][j] to the handle's workspace.
//   expert_down_mma  CTA b owns a block of <= 16 output columns. For every union expert
//                    it bulk-copies the contiguous [columns x d_e] slab of D and the
//                    expert's h chunk, accumulates out[t][c] over all experts on the
//                    tensor cores and writes each output element exactly once
//                    (no atomics; results are run-to-run identical).
//
// The D slabs (and, for calls flagged independent, the U rows) are requested before
// griddepcontrol.wait, i.e. while the previous kernel is still running; everything a
// previous kernel may have produced (x, h, out) is touched only after it.
//
// The k index of each 32-wide block is permuted identically for both mma operands
// (lane tg owns 8 consecutive k), so every fragment is one 128-bit shared-memory load.
// Every wait on an mbarrier is bounded: on expiry the kernel sets
// BLOCKFFN_DEV_WAIT_EXPIRED, keeps its control flow (so all barriers are met), drains
// its own outstanding copies with a bound and returns.
#include "common.cuh"

namespace {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;  // + one producer warp
constexpr int kKC = 512;                         // k columns per up-projection stage
constexpr int kPad = 64;                         // padding bytes per staged row (bank skew)
constexpr int kMaxStages = 32;
constexpr long long kWaitCycles = 2000000000ll;  // about one second
constexpr int kSmemMax = 232448;                 // 227 KB per CTA
constexpr int kSmemHalf = 113 * 1024;            // lets an up and a down CTA share one SM

// ---- shared-memory layout ----------------------------------------------------
__host__ __device__ inline int align128(int v) { return (v + 127) & ~127; }

struct SmemLayout {
  int off_ctl, off_ids, off_red, off_x, off_ring, slot_bytes, slot_h_off, total;
};
// bars: full[kMaxStages], empty[kMaxStages], xbar
constexpr int kOffBars = 0;
constexpr int kBarBytes = 1024;
constexpr int kCtlBytes = 512;  // ints: [0] nu, [1] abort, [2] n_active, [3] bad bits, [5] abort of the
                                // final drain; [8..40) union mask words; [40..72), [72..104) scratch

__host__ __device__ inline SmemLayout up_layout(int d, int E, int NT, int ns) {
  SmemLayout s;
  s.off_ctl = kBarBytes;
  s.off_ids = s.off_ctl + kCtlBytes;
  s.off_red = s.off_ids + align128(E * 4);
  s.off_x = s.off_red + kConsumerWarps * 16 * 8 * NT * 4;
  s.off_ring = s.off_x + align128(8 * NT * (2 * d + kPad));
  s.slot_bytes = 16 * (2 * kKC + kPad);
  s.slot_h_off = 0;
  s.total = s.off_ring + ns * s.slot_bytes;
  return s;
}

__host__ __device__ inline SmemLayout down_layout(int d_e, int E, int NT, int ns) {
  SmemLayout s;
  s.off_ctl = kBarBytes;
  s.off_ids = s.off_ctl + kCtlBytes;
  s.off_red = s.off_ids + align128(E * 4);
  s.off_x = s.off_red + kConsumerWarps * 16 * 8 * NT * 4;
  s.off_ring = s.off_x;
  s.slot_h_off = align128(16 * 2 * d_e);
  s.slot_bytes = s.slot_h_off + align128(8 * NT * (2 * d_e + kPad));
  s.total = s.off_ring + ns * s.slot_bytes;
  return s;
}

// ---- PTX wrappers --------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait. Returns false if it gave up (or another thread already had).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* ctl,
                                          uint32_t* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if (ctl[1]) return false;
    if (clock64() - t0 > kWaitCycles) {
      ctl[1] = 1;
      atomicOr(status, BLOCKFFN_DEV_WAIT_EXPIRED);
      return false;
    }
  }
}
// 1-D bulk async copy global -> shared, completion counted in bytes on an mbarrier.
// dst, src and bytes are multiples of 16.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes,
                                         uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::
          "r"(dst),
      "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void consumer_sync() {
  asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "r"(addr));
  return v;
}
// D(16x8, f32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                         uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
      "{%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// ---- Union(x) inside the CTA -----------------------------------------------------
// Fills ids_sm[0 .. nu) with the ascending valid expert ids and returns nu.
// ids_in == NULL: derived from the nonzero pattern of scores (Sec. 3.3); ctl[2] then holds
// the number of active (token, expert) pairs and ctl[8 ..] the union mask words.
// ids_in != NULL: taken from the caller's list; entries out of range are dropped and
// reported, a count out of range is clamped and reported.
__device__ int derive_union(const float* scores, const int32_t* ids_in, const int32_t* n_in,
                            int L, int E, int* ids_sm, int* ctl, uint32_t* status) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nwarps = blockDim.x >> 5;
  const int words = (E + 31) >> 5;
  int* cnt = ctl + 40;
  int* act = ctl + 72;
  if (ids_in == nullptr) {
    uint32_t* um = reinterpret_cast<uint32_t*>(ctl + 8);
    for (int w = warp; w < words; w += nwarps) {
      const int e = 32 * w + lane;
      uint32_t un = 0;
      int nact = 0;
      for (int t = 0; t < L; ++t) {
        const float v = (e < E) ? __ldcg(scores + (size_t)t * E + e) : 0.0f;
        const uint32_t m = __ballot_sync(0xffffffffu, v != 0.0f);
        un |= m;
        nact += __popc(m);
      }
      if (lane == 0) {
        cnt[w] = __popc(un);
        act[w] = nact;
        um[w] = un;
      }
    }
    __syncthreads();
    int total = 0, total_act = 0;
    for (int w = 0; w < words; ++w) {
      total += cnt[w];
      total_act += act[w];
    }
    for (int w = warp; w < words; w += nwarps) {
      int off = 0;
      for (int v = 0; v < w; ++v) off += cnt[v];
      const uint32_t un = um[w];
      if ((un >> lane) & 1u) ids_sm[off + __popc(un & ((1u << lane) - 1u))] = 32 * w + lane;
    }
    if (threadIdx.x == 0) {
      ctl[0] = total;
      ctl[2] = total_act;
    }
  } else {
    if (threadIdx.x == 0) {
      int n = __ldcg(n_in), bad = 0;
      if (n < 0 || n > E) {
        bad |= BLOCKFFN_DEV_BAD_UNION_COUNT;
        n = n < 0 ? 0 : E;
      }
      int k = 0;
      for (int q = 0; q < n; ++q) {
        const int id = __ldcg(ids_in + q);
        if (id < 0 || id >= E)
          bad |= BLOCKFFN_DEV_BAD_UNION_ID;
        else
          ids_sm[k++] = id;
      }
      ctl[0] = k;
      ctl[3] = bad;
    }
  }
  __syncthreads();
  return ctl[0];
}

// ---- up projection ---------------------------------------------------------------
struct UpParams {
  const uint16_t* x;       // bf16 [L][d]
  const uint16_t* U;       // bf16 [E][d_e][d]
  const float* scores;     // f32 [L][E]
  const int32_t* ids_in;   // caller's union list, or NULL: derive from scores
  const int32_t* n_in;
  uint16_t* h;             // bf16 [q][L][d_e + 32] intermediate
  int L, d, E, d_e, ns, early;
  uint32_t* status;
  // what CTA 0 publishes when it derived the union itself (each may be NULL)
  uint32_t* pub_mask;
  int32_t* pub_ids;
  int32_t* pub_n;
  blockffn_stats* stats;
};

template <int NT>
__global__ void __launch_bounds__(kThreads, 1) expert_up_mma_kernel(const UpParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const SmemLayout lay = up_layout(p.d, p.E, NT, p.ns);
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bar_full = sbase + kOffBars, bar_empty = bar_full + 8 * kMaxStages,
                 bar_x = bar_empty + 8 * kMaxStages;
  int* ctl = reinterpret_cast<int*>(smem + lay.off_ctl);
  int* ids_sm = reinterpret_cast<int*>(smem + lay.off_ids);
  float* red = reinterpret_cast<float*>(smem + lay.off_red);
  const int d = p.d, d_e = p.d_e, L = p.L, ns = p.ns;
  const int XS = 2 * d + kPad, RS = 2 * kKC + kPad;

  if (tid == 0) {
    for (int s = 0; s < ns; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, kConsumerWarps);
    }
    mbar_init(bar_x, 1);
    for (int v = 0; v < 8; ++v) ctl[v] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (p.early) {
    pdl_trigger();       // the next kernel may start fetching its weights right away
  } else {
    pdl_wait();          // scores / ids may come from the kernel just before
    pdl_trigger();
  }
  __syncthreads();
  const int nu = derive_union(p.scores, p.ids_in, p.n_in, L, p.E, ids_sm, ctl, p.status);

  const long long R = (long long)nu * d_e;
  const int r0 = (int)(R * blockIdx.x / gridDim.x), r1 = (int)(R * (blockIdx.x + 1) / gridDim.x);
  const int nrows = r1 - r0;
  const int mt = (nrows + 15) >> 4;
  const int nkc = (d + kKC - 1) / kKC;
  const int nstages = mt * nkc;

  if (warp == kConsumerWarps) {
    // ===== producer warp: lane m copies row m of the stage's tile =====
    auto issue = [&](int s) {
      const int slot = s % ns, tile = s / nkc, kc = s - tile * nkc;
      const int k0 = kc * kKC, klen = min(kKC, d - k0);
      const int rows = min(16, nrows - tile * 16);
      if (lane == 0) mbar_expect_tx(bar_full + 8 * slot, (uint32_t)(rows * klen * 2));
      __syncwarp();
      if (lane < rows) {
        const int r = r0 + tile * 16 + lane;
        const int q = r / d_e, j = r - q * d_e;
        const uint16_t* src = p.U + ((size_t)ids_sm[q] * d_e + j) * d + k0;
        bulk_g2s(sbase + lay.off_ring + slot * lay.slot_bytes + lane * RS, src,
                 (uint32_t)(klen * 2), bar_full + 8 * slot);
      }
    };
    const int s_pre = p.early ? min(nstages, ns) : 0;
    for (int s = 0; s < s_pre; ++s) issue(s);
    pdl_wait();          // x may come from the kernel just before
    if (nstages > 0) {
      if (lane == 0) mbar_expect_tx(bar_x, (uint32_t)(L * d * 2));
      __syncwarp();
      for (int t = lane; t < L; t += 32)
        bulk_g2s(sbase + lay.off_x + t * XS, p.x + (size_t)t * d, (uint32_t)(d * 2), bar_x);
    }
    for (int s = s_pre; s < nstages; ++s) {
      if (s >= ns) mbar_wait(bar_empty + 8 * (s % ns), ((s / ns) - 1) & 1, ctl, p.status);
      issue(s);
    }
    // Outstanding copies: every stage issued is also awaited by the consumers; if they
    // gave up, wait here (bounded) so that no copy lands after the CTA is gone.
    if (ctl[1]) {
      for (int s = max(0, nstages - ns); s < nstages; ++s)
        mbar_wait(bar_full + 8 * (s % ns), (s / ns) & 1, ctl + 4, p.status);
      if (nstages > 0) mbar_wait(bar_x, 0, ctl + 4, p.status);
    }
  } else {
    // ===== consumer warps =====
    pdl_wait();
    const int g = lane >> 2, tg = lane & 3;
    if (nstages > 0) mbar_wait(bar_x, 0, ctl, p.status);
    for (int tile = 0; tile < mt; ++tile) {
      float acc[NT][4];
#pragma unroll
      for (int n = 0; n < NT; ++n)
#pragma unroll
        for (int v = 0; v < 4; ++v) acc[n][v] = 0.0f;
      for (int kc = 0; kc < nkc; ++kc) {
        const int s = tile * nkc + kc, slot = s % ns;
        const int k0 = kc * kKC, nsb = min(kKC, d - k0) >> 5;
        mbar_wait(bar_full + 8 * slot, (s / ns) & 1, ctl, p.status);
        const uint32_t a_base = sbase + lay.off_ring + slot * lay.slot_bytes + g * RS + tg * 16;
        const uint32_t b_base = sbase + lay.off_x + g * XS + k0 * 2 + tg * 16;
#pragma unroll 2
        for (int sb = warp; sb < nsb; sb += kConsumerWarps) {
          const uint4 ra = lds128(a_base + sb * 64);
          const uint4 rb = lds128(a_base + 8 * RS + sb * 64);
#pragma unroll
          for (int n = 0; n < NT; ++n) {
            const uint4 xb = lds128(b_base + n * 8 * XS + sb * 64);
            mma_bf16(acc[n], ra.x, rb.x, ra.y, rb.y, xb.x, xb.y);
            mma_bf16(acc[n], ra.z, rb.z, ra.w, rb.w, xb.z, xb.w);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_empty + 8 * slot);
      }
      // cross-warp reduction of the K split, then Swish, score, store
      float* mine = red + warp * (16 * 8 * NT);
#pragma unroll
      for (int n = 0; n < NT; ++n) {
        const int t = 8 * n + 2 * tg;
        mine[t * 16 + g] = acc[n][0];
        mine[(t + 1) * 16 + g] = acc[n][1];
        mine[t * 16 + g + 8] = acc[n][2];
        mine[(t + 1) * 16 + g + 8] = acc[n][3];
      }
      consumer_sync();
      const int rows = min(16, nrows - tile * 16);
      for (int e = tid; e < 16 * 8 * NT; e += kConsumerThreads) {
        const int t = e >> 4, m = e & 15;
        if (t < L && m < rows) {
          float v = 0.0f;
#pragma unroll
          for (int w = 0; w < kConsumerWarps; ++w) v += red[w * (16 * 8 * NT) + e];
          const int r = r0 + tile * 16 + m;
          const int q = r / d_e, j = r - q * d_e;
          const float s = __ldcg(p.scores + (size_t)t * p.E + ids_sm[q]);
          p.h[((size_t)q * L + t) * (d_e + 32) + j] = (uint16_t)f32_to_bf16_bits(s * swish(v));
        }
      }
      consumer_sync();
    }
    // CTA 0 publishes the routing it derived (after the wait: earlier readers are done)
    if (blockIdx.x == 0) {
      if (p.ids_in == nullptr) {
        const int words = (p.E + 31) >> 5;
        const uint32_t* um = reinterpret_cast<const uint32_t*>(ctl + 8);
        for (int e = tid; e < p.E; e += kConsumerThreads) {
          if (p.pub_ids) p.pub_ids[e] = e < nu ? ids_sm[e] : -1;
          if (p.pub_mask && e < words) p.pub_mask[e] = um[e];
        }
        if (tid == 0) {
          if (p.pub_n) *p.pub_n = nu;
          if (p.stats) {
            atomicAdd(reinterpret_cast<unsigned long long*>(&p.stats->n_tokens),
                      (unsigned long long)L);
            atomicAdd(reinterpret_cast<unsigned long long*>(&p.stats->n_active),
                      (unsigned long long)ctl[2]);
            atomicAdd(reinterpret_cast<unsigned long long*>(&p.stats->n_chunks), 1ull);
            atomicAdd(reinterpret_cast<unsigned long long*>(&p.stats->n_union),
                      (unsigned long long)nu);
          }
        }
      } else if (tid == 0 && ctl[3]) {
        atomicOr(p.status, (uint32_t)ctl[3]);
      }
    }
  }
}

// ---- down projection ---------------------------------------------------------------
struct DownParams {
  const uint16_t* D;       // bf16 [E][d][d_e]
  const uint16_t* h;       // bf16 [q][L][d_e + 32]
  const float* scores;
  const int32_t* ids_in;
  const int32_t* n_in;
  float* out;              // f32 [L][d]
  uint16_t* x_next;        // bf16 [L][d] or NULL
  int L, d, E, d_e, ns, accumulate;
  uint32_t* status;
};

template <int NT>
__global__ void __launch_bounds__(kThreads, 1) expert_down_mma_kernel(const DownParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const SmemLayout lay = down_layout(p.d_e, p.E, NT, p.ns);
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bar_full = sbase + kOffBars, bar_empty = bar_full + 8 * kMaxStages;
  int* ctl = reinterpret_cast<int*>(smem + lay.off_ctl);
  int* ids_sm = reinterpret_cast<int*>(smem + lay.off_ids);
  float* red = reinterpret_cast<float*>(smem + lay.off_red);
  const int d = p.d, d_e = p.d_e, L = p.L, ns = p.ns;
  const int DS = 2 * d_e, HS = 2 * d_e + kPad;   // bytes per staged D row / h row
  const uint32_t h_bytes = (uint32_t)(L * HS);

  if (tid == 0) {
    for (int s = 0; s < ns; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, kConsumerWarps);
    }
    for (int v = 0; v < 8; ++v) ctl[v] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  pdl_trigger();
  __syncthreads();
  // The routing inputs were final before the up kernel of this call passed its own wait.
  const int nu = derive_union(p.scores, p.ids_in, p.n_in, L, p.E, ids_sm, ctl, p.status);

  // column tiles: W = G * ceil(d / 16G) tiles of at most 16 columns, tile w -> CTA w % G
  const int G = gridDim.x;
  const int per = (d + 16 * G - 1) / (16 * G);
  const long long W = (long long)G * per;
  auto tile_c0 = [&](int ti) { return (int)((long long)d * (blockIdx.x + (long long)ti * G) / W); };
  auto tile_c1 = [&](int ti) {
    return (int)((long long)d * (blockIdx.x + (long long)ti * G + 1) / W);
  };
  const int nstages = per * nu;   // empty tiles keep their stages (h only), which is rare

  if (warp == kConsumerWarps) {
    // ===== producer lane =====
    if (lane == 0) {
      auto issue_d = [&](int s) {
        const int slot = s % ns, ti = s / nu, q = s - ti * nu;
        const int c0 = tile_c0(ti), ncols = tile_c1(ti) - c0;
        const uint32_t d_bytes = (uint32_t)(ncols * DS);
        mbar_expect_tx(bar_full + 8 * slot, d_bytes + h_bytes);
        if (ncols > 0)
          bulk_g2s(sbase + lay.off_ring + slot * lay.slot_bytes,
                   p.D + ((size_t)ids_sm[q] * d + c0) * d_e, d_bytes, bar_full + 8 * slot);
      };
      auto issue_h = [&](int s) {
        const int slot = s % ns, q = s % nu;
        bulk_g2s(sbase + lay.off_ring + slot * lay.slot_bytes + lay.slot_h_off,
                 p.h + (size_t)q * L * (d_e + 32), h_bytes, bar_full + 8 * slot);
      };
      const int s_pre = min(nstages, ns);
      for (int s = 0; s < s_pre; ++s) issue_d(s);
      pdl_wait();        // h is complete and visible from here on
      for (int s = 0; s < s_pre; ++s) issue_h(s);
      for (int s = s_pre; s < nstages; ++s) {
        mbar_wait(bar_empty + 8 * (s % ns), ((s / ns) - 1) & 1, ctl, p.status);
        issue_d(s);
        issue_h(s);
      }
      if (ctl[1]) {
        for (int s = max(0, nstages - ns); s < nstages; ++s)
          mbar_wait(bar_full + 8 * (s % ns), (s / ns) & 1, ctl + 4, p.status);
      }
    }
  } else {
    // ===== consumer warps =====
    pdl_wait();
    const int g = lane >> 2, tg = lane & 3;
    const int nsb = d_e >> 5;            // 32-wide k blocks per expert
    for (int ti = 0; ti < per; ++ti) {
      const int c0 = tile_c0(ti), ncols = tile_c1(ti) - c0;
      float acc[NT][4];
#pragma unroll
      for (int n = 0; n < NT; ++n)
#pragma unroll
        for (int v = 0; v < 4; ++v) acc[n][v] = 0.0f;
      for (int q = 0; q < nu; ++q) {
        const int s = ti * nu + q, slot = s % ns;
        mbar_wait(bar_full + 8 * slot, (s / ns) & 1, ctl, p.status);
        const uint32_t a_base = sbase + lay.off_ring + slot * lay.slot_bytes + g * DS + tg * 16;
        const uint32_t b_base =
            sbase + lay.off_ring + slot * lay.slot_bytes + lay.slot_h_off + g * HS + tg * 16;
        // k blocks of all experts are dealt round-robin to the warps
        for (int sb = (warp - q * nsb) & (kConsumerWarps - 1); sb < nsb; sb += kConsumerWarps) {
          const uint4 ra = lds128(a_base + sb * 64);
          const uint4 rb = lds128(a_base + 8 * DS + sb * 64);
#pragma unroll
          for (int n = 0; n < NT; ++n) {
            const uint4 xb = lds128(b_base + n * 8 * HS + sb * 64);
            mma_bf16(acc[n], ra.x, rb.x, ra.y, rb.y, xb.x, xb.y);
            mma_bf16(acc[n], ra.z, rb.z, ra.w, rb.w, xb.z, xb.w);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_empty + 8 * slot);
      }
      float* mine = red + warp * (16 * 8 * NT);
#pragma unroll
      for (int n = 0; n < NT; ++n) {
        const int t = 8 * n + 2 * tg;
        mine[t * 16 + g] = acc[n][0];
        mine[(t + 1) * 16 + g] = acc[n][1];
        mine[t * 16 + g + 8] = acc[n][2];
        mine[(t + 1) * 16 + g + 8] = acc[n][3];
      }
      consumer_sync();
      for (int e = tid; e < 16 * 8 * NT; e += kConsumerThreads) {
        const int t = e >> 4, m = e & 15;
        if (t < L && m < ncols) {
          float v = 0.0f;
#pragma unroll
          for (int w = 0; w < kConsumerWarps; ++w) v += red[w * (16 * 8 * NT) + e];
          const size_t o = (size_t)t * d + c0 + m;
          if (p.accumulate) v += __ldcg(p.out + o);
          p.out[o] = v;
          if (p.x_next) p.x_next[o] = (uint16_t)f32_to_bf16_bits(v);
        }
      }
      consumer_sync();
    }
  }
}

// ---- host side -----------------------------------------------------------------------
struct MmaPlan {
  int NT, ns_up, ns_down, smem_up, smem_down;
  bool ok;
};

MmaPlan make_plan(const blockffn_config& cfg, int L) {
  MmaPlan pl{};
  pl.ok = false;
  if (L < 1 || L > 32) return pl;
  if (cfg.d % 32 || cfg.d_e % 32 || cfg.E > 1024) return pl;
  if (cfg.d_e > 2048 || cfg.d > 65536) return pl;
  if ((long long)32 * (2 * cfg.d_e + kPad) + 16 * 2 * cfg.d_e >= (1 << 20)) return pl;  // tx count
  pl.NT = (L + 7) / 8;
  const int want_up = cfg.flags & 0xff, want_down = (cfg.flags >> 8) & 0xff;
  auto pick = [&](auto layout_of, int want) {
    const SmemLayout one = layout_of(1);
    const int base = one.total - one.slot_bytes;
    int ns = (kSmemHalf - base) / one.slot_bytes;        // share the SM with the other kernel
    if (ns < 2) ns = (kSmemMax - base) / one.slot_bytes; // or take it alone
    if (want) ns = want;
    if (ns > kMaxStages) ns = kMaxStages;
    if (base + ns * one.slot_bytes > kSmemMax) ns = (kSmemMax - base) / one.slot_bytes;
    return ns;
  };
  pl.ns_up = pick([&](int ns) { return up_layout(cfg.d, cfg.E, pl.NT, ns); }, want_up);
  pl.ns_down = pick([&](int ns) { return down_layout(cfg.d_e, cfg.E, pl.NT, ns); }, want_down);
  if (pl.ns_up < 2 || pl.ns_down < 2) return pl;
  if (pl.ns_up > 8) pl.ns_up = want_up ? pl.ns_up : 8;
  pl.smem_up = up_layout(cfg.d, cfg.E, pl.NT, pl.ns_up).total;
  pl.smem_down = down_layout(cfg.d_e, cfg.E, pl.NT, pl.ns_down).total;
  pl.ok = true;
  return pl;
}

template <int NT>
cudaError_t set_attrs() {
  cudaError_t e = cudaFuncSetAttribute(expert_up_mma_kernel<NT>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(expert_down_mma_kernel<NT>,
                              cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax);
}

template <int NT>
cudaError_t launch_nt(const MmaPlan& pl, int grid, const UpParams& up, const DownParams& dn,
                      cudaStream_t st) {
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t lc{};
  lc.gridDim = dim3(grid);
  lc.blockDim = dim3(kThreads);
  lc.stream = st;
  lc.attrs = attr;
  lc.numAttrs = 1;
  lc.dynamicSmemBytes = pl.smem_up;
  cudaError_t e = cudaLaunchKernelEx(&lc, expert_up_mma_kernel<NT>, up);
  if (e != cudaSuccess) return e;
  lc.dynamicSmemBytes = pl.smem_down;
  return cudaLaunchKernelEx(&lc, expert_down_mma_kernel<NT>, dn);
}

}  // namespace

bool expert_mma_supported(const blockffn_ctx* c, int L) { return make_plan(c->cfg, L).ok; }

size_t expert_mma_h_bytes(const blockffn_config* cfg) {
  return sizeof(uint16_t) * (size_t)cfg->E * cfg->L_max * (cfg->d_e + 32) + 256;
}

cudaError_t expert_mma_setup(blockffn_ctx*) {
  cudaError_t e = set_attrs<1>();
  if (e == cudaSuccess) e = set_attrs<2>();
  if (e == cudaSuccess) e = set_attrs<3>();
  if (e == cudaSuccess) e = set_attrs<4>();
  return e;
}

cudaError_t launch_expert_mma(blockffn_ctx* c, const blockffn_weights* w, const void* x,
                              const float* scores, int L, const int32_t* union_ids,
                              const int32_t* n_union, float* out, void* x_next, int call_flags,
                              const RoutingOut* pub, cudaStream_t st) {
  const MmaPlan pl = make_plan(c->cfg, L);
  if (!pl.ok) return cudaErrorNotSupported;
  UpParams up{};
  up.x = static_cast<const uint16_t*>(x);
  up.U = static_cast<const uint16_t*>(w->U);
  up.scores = scores;
  up.ids_in = union_ids;
  up.n_in = n_union;
  up.h = static_cast<uint16_t*>(c->h16);
  up.L = L;
  up.d = c->cfg.d;
  up.E = c->cfg.E;
  up.d_e = c->cfg.d_e;
  up.ns = pl.ns_up;
  up.early = (call_flags & BLOCKFFN_CALL_INDEPENDENT) ? 1 : 0;
  up.status = c->status;
  if (pub) {
    up.pub_mask = pub->union_mask;
    up.pub_ids = pub->union_ids;
    up.pub_n = pub->n_union;
    up.stats = pub->stats;
  }
  DownParams dn{};
  dn.D = static_cast<const uint16_t*>(w->D);
  dn.h = up.h;
  dn.scores = scores;
  dn.ids_in = union_ids;
  dn.n_in = n_union;
  dn.out = out;
  dn.x_next = static_cast<uint16_t*>(x_next);
  dn.L = L;
  dn.d = c->cfg.d;
  dn.E = c->cfg.E;
  dn.d_e = c->cfg.d_e;
  dn.ns = pl.ns_down;
  dn.accumulate = (call_flags & BLOCKFFN_CALL_ACCUMULATE) ? 1 : 0;
  dn.status = c->status;
  cudaError_t e;
  switch (pl.NT) {
    case 1: e = launch_nt<1>(pl, c->num_sms, up, dn, st); break;
    case 2: e = launch_nt<2>(pl, c->num_sms, up, dn, st); break;
    case 3: e = launch_nt<3>(pl, c->num_sms, up, dn, st); break;
    default: e = launch_nt<4>(pl, c->num_sms, up, dn, st); break;
  }
  if (e == cudaSuccess) c->launches += 2;
  return e;
}
