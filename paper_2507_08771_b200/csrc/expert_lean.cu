// Expert stage (Eq. 1, Eq. 2 restricted to Union(x), Sec. 3.3) as one kernel per call, for
// calls whose inputs are all stable (x included), so that several calls are in flight per SM.
// expert_lean_kernel takes chunks of up to 8 tokens, expert_wide_kernel (expert_wide.cuh) chunks
// of 9 to 32.
//
// A call lasts a few microseconds, most of which is memory latency: the routing inputs, then
// the weights they select, then the intermediate every CTA needs from every other. What the
// device sustains is therefore set by how many calls are in flight per SM, i.e. by how little
// shared memory and how few registers one CTA holds, and by how few instructions and bytes from
// L2 a call spends next to its weight stream. This kernel keeps only the weights in shared
// memory; the small operands (x for the up projection, the intermediate h for the down
// projection) go from L2 straight into the registers of the one warp that uses them: with K
// split over the warps no two warps read the same element, so a shared tile would only be a
// detour. Three CTAs (of three different calls) fit one SM, and a call runs on about a third of
// the SMs (see lean_plan), so that seven to nine calls are in flight.
//
//   CTA b, call n:
//     ticket           one atomic per CTA on the ring's call counter; ticket / CTAs per call is
//                      the call's index n (all CTAs of a call take theirs before any CTA of the
//                      next call exists, see below), n mod 16 its slot in the ring of h buffers
//     Union(x)         derived by every CTA from the scores, the caller's list or raw logits;
//                      thread 0 releases the dependent launch while those loads are in flight
//     up projection    the CTA's share of the union's neuron rows -> shared memory (16-byte
//                      asynchronous copies, in stages when the share exceeds the region), K split
//                      over the 8 warps, mma.sync m16n8k16 with the weights as the M operand and
//                      the tokens as N, cross-warp sum, Swish, router score, bf16 -> h ring slot
//                      (global, L2)
//     hand-over        one arrival per CTA on the slot's counter (after a fence); the D slabs of
//                      the CTA's output columns are requested into the same shared memory; then
//                      one thread polls the counter until all CTAs of the call have arrived
//                      (bounded: BLOCKFFN_DEV_WAIT_EXPIRED) and the warps fetch their h fragments
//     down projection  out[t][c] over all union experts for the CTA's columns (up to three tiles
//                      of 16), one writer per element, fixed summation order
//     griddepcontrol.wait before out is touched (and before the kernel ends)
//
// Ordering between calls. Kernels are chained by programmatic dependent launch and trigger
// their dependents only once the CTA holds its ticket, so tickets of successive calls never
// interleave. Every kernel waits for its predecessor before it ends, so no CTA of a call exits
// while an earlier call is incomplete: when a CTA of call n + R exists and call n is incomplete,
// all CTAs of calls n + 1 .. n + R - 1 are resident, plus one of each end, i.e.
// (R - 1) grid + 2 <= 3 SMs CTAs (at most three CTAs fit one SM: every launch asks for more than
// a quarter of its shared memory). A shared grid is never smaller than a quarter of the SMs, which
// allows R <= 12; the ring has 16 slots, so a slot is never reused while a CTA of its earlier call is alive, and
// its arrival counter is an exact multiple of the call's CTA count when a call starts: the
// counters only ever grow, nothing is reset, graph replays need no host state. A ticket
// identifies a call only if every call drawing from the counter has the same number of CTAs, so
// each kind of call (whole device; part of it with up to 8, up to 16, up to 32 tokens) has a
// ring and a counter of its own. The hand-over also needs all CTAs of a call resident at once:
// lean_plan refuses grids for which that is not guaranteed.
// The polling thread issues no asynchronous copies: a fence or an acquire by a thread waits
// for that thread's own copies in flight.
#include "mma_tiles.cuh"

namespace {

constexpr int kHRing = 16;           // h buffers and arrival counters per ring (see the bound above)
constexpr int kRings = 4;            // kinds of calls that count their own tickets (see below)
constexpr int kMinSmem = 60 * 1024;  // four such CTAs do not fit one SM (228 KB, 1 KB reserved each)
constexpr int kSyncThread = kThreads - 1;
constexpr int kCopyThreads = kThreads - 32;   // the last warp (the polling thread's) issues no D copies
constexpr int kMaxKB = 4;            // 64-wide k blocks of x per warp: d <= 8 * 64 * kMaxKB

struct LeanLayout {
  int off_red, off_w, total;
};
// red: cross-warp partial tiles, f32. The long-chunk kernel keeps them [token][warp][row]: a
// warp's rows are ws = rows rounded up to even apart, a token is ts = 8 ws + 4 words further.
// The 32 lanes of a partial store (tokens 2 tg (+ 1), rows g (+ 8)) then fall into 32 different banks, and the eight partials
// of an element are read by consecutive lanes from consecutive words. (With the warp index
// innermost every such store was an 8-way bank conflict: a third of the shared-memory
// wavefronts of a stage.) The 8-token kernel keeps [token][row][warp] inside the same region
// (see there). rows = red_rows in the up projection, 16 per column tile in the down projection;
// red_rows is at least 16 (16 per column tile); groups: token groups of 8.
__host__ __device__ inline int red_ws(int rows) { return (rows + 1) & ~1; }
__host__ __device__ inline int red_ts(int rows) { return kWarps * red_ws(rows) + 4; }
__host__ __device__ inline LeanLayout lean_layout(int E, int red_rows, int groups, int cap_bytes) {
  LeanLayout s;
  s.off_red = kOffIds + align128(E * 4);
  const int red = groups == 1 ? kWarps * 8 * 4 * red_rows              // [token][row][warp]
                              : groups * 8 * red_ts(red_rows) * 4;     // [token][warp][row]
  s.off_w = s.off_red + align128(red);
  s.total = s.off_w + cap_bytes;
  return s;
}
// sum of an element's eight partials, e: the first one, ws apart (fixed order)
__device__ __forceinline__ float red_sum(const float* e, int ws) {
  return ((e[0] + e[ws]) + (e[2 * ws] + e[3 * ws])) + ((e[4 * ws] + e[5 * ws]) + (e[6 * ws] + e[7 * ws]));
}

struct LeanParams {
  const uint16_t* x;       // bf16 [L][d]
  const uint16_t* U;       // bf16 [E][d_e][d]
  const uint16_t* D;       // bf16 [E][d][d_e]
  const float* scores;
  RouterLogits lg;
  const int32_t* ids_in;
  const int32_t* n_in;
  const uint16_t* W_r;     // MODE 3: router weight bf16 [E][d], bias f32 [E] or NULL (Eq. 3)
  const float* bias;
  float* logit_ring;       // MODE 3: kHRing buffers of logit_slot floats, each f32 [L][E]
  size_t logit_slot;
  uint16_t* h_ring;        // kHRing buffers of h_slot elements, each bf16 [q][L][d_e]
  size_t h_slot;
  unsigned long long* seq;     // tickets: one per CTA per call
  unsigned long long* ready;   // [kHRing] arrivals, never reset
  unsigned long long* ready2;  // MODE 3: [kHRing] arrivals of the logit hand-over, likewise
  float* out;
  uint16_t* x_next;
  int L, d, E, d_e, de_shift;
  int cap_bytes, red_rows;     // weight region; rows the up partial tile is sized for
  int cap_rows, cap_slabs;     // rows of U / slabs of D the region holds (paddings included)
  uint32_t magic_g;            // ceil(2^32 / grid): R / grid = mulhi(R, magic_g) for R < 2^24
  uint32_t magic_cpr;          // ceil(2^16 / (d / 8)): tid / (d / 8) = tid * magic_cpr >> 16
  int max_cols, cols_q, cols_rem;
  int accumulate;
  int dep;                     // x comes from the call before on the stream: wait before reading it
  int hold;                    // test aid: wait for an arrival that never comes
  unsigned long long wait_ns;  // bound of the hand-over wait
  uint32_t* status;
  uint32_t* pub_mask;
  int32_t* pub_ids;
  int32_t* pub_n;
  blockffn_stats* stats;
  float* pub_scores;
  uint32_t* pub_tok;
};

__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
// Asks L2 for the 128-byte lines that hold [p, p + bytes) (whole lines that contain a valid byte:
// never beyond the page of the range), shared out over the CTA's threads.
__device__ __forceinline__ void prefetch_l2(const void* p, int bytes) {
  const unsigned long long a = reinterpret_cast<unsigned long long>(p);
  const unsigned long long a0 = a & ~127ull;
  const int lines = (int)((a + (unsigned long long)bytes - a0 + 127ull) >> 7);
  for (int i = threadIdx.x; i < lines; i += blockDim.x)
    asm volatile("prefetch.global.L2 [%0];" ::"l"(a0 + 128ull * (unsigned)i));
}
// A 64-wide k block of a small operand row straight from global memory (L2): this lane's 8
// consecutive k of each 32-wide half, the same k permutation load_frag64 applies to the
// shared-memory operand.
// (volatile: the loads are issued where they are written, long before their first use, and must
// not be sunk to it)
__device__ __forceinline__ uint4 ld_cg_v4(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.cg.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p)
               : "memory");
  return v;
}
// ---- instruction-lean building blocks ----------------------------------------------------
// A call's 2000-odd warp instructions per warp were what limited three resident CTAs, not the
// memory system: four schedulers issue for 24 warps. Everything below is written to spend few
// instructions: 32-bit shared-memory addresses with constant offsets, 32-bit element indices
// into global memory (one mad.wide per address), no select in the fragment path.
//
// Rows of an operand tile are stored even rows first, then 64 bytes of padding, then the odd
// rows: the two rows a quarter-warp reads together (g and g + 1) then sit 64 bytes apart modulo
// 128, i.e. on disjoint halves of the 32 banks, and a fragment is two plain 128-bit loads.
__device__ __forceinline__ uint4 lds128(uint32_t a) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "r"(a));
  return v;
}
// global address = base + 16 * idx16 (idx16 < 2^32)
__device__ __forceinline__ const void* at16(const void* base, uint32_t idx16) {
  unsigned long long a;
  asm("mad.wide.u32 %0, %1, 16, %2;" : "=l"(a) : "r"(idx16), "l"(base));
  return reinterpret_cast<const void*>(a);
}
// the four mma of one 64-wide k block: a = rows g (lo/hi half), b = rows g + 8, x = the tokens
__device__ __forceinline__ void mma64(float (&c0)[4], float (&c1)[4], const uint4& alo,
                                      const uint4& ahi, const uint4& blo, const uint4& bhi,
                                      const Frag64& x) {
  mma_bf16(c0, alo.x, blo.x, alo.y, blo.y, x.lo.x, x.lo.y);
  mma_bf16(c1, ahi.x, bhi.x, ahi.y, bhi.y, x.hi.x, x.hi.y);
  mma_bf16(c0, alo.z, blo.z, alo.w, blo.w, x.lo.z, x.lo.w);
  mma_bf16(c1, ahi.z, bhi.z, ahi.w, bhi.w, x.hi.z, x.hi.w);
}

// KB: 64-wide k blocks of x per warp (ceil(d / 512)); NC: 16-column tiles of out per CTA
// (1 .. 4); MODE as derive_union, or 3: the router runs inside the kernel (Eq. 3). CTA b then
// computes the logits of experts b, b + grid, ... for all tokens (the arithmetic of the router
// kernel: one 16-byte piece of the rows per thread, fp32 FMAs, warp shuffles, the eight warp sums
// added in order), stores them in the call's slot of a ring of logit buffers, arrives on that
// slot's counter and waits (bounded) until all CTAs of the call have: a first hand-over of the
// same kind as the one for h. Then every CTA finishes Eq. 3 as in MODE 2.
// Everything the call reads is stable (x included): nothing waits for the kernel before it
// until out is touched.
template <int KB, int NC, int MODE>
__global__ void __launch_bounds__(kThreads, 3) expert_lean_kernel(const LeanParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int d = p.d, d_e = p.d_e, L = p.L;
  const LeanLayout lay = lean_layout(p.E, p.red_rows, 1, p.cap_bytes);
  const uint32_t sbase = smem_u32(smem);
  const uint32_t wbase = sbase + lay.off_w;
  int* ctl = reinterpret_cast<int*>(smem + kOffCtl);
  int* ids_sm = reinterpret_cast<int*>(smem + kOffIds);
  float* red = reinterpret_cast<float*>(smem + lay.off_red);
  const int g = lane >> 2, tg = lane & 3;
  const int wpos = (warp + 2 * tg + (g >> 2)) & 7;   // where this warp's partial of an element sits
  const int G = gridDim.x, bx = blockIdx.x;

  if (tid < 8) ctl[tid] = 0;
  unsigned long long ticket = 0;
  if (tid == 0) ticket = atomicAdd(p.seq, 1ull);
  __syncthreads();
  // Thread 0 turns its ticket into the call's ring slot and lets the dependents go while the
  // routing loads are in flight: every CTA of this call then holds its ticket before a CTA of
  // the next call exists, and the next call starts as early as that allows.
  auto on_ticket = [&]() {
    const unsigned long long n = ticket / (unsigned)G;
    ctl[6] = (int)(n & (kHRing - 1));
    *reinterpret_cast<unsigned long long*>(ctl + 138) =
        p.hold ? ~0ull : (n / kHRing + 1ull) * (unsigned)G;
    pdl_trigger();
  };
  // With the caller's union list the scores are first read when the first stage is finished:
  // their lines are requested now, or that read waits for DRAM in the middle of the up projection.
  if constexpr (MODE == 1) prefetch_l2(p.scores, L * p.E * 4);
  RouterLogits lg3 = p.lg;       // MODE 3 only: the logits are this call's slot of the logit ring
  if constexpr (MODE == 3) {
    if (tid == 0) on_ticket();
    __syncthreads();
    // In a dependent chain x (and, without any promise, everything else) is what the call
    // before leaves: nothing has been read so far, and nothing is before that call is done.
    if (p.dep) pdl_wait();
    const int rslot = ctl[6];
    float* a0 = p.logit_ring + (size_t)rslot * p.logit_slot;
    lg3.a0 = a0;
    const int chunks = d >> 3;                 // 16-byte pieces of a row (<= 256: one per thread)
    float* wsum = red;                         // [8 warps][8 tokens]
    for (int e = bx; e < p.E; e += G) {
      float acc[8];
#pragma unroll
      for (int t = 0; t < 8; ++t) acc[t] = 0.0f;
      if (tid < chunks) {
        const uint4 wv = __ldg(reinterpret_cast<const uint4*>(p.W_r + (size_t)e * d) + tid);
        const uint32_t wp[4] = {wv.x, wv.y, wv.z, wv.w};
        uint4 xv[8];
#pragma unroll
        for (int t = 0; t < 8; ++t)
          xv[t] = t < L ? __ldcg(reinterpret_cast<const uint4*>(p.x + (size_t)t * d) + tid)
                        : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          const uint32_t xp[4] = {xv[t].x, xv[t].y, xv[t].z, xv[t].w};
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            acc[t] = fmaf(bf16_lo(wp[q]), bf16_lo(xp[q]), acc[t]);
            acc[t] = fmaf(bf16_hi(wp[q]), bf16_hi(xp[q]), acc[t]);
          }
        }
      }
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        float v = acc[t];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) wsum[warp * 8 + t] = v;
      }
      __syncthreads();
      if (tid < L) {
        float v = p.bias ? p.bias[e] : 0.0f;
#pragma unroll
        for (int w8 = 0; w8 < kWarps; ++w8) v += wsum[w8 * 8 + tid];
        a0[(size_t)tid * p.E + e] = v;
      }
      __syncthreads();
    }
    if (tid == kSyncThread) {
      __threadfence();
      asm volatile("red.relaxed.gpu.global.add.u64 [%0], 1;" ::"l"(p.ready2 + rslot) : "memory");
      const unsigned long long target = *reinterpret_cast<const unsigned long long*>(ctl + 138);
      const unsigned long long t0 = global_ns();
      const unsigned long long limit = p.hold ? 2000000ull : p.wait_ns;
      while (ld_acquire_u64(p.ready2 + rslot) < target) {
        if (global_ns() - t0 > limit) {
          ctl[5] = 1;
          atomicOr(p.status, BLOCKFFN_DEV_WAIT_EXPIRED);
          break;
        }
      }
    }
    __syncthreads();
  }
  // (the other modes read the kernel parameter where they need it: nothing to keep in registers)
  const RouterLogits& lg = MODE == 3 ? lg3 : p.lg;
  int nu_;
  if constexpr (MODE == 3)       // (the dependents were released above)
    nu_ = derive_union<2>(p.scores, lg, p.ids_in, p.n_in, L, p.E, ids_sm, ctl,
                          reinterpret_cast<uint32_t*>(red));
  else
    nu_ = derive_union<MODE>(p.scores, lg, p.ids_in, p.n_in, L, p.E, ids_sm, ctl,
                             reinterpret_cast<uint32_t*>(red), on_ticket);
  const int nu = nu_;

  // ---- up projection ---------------------------------------------------------------------
  const int R = nu * d_e;
  const int rq = (int)__umulhi((unsigned)R, p.magic_g), rrem = R - rq * G;
  const int r0 = bx * rq + min(bx, rrem), nrows = rq + (bx < rrem ? 1 : 0), r1 = r0 + nrows;
  const int row_bytes = 2 * d;
  const int cap_rows = p.cap_rows;
  // one stage when the share fits (the usual case: no division on that path), else stages of
  // half the region that are refilled as they free
  const int ldr = min(p.red_rows, 32);       // a stage is at most two row tiles
  const bool single = nrows <= min(ldr, cap_rows);
  const int slot_rows = single ? max(nrows, 1) : min(ldr, cap_rows / 2);
  const int ngroups = single ? (nrows > 0 ? 1 : 0) : (nrows + slot_rows - 1) / slot_rows;
  const int rpg = single ? nrows : (nrows + ngroups - 1) / ngroups;
  const int half_u = ((slot_rows + 1) >> 1) * row_bytes + 64;   // where the odd rows start
  const int slot_bytes = slot_rows * row_bytes + 64;
  const int sh = p.de_shift;
  // This thread's part of a row copy: 16-byte chunk my_c of the rows my_sub, my_sub + rpi, ...
  const int cpr = d >> 3;                       // chunks per row (<= 256)
  const int rpi = cpr > 128 ? 1 : kThreads / cpr;   // rows the CTA copies per step
  const int my_sub = (tid * p.magic_cpr) >> 16, my_c = tid - my_sub * cpr;
  const bool copies_u = my_sub < rpi;
  // stage gi: rows [r0 + gi rpg, ...) -> slot gi & 1, row m of the stage at
  // (m >> 1) row_bytes + (m & 1) half_u
  auto issue_u = [&](int gi) {
    const int ra = r0 + gi * rpg;
    const int rows = min(r1, ra + rpg) - ra;
    const uint32_t slot0 = wbase + (gi & 1) * slot_bytes + my_c * 16;
    if (!copies_u) return;
    if (rpi == 1) {
      // every thread walks all rows: two running destinations (even rows, odd rows), the
      // source index steps by one row inside an expert and jumps at an expert's end
      uint32_t de = slot0, dd = slot0 + half_u;
      int m = 0;
      while (m < rows) {
        const int r = ra + m, q = r >> sh;
        const int seg_end = min(rows, ((q + 1) << sh) - ra);     // rows of this expert end here
        uint32_t idx = (uint32_t)(ids_sm[q] * d_e + (r - (q << sh))) * (uint32_t)cpr + my_c;
        if (m & 1) {               // start on an even row of the stage
          cp_async16(dd, at16(p.U, idx));
          dd += row_bytes;
          idx += cpr;
          ++m;
        }
#pragma unroll 2
        for (; m + 1 < seg_end; m += 2, idx += 2 * cpr, de += row_bytes, dd += row_bytes) {
          cp_async16(de, at16(p.U, idx));
          cp_async16(dd, at16(p.U, idx + cpr));
        }
        if (m < seg_end) {
          cp_async16(de, at16(p.U, idx));
          de += row_bytes;
          ++m;
        }
      }
    } else {
      int m = my_sub;
      while (m < rows) {
        const int r = ra + m, q = r >> sh;
        const int seg_end = min(rows, ((q + 1) << sh) - ra);
        uint32_t idx = (uint32_t)(ids_sm[q] * d_e + (r - (q << sh))) * (uint32_t)cpr + my_c;
        const uint32_t step = (uint32_t)rpi * cpr;
        for (; m < seg_end; m += rpi, idx += step)
          cp_async16(slot0 + (m >> 1) * row_bytes + (m & 1) * half_u, at16(p.U, idx));
      }
    }
  };
  // score, expert slot and neuron of the h element this thread finishes in a stage
  // (token tid / 32, row tid % 32 of the stage)
  float sc = 0.0f;
  int hidx = -1;        // element index into the h buffer, -1: nothing to finish
  auto prepare = [&](int gi) {
    const int ra = r0 + gi * rpg, rows = min(r1, ra + rpg) - ra;
    const int t = tid >> 5, m = tid & 31;
    sc = 0.0f;
    hidx = -1;
    if (t < L && m < rows) {
      const int hq = (ra + m) >> sh;
      hidx = (hq * L + t) * d_e + (ra + m - (hq << sh));
      const int id = ids_sm[hq];
      if constexpr (MODE >= 2) {
        float v = __ldcg(lg.a0 + t * p.E + id);
        v = v > 0.0f ? v : 0.0f;
        sc = __ldg(lg.gain + id) * v * reinterpret_cast<const float*>(ctl + 104)[t];
      } else {
        sc = __ldcg(p.scores + t * p.E + id);
      }
    }
  };
  // x: this warp's k blocks (warp + 8 i) of the token row this lane feeds to the mma
  const int npx = d >> 6;
  Frag64 fx[KB];
  auto load_x = [&]() {
    const uint4* xp = reinterpret_cast<const uint4*>(p.x + min(g, L - 1) * d + 64 * warp) + tg;
#pragma unroll
    for (int i = 0; i < KB; ++i) {
      if (warp + kWarps * i < npx) {
        fx[i].lo = ld_cg_v4(xp + 64 * i);          // 64 k blocks of 128 bytes = 8 warps further
        fx[i].hi = ld_cg_v4(xp + 64 * i + 4);
      } else {
        fx[i].lo = fx[i].hi = make_uint4(0, 0, 0, 0);
      }
    }
  };
  // x goes first: its short round trip then runs under the long issue of the weights instead
  // of behind it
  load_x();
  if (ngroups > 0) issue_u(0);
  cp_async_commit();
  if (ngroups > 1) issue_u(1);
  cp_async_commit();
  if (ngroups > 0) prepare(0);
  const int slot = ctl[6];       // (written before the barriers inside derive_union)
  uint16_t* hbuf = p.h_ring + (size_t)slot * p.h_slot;

  for (int gi = 0; gi < ngroups; ++gi) {
    const int rows = min(r1, r0 + (gi + 1) * rpg) - (r0 + gi * rpg);
    // fragment addresses of rows g and g + 8 (same parity) of the two 16-row tiles, at this
    // warp's first k block; rows beyond the stage read its last row (their results are dropped)
    auto row_addr = [&](int m) {
      m = min(m, rows - 1);
      return wbase + (gi & 1) * slot_bytes + (m >> 1) * row_bytes + (m & 1) * half_u + 128 * warp +
             16 * tg;
    };
    const uint32_t a0 = row_addr(g), b0 = row_addr(g + 8);
    cp_async_wait_group<1>();      // all but the newest group: this stage has landed
    __syncthreads();
    // partial tiles -> red[t][m][.]: the eight partials of an element are 32 contiguous bytes
    // (two 128-bit loads: this kernel is bound by its instruction count, and the layout of the
    // long-chunk kernel costs six more loads per element). Warp w's partial sits at position
    // (w + 2 tg + g / 4) mod 8 of those eight words: the 32 lanes of a store then fall into 32
    // different banks (with w itself as the position they fell into four), and the reader adds
    // all eight words anyway.
    float* mine = red + (2 * tg * ldr + g) * kWarps + wpos;
    const int nt = ldr * kWarps;           // one token further
    {
      float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int i = 0; i < KB; ++i) {
        if (warp + kWarps * i < npx) {
          const uint4 alo = lds128(a0 + 1024 * i), ahi = lds128(a0 + 1024 * i + 64);
          const uint4 blo = lds128(b0 + 1024 * i), bhi = lds128(b0 + 1024 * i + 64);
          mma64(c0, c1, alo, ahi, blo, bhi, fx[i]);
        }
      }
      if (g < ldr) {
        mine[0] = c0[0] + c1[0];
        mine[nt] = c0[1] + c1[1];
      }
      if (g + 8 < ldr) {
        mine[8 * kWarps] = c0[2] + c1[2];
        mine[nt + 8 * kWarps] = c0[3] + c1[3];
      }
    }
    if (rows > 16) {               // second tile of 16 rows
      const uint32_t a1 = row_addr(g + 16), b1 = row_addr(g + 24);
      float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int i = 0; i < KB; ++i) {
        if (warp + kWarps * i < npx) {
          const uint4 alo = lds128(a1 + 1024 * i), ahi = lds128(a1 + 1024 * i + 64);
          const uint4 blo = lds128(b1 + 1024 * i), bhi = lds128(b1 + 1024 * i + 64);
          mma64(c0, c1, alo, ahi, blo, bhi, fx[i]);
        }
      }
      if (g + 16 < ldr) {
        mine[16 * kWarps] = c0[0] + c1[0];
        mine[nt + 16 * kWarps] = c0[1] + c1[1];
      }
      if (g + 24 < ldr) {
        mine[24 * kWarps] = c0[2] + c1[2];
        mine[nt + 24 * kWarps] = c0[3] + c1[3];
      }
    }
    __syncthreads();               // partials complete; every warp is done with the slot
    if (gi + 2 < ngroups) issue_u(gi + 2);
    cp_async_commit();
    if (hidx >= 0) {
      const float4* part = reinterpret_cast<const float4*>(red + ((tid >> 5) * ldr + (tid & 31)) * kWarps);
      const float4 lo = part[0], hi = part[1];
      const float v = ((lo.x + lo.y) + (lo.z + lo.w)) + ((hi.x + hi.y) + (hi.z + hi.w));
      hbuf[hidx] = (uint16_t)f32_to_bf16_bits(sc * swish_fast(v));
    }
    if (gi + 1 < ngroups) prepare(gi + 1);
    // the next stage starts with a wait and a barrier, which also protects red
  }
  cp_async_wait_all();
  __syncthreads();                 // every h element of this CTA has been stored
  if (tid == kSyncThread) {
    __threadfence();
    asm volatile("red.relaxed.gpu.global.add.u64 [%0], 1;" ::"l"(p.ready + slot) : "memory");
    // the counters of the logit hand-over advance in step with these, whether or not the call
    // has one: a slot's two counters then always agree on how often the slot has been used
    static_assert(kHRing * sizeof(unsigned long long) == 128, "offset of ready2 below");
    if constexpr (MODE != 3)     // (ready2 = ready + kHRing)
      asm volatile("red.relaxed.gpu.global.add.u64 [%0 + 128], 1;" ::"l"(p.ready + slot) : "memory");
  }

  // ---- down projection -------------------------------------------------------------------
  // Slab of one expert: the CTA's columns (at most 16 NC, NC mma row tiles) as rows of 2 d_e
  // bytes, even columns first, 64 bytes of padding, odd columns.
  const int drow = 2 * d_e;
  const int half_d = ((p.max_cols + 1) >> 1) * drow + 64;
  const int slot_d = p.max_cols * drow + 64;
  const int cap_slabs = p.cap_slabs;
  const bool one_round = nu <= cap_slabs;
  const int rsz = one_round ? max(nu, 1) : max(1, cap_slabs / 2);
  const int nrounds = one_round ? (nu > 0 ? 1 : 0) : (nu + rsz - 1) / rsz;
  const int c0 = bx * p.cols_q + min(bx, p.cols_rem);
  const int ncols = p.cols_q + (bx < p.cols_rem ? 1 : 0);
  // A slab is ncols << kshift chunks of 16 bytes; chunk c = column c >> kshift, piece
  // c & (2^kshift - 1). Thread tid copies chunks tid, tid + kCopyThreads, ... of every expert.
  const int kshift = sh - 3;                    // log2(chunks per D row)
  const uint32_t estride16 = (uint32_t)d << kshift;
  const int nchunks = tid < kCopyThreads ? ncols << kshift : 0;
  auto issue_d = [&](int r) {
    const int q0 = r * rsz, n = min(rsz, nu - q0);
    for (int c = tid; c < nchunks; c += kCopyThreads) {
      const int cc = c >> kshift, k = c & ((1 << kshift) - 1);
      const uint32_t src0 = ((uint32_t)(c0 + cc) << kshift) + k;          // + id * d << kshift
      uint32_t dst = wbase + (r & 1) * rsz * slot_d + (cc >> 1) * drow + (cc & 1) * half_d + k * 16;
#pragma unroll 4
      for (int i = 0; i < n; ++i, dst += slot_d)
        cp_async16(dst, at16(p.D, src0 + (uint32_t)ids_sm[q0 + i] * estride16));
    }
  };
  if (nrounds > 0) issue_d(0);
  cp_async_commit();
  if (nrounds > 1) issue_d(1);
  cp_async_commit();
  const int ot = tid >> 5, om = tid & 31;   // this thread's outputs: token ot, columns om (+ 32)
  // hand-over: all CTAs of this call have stored their part of h
  if (tid == kSyncThread) {
    const unsigned long long target = *reinterpret_cast<const unsigned long long*>(ctl + 138);
    const unsigned long long t0 = global_ns();
    // once a wait has run out on this handle the later ones give up quickly, until the caller
    // has read and cleared the status word
    const bool before = (*reinterpret_cast<volatile uint32_t*>(p.status) & BLOCKFFN_DEV_WAIT_EXPIRED) != 0;
    const unsigned long long limit = p.hold ? 2000000ull : before ? 1000000ull : p.wait_ns;
    int expired = 0;
    while (ld_acquire_u64(p.ready + slot) < target) {
      if (global_ns() - t0 > limit) {
        expired = 1;
        break;
      }
    }
    if (expired) {
      ctl[5] = 1;
      atomicOr(p.status, BLOCKFFN_DEV_WAIT_EXPIRED);
    }
  }
  __syncthreads();
  const bool dead = ctl[5] != 0;    // the wait ran out: out is left untouched

  const int npairs = d_e >> 6;      // 64-wide k blocks per expert (a power of two)
  const int pshift = sh - 6;
  float acc[NC][2][4];
#pragma unroll
  for (int c = 0; c < NC; ++c)
#pragma unroll
    for (int v = 0; v < 4; ++v) acc[c][0][v] = acc[c][1][v] = 0.0f;
  // rows (columns of out) g, g + 8 (, g + 16, g + 24) of a slab, clamped to the CTA's columns
  auto col_off = [&](int m) {
    m = min(m, max(ncols, 1) - 1);
    return (m >> 1) * drow + (m & 1) * half_d + 16 * tg;
  };
  uint32_t offs[NC][2];
#pragma unroll
  for (int c = 0; c < NC; ++c) {
    offs[c][0] = col_off(g + 16 * c);
    offs[c][1] = col_off(g + 16 * c + 8);
  }
  const uint4* hrow = reinterpret_cast<const uint4*>(hbuf + min(g, L - 1) * d_e) + tg;
  const uint32_t hstep16 = (uint32_t)(L * d_e) >> 3;         // one expert further, in 16 bytes
  for (int r = 0; r < nrounds && !dead; ++r) {
    const int q0 = r * rsz, n = min(rsz, nu - q0);
    const int nblk = n << pshift;
    const uint32_t d_base = wbase + (r & 1) * rsz * slot_d;
    // this warp's k blocks b = warp + 8 i of the round, in batches whose h fragments are all
    // requested before the first is used; block b = expert b >> pshift, k block b & (npairs - 1)
    // (fewer per batch with more column tiles: their accumulators need the registers, and a
    // round then holds fewer experts anyway)
    constexpr int kHB = NC == 1 ? 5 : NC == 2 ? 3 : 2;
    Frag64 fh[kHB];
    auto load_h = [&](int b0) {
#pragma unroll
      for (int i = 0; i < kHB; ++i) {
        const int b = b0 + kWarps * i;
        if (b < nblk) {
          const uint4* hp = hrow + (uint32_t)(q0 + (b >> pshift)) * hstep16 + 8 * (b & (npairs - 1));
          fh[i].lo = ld_cg_v4(hp);
          fh[i].hi = ld_cg_v4(hp + 4);
        }
      }
    };
    load_h(warp);
    cp_async_wait_group<1>();      // all but the newest group: this round's slabs have landed
    __syncthreads();
    for (int b0 = warp; b0 < nblk; b0 += kWarps * kHB) {
      if (b0 != warp) load_h(b0);
#pragma unroll
      for (int i = 0; i < kHB; ++i) {
        const int b = b0 + kWarps * i;
        if (b < nblk) {
          const uint32_t da = d_base + (b >> pshift) * slot_d + 128 * (b & (npairs - 1));
#pragma unroll
          for (int c = 0; c < NC; ++c) {
            const uint4 alo = lds128(da + offs[c][0]), ahi = lds128(da + offs[c][0] + 64);
            const uint4 blo = lds128(da + offs[c][1]), bhi = lds128(da + offs[c][1] + 64);
            mma64(acc[c][0], acc[c][1], alo, ahi, blo, bhi, fh[i]);
          }
        }
      }
    }
    __syncthreads();               // every warp is done with this round's slabs
    if (r + 2 < nrounds) issue_d(r + 2);
    cp_async_commit();
  }
  cp_async_wait_all();
  pdl_wait();                      // out (and x_next) may still be in use by the call before
  if (!dead) {
    if (nu > 0) {
      // partial tiles -> red[t][m][warp] (m < 16 NC), then one thread per output element
      float* mine = red + (2 * tg * (16 * NC) + g) * kWarps + wpos;
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        mine[(16 * c) * kWarps] = acc[c][0][0] + acc[c][1][0];
        mine[(16 * NC + 16 * c) * kWarps] = acc[c][0][1] + acc[c][1][1];
        mine[(16 * c + 8) * kWarps] = acc[c][0][2] + acc[c][1][2];
        mine[(16 * NC + 16 * c + 8) * kWarps] = acc[c][0][3] + acc[c][1][3];
      }
      __syncthreads();
      if (ot < L) {
#pragma unroll
        for (int k = 0; k < (NC + 1) / 2; ++k) {
          const int m = om + 32 * k;
          if (m < ncols) {
            const float4* part = reinterpret_cast<const float4*>(red + (ot * (16 * NC) + m) * kWarps);
            const float4 lo = part[0], hi = part[1];
            float v = ((lo.x + lo.y) + (lo.z + lo.w)) + ((hi.x + hi.y) + (hi.z + hi.w));
            const int o = ot * d + c0 + m;
            if (p.accumulate) v += __ldcg(p.out + o);
            p.out[o] = v;
            if (p.x_next) p.x_next[o] = (uint16_t)f32_to_bf16_bits(v);
          }
        }
      }
    } else if (ot < L) {           // empty union: FFN(x) = 0
      for (int m = om; m < ncols; m += 32) {
        const int o = ot * d + c0 + m;
        const float v = p.accumulate ? __ldcg(p.out + o) : 0.0f;
        p.out[o] = v;
        if (p.x_next) p.x_next[o] = (uint16_t)f32_to_bf16_bits(v);
      }
    }
  }
  // CTA 0 publishes the routing it derived (after the wait: earlier readers are done)
  if (blockIdx.x == 0) {
    if (lg.a0 != nullptr && p.pub_scores != nullptr) {
      const int words = (p.E + 31) >> 5;
      const float* rinv = reinterpret_cast<const float*>(ctl + 104);
      for (int t = warp; t < L; t += kWarps) {
        for (int w = 0; w < words; ++w) {
          const int e = 32 * w + lane;
          float sv = 0.0f;
          if (e < p.E) {
            float v = __ldcg(lg.a0 + (size_t)t * p.E + e);
            v = v > 0.0f ? v : 0.0f;
            sv = __ldg(lg.gain + e) * v * rinv[t];
            p.pub_scores[(size_t)t * p.E + e] = sv;
          }
          const uint32_t m = __ballot_sync(0xffffffffu, sv != 0.0f);
          if (p.pub_tok && lane == 0) p.pub_tok[(size_t)t * words + w] = m;
        }
      }
    }
    if (p.ids_in == nullptr) {
      const int words = (p.E + 31) >> 5;
      const uint32_t* um = reinterpret_cast<const uint32_t*>(ctl + 8);
      for (int e = tid; e < p.E; e += kThreads) {
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

#include "expert_wide.cuh"   // expert_wide_kernel: the same for chunks of 9 .. 32 tokens

// ---- host side ---------------------------------------------------------------------------
struct LeanPlan {
  int grid, teams, nc, ntg, cap_bytes, red_rows, max_cols, cols_q, cols_rem, smem, kb, slot_d;
  bool ok;
};

// Shapes: d a multiple of 64 up to 2048 (x fragments of a warp fit its registers); d_e a power
// of two >= 64; L <= 32 (up to 8 tokens: one token group; 9 .. 16: two; 17 .. 32: two teams of
// two; more than 8 only for calls that share the device and do not come with raw router logits).
//
// How many CTAs a call gets. Every CTA reads all of x and all of h from L2, whatever its share
// of the weights: with one CTA per SM that broadcast is half as many bytes again as the weights
// themselves, and an SM takes bytes in from L2 only about one and a half times as fast as its
// share of the HBM stream. A call therefore runs on a fraction of the SMs (grid = SMs / split),
// each CTA with a `split` times larger share (up to three column tiles of out), and `split`
// times as many calls are in flight to cover the rest of the device.
//
// shared: the call may share the device with its neighbours (it depends on none of them)
LeanPlan lean_plan(const blockffn_config& cfg, int L, int sms, bool shared) {
  LeanPlan pl{};
  pl.ok = false;
  const int d = cfg.d, d_e = cfg.d_e, E = cfg.E;
  if (L < 1 || L > 32 || sms < 1) return pl;
  if (d % 64 || d > 512 * kMaxKB || d_e % 64 || (d_e & (d_e - 1)) || d_e > 4096 || E > 1024)
    return pl;
  pl.kb = (d / 64 + kWarps - 1) / kWarps;
  pl.teams = L > 16 ? 2 : 1;          // more than 16 tokens: two teams of 8 warps in one CTA
  pl.ntg = L <= 8 ? 1 : 2;            // longer chunks: 16 tokens per team, two groups each
  int u_exp = (cfg.flags >> 17) & 0x7ff;
  if (u_exp == 0) u_exp = (L == 1 ? E + 4 : 3 * E + 5) / (L == 1 ? 8 : 10);
  if (u_exp < 1) u_exp = 1;
  if (u_exp > E) u_exp = E;
  // measured on B200 (d = 1536 and 2048, unions of 30 %): a third of the SMs per call is best
  // for calls that do not depend on one another; a call in a dependent chain is alone on the
  // device and takes all of it
  int split = shared && !(cfg.flags & BLOCKFFN_CFG_NO_SPLIT) ? 3 : 1;
  for (;; --split) {                               // at most three column tiles per CTA
    // Chunks of more than 8 tokens run one or two CTAs per SM; their grid is rounded down, so
    // that whole calls fill the SMs (three calls of 49 CTAs on 148 SMs at one CTA per SM, six at
    // two). With 50 the last call resident is short of two CTAs until an earlier call has ended,
    // and its hand-over waits for them: measured 12.3 against 8.6 us per call at 32 tokens, 6.0
    // against 5.2 at 16 (d = 2048, union 19). At three CTAs per SM nine calls are in flight either
    // way and the slightly smaller share per CTA wins (4.18 against 4.37 us at 8 tokens).
    pl.grid = pl.ntg == 1 ? (sms + split - 1) / split : sms / split;
    pl.nc = (d + 16 * pl.grid - 1) / (16 * pl.grid);
    if (pl.nc <= 3 || split == 1) break;
  }
  if (pl.nc > 3) return pl;
  // Chunks of up to 8 tokens that share the device: a grid that gives every CTA whole 16-column
  // tiles of out (d = 16 nc grid), if one lies between a quarter and half of the SMs, rather
  // than exactly a third. A ragged last tile costs its mma and fragment loads all the same:
  // measured 2.31 -> 2.23 us per call at d = 1536 (48 CTAs with two tiles instead of 50 with
  // 31 columns), 4.18 -> 3.95 at d = 2048 (64 CTAs with two tiles instead of 50 with 41 columns),
  // 12.7 -> 11.7 for the dense layer of that shape.
  if (pl.ntg == 1 && split > 1) {
    int best = 0;
    for (int nc = 1; nc <= 3; ++nc) {
      if (d % (16 * nc)) continue;
      const int g = d / (16 * nc);
      if (4 * g < sms || 2 * g > sms) continue;
      if (best == 0 || abs(split * g - sms) < abs(split * best - sms)) best = g;
    }
    if (best) {
      pl.grid = best;
      pl.nc = d / (16 * best);
    }
  }
  // Longer chunks that share the device: the smallest grid, down to a quarter of the SMs, that
  // still lets whole calls fill the SMs (a whole number of calls on one CTA per SM, whatever the
  // kernel ends up with) and keeps a CTA within three column tiles. Fewer, larger CTAs read x
  // and h less often; measured at d = 1536: 37 instead of 49 CTAs, 2.91 -> 2.76 us at 16 tokens,
  // 5.11 -> 4.70 at 32 (42 CTAs, three and a half calls: 5.46). At d = 2048 it stays 49.
  if (pl.ntg == 2 && split > 1) {
    const int step = pl.teams == 2 ? 1 : 2;
    for (int k = 8; k >= 2; k -= step) {
      const int g = (pl.teams == 2 ? sms : 2 * sms) / k;
      if (4 * g < sms) continue;
      const int nc = (d + 16 * g - 1) / (16 * g);
      if (nc > 3) continue;
      pl.grid = g;
      pl.nc = nc;
      break;
    }
  }
  pl.cols_q = d / pl.grid;
  pl.cols_rem = d % pl.grid;
  pl.max_cols = pl.cols_q + (pl.cols_rem ? 1 : 0);
  const int rows_exp = (u_exp * d_e + pl.grid - 1) / pl.grid;
  // an expert's slot in the down projection: its slab of D (columns split even / odd around
  // 64 bytes) and, with two teams, its h tile
  pl.slot_d = pl.max_cols * 2 * d_e + 64 + (pl.teams == 2 ? 8 * pl.ntg * pl.teams * 2 * d_e + 64 : 0);
  const int need = max(min(rows_exp, 32) * 2 * d + 64, min(u_exp, 16) * pl.slot_d);
  // the partial tile (and a stage) is as wide as the expected share, between one row tile per
  // column tile and two row tiles
  int red_rows = rows_exp < 32 ? rows_exp : 32;
  if (red_rows < 16 * pl.nc) red_rows = 16 * pl.nc;
  const int fixed = lean_layout(E, red_rows, pl.ntg * pl.teams, 0).total;
  // A call that owns the device gets the most CTAs per SM (three at most) whose shared memory
  // still holds the expected share in one stage; calls that share the device always run three
  // to an SM and stream their larger shares through in stages; chunks of more than 8 tokens
  // take a whole SM (their registers allow no more).
  for (int n = pl.teams == 2 ? 1 : pl.ntg == 2 ? 2 : 3; n >= 1; --n) {
    const int budget = (n == 1 ? kSmemMax : (kSmemMax + 1024) / n - 1024) & ~127;
    const int cap = (budget - fixed) & ~127;
    if (cap < need && n > 1 && split == 1) continue;
    if (cap < 2 * 4 * 2 * d + 128 || cap < 2 * pl.slot_d) {   // two stages of four rows, two slots
      if (n > 1) continue;
      if (cap < 2 * 2 * d + 128 || cap < 2 * pl.slot_d) return pl;
    }
    if (pl.ntg > 1 && cap < pl.teams * 8 * pl.ntg * red_ts(16 * pl.nc) * 4) {    // the final partials
      if (n > 1) continue;
      return pl;
    }
    // The hand-over inside the kernel needs every CTA of the call resident at once: n CTAs fit
    // an SM (by shared memory here, and the kernels are compiled for at least as many by
    // registers), so the call must not have more than n per SM.
    if (pl.grid > sms * n) return pl;
    pl.cap_bytes = cap;
    pl.red_rows = red_rows;
    pl.smem = lean_layout(E, red_rows, pl.ntg * pl.teams, cap).total;
    pl.ok = true;
    return pl;
  }
  return pl;
}

template <int KB, int NC, int NTG, int MODE, int TEAMS = 1>
cudaError_t lean_attr() {
  const void* f;
  if constexpr (NTG == 1)
    f = reinterpret_cast<const void*>(&expert_lean_kernel<KB, NC, MODE>);
  else
    f = reinterpret_cast<const void*>(&expert_wide_kernel<KB, NC, NTG, MODE, TEAMS>);
  cudaError_t e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(f, cudaFuncAttributePreferredSharedMemoryCarveout,
                              cudaSharedmemCarveoutMaxShared);
}
template <int KB, int NC>
cudaError_t lean_attrs_kb() {
  cudaError_t e = lean_attr<KB, NC, 1, 0>();
  if (e == cudaSuccess) e = lean_attr<KB, NC, 1, 1>();
  if (e == cudaSuccess) e = lean_attr<KB, NC, 1, 2>();
  if (e == cudaSuccess) e = lean_attr<KB, NC, 1, 3>();
  if (e == cudaSuccess) e = lean_attr<KB, NC, 2, 0>();
  if (e == cudaSuccess) e = lean_attr<KB, NC, 2, 1>();
  if (e == cudaSuccess) e = lean_attr<KB, NC, 2, 0, 2>();
  if (e == cudaSuccess) e = lean_attr<KB, NC, 2, 1, 2>();
  if (e == cudaSuccess) e = lean_attr<KB, NC, 2, 3>();
  if (e == cudaSuccess) e = lean_attr<KB, NC, 2, 3, 2>();
  return e;
}

template <int KB, int NC>
cudaError_t lean_launch_kb(const cudaLaunchConfig_t& lc, const LeanParams& p, int ntg, int teams,
                           int mode) {
  if (ntg == 1)
    return mode == 3   ? cudaLaunchKernelEx(&lc, expert_lean_kernel<KB, NC, 3>, p)
           : mode == 2 ? cudaLaunchKernelEx(&lc, expert_lean_kernel<KB, NC, 2>, p)
           : mode == 1 ? cudaLaunchKernelEx(&lc, expert_lean_kernel<KB, NC, 1>, p)
                       : cudaLaunchKernelEx(&lc, expert_lean_kernel<KB, NC, 0>, p);
  if (mode == 2) return cudaErrorNotSupported;
  if (teams == 2)
    return mode == 3   ? cudaLaunchKernelEx(&lc, expert_wide_kernel<KB, NC, 2, 3, 2>, p)
           : mode == 1 ? cudaLaunchKernelEx(&lc, expert_wide_kernel<KB, NC, 2, 1, 2>, p)
                       : cudaLaunchKernelEx(&lc, expert_wide_kernel<KB, NC, 2, 0, 2>, p);
  return mode == 3   ? cudaLaunchKernelEx(&lc, expert_wide_kernel<KB, NC, 2, 3, 1>, p)
         : mode == 1 ? cudaLaunchKernelEx(&lc, expert_wide_kernel<KB, NC, 2, 1, 1>, p)
                     : cudaLaunchKernelEx(&lc, expert_wide_kernel<KB, NC, 2, 0, 1>, p);
}
template <int NC>
cudaError_t lean_launch_nc(int kb, const cudaLaunchConfig_t& lc, const LeanParams& p, int ntg,
                           int teams, int mode) {
  switch (kb) {
    case 1: return lean_launch_kb<1, NC>(lc, p, ntg, teams, mode);
    case 2: return lean_launch_kb<2, NC>(lc, p, ntg, teams, mode);
    case 3: return lean_launch_kb<3, NC>(lc, p, ntg, teams, mode);
    default: return lean_launch_kb<4, NC>(lc, p, ntg, teams, mode);
  }
}

// (router inside the kernel) the logits of a chunk: f32 [L_max][E]; the logit rings follow the
// h rings in the workspace
size_t lean_logit_slot_bytes(const blockffn_config& cfg) {
  return ((size_t)cfg.L_max * cfg.E * sizeof(float) + 255) & ~(size_t)255;
}
size_t lean_h_slot_bytes(const blockffn_config& cfg) {
  return ((size_t)cfg.E * cfg.L_max * cfg.d_e * sizeof(uint16_t) + 255) & ~(size_t)255;
}

}  // namespace

// Whether a call of L tokens whose x is stable takes the one-kernel form (with_logits: it comes
// with raw router logits, i.e. it is the expert stage of a router-on layer call).
// (inside: the logits are computed in the kernel, which every chunk length can; logits from a
// router kernel are taken by the 8-token kernel only)
bool expert_lean_supported(const blockffn_ctx* c, int L, bool with_logits, bool shared, bool inside) {
  if (c->lean_ring == nullptr || (c->cfg.flags & BLOCKFFN_CFG_TWO_KERNELS)) return false;
  if (with_logits && !inside && L > 8) return false;
  return lean_plan(c->cfg, L, c->num_sms, shared).ok;
}

// Four rings (calls that own the device; calls that share it with up to 8, up to 16, up to 32
// tokens: their grids differ, so each kind counts its own tickets) of kHRing intermediates of a
// chunk of L_max tokens; 0 when the shape never takes this kernel (or the rings would be
// unreasonably large).
size_t expert_lean_ws_bytes(const blockffn_config* cfg, int sms) {
  const int L = cfg->L_max < 8 ? cfg->L_max : 8;
  if (!lean_plan(*cfg, L, sms, false).ok || !lean_plan(*cfg, L, sms, true).ok) return 0;
  const size_t slot = lean_h_slot_bytes(*cfg) + lean_logit_slot_bytes(*cfg);
  if (kRings * kHRing * slot > ((size_t)256 << 20)) return 0;
  return kRings * kHRing * slot;
}

cudaError_t expert_lean_setup(blockffn_ctx* c) {
  (void)c;
  cudaError_t e = lean_attrs_kb<1, 1>();
  if (e == cudaSuccess) e = lean_attrs_kb<2, 1>();
  if (e == cudaSuccess) e = lean_attrs_kb<3, 1>();
  if (e == cudaSuccess) e = lean_attrs_kb<4, 1>();
  if (e == cudaSuccess) e = lean_attrs_kb<1, 2>();
  if (e == cudaSuccess) e = lean_attrs_kb<2, 2>();
  if (e == cudaSuccess) e = lean_attrs_kb<3, 2>();
  if (e == cudaSuccess) e = lean_attrs_kb<4, 2>();
  if (e == cudaSuccess) e = lean_attrs_kb<1, 3>();
  if (e == cudaSuccess) e = lean_attrs_kb<2, 3>();
  if (e == cudaSuccess) e = lean_attrs_kb<3, 3>();
  if (e == cudaSuccess) e = lean_attrs_kb<4, 3>();
  return e;
}

cudaError_t launch_expert_lean(blockffn_ctx* c, const blockffn_weights* w, const void* x,
                               const float* scores, int L, const int32_t* union_ids,
                               const int32_t* n_union, float* out, void* x_next, int call_flags,
                               const RoutingOut* pub, const RouterLogits* logits, bool logits_final,
                               cudaStream_t st) {
  // For calls whose x is stable (for a router-on call: whose router has finished), and for
  // chunks of more than 8 tokens in a dependent chain (weights and scores stable, x from the
  // call before): those wait for their predecessor before they read x.
  // A router-on call of up to 8 tokens whose router runs inside the kernel (logits->a0 == NULL)
  // may be dependent as well, with or without promises: it waits before it reads anything.
  const bool inside = logits && logits->a0 == nullptr;
  const bool x_stable = logits ? logits_final : (call_flags & BLOCKFFN_CALL_INDEPENDENT_X) != 0;
  const bool dep = !x_stable &&
                   (inside || (!logits && (call_flags & BLOCKFFN_CALL_INDEPENDENT) && L > 8));
  if (!x_stable && !dep) return cudaErrorNotSupported;
  // Nothing consumed from its predecessors: the call shares the device with them (a router-on
  // call is ordered behind its own router by an event, and the routers run far enough ahead on
  // streams of the handle's own); a dependent call runs alone anyway.
  const bool shared = x_stable;
  if (!expert_lean_supported(c, L, logits != nullptr, shared, inside)) return cudaErrorNotSupported;
  const LeanPlan pl = lean_plan(c->cfg, L, c->num_sms, shared);
  if (!pl.ok) return cudaErrorNotSupported;
  LeanParams p{};
  p.x = static_cast<const uint16_t*>(x);
  p.U = static_cast<const uint16_t*>(w->U);
  p.D = static_cast<const uint16_t*>(w->D);
  p.scores = scores;
  if (logits) p.lg = *logits;
  const bool router_inside = inside;
  if (router_inside && !w->W_r) return cudaErrorNotSupported;
  p.W_r = static_cast<const uint16_t*>(w->W_r);
  p.bias = w->bias;
  p.ids_in = union_ids;
  p.n_in = n_union;
  p.h_slot = lean_h_slot_bytes(c->cfg) / 2;
  // a ring and a ticket counter per kind of call: tickets only identify a call when every call
  // that draws from the counter has the same number of CTAs
  const int ring = !shared ? 0 : L <= 8 ? 1 : L <= 16 ? 2 : 3;
  p.h_ring = static_cast<uint16_t*>(c->lean_ring) + (size_t)ring * kHRing * p.h_slot;
  p.seq = c->lean_seq + 64 * ring;
  p.ready = p.seq + 1;
  p.ready2 = p.seq + 1 + kHRing;
  p.logit_slot = lean_logit_slot_bytes(c->cfg) / sizeof(float);
  p.logit_ring = reinterpret_cast<float*>(static_cast<char*>(c->lean_ring) +
                                          kRings * kHRing * lean_h_slot_bytes(c->cfg)) +
                 (size_t)ring * kHRing * p.logit_slot;
  p.out = out;
  p.x_next = static_cast<uint16_t*>(x_next);
  p.L = L;
  p.d = c->cfg.d;
  p.E = c->cfg.E;
  p.d_e = c->cfg.d_e;
  p.de_shift = __builtin_ctz(c->cfg.d_e);
  p.cap_bytes = pl.cap_bytes;
  p.red_rows = pl.red_rows;
  p.cap_rows = (pl.cap_bytes - 256) / (2 * c->cfg.d);     // up to three stages, 64 bytes of padding each
  if (p.cap_rows > 96) p.cap_rows = 96;
  p.cap_slabs = pl.cap_bytes / pl.slot_d;
  p.magic_g = (uint32_t)((0x100000000ull + (unsigned)pl.grid - 1) / (unsigned)pl.grid);
  p.magic_cpr = (uint32_t)((0x10000u + (unsigned)(c->cfg.d / 8) - 1) / (unsigned)(c->cfg.d / 8));
  p.max_cols = pl.max_cols;
  p.cols_q = pl.cols_q;
  p.cols_rem = pl.cols_rem;
  p.accumulate = (call_flags & BLOCKFFN_CALL_ACCUMULATE) ? 1 : 0;
  p.dep = dep ? 1 : 0;
  p.hold = (c->cfg.flags & BLOCKFFN_CFG_TEST_EXPIRE_WAIT) ? 1 : 0;
  p.wait_ns = 1000000000ull;      // one second
  p.status = c->status;
  if (pub) {
    p.pub_mask = pub->union_mask;
    p.pub_ids = pub->union_ids;
    p.pub_n = pub->n_union;
    p.stats = pub->stats;
    p.pub_scores = pub->scores;
    p.pub_tok = pub->tok_mask;
  }
  const bool chained = !(c->cfg.flags & BLOCKFFN_CFG_NO_CHAINING);
  const int mode = router_inside ? 3 : logits ? 2 : union_ids ? 1 : 0;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t lc{};
  lc.gridDim = dim3(pl.grid);
  lc.blockDim = dim3(kThreads * pl.teams);
  lc.stream = st;
  lc.attrs = attr;
  lc.numAttrs = chained ? 1 : 0;
  // never less than a quarter of an SM's shared memory: at most three CTAs then fit one SM,
  // whatever the shape, which is what the size of the ring rests on
  lc.dynamicSmemBytes = pl.smem > kMinSmem ? pl.smem : kMinSmem;
  const cudaError_t e = pl.nc == 3   ? lean_launch_nc<3>(pl.kb, lc, p, pl.ntg, pl.teams, mode)
                        : pl.nc == 2 ? lean_launch_nc<2>(pl.kb, lc, p, pl.ntg, pl.teams, mode)
                                     : lean_launch_nc<1>(pl.kb, lc, p, pl.ntg, pl.teams, mode);
  if (e == cudaSuccess) c->launches += 1;
  return e;
}
