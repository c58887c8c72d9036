// Expert stage (Eq. 1, Eq. 2 restricted to Union(x), Sec. 3.3): asynchronously staged,
// tensor-core variant.
//
// Two kernels per call, one CTA per SM each, chained by programmatic dependent
// launch so that the weight fetch of a kernel overlaps the tail of the one before:
//
//   expert_up_mma    CTA b owns an equal share of the union's neuron rows (u * d_e
//                    rows of U, d contiguous bf16 each). All 256 threads gather the
//                    share into shared memory with 16-byte asynchronous copies
//                    (cp.async, L2 only), a few rows per stage; the eight warps split K,
//                    multiply a stage of up to 16
//                    rows with all L tokens on mma.sync m16n8k16 (weights are the M
//                    operand, tokens the N operand), reduce across warps, apply Swish
//                    and the token's router score and store the bf16 intermediate
//                    h[q][t][j] to the handle's workspace.
//   expert_down_mma  CTA b owns a block of <= 16 output columns. For every union expert
//                    it stages the contiguous [columns x d_e] slab of D and the expert's
//                    h rows, accumulates out[t][c] over all experts on the tensor cores
//                    and writes each output element exactly once (no atomics; results
//                    are run-to-run identical).
//
// The D slabs (and, for calls flagged independent, the U rows) are requested before
// griddepcontrol.wait, i.e. while the previous kernel is still running; everything a
// previous kernel may have produced (x, h, out) is touched only after it.
//
// Why cp.async and not bulk (TMA) copies: the pieces are small (a D slab is
// columns * 2 d_e bytes, 3.5 KB at d = 2048) and a bulk copy costs its issuing thread a
// few hundred nanoseconds whatever its size, which measured 0.56 / 2.2 / 7.0 TB/s device
// wide for 1 / 4 / 16 KB pieces; 16-byte cp.async from 256 threads with 64 KB in flight
// per SM measured 7.2 TB/s.
//
// Fragments: the k index of each 64-wide block is permuted identically for both mma
// operands (lane tg owns 8 consecutive k of each 32-wide half), so a fragment is a
// 128-bit shared-memory load; rows are staged unpadded (row strides are multiples of
// 128 bytes) and lanes of odd rows read the two halves in the opposite order, which
// keeps every quarter-warp on 32 distinct banks.
// Completion is tracked with cp.async commit groups and CTA barriers only: no thread ever
// spins on memory, so nothing here can wait forever.
#include "mma_tiles.cuh"

namespace {

// ---- up projection ---------------------------------------------------------------
struct UpParams {
  const uint16_t* x;       // bf16 [L][d]
  const uint16_t* U;       // bf16 [E][d_e][d]
  const float* scores;     // f32 [L][E] (unused when lg.a0 is set)
  RouterLogits lg;         // raw router logits to finish here, or a0 == NULL
  const int32_t* ids_in;   // caller's union list, or NULL: derive from scores / logits
  const int32_t* n_in;
  uint16_t* h;             // bf16 [q][L][d_e] intermediate
  int L, d, E, d_e, de_shift, ring_rows;   // de_shift: log2(d_e)
  uint32_t* status;
  // what CTA 0 publishes when it derived the union itself (each may be NULL)
  uint32_t* pub_mask;
  int32_t* pub_ids;
  int32_t* pub_n;
  blockffn_stats* stats;
  float* pub_scores;       // logits mode only
  uint32_t* pub_tok;
};

// Chunks longer than 8 tokens go through the math in groups of 8 tokens (one mma n tile): the
// weights stay in shared memory, the x tile of the next group replaces the current one. That
// keeps the kernel within half an SM's shared memory for every L, which is what lets it run
// next to the down kernel of the call before.
// MULTI: the chunk has more than one token group (L > 8)
// EARLY: 0 wait first; 1 routing inputs and weights before the wait; 2 x as well
template <bool MULTI, int MODE, int EARLY>
__global__ void __launch_bounds__(kThreads, 2) expert_up_mma_kernel(const UpParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int NT = 1;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int d = p.d, d_e = p.d_e, L = p.L;
  constexpr int ns = kUpStages;
  const UpLayout lay = up_layout(d, p.E, p.ring_rows);
  const uint32_t sbase = smem_u32(smem);
  int* ctl = reinterpret_cast<int*>(smem + kOffCtl);
  int* ids_sm = reinterpret_cast<int*>(smem + kOffIds);
  float* red = reinterpret_cast<float*>(smem + lay.off_red);
  const int row_bytes = 2 * d;
  const int ntg = MULTI ? (L + 7) >> 3 : 1;   // token groups

  if (tid < 8) ctl[tid] = 0;
  if constexpr (EARLY != 0) {
    pdl_trigger();       // the next kernel may start fetching its weights right away
  } else {
    if constexpr (MODE == 2) {   // the gains are weights: have them in L2 when the wait is over
      if (tid * 32 < p.E) asm volatile("prefetch.global.L2 [%0];" ::"l"(p.lg.gain + tid * 32));
    }
    pdl_wait();          // scores / ids may come from the kernel just before
    pdl_trigger();
  }
  __syncthreads();
  const int nu = derive_union<MODE>(p.scores, p.lg, p.ids_in, p.n_in, L, p.E, ids_sm, ctl,
                              reinterpret_cast<uint32_t*>(red));

  // This CTA's rows [r0, r1) of the u * d_e union rows (balanced: the first R % G CTAs take
  // one row more). They are one stage when they fit the ring (the usual case), else stages
  // of a third of the ring that are refilled as they free.
  const int R = nu * d_e, G = gridDim.x, bx = blockIdx.x;
  const int rq = R / G, rrem = R - rq * G;
  const int r0 = bx * rq + min(bx, rrem), nrows = rq + (bx < rrem ? 1 : 0), r1 = r0 + nrows;
  const bool single = nrows <= min(32, p.ring_rows);
  const int slot_rows = single ? max(nrows, 1) : min(32, p.ring_rows / ns);
  const int ngroups = (nrows + slot_rows - 1) / slot_rows;
  const int rpg = ngroups ? (nrows + ngroups - 1) / ngroups : 0;
  const int slot_bytes = slot_rows * row_bytes;
  const int sh = p.de_shift;
  auto row_q = [&](int r) { return r >> sh; };   // d_e is a power of two

  // stage gi: rows [r0 + gi rpg, ...) -> slot gi % ns; one run per expert the rows fall in
  auto issue = [&](int gi) {
    int ra = r0 + gi * rpg;
    const int rb = min(r1, ra + rpg);
    uint32_t dst = sbase + lay.off_ring + (gi % ns) * slot_bytes;
    int q = row_q(ra), j = ra - q * d_e;
    while (ra < rb) {
      const int n = min(rb - ra, d_e - j);
      copy_run(dst, p.U + ((size_t)ids_sm[q] * d_e + j) * d, n * row_bytes);
      dst += n * row_bytes;
      ra += n;
      ++q;
      j = 0;
    }
  };
  // x tile of token group tgi: tokens [8 tgi, 8 tgi + 8) of the chunk
  auto issue_x = [&](int tgi) {
    const int nt = min(8, L - 8 * tgi);
    copy_run(sbase + lay.off_x, p.x + (size_t)8 * tgi * d, nt * row_bytes);
  };
  // The router score, expert slot and neuron of the element this thread finishes in a pass
  // (element e = t * 32 + m: token t of the group, row m of the stage).
  float sc = 0.0f;
  int hq = -1, hj = 0;
  uint16_t held[4] = {0, 0, 0, 0};
  auto prepare = [&](int gi, int tgi) {
    const int ra = r0 + gi * rpg, rows = min(r1, ra + rpg) - ra;
    const int t = 8 * tgi + (tid >> 5), m = tid & 31;
    sc = 0.0f;
    hq = -1;
    if (m < rows) {          // the row is this thread's for every token group of the stage
      hq = row_q(ra + m);
      hj = ra + m - hq * d_e;
    }
    if (t < L && m < rows) {
      const int id = ids_sm[hq];
      if constexpr (MODE == 2) {     // gain * ReLU(logit) / rms, as in derive_union
        float v = __ldcg(p.lg.a0 + (size_t)t * p.E + id);
        v = v > 0.0f ? v : 0.0f;
        sc = __ldg(p.lg.gain + id) * v * reinterpret_cast<const float*>(ctl + 104)[t];
      } else {
        sc = __ldcg(p.scores + (size_t)t * p.E + id);
      }
    }
  };
  const int g = lane >> 2, tg = lane & 3, par = g & 1;
  const int npairs = d >> 6;   // 64-wide k blocks

  const int g_first = min(ngroups, ns);
  // DEEP (one token group, x not later than the weights): every stage is a commit group of its
  // own, x rides with the first, and a pass waits for its own stage only, so that up to
  // ns - 1 later stages stay in flight under its math. Otherwise the first pass waits for
  // everything requested so far and later passes for all but the newest group.
  constexpr bool DEEP = !MULTI && EARLY != 1;
  if constexpr (DEEP) {
    if constexpr (EARLY == 0) pdl_wait();   // x may come from the kernel just before
    if (ngroups > 0) {
      issue_x(0);
      issue(0);
    }
    cp_async_commit();
    for (int gi = 1; gi < g_first; ++gi) {
      issue(gi);
      cp_async_commit();
    }
    if (ngroups > 0) prepare(0, 0);
  } else {
    // (x, when it is stable, goes first: its short round trip then runs under the long issue
    // of the weights instead of behind it)
    if constexpr (EARLY == 2) {
      if (ngroups > 0) issue_x(0);
    }
    if constexpr (EARLY != 0) {
      for (int gi = 0; gi < g_first; ++gi) issue(gi);
      if (ngroups > 0) prepare(0, 0);
    }
    if constexpr (EARLY < 2) pdl_wait();   // x may come from the kernel just before
    if constexpr (EARLY < 2) {
      if (ngroups > 0) issue_x(0);
    }
    if constexpr (EARLY == 0) {
      for (int gi = 0; gi < g_first; ++gi) issue(gi);
      if (ngroups > 0) prepare(0, 0);
    }
    cp_async_commit();
  }

  for (int gi = 0; gi < ngroups; ++gi) {
    const int rows = min(r1, r0 + (gi + 1) * rpg) - (r0 + gi * rpg);
    const unsigned char* slot = smem + lay.off_ring + (gi % ns) * slot_bytes;
    const bool two = rows > 16;   // second block of 16 rows
    const unsigned char* ra0 = slot + min(g, rows - 1) * row_bytes;
    const unsigned char* rb0 = slot + min(g + 8, rows - 1) * row_bytes;
    const unsigned char* ra1 = slot + min(g + 16, rows - 1) * row_bytes;
    const unsigned char* rb1 = slot + min(g + 24, rows - 1) * row_bytes;
    for (int tgi = 0; tgi < ntg; ++tgi) {
      const int nt = min(8, L - 8 * tgi);
      const unsigned char* x_row = smem + lay.off_x + min(g, nt - 1) * row_bytes;
      // Every pass ends with two commit groups: the next x tile, then the refill of a ring slot
      // (either may be empty). The refill is only needed stages later, so all but the newest
      // group have to have landed; the very first pass waits for everything requested so far.
      if constexpr (DEEP) {
        // one group per stage and per pass: all but the g_first - 1 newest have to have landed
        if (g_first >= 3) cp_async_wait_group<2>();
        else if (g_first == 2) cp_async_wait_group<1>();
        else cp_async_wait_group<0>();
      } else {
        if (gi == 0 && tgi == 0) cp_async_wait_group<0>(); else cp_async_wait_group<1>();
      }
      __syncthreads();
      float a00[NT][4], a01[NT][4], a10[NT][4], a11[NT][4];
      zero_acc<NT>(a00);
      zero_acc<NT>(a01);
      zero_acc<NT>(a10);
      zero_acc<NT>(a11);
#pragma unroll 1
      for (int pp = warp; pp < npairs; pp += kWarps) {
        Frag64 fx[NT];
        fx[0] = load_frag64(x_row + 128 * pp, par, tg);
        const Frag64 fa = load_frag64(ra0 + 128 * pp, par, tg);
        const Frag64 fb = load_frag64(rb0 + 128 * pp, par, tg);
        mma_block64<NT>(a00, a01, fa, fb, fx);
        if (two) {
          const Frag64 fc = load_frag64(ra1 + 128 * pp, par, tg);
          const Frag64 fd = load_frag64(rb1 + 128 * pp, par, tg);
          mma_block64<NT>(a10, a11, fc, fd, fx);
        }
      }
      // cross-warp reduction of the K split, then Swish, score, store
      float* mine = red + warp * (32 * 8);
      store_partial<NT>(mine, 32, 0, a00, a01, g, tg);
      if (two) store_partial<NT>(mine, 32, 16, a10, a11, g, tg);
      __syncthreads();     // every warp is done with the x tile (and, after the last group, the slot)
      const bool last_tg = tgi + 1 == ntg;
      if constexpr (!DEEP) {
        if (!last_tg) issue_x(tgi + 1);
        else if (gi + 1 < ngroups && ntg > 1) issue_x(0);
        cp_async_commit();
      }
      if (last_tg && gi + ns < ngroups) issue(gi + ns);
      cp_async_commit();
      // h may still be read by the down kernel of the call before: when this kernel runs ahead
      // of it (early == 2), the first stage keeps its results in registers until all its token
      // groups are done, so that all of that math happens before the wait.
      const bool hold = MULTI && EARLY == 2 && gi == 0;
      if (!MULTI && EARLY == 2 && gi == 0) pdl_wait();
      uint16_t hval = 0;
      const bool tok_ok = 8 * tgi + (tid >> 5) < L;
      if (hq >= 0 && tok_ok) {
        float v = 0.0f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) v += red[w * (32 * 8) + tid];
        hval = (uint16_t)f32_to_bf16_bits(sc * swish_fast(v));
      }
      if (hold) {
        if (tgi == 0) held[0] = hval;
        else if (tgi == 1) held[1] = hval;
        else if (tgi == 2) held[2] = hval;
        else held[3] = hval;
        if (last_tg) {
          pdl_wait();
          if (hq >= 0) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
              if (i < ntg && 8 * i + (tid >> 5) < L)
                p.h[((size_t)hq * L + 8 * i + (tid >> 5)) * d_e + hj] = held[i];
          }
        }
      } else if (hq >= 0 && tok_ok) {
        p.h[((size_t)hq * L + 8 * tgi + (tid >> 5)) * d_e + hj] = hval;
      }
      if (!last_tg) prepare(gi, tgi + 1);
      else if (gi + 1 < ngroups) prepare(gi + 1, 0);
      // the next pass starts with a wait and a barrier, which also protects red
    }
  }
  if (EARLY == 2 && ngroups == 0) pdl_wait();   // every kernel waits before it ends
  // CTA 0 publishes the routing it derived (after the wait: earlier readers are done)
  if (blockIdx.x == 0) {
    if (p.lg.a0 != nullptr && p.pub_scores != nullptr) {   // the scores and masks it computed
      const int words = (p.E + 31) >> 5;
      const float* rinv = reinterpret_cast<const float*>(ctl + 104);
      for (int t = warp; t < L; t += kWarps) {
        for (int w = 0; w < words; ++w) {
          const int e = 32 * w + lane;
          float sv = 0.0f;
          if (e < p.E) {
            float v = __ldcg(p.lg.a0 + (size_t)t * p.E + e);
            v = v > 0.0f ? v : 0.0f;
            sv = __ldg(p.lg.gain + e) * v * rinv[t];
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
  cp_async_wait_all();
}

// ---- down projection ---------------------------------------------------------------
struct DownParams {
  const uint16_t* D;       // bf16 [E][d][d_e]
  const uint16_t* h;       // bf16 [q][L][d_e]
  const float* scores;
  RouterLogits lg;
  const int32_t* ids_in;
  const int32_t* n_in;
  float* out;              // f32 [L][d]
  uint16_t* x_next;        // bf16 [L][d] or NULL
  int L, d, E, d_e, ns, max_cols, per, accumulate;
  int cols_q, cols_rem;    // the d columns over G * per tiles: tile w has cols_q + (w < cols_rem)
  uint32_t* status;
};

// NTG: token groups of 8 in the chunk (1 .. 4), each with its own accumulators
template <int NTG, int MODE>
__global__ void __launch_bounds__(kThreads, 2) expert_down_mma_kernel(const DownParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int NT = 1;
  constexpr int kMaxTg = NTG;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int d = p.d, d_e = p.d_e, L = p.L, per = p.per;
  const DownLayout lay = down_layout(d_e, p.E, p.ns, p.max_cols);
  const uint32_t sbase = smem_u32(smem);
  int* ctl = reinterpret_cast<int*>(smem + kOffCtl);
  int* ids_sm = reinterpret_cast<int*>(smem + kOffIds);
  float* red = reinterpret_cast<float*>(smem + lay.off_red);
  const int row_bytes = 2 * d_e;
  constexpr int ntg = NTG;

  if (tid < 8) ctl[tid] = 0;
  pdl_trigger();
  __syncthreads();
  // The routing inputs were final before the up kernel of this call passed its own wait.
  const int nu = derive_union<MODE>(p.scores, p.lg, p.ids_in, p.n_in, L, p.E, ids_sm, ctl,
                              reinterpret_cast<uint32_t*>(red));

  // Column tiles: G * per tiles of at most max_cols (<= 16) columns, tile w -> CTA w % G,
  // tile w = columns [w cols_q + min(w, cols_rem), ...). Per tile, the experts go through
  // the ring in rounds: all of them at once when they fit (the usual case), else half a
  // ring per round, the next round in flight during the math. Within a round the chunk's
  // tokens go through the math in groups of 8, each with its own h tile and accumulators.
  const int G = gridDim.x;
  const int rsz = (per == 1 && nu <= p.ns) ? max(nu, 1) : max(1, min(nu, p.ns / 2));
  const int rpt = (nu + rsz - 1) / rsz;                  // rounds per tile
  const int nrounds = per * rpt;
  const char* dptr = reinterpret_cast<const char*>(p.D);
  const size_t estride = (size_t)d * d_e * 2;
  const char* hptr = reinterpret_cast<const char*>(p.h);
  auto tile_c0 = [&](int ti) {
    const int w = blockIdx.x + ti * G;
    return w * p.cols_q + min(w, p.cols_rem);
  };
  auto tile_nc = [&](int ti) { return p.cols_q + ((int)blockIdx.x + ti * G < p.cols_rem ? 1 : 0); };
  int i_r = 0, i_ti = 0, i_rr = 0;      // the next round to request: index, tile, round in tile
  auto issue_d = [&]() {
    const int q0 = i_rr * rsz, n = min(rsz, nu - q0);
    const char* base = dptr + (size_t)tile_c0(i_ti) * row_bytes;
    copy_pieces(sbase + lay.off_d + (i_r & 1) * rsz * lay.slot_d, lay.slot_d, n,
                tile_nc(i_ti) * row_bytes,
                [&](int i) { return base + (size_t)ids_sm[q0 + i] * estride; });
    ++i_r;
    if (++i_rr == rpt) {
      i_rr = 0;
      ++i_ti;
    }
  };
  // h tile of (round-in-tile rr, token group tgi): tokens [8 tgi, ..) of the round's experts
  // (a chunk of at most 8 tokens has one group, and its tiles are one run in memory: they are
  // kept at the chunk's own stride so that all threads share one long copy)
  const int hstride = ntg == 1 ? L * row_bytes : lay.slot_h;
  auto issue_h = [&](int rr, int tgi) {
    const int q0 = rr * rsz, n = min(rsz, nu - q0), nt = min(8, L - 8 * tgi);
    const char* base = hptr + ((size_t)q0 * L + 8 * tgi) * row_bytes;
    if (ntg == 1) {
      copy_run(sbase + lay.off_h, base, n * hstride);
    } else {
      const size_t qstride = (size_t)L * row_bytes;
      copy_pieces(sbase + lay.off_h, hstride, n, nt * row_bytes,
                  [&](int i) { return base + (size_t)i * qstride; });
    }
  };
  const int g = lane >> 2, tg = lane & 3, par = g & 1;
  const int npairs = d_e >> 6;         // 64-wide k blocks per expert
  const int pshift = __ffs(npairs) - 1;   // d_e, hence npairs, is a power of two

  // before the wait: the weights of the first two rounds
  const int npre = min(nrounds, 2);
  for (int r = 0; r < npre; ++r) {
    issue_d();
    cp_async_commit();
  }
  pdl_wait();            // h, out and x_next are safe to touch from here on
  if (nrounds > 0) {
    issue_h(0, 0);
    cp_async_commit();
  }
  // the residual the first tile's first token group is added to: asked for now, used in the
  // epilogue (one memory round trip off the tail of the kernel)
  float resid = 0.0f;
  if (p.accumulate && tid < 128) {
    const int t = tid >> 4, m = tid & 15;
    if (t < L && m < tile_nc(0)) resid = __ldcg(p.out + (size_t)t * d + tile_c0(0) + m);
  }

  float acc0[kMaxTg][4], acc1[kMaxTg][4];
  int c_ti = 0, c_rr = 0;
  for (int r = 0; r < nrounds; ++r) {
    const int q0 = c_rr * rsz, n = min(rsz, nu - q0);
    const int c0 = tile_c0(c_ti), ncols = tile_nc(c_ti);
    const int off_a = min(g, max(ncols, 1) - 1) * row_bytes;
    const int off_b = min(g + 8, max(ncols, 1) - 1) * row_bytes;
    const unsigned char* d_base = smem + lay.off_d + (r & 1) * rsz * lay.slot_d;
    const unsigned char* h_base = smem + lay.off_h;
    const int nblk = n * npairs;
    if (c_rr == 0) {
      zero_acc<kMaxTg>(acc0);
      zero_acc<kMaxTg>(acc1);
    }
#pragma unroll
    for (int tgi = 0; tgi < kMaxTg; ++tgi) {
      if (tgi < ntg) {
        const int nt = min(8, L - 8 * tgi);
        const int h_off = min(g, nt - 1) * row_bytes;
        // Every pass ends with two commit groups: the next h tile, then the refill of half
        // the D ring (either may be empty). The refill is only needed two rounds later, so all
        // but the newest group have to have landed; the first pass waits for everything.
        if (r == 0 && tgi == 0) cp_async_wait_group<0>(); else cp_async_wait_group<1>();
        __syncthreads();
        if (ncols > 0) {
          // the 64-wide k blocks of the round's experts are dealt round-robin to the warps
#pragma unroll 1
          for (int b = warp; b < nblk; b += kWarps) {
            const int i = b >> pshift, pp = b - i * npairs;
            const unsigned char* da = d_base + i * lay.slot_d + 128 * pp;
            const unsigned char* ha = h_base + i * hstride + 128 * pp;
            const Frag64 fa = load_frag64(da + off_a, par, tg);
            const Frag64 fb = load_frag64(da + off_b, par, tg);
            Frag64 fx[NT];
            fx[0] = load_frag64(ha + h_off, par, tg);
            float (&b0)[1][4] = reinterpret_cast<float (&)[1][4]>(acc0[tgi]);
            float (&b1)[1][4] = reinterpret_cast<float (&)[1][4]>(acc1[tgi]);
            mma_block64<NT>(b0, b1, fa, fb, fx);
          }
        }
        const bool last_tg = tgi + 1 == ntg;
        if (!last_tg || r + 1 < nrounds) {   // more to fetch into what this pass has read
          __syncthreads();   // every warp is done with the h tile (and, after the last group, the slabs)
          if (!last_tg) issue_h(c_rr, tgi + 1);
          else issue_h(c_rr + 1 == rpt ? 0 : c_rr + 1, 0);
          cp_async_commit();
          if (last_tg && r + 2 < nrounds) issue_d();        // refill this round's half of the ring
          cp_async_commit();
        }
      }
    }
    if (c_rr == rpt - 1) {       // the tile is complete: reduce across warps and store
#pragma unroll
      for (int tgi = 0; tgi < kMaxTg; ++tgi) {
        if (tgi < ntg) {
          float (&b0)[1][4] = reinterpret_cast<float (&)[1][4]>(acc0[tgi]);
          float (&b1)[1][4] = reinterpret_cast<float (&)[1][4]>(acc1[tgi]);
          store_partial<NT>(red + warp * 128, 16, 0, b0, b1, g, tg);
          __syncthreads();
          if (tid < 128) {
            const int t = 8 * tgi + (tid >> 4), m = tid & 15;
            if (t < L && m < ncols) {
              float v = 0.0f;
#pragma unroll
              for (int w = 0; w < kWarps; ++w) v += red[w * 128 + tid];
              const size_t o = (size_t)t * d + c0 + m;
              if (p.accumulate) v += (c_ti == 0 && tgi == 0) ? resid : __ldcg(p.out + o);
              p.out[o] = v;
              if (p.x_next) p.x_next[o] = (uint16_t)f32_to_bf16_bits(v);
            }
          }
          __syncthreads();
        }
      }
    }
    if (++c_rr == rpt) {
      c_rr = 0;
      ++c_ti;
    }
  }
  if (nu == 0) {               // empty union: FFN(x) = 0
    for (int ti = 0; ti < per; ++ti) {
      const int c0 = tile_c0(ti), ncols = tile_nc(ti);
      for (int e = tid; e < L * ncols; e += kThreads) {
        const int t = e / ncols, m = e - t * ncols;
        const size_t o = (size_t)t * d + c0 + m;
        const float v = p.accumulate ? __ldcg(p.out + o) : 0.0f;
        p.out[o] = v;
        if (p.x_next) p.x_next[o] = (uint16_t)f32_to_bf16_bits(v);
      }
    }
  }
  cp_async_wait_all();
}

// ---- host side -----------------------------------------------------------------------
struct MmaPlan {
  int ring_rows, ns_down, max_cols, per, cols_q, cols_rem, smem_up, smem_down;
  bool ok;
};

// Shapes the kernels take: d a multiple of 64 and d_e a power of two >= 64 (whole 64-wide k
// blocks, row strides multiples of 128 bytes, shifts instead of divisions) and, within half an SM's shared memory, an x tile plus a few rows
// of U (up) and a few expert slabs with their h tiles (down).
MmaPlan make_plan(const blockffn_config& cfg, int L, int grid) {
  MmaPlan pl{};
  pl.ok = false;
  const int d = cfg.d, d_e = cfg.d_e, E = cfg.E;
  if (L < 1 || L > 32 || grid < 1) return pl;
  if (d % 64 || d_e % 64 || (d_e & (d_e - 1)) || E > 1024 || d > 32768 || d_e > 4096) return pl;
  const int want_up = cfg.flags & 0xff, want_down = (cfg.flags >> 8) & 0xff;
  // down: column tiles
  pl.per = (d + 16 * grid - 1) / (16 * grid);
  const int W = grid * pl.per;
  pl.cols_q = d / W;
  pl.cols_rem = d % W;
  pl.max_cols = pl.cols_q + (pl.cols_rem ? 1 : 0);
  const int up_base = up_layout(d, E, 0).total;
  const int down_base = down_layout(d_e, E, 0, pl.max_cols).total;
  const int slot_dn = 8 * 2 * d_e + pl.max_cols * 2 * d_e;
  // Paired: an up and a down CTA share an SM (half its shared memory each), so that consecutive
  // launches overlap. That pays as long as the share of the union a CTA works on fits the half:
  // otherwise each kernel goes through many short stages, and a whole SM per kernel (fewer,
  // larger stages, no overlap) is faster. The union is not known at launch time, so the choice
  // follows the caller's hint, or else the paper's sparsity: 30 % of the experts for a chunk,
  // 12.5 % for a single token.
  int u_exp = (cfg.flags >> 17) & 0x7ff;
  if (u_exp == 0) u_exp = (L == 1 ? E + 4 : 3 * E + 5) / (L == 1 ? 8 : 10);
  if (u_exp < 1) u_exp = 1;
  if (u_exp > E) u_exp = E;
  const int rows_exp = (u_exp * d_e + grid - 1) / grid;
  const int half_rows = (kSmemHalf - up_base) / (2 * d);
  const int half_slots = (kSmemHalf - down_base - 128) / slot_dn;
  const bool fits_half = up_base + 12 * 2 * d <= kSmemHalf && down_base + 4 * slot_dn <= kSmemHalf;
  const bool paired = fits_half && rows_exp <= half_rows && u_exp <= half_slots;
  const int budget = paired ? kSmemHalf : kSmemMax;
  pl.ring_rows = (budget - up_base) / (2 * d);
  if (want_up && want_up < pl.ring_rows) pl.ring_rows = want_up;
  if (pl.ring_rows > 96) pl.ring_rows = 96;
  if (pl.ring_rows < kUpStages) return pl;
  pl.ns_down = (budget - down_base - 128) / slot_dn;
  if (want_down) pl.ns_down = want_down;
  if (pl.ns_down > kMaxStages) pl.ns_down = kMaxStages;
  if (pl.ns_down > E) pl.ns_down = E < 2 ? 2 : E;
  if (pl.ns_down < 2) return pl;
  pl.smem_up = up_layout(d, E, pl.ring_rows).total;
  pl.smem_down = down_layout(d_e, E, pl.ns_down, pl.max_cols).total;
  if (pl.smem_up > kSmemMax || pl.smem_down > kSmemMax) return pl;
  pl.ok = true;
  return pl;
}

// Both kernels ask for the largest shared-memory carve-out: an SM keeps its carve-out while
// any CTA runs on it, so a down CTA can only join an up CTA (and the next call's up CTA the
// down CTA) if the first of them already configured the SM for both.
cudaError_t set_one(const void* f) {
  cudaError_t e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(f, cudaFuncAttributePreferredSharedMemoryCarveout,
                              cudaSharedmemCarveoutMaxShared);
}

template <int MODE, int EARLY>
cudaError_t set_attrs_up() {
  cudaError_t e = set_one(reinterpret_cast<const void*>(&expert_up_mma_kernel<false, MODE, EARLY>));
  if (e != cudaSuccess) return e;
  return set_one(reinterpret_cast<const void*>(&expert_up_mma_kernel<true, MODE, EARLY>));
}

template <int MODE>
cudaError_t set_attrs_down() {
  const void* fns[4] = {reinterpret_cast<const void*>(&expert_down_mma_kernel<1, MODE>),
                        reinterpret_cast<const void*>(&expert_down_mma_kernel<2, MODE>),
                        reinterpret_cast<const void*>(&expert_down_mma_kernel<3, MODE>),
                        reinterpret_cast<const void*>(&expert_down_mma_kernel<4, MODE>)};
  for (const void* f : fns) {
    const cudaError_t e = set_one(f);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

cudaError_t set_attrs() {
  cudaError_t e = set_attrs_down<0>();
  if (e == cudaSuccess) e = set_attrs_down<1>();
  if (e == cudaSuccess) e = set_attrs_down<2>();
  if (e == cudaSuccess) e = set_attrs_up<0, 0>();
  if (e == cudaSuccess) e = set_attrs_up<0, 1>();
  if (e == cudaSuccess) e = set_attrs_up<0, 2>();
  if (e == cudaSuccess) e = set_attrs_up<1, 0>();
  if (e == cudaSuccess) e = set_attrs_up<1, 1>();
  if (e == cudaSuccess) e = set_attrs_up<1, 2>();
  if (e == cudaSuccess) e = set_attrs_up<2, 0>();   // raw logits come from the kernel just before
  if (e == cudaSuccess) e = set_attrs_up<2, 2>();   // ... or from a router that has finished
  return e;
}

// One call: the up kernel, then the down kernel, both with the routing mode compiled in.
template <int MODE, int EARLY>
cudaError_t launch_pair(const MmaPlan& pl, int grid, const UpParams& up, const DownParams& dn,
                        bool chained, cudaStream_t st) {
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t lc{};
  lc.gridDim = dim3(grid);
  lc.blockDim = dim3(kThreads);
  lc.stream = st;
  lc.attrs = attr;
  lc.numAttrs = chained ? 1 : 0;
  lc.dynamicSmemBytes = pl.smem_up;
  cudaError_t e = up.L > 8 ? cudaLaunchKernelEx(&lc, expert_up_mma_kernel<true, MODE, EARLY>, up)
                           : cudaLaunchKernelEx(&lc, expert_up_mma_kernel<false, MODE, EARLY>, up);
  if (e != cudaSuccess) return e;
  lc.dynamicSmemBytes = pl.smem_down;
  switch ((dn.L + 7) / 8) {
    case 1: return cudaLaunchKernelEx(&lc, expert_down_mma_kernel<1, MODE>, dn);
    case 2: return cudaLaunchKernelEx(&lc, expert_down_mma_kernel<2, MODE>, dn);
    case 3: return cudaLaunchKernelEx(&lc, expert_down_mma_kernel<3, MODE>, dn);
    default: return cudaLaunchKernelEx(&lc, expert_down_mma_kernel<4, MODE>, dn);
  }
}

}  // namespace

bool expert_mma_supported(const blockffn_ctx* c, int L) {
  return make_plan(c->cfg, L, c->num_sms).ok;
}

size_t expert_mma_h_bytes(const blockffn_config* cfg) {
  return sizeof(uint16_t) * (size_t)cfg->E * cfg->L_max * cfg->d_e + 256;
}

cudaError_t expert_mma_setup(blockffn_ctx*) { return set_attrs(); }

cudaError_t launch_expert_mma(blockffn_ctx* c, const blockffn_weights* w, const void* x,
                              const float* scores, int L, const int32_t* union_ids,
                              const int32_t* n_union, float* out, void* x_next, int call_flags,
                              const RoutingOut* pub, const RouterLogits* logits, bool logits_final,
                              cudaStream_t st) {
  const MmaPlan pl = make_plan(c->cfg, L, c->num_sms);
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
  up.ring_rows = pl.ring_rows;
  up.de_shift = __builtin_ctz(c->cfg.d_e);
  up.status = c->status;
  if (pub) {
    up.pub_mask = pub->union_mask;
    up.pub_ids = pub->union_ids;
    up.pub_n = pub->n_union;
    up.stats = pub->stats;
    up.pub_scores = pub->scores;
    up.pub_tok = pub->tok_mask;
  }
  if (logits) up.lg = *logits;
  DownParams dn{};
  dn.D = static_cast<const uint16_t*>(w->D);
  dn.h = up.h;
  dn.scores = scores;
  if (logits) dn.lg = *logits;
  dn.ids_in = union_ids;
  dn.n_in = n_union;
  dn.out = out;
  dn.x_next = static_cast<uint16_t*>(x_next);
  dn.L = L;
  dn.d = c->cfg.d;
  dn.E = c->cfg.E;
  dn.d_e = c->cfg.d_e;
  dn.ns = pl.ns_down;
  dn.max_cols = pl.max_cols;
  dn.per = pl.per;
  dn.cols_q = pl.cols_q;
  dn.cols_rem = pl.cols_rem;
  dn.accumulate = (call_flags & BLOCKFFN_CALL_ACCUMULATE) ? 1 : 0;
  dn.status = c->status;
  const bool chained = !(c->cfg.flags & BLOCKFFN_CFG_NO_CHAINING);
  // logits_final: the router finished before these kernels could start and x is stable
  const int early = logits ? (logits_final ? 2 : 0)
                    : (call_flags & BLOCKFFN_CALL_INDEPENDENT_X) ? 2
                    : (call_flags & BLOCKFFN_CALL_INDEPENDENT)   ? 1
                                                                 : 0;
  const int grid = c->num_sms;
  cudaError_t e;
  if (logits) {
    e = early == 2 ? launch_pair<2, 2>(pl, grid, up, dn, chained, st)
                   : launch_pair<2, 0>(pl, grid, up, dn, chained, st);
  } else if (union_ids) {
    e = early == 2   ? launch_pair<1, 2>(pl, grid, up, dn, chained, st)
        : early == 1 ? launch_pair<1, 1>(pl, grid, up, dn, chained, st)
                     : launch_pair<1, 0>(pl, grid, up, dn, chained, st);
  } else {
    e = early == 2   ? launch_pair<0, 2>(pl, grid, up, dn, chained, st)
        : early == 1 ? launch_pair<0, 1>(pl, grid, up, dn, chained, st)
                     : launch_pair<0, 0>(pl, grid, up, dn, chained, st);
  }
  if (e == cudaSuccess) c->launches += 2;
  return e;
}
