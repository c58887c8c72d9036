// One-kernel expert stage for chunks of 9 .. 32 tokens (Eq. 1, Eq. 2 over Union(x), Sec. 3.3).
// Included by expert_lean.cu inside its unnamed namespace: it shares that file's parameters,
// shared-memory layout, ring of h buffers and helpers.
#pragma once

// The kernel of expert_lean.cu for chunks of 9 .. 32 tokens: NTG = 2 groups of 8 tokens per
// weight fragment. (A kernel of its own rather than NTG = 1 of this template: written for any
// NTG the single-group case kept a few more values live and spilled, which cost 15 % at 8 tokens.)
//
// The x fragments of both token groups stay in registers (up to 64 of them; 128 registers per
// thread, two CTAs per SM) and every weight fragment read from shared memory is used for both
// groups. In the down projection the fragments of the intermediate h come from L2 straight into
// registers, a few k blocks ahead of their use, in the registers the x fragments have left
// (measured at 16 tokens, d = 2048, union 19: 5.04 us per call against 5.25 with h staged in
// shared memory).
//
// TEAMS = 2 (chunks of 17 .. 32 tokens): a CTA of 512 threads, two teams of 8 warps. Both teams
// work on the same weights in shared memory (copied once, by all 512 threads) and differ in their
// tokens: team 0 takes tokens 0 .. 15, team 1 the rest, each with NTG = 2 groups in registers.
// Within a team everything is as in the one-team kernel: K split over the team's 8 warps and
// partial tiles of its own, except that the intermediate h of a round's experts is staged in
// shared memory next to their slabs of D: with one CTA per SM nothing else runs under the round
// trips of direct fragment loads (measured at 32 tokens: 9.4 us per call direct, 8.6 staged).
template <int KB, int NC, int NTG, int MODE, int TEAMS>
__global__ void __launch_bounds__(kThreads * TEAMS, (NTG == 2 && TEAMS == 1) ? 2 : 1)
expert_wide_kernel(const LeanParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int kNT = kThreads * TEAMS;              // threads of the CTA
  const int tid = threadIdx.x, lane = tid & 31;
  const int team = TEAMS == 2 ? tid >> 8 : 0;        // which 16 tokens
  const int ttid = tid & (kThreads - 1);             // thread within the team
  const int warp = ttid >> 5;                        // warp within the team: its share of K
  // Lf: tokens of the chunk; tok0, L: the team's first token and token count.
  const int d = p.d, d_e = p.d_e, Lf = p.L;
  const int tok0 = team * 16, L = min(16, Lf - tok0);
  const LeanLayout lay = lean_layout(p.E, p.red_rows, NTG * TEAMS, p.cap_bytes);
  const uint32_t sbase = smem_u32(smem);
  const uint32_t wbase = sbase + lay.off_w;
  int* ctl = reinterpret_cast<int*>(smem + kOffCtl);
  int* ids_sm = reinterpret_cast<int*>(smem + kOffIds);
  float* red0 = reinterpret_cast<float*>(smem + lay.off_red);     // (the union derivation's scratch)
  float* red = red0 + team * (8 * NTG * red_ts(p.red_rows));      // this team's partial tiles
  const int g = lane >> 2, tg = lane & 3;
  const int G = gridDim.x, bx = blockIdx.x;   // the weights are shared out over the CTAs of the call
  const unsigned Gt = gridDim.x;

  if (tid < 8) ctl[tid] = 0;
  unsigned long long ticket = 0;
  if (tid == 0) ticket = atomicAdd(p.seq, 1ull);
  __syncthreads();
  // Thread 0 turns its ticket into the call's ring slot and lets the dependents go while the
  // routing loads are in flight: every CTA of this call then holds its ticket before a CTA of
  // the next call exists, and the next call starts as early as that allows.
  auto on_ticket = [&]() {
    const unsigned long long n = ticket / Gt;
    ctl[6] = (int)(n & (kHRing - 1));
    *reinterpret_cast<unsigned long long*>(ctl + 138) =
        p.hold ? ~0ull : (n / kHRing + 1ull) * Gt;
    pdl_trigger();
  };
  // (the caller's union list: the scores are first read at the end of the first stage)
  if constexpr (MODE == 1) prefetch_l2(p.scores, Lf * p.E * 4);
  // MODE 3: the router inside the kernel, as in expert_lean_kernel, 8 tokens per pass and team
  // (a row has at most 256 pieces of 16 bytes: one per thread of a team).
  RouterLogits lg3 = p.lg;
  if constexpr (MODE == 3) {
    if (tid == 0) on_ticket();
    __syncthreads();
    if (p.dep) pdl_wait();
    const int rslot = ctl[6];
    float* a0 = p.logit_ring + (size_t)rslot * p.logit_slot;
    lg3.a0 = a0;
    const int chunks = d >> 3;
    // Work units: (expert, pass of 8 tokens), dealt out over the teams of all CTAs, so that the
    // router part of a 32-token chunk is as many short steps per team as it takes (with whole
    // experts per CTA the CTAs that get two of them held everyone up at the hand-over).
    float* wsum = red0 + team * 64;            // [8 warps][8 tokens] per team
    const int npass = (Lf + 7) >> 3;
    const int units = p.E * npass, stride = G * TEAMS;
    const int rounds = (units + stride - 1) / stride;      // the same for every thread: barriers inside
    for (int k = 0; k < rounds; ++k) {
      const int u = k * stride + bx * TEAMS + team;
      const bool live = u < units;
      const int e = live ? u / npass : 0, t0 = live ? 8 * (u - e * npass) : 0;
      float acc[8];
#pragma unroll
      for (int t = 0; t < 8; ++t) acc[t] = 0.0f;
      if (live && ttid < chunks) {
        const uint4 wv = __ldg(reinterpret_cast<const uint4*>(p.W_r + (size_t)e * d) + ttid);
        const uint32_t wp[4] = {wv.x, wv.y, wv.z, wv.w};
        uint4 xv[8];
#pragma unroll
        for (int t = 0; t < 8; ++t)
          xv[t] = t0 + t < Lf ? __ldcg(reinterpret_cast<const uint4*>(p.x + (size_t)(t0 + t) * d) + ttid)
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
      if (live && ttid < 8 && t0 + ttid < Lf) {
        float v = p.bias ? p.bias[e] : 0.0f;
#pragma unroll
        for (int q = 0; q < kWarps; ++q) v += wsum[q * 8 + ttid];
        a0[(size_t)(t0 + ttid) * p.E + e] = v;
      }
      __syncthreads();
    }
    if (tid == kNT - 1) {
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
  const RouterLogits& lg = MODE == 3 ? lg3 : p.lg;
  int nu_;
  if constexpr (MODE == 3)
    nu_ = derive_union<2>(p.scores, lg, p.ids_in, p.n_in, Lf, p.E, ids_sm, ctl,
                          reinterpret_cast<uint32_t*>(red0));
  else
    nu_ = derive_union<MODE>(p.scores, lg, p.ids_in, p.n_in, Lf, p.E, ids_sm, ctl,
                             reinterpret_cast<uint32_t*>(red0), on_ticket);
  const int nu = nu_;

  // ---- up projection ---------------------------------------------------------------------
  const int R = nu * d_e;
  const int rq = (int)__umulhi((unsigned)R, p.magic_g), rrem = R - rq * G;
  const int r0 = bx * rq + min(bx, rrem), nrows = rq + (bx < rrem ? 1 : 0), r1 = r0 + nrows;
  const int row_bytes = 2 * d;
  const int cap_rows = p.cap_rows;
  // one stage when the share fits (the usual case: no division on that path), else stages of
  // half the region that are refilled as they free
  // (chunks of more than 8 tokens have a whole SM's shared memory: three stages in the ring, so
  // that two are in flight under the math of the third)
  constexpr int NS = (NTG <= 2 && TEAMS == 1) ? 2 : 3;
  const int ldr = min(p.red_rows, 32);       // a stage is at most two row tiles
  const bool single = nrows <= min(ldr, cap_rows);
  const int slot_rows = single ? max(nrows, 1) : min(ldr, cap_rows / NS);
  const int ngroups = single ? (nrows > 0 ? 1 : 0) : (nrows + slot_rows - 1) / slot_rows;
  const int rpg = single ? nrows : (nrows + ngroups - 1) / ngroups;
  const int half_u = ((slot_rows + 1) >> 1) * row_bytes + 64;   // where the odd rows start
  const int slot_bytes = slot_rows * row_bytes + 64;
  const int sh = p.de_shift;
  // This thread's part of a row copy: 16-byte chunk my_c of the rows my_sub, my_sub + rpi, ...
  const int cpr = d >> 3;                       // chunks per row (<= 256)
  const int rpi = cpr > kNT / 2 ? 1 : kNT / cpr;    // rows the CTA copies per step
  // (the reciprocal multiply is exact for tid < 256 only)
  const int my_sub = TEAMS == 2 ? tid / cpr : (int)((tid * p.magic_cpr) >> 16);
  const int my_c = tid - my_sub * cpr;
  const bool copies_u = my_sub < rpi;
  // stage gi: rows [r0 + gi rpg, ...) -> slot gi % NS, row m of the stage at
  // (m >> 1) row_bytes + (m & 1) half_u
  auto issue_u = [&](int gi) {
    const int ra = r0 + gi * rpg;
    const int rows = min(r1, ra + rpg) - ra;
    const uint32_t slot0 = wbase + (gi % NS) * slot_bytes + my_c * 16;
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
  // score and h element (expert slot, token, neuron) this thread finishes in a stage, per token
  // group: token 8 n + ttid / 32 of the team, row tid % 32 of the stage
  float sc[NTG];
  int hidx[NTG];        // element index into the h buffer, -1: nothing to finish
  auto prepare = [&](int gi) {
    const int ra = r0 + gi * rpg, rows = min(r1, ra + rpg) - ra;
    const int m = tid & 31;
    const int hq = (ra + m) >> sh;
    const int id = m < rows ? ids_sm[hq] : 0;
#pragma unroll
    for (int n = 0; n < NTG; ++n) {
      const int t = 8 * n + (ttid >> 5);
      sc[n] = 0.0f;
      hidx[n] = -1;
      if (t < L && m < rows) {
        hidx[n] = (hq * Lf + tok0 + t) * d_e + (ra + m - (hq << sh));
        if constexpr (MODE >= 2) {
          float v = __ldcg(lg.a0 + (tok0 + t) * p.E + id);
          v = v > 0.0f ? v : 0.0f;
          sc[n] = __ldg(lg.gain + id) * v * reinterpret_cast<const float*>(ctl + 104)[tok0 + t];
        } else {
          sc[n] = __ldcg(p.scores + (tok0 + t) * p.E + id);
        }
      }
    }
  };
  // x: this warp's k blocks (warp + 8 i) of the token rows this lane feeds to the mma
  const int npx = d >> 6;
  Frag64 fx[NTG][KB];
  auto load_x = [&]() {
#pragma unroll
    for (int n = 0; n < NTG; ++n) {
      const uint4* xp = reinterpret_cast<const uint4*>(p.x + (tok0 + min(8 * n + g, L - 1)) * d + 64 * warp) + tg;
#pragma unroll
      for (int i = 0; i < KB; ++i) {
        if (warp + kWarps * i < npx) {
          fx[n][i].lo = ld_cg_v4(xp + 64 * i);       // 64 k blocks of 128 bytes = 8 warps further
          fx[n][i].hi = ld_cg_v4(xp + 64 * i + 4);
        } else {
          fx[n][i].lo = fx[n][i].hi = make_uint4(0, 0, 0, 0);
        }
      }
    }
  };
  // x goes first: its short round trip then runs under the long issue of the weights instead
  // of behind it. In a dependent chain x is what the call before leaves: the weights (stable)
  // are requested under that call, then the kernel waits for it and reads x.
  if (!p.dep) load_x();
#pragma unroll
  for (int gi = 0; gi < NS; ++gi) {          // one commit group per stage, empty ones included
    if (gi < ngroups) issue_u(gi);
    cp_async_commit();
  }
  if (p.dep) {
    pdl_wait();
    load_x();
  }
  if (ngroups > 0) prepare(0);
  const int slot = ctl[6];       // (written before the barriers inside derive_union)
  uint16_t* hbuf = p.h_ring + (size_t)slot * p.h_slot;

  for (int gi = 0; gi < ngroups; ++gi) {
    const int rows = min(r1, r0 + (gi + 1) * rpg) - (r0 + gi * rpg);
    // fragment addresses of rows g and g + 8 (same parity) of the two 16-row tiles, at this
    // warp's first k block; rows beyond the stage read its last row (their results are dropped)
    auto row_addr = [&](int m) {
      m = min(m, rows - 1);
      return wbase + (gi % NS) * slot_bytes + (m >> 1) * row_bytes + (m & 1) * half_u + 128 * warp +
             16 * tg;
    };
    cp_async_wait_group<NS - 1>(); // all but the NS - 1 newest groups: this stage has landed
    __syncthreads();
    // partial tiles -> red[t][warp][m]
    const int ws = red_ws(ldr), nt = red_ts(ldr);      // one warp, one token further
    float* mine = red + 2 * tg * nt + warp * ws + g;
    auto do_tile = [&](const int tile) {
      const uint32_t a0 = row_addr(g + 16 * tile), b0 = row_addr(g + 16 * tile + 8);
      float c0[NTG][4], c1[NTG][4];
#pragma unroll
      for (int n = 0; n < NTG; ++n)
#pragma unroll
        for (int v = 0; v < 4; ++v) c0[n][v] = c1[n][v] = 0.0f;
#pragma unroll
      for (int i = 0; i < KB; ++i) {
        if (warp + kWarps * i < npx) {
          const uint4 alo = lds128(a0 + 1024 * i), ahi = lds128(a0 + 1024 * i + 64);
          const uint4 blo = lds128(b0 + 1024 * i), bhi = lds128(b0 + 1024 * i + 64);
#pragma unroll
          for (int n = 0; n < NTG; ++n) mma64(c0[n], c1[n], alo, ahi, blo, bhi, fx[n][i]);
        }
      }
      const int m0 = g + 16 * tile;
#pragma unroll
      for (int n = 0; n < NTG; ++n) {
        float* o = mine + 8 * n * nt + 16 * tile;
        if (m0 < ldr) {
          o[0] = c0[n][0] + c1[n][0];
          o[nt] = c0[n][1] + c1[n][1];
        }
        if (m0 + 8 < ldr) {
          o[8] = c0[n][2] + c1[n][2];
          o[nt + 8] = c0[n][3] + c1[n][3];
        }
      }
    };
    do_tile(0);
    if (rows > 16) do_tile(1);     // second tile of 16 rows
    __syncthreads();               // partials complete; every warp is done with the slot
    if (gi + NS < ngroups) issue_u(gi + NS);
    cp_async_commit();
#pragma unroll
    for (int n = 0; n < NTG; ++n) {
      if (hidx[n] >= 0) {
        const float v = red_sum(red + (8 * n + (ttid >> 5)) * red_ts(ldr) + (tid & 31), red_ws(ldr));
        hbuf[hidx[n]] = (uint16_t)f32_to_bf16_bits(sc[n] * swish_fast(v));
      }
    }
    if (gi + 1 < ngroups) prepare(gi + 1);
    // the next stage starts with a wait and a barrier, which also protects red
  }
  cp_async_wait_all();
  __syncthreads();                 // every h element of this CTA has been stored
  if (tid == kNT - 1) {
    __threadfence();
    asm volatile("red.relaxed.gpu.global.add.u64 [%0], 1;" ::"l"(p.ready + slot) : "memory");
    // (the slot's counter of the logit hand-over advances in step, see expert_lean_kernel)
    if constexpr (MODE != 3)
      asm volatile("red.relaxed.gpu.global.add.u64 [%0], 1;" ::"l"(p.ready2 + slot) : "memory");
  }

  // ---- down projection -------------------------------------------------------------------
  // Slab of one expert: the CTA's columns (at most 16 NC, NC mma row tiles) as rows of 2 d_e
  // bytes, even columns first, 64 bytes of padding, odd columns. With two teams the expert's
  // h tile follows its slab: token rows of 2 d_e bytes, split even / odd the same way.
  const int drow = 2 * d_e;
  const int half_d = ((p.max_cols + 1) >> 1) * drow + 64;
  const int half_h = 4 * NTG * TEAMS * drow + 64;
  const int slot_d = p.max_cols * drow + 64 + (TEAMS == 2 ? 8 * NTG * TEAMS * drow + 64 : 0);
  const int h_off = p.max_cols * drow + 64;     // the h tile inside an expert's slot
  const int cap_slabs = p.cap_slabs;
  const bool one_round = nu <= cap_slabs;
  const int rsz = one_round ? max(nu, 1) : max(1, cap_slabs / 2);
  const int nrounds = one_round ? (nu > 0 ? 1 : 0) : (nu + rsz - 1) / rsz;
  const int c0 = bx * p.cols_q + min(bx, p.cols_rem);
  const int ncols = p.cols_q + (bx < p.cols_rem ? 1 : 0);
  // A slab is ncols << kshift chunks of 16 bytes; chunk c = column c >> kshift, piece
  // c & (2^kshift - 1). Thread tid copies chunks tid, tid + kDCopy, ... of every expert; the
  // last warp (the polling thread's) copies none.
  const int kshift = sh - 3;                    // log2(chunks per D row)
  const uint32_t estride16 = (uint32_t)d << kshift;
  constexpr int kDCopy = kNT - 32;
  const int nchunks = tid < kDCopy ? ncols << kshift : 0;
  auto issue_d = [&](int r) {
    const int q0 = r * rsz, n = min(rsz, nu - q0);
    for (int c = tid; c < nchunks; c += kDCopy) {
      const int cc = c >> kshift, k = c & ((1 << kshift) - 1);
      const uint32_t src0 = ((uint32_t)(c0 + cc) << kshift) + k;          // + id * d << kshift
      uint32_t dst = wbase + (r & 1) * rsz * slot_d + (cc >> 1) * drow + (cc & 1) * half_d + k * 16;
#pragma unroll 4
      for (int i = 0; i < n; ++i, dst += slot_d)
        cp_async16(dst, at16(p.D, src0 + (uint32_t)ids_sm[q0 + i] * estride16));
    }
  };
  // (two teams) the h tiles of a round's experts: L rows of 2 d_e bytes per expert,
  // contiguous in the h buffer; chunk c = token c >> kshift, piece c & (2^kshift - 1). Each team
  // fetches its own tokens into its own rows of the tile (team 1: rows 16 ..).
  auto issue_h = [&](int r) {
    const int q0 = r * rsz, n = min(rsz, nu - q0);
    const uint32_t hstep16 = (uint32_t)(Lf * d_e) >> 3;
    for (int c = ttid; c < (L << kshift); c += kThreads) {
      const int t = c >> kshift, k = c & ((1 << kshift) - 1);
      uint32_t dst = wbase + (r & 1) * rsz * slot_d + h_off + (8 * team + (t >> 1)) * drow +
                     (t & 1) * half_h + k * 16;
      uint32_t src = (uint32_t)q0 * hstep16 + ((uint32_t)tok0 << kshift) + c;
      for (int i = 0; i < n; ++i, dst += slot_d, src += hstep16) cp_async16(dst, at16(hbuf, src));
    }
  };
  if (nrounds > 0) issue_d(0);
  cp_async_commit();
  if (nrounds > 1) issue_d(1);
  cp_async_commit();
  const int ot = ttid >> 5, om = tid & 31;  // this thread's outputs: tokens ot (+ 8), columns om (+ 32)
  // hand-over: all CTAs of this call have stored their part of h
  if (tid == kNT - 1) {
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
  if constexpr (TEAMS == 2) {
    if (!dead) {
      if (nrounds > 0) issue_h(0);
      cp_async_commit();
      if (nrounds > 1) issue_h(1);
      cp_async_commit();
    }
  }

  const int npairs = d_e >> 6;      // 64-wide k blocks per expert (a power of two)
  const int pshift = sh - 6;
  float acc[NC][NTG][2][4];
#pragma unroll
  for (int c = 0; c < NC; ++c)
#pragma unroll
    for (int n = 0; n < NTG; ++n)
#pragma unroll
      for (int v = 0; v < 4; ++v) acc[c][n][0][v] = acc[c][n][1][v] = 0.0f;
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
  // token rows 8 n + g of this team in the h buffer (rows beyond the chunk repeat its last one:
  // their columns of the result are dropped)
  const uint4* hrow[NTG];
#pragma unroll
  for (int n = 0; n < NTG; ++n)
    hrow[n] = reinterpret_cast<const uint4*>(hbuf + (tok0 + min(8 * n + g, L - 1)) * d_e) + tg;
  const uint32_t hstep16 = (uint32_t)(Lf * d_e) >> 3;        // one expert further, in 16 bytes
  // (two teams) token rows 8 n + g of an h tile in shared memory (rows beyond the chunk hold
  // whatever the buffer held: their columns of the result are dropped)
  const uint32_t hs_off = h_off + (8 * team + (g >> 1)) * drow + (g & 1) * half_h + 16 * tg;
  for (int r = 0; r < nrounds && !dead; ++r) {
    const int q0 = r * rsz, n = min(rsz, nu - q0);
    const int nblk = n << pshift;
    const uint32_t d_base = wbase + (r & 1) * rsz * slot_d;
    if constexpr (TEAMS == 1) {
      // this warp's k blocks b = warp + 8 i of the round, in batches whose h fragments are all
      // requested before the first is used; block b = expert b >> pshift, k block b & (npairs - 1)
      // (fewer per batch with more column tiles: their accumulators need the registers)
      constexpr int kHB = NC == 1 ? 4 : NC == 2 ? 3 : 2;
      Frag64 fh[kHB][NTG];
      auto load_h = [&](int b0) {
#pragma unroll
        for (int i = 0; i < kHB; ++i) {
          const int b = b0 + kWarps * i;
          if (b < nblk) {
            const uint32_t ho = (uint32_t)(q0 + (b >> pshift)) * hstep16 + 8 * (b & (npairs - 1));
#pragma unroll
            for (int n2 = 0; n2 < NTG; ++n2) {
              fh[i][n2].lo = ld_cg_v4(hrow[n2] + ho);
              fh[i][n2].hi = ld_cg_v4(hrow[n2] + ho + 4);
            }
          }
        }
      };
      load_h(warp);
      cp_async_wait_group<1>();    // all but the newest group: this round's slabs have landed
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
#pragma unroll
              for (int n2 = 0; n2 < NTG; ++n2)
                mma64(acc[c][n2][0], acc[c][n2][1], alo, ahi, blo, bhi, fh[i][n2]);
            }
          }
        }
      }
    } else {
      cp_async_wait_group<1>();    // this round's slabs and h tiles have landed
      __syncthreads();
#pragma unroll 1
      for (int b = warp; b < nblk; b += kWarps) {
        const uint32_t da = d_base + (b >> pshift) * slot_d + 128 * (b & (npairs - 1));
        Frag64 fh[NTG];
#pragma unroll
        for (int n2 = 0; n2 < NTG; ++n2) {
          fh[n2].lo = lds128(da + hs_off + 4 * n2 * drow);      // 8 token rows = 4 row pairs further
          fh[n2].hi = lds128(da + hs_off + 4 * n2 * drow + 64);
        }
#pragma unroll
        for (int c = 0; c < NC; ++c) {
          const uint4 alo = lds128(da + offs[c][0]), ahi = lds128(da + offs[c][0] + 64);
          const uint4 blo = lds128(da + offs[c][1]), bhi = lds128(da + offs[c][1] + 64);
#pragma unroll
          for (int n2 = 0; n2 < NTG; ++n2)
            mma64(acc[c][n2][0], acc[c][n2][1], alo, ahi, blo, bhi, fh[n2]);
        }
      }
    }
    __syncthreads();               // every warp is done with this round's slabs
    if (r + 2 < nrounds) {
      issue_d(r + 2);
      if constexpr (TEAMS == 2) issue_h(r + 2);
    }
    cp_async_commit();
  }
  cp_async_wait_all();
  pdl_wait();                      // out (and x_next) may still be in use by the call before
  if (!dead) {
    if (nu > 0) {
      // partial tiles -> part[t][warp][m] (m < 16 NC), then one thread per output element; the
      // partials take the weight region, which is free by now
      constexpr int ws2 = 16 * NC, ts2 = kWarps * ws2 + 4;
      float* part0 = reinterpret_cast<float*>(smem + lay.off_w) + team * (8 * NTG * ts2);
      float* mine = part0 + 2 * tg * ts2 + warp * ws2 + g;
#pragma unroll
      for (int n = 0; n < NTG; ++n) {
#pragma unroll
        for (int c = 0; c < NC; ++c) {
          float* o = mine + 8 * n * ts2 + 16 * c;
          o[0] = acc[c][n][0][0] + acc[c][n][1][0];
          o[ts2] = acc[c][n][0][1] + acc[c][n][1][1];
          o[8] = acc[c][n][0][2] + acc[c][n][1][2];
          o[ts2 + 8] = acc[c][n][0][3] + acc[c][n][1][3];
        }
      }
      __syncthreads();
#pragma unroll
      for (int n = 0; n < NTG; ++n) {
        const int t = ot + 8 * n;
        if (t < L) {
#pragma unroll
          for (int k = 0; k < (NC + 1) / 2; ++k) {
            const int m = om + 32 * k;
            if (m < ncols) {
              float v = red_sum(part0 + t * ts2 + m, ws2);
              const int o = (tok0 + t) * d + c0 + m;
              if (p.accumulate) v += __ldcg(p.out + o);
              p.out[o] = v;
              if (p.x_next) p.x_next[o] = (uint16_t)f32_to_bf16_bits(v);
            }
          }
        }
      }
    } else {                       // empty union: FFN(x) = 0
      for (int t = ot; t < L; t += 8) {
        for (int m = om; m < ncols; m += 32) {
          const int o = (tok0 + t) * d + c0 + m;
          const float v = p.accumulate ? __ldcg(p.out + o) : 0.0f;
          p.out[o] = v;
          if (p.x_next) p.x_next[o] = (uint16_t)f32_to_bf16_bits(v);
        }
      }
    }
  }
  // CTA 0 publishes the routing it derived (after the wait: earlier readers are done)
  if (blockIdx.x == 0) {
    if (lg.a0 != nullptr && p.pub_scores != nullptr) {
      const int words = (p.E + 31) >> 5;
      const float* rinv = reinterpret_cast<const float*>(ctl + 104);
      for (int t = tid >> 5; t < Lf; t += kNT / 32) {
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
      for (int e = tid; e < p.E; e += kNT) {
        if (p.pub_ids) p.pub_ids[e] = e < nu ? ids_sm[e] : -1;
        if (p.pub_mask && e < words) p.pub_mask[e] = um[e];
      }
      if (tid == 0) {
        if (p.pub_n) *p.pub_n = nu;
        if (p.stats) {
          atomicAdd(reinterpret_cast<unsigned long long*>(&p.stats->n_tokens),
                    (unsigned long long)Lf);
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

