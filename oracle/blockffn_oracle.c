/*
 * BlockFFN chunk-verify FFN forward: the CPU oracle.
 *
 * TEST INFRASTRUCTURE, NOT PRODUCT. This file is the slow, plain statement of
 * what the layer computes, written from the paper's definitions. Only the test
 * suite, the smoke check and the benchmark's CPU-baseline leg may call it; the
 * CUDA library never does, and the two share no code (this file carries its own
 * bf16 helpers on purpose).
 *
 * Arithmetic: every bf16 input is widened exactly (a 16-bit shift) and all sums
 * run in IEEE double, sequentially, in index order. No blocking, no fusion, no
 * skipping beyond what the cited passage states.
 *
 * Layouts (row-major, C order):
 *   x      bf16 [L][d]          hidden states of the chunk's L tokens
 *   W_r    bf16 [E][d]          router weight, row i = column i of W_router   (Eq. 3)
 *   gain   f32  [E]             RMSNorm per-expert gain
 *   bias   f32  [E] or NULL     optional additive shift on the router logits
 *                               (NULL is the paper's Eq. 3; the shift exists only
 *                               so a synthetic router can hit a target sparsity)
 *   U      bf16 [E][d_e][d]     U[i][j][k] = W_up^(i)[k][j]                   (Eq. 2)
 *   D      bf16 [E][d][d_e]     D[i][c][j] = W_down^(i)[j][c]                 (Eq. 2)
 *   scores f64  [L][E]          A(x), the router activation values            (Eq. 3)
 *   out    f64  [L][d]          FFN(x_t)                                      (Eq. 1)
 *
 * Readings where the paper is silent (also listed in the design document):
 *   - RMSNorm carries a per-expert gain and an eps inside the square root, the
 *     mean square runs over all E entries (zeros included);
 *   - Swish is z * sigmoid(z) (beta = 1), experts are not gated;
 *   - an expert is "activated" by a token iff its final score is nonzero by
 *     value (-0.0 is zero, NaN counts as nonzero);
 *   - the score multiplies the activated intermediate, before the down
 *     projection;
 *   - the union id list is in ascending expert order;
 *   - the router without RMSNorm (Sec. 4.2.3) has no gain either: its scores are
 *     the ReLU of the logits;
 *   - the reuse ratio (Sec. 4.1.2) leaves out a pair whose first token activates
 *     no expert (its ratio is 0/0).
 * "parity unpinned" (no independent source fixes them): the eps value, beta = 1,
 * the place where the score multiplies. Everything else is pinned by the CPU
 * tests (brute force, closed forms, library reductions, invariants).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_API __attribute__((visibility("default")))

static double widen_bf16(uint16_t b) {
  uint32_t w = ((uint32_t)b) << 16;
  float f;
  memcpy(&f, &w, sizeof f);
  return (double)f;
}

/* float -> bf16, round to nearest even; NaN stays NaN (quiet). */
static uint16_t narrow_to_bf16(float f) {
  uint32_t w;
  memcpy(&w, &f, sizeof w);
  if ((w & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((w >> 16) | 0x0040u);
  uint32_t lsb = (w >> 16) & 1u;
  w += 0x7fffu + lsb;
  return (uint16_t)(w >> 16);
}

static int mask_words(int E) { return (E + 31) / 32; }

/* Eq. 3: A0 = W_router^T x ; A1 = ReLU(A0) ; A = RMSNorm(A1) (gain, eps).
 * a0 (may be NULL) receives the pre-ReLU logits. */
ORACLE_API void oracle_router(const uint16_t* x, const uint16_t* W_r, const float* gain,
                              const float* bias, int L, int d, int E, double eps,
                              double* a0, double* scores) {
  double* a1 = (double*)malloc(sizeof(double) * (size_t)E);
  for (int t = 0; t < L; ++t) {
    for (int i = 0; i < E; ++i) {
      double acc = bias ? (double)bias[i] : 0.0;
      for (int k = 0; k < d; ++k)
        acc += widen_bf16(x[(size_t)t * d + k]) * widen_bf16(W_r[(size_t)i * d + k]);
      if (a0) a0[(size_t)t * E + i] = acc;
      a1[i] = acc > 0.0 ? acc : 0.0;
    }
    double sumsq = 0.0;
    for (int i = 0; i < E; ++i) sumsq += a1[i] * a1[i];
    double r = 1.0 / sqrt(sumsq / (double)E + eps);
    for (int i = 0; i < E; ++i) scores[(size_t)t * E + i] = (double)gain[i] * a1[i] * r;
  }
  free(a1);
}

/* The router of the RMSNorm ablation (Sec. 4.2.3, the ReMoE-style router of Table 1): the
 * activation values are the ReLU of the logits themselves, A = ReLU(W_router^T x); no
 * normalisation, hence no gain and no eps. */
ORACLE_API void oracle_router_relu_only(const uint16_t* x, const uint16_t* W_r, const float* bias,
                                        int L, int d, int E, double* a0, double* scores) {
  for (int t = 0; t < L; ++t)
    for (int i = 0; i < E; ++i) {
      double acc = bias ? (double)bias[i] : 0.0;
      for (int k = 0; k < d; ++k)
        acc += widen_bf16(x[(size_t)t * d + k]) * widen_bf16(W_r[(size_t)i * d + k]);
      if (a0) a0[(size_t)t * E + i] = acc;
      scores[(size_t)t * E + i] = acc > 0.0 ? acc : 0.0;
    }
}

/* The sparse pattern of A(x) (Sec. 3.3): bit i of token t's mask is set iff the
 * score is nonzero. Bits at and beyond E are zero. */
ORACLE_API void oracle_token_masks(const double* scores, int L, int E, uint32_t* tok_mask) {
  int W = mask_words(E);
  for (int t = 0; t < L; ++t) {
    for (int w = 0; w < W; ++w) tok_mask[(size_t)t * W + w] = 0u;
    for (int i = 0; i < E; ++i)
      if (scores[(size_t)t * E + i] != 0.0) tok_mask[(size_t)t * W + i / 32] |= 1u << (i % 32);
  }
}

/* Union(x) (Sec. 3.3): the experts activated by any token of the chunk, as a
 * bitmask and as the ascending id list (tail filled with -1), and the counters
 * behind TLS and CLS_L (Sec. 2.1):
 *   stats[0] += L (tokens), stats[1] += sum_t |active(t)|,
 *   stats[2] += 1 (chunks), stats[3] += |Union|.                              */
ORACLE_API void oracle_chunk_union(const uint32_t* tok_mask, int L, int E, uint32_t* union_mask,
                                   int32_t* union_ids, int32_t* n_union, uint64_t* stats) {
  int W = mask_words(E);
  for (int w = 0; w < W; ++w) union_mask[w] = 0u;
  uint64_t n_active = 0;
  for (int t = 0; t < L; ++t)
    for (int i = 0; i < E; ++i)
      if ((tok_mask[(size_t)t * W + i / 32] >> (i % 32)) & 1u) {
        union_mask[i / 32] |= 1u << (i % 32);
        n_active += 1;
      }
  int n = 0;
  for (int i = 0; i < E; ++i)
    if ((union_mask[i / 32] >> (i % 32)) & 1u) union_ids[n++] = i;
  for (int i = n; i < E; ++i) union_ids[i] = -1;
  *n_union = n;
  if (stats) {
    stats[0] += (uint64_t)L;
    stats[1] += n_active;
    stats[2] += 1;
    stats[3] += (uint64_t)n;
  }
}

/* TLS = mean fraction of experts a token leaves inactive; CLS_L = fraction of
 * experts inactive for every token of a chunk (Sec. 2.1). */
ORACLE_API double oracle_tls(const uint64_t* stats, int E) {
  return 1.0 - (double)stats[1] / ((double)stats[0] * (double)E);
}
ORACLE_API double oracle_cls(const uint64_t* stats, int E) {
  return 1.0 - (double)stats[3] / ((double)stats[2] * (double)E);
}

/* Reuse ratio (Sec. 4.1.2): with S_i the experts token i of a sequence activates, the ratio of
 * the sequence is the mean over its L - 1 successive pairs of |S_i n S_{i+1}| / |S_i|.
 * acc[0] += the sum of the pairs' ratios, in token order; acc[1] += the number of pairs
 * counted. A token that activates no expert has no ratio: its pair is left out of both. */
ORACLE_API void oracle_reuse_ratio(const double* scores, int L, int E, double* acc) {
  for (int i = 0; i + 1 < L; ++i) {
    int n_i = 0, n_both = 0;
    for (int e = 0; e < E; ++e) {
      int now = scores[(size_t)i * E + e] != 0.0;
      int next = scores[(size_t)(i + 1) * E + e] != 0.0;
      n_i += now;
      n_both += now && next;
    }
    if (n_i == 0) continue;
    acc[0] += (double)n_both / (double)n_i;
    acc[1] += 1.0;
  }
}

/* Eq. 1 with Eq. 2:  out[t] = sum_i A_i(x_t) * W_down^(i)T Swish(W_up^(i)T x_t).
 * expert_ids == NULL: the sum runs over ALL E experts (the definition).
 * expert_ids != NULL: the sum runs over those n_ids experts only, in list order
 * (the union-restricted evaluation of Sec. 3.3; entries < 0 are skipped).       */
ORACLE_API void oracle_expert_ffn(const uint16_t* x, const double* scores, const uint16_t* U,
                                  const uint16_t* D, int L, int d, int E, int d_e,
                                  const int32_t* expert_ids, int n_ids, double* out) {
  double* xt = (double*)malloc(sizeof(double) * (size_t)d);
  double* hcol = (double*)malloc(sizeof(double) * (size_t)d_e);
  int n = expert_ids ? n_ids : E;
  for (int t = 0; t < L; ++t) {
    for (int k = 0; k < d; ++k) xt[k] = widen_bf16(x[(size_t)t * d + k]);
    for (int c = 0; c < d; ++c) out[(size_t)t * d + c] = 0.0;
    for (int q = 0; q < n; ++q) {
      int i = expert_ids ? expert_ids[q] : q;
      if (i < 0) continue;
      const uint16_t* Ui = U + (size_t)i * d_e * d;
      const uint16_t* Di = D + (size_t)i * d * d_e;
      double s = scores[(size_t)t * E + i];
      for (int j = 0; j < d_e; ++j) {
        double m = 0.0;
        for (int k = 0; k < d; ++k) m += xt[k] * widen_bf16(Ui[(size_t)j * d + k]);
        double swish = m / (1.0 + exp(-m));
        hcol[j] = s * swish;
      }
      for (int c = 0; c < d; ++c) {
        double acc = 0.0;
        for (int j = 0; j < d_e; ++j) acc += hcol[j] * widen_bf16(Di[(size_t)c * d_e + j]);
        out[(size_t)t * d + c] += acc;
      }
    }
  }
  free(xt);
  free(hcol);
}

/* Whole layer from precomputed scores (f32 as the caller hands them in):
 * masks -> union -> counters -> FFN. union_only != 0 restricts the expert sum
 * to Union(x); 0 evaluates the plain definition over all experts.             */
ORACLE_API void oracle_layer_forward_scores(const uint16_t* x, const float* scores_f32,
                                            const uint16_t* U, const uint16_t* D, int L, int d,
                                            int E, int d_e, int union_only, double* scores,
                                            uint32_t* tok_mask, uint32_t* union_mask,
                                            int32_t* union_ids, int32_t* n_union, uint64_t* stats,
                                            double* out) {
  for (size_t p = 0; p < (size_t)L * E; ++p) scores[p] = (double)scores_f32[p];
  oracle_token_masks(scores, L, E, tok_mask);
  oracle_chunk_union(tok_mask, L, E, union_mask, union_ids, n_union, stats);
  if (union_only)
    oracle_expert_ffn(x, scores, U, D, L, d, E, d_e, union_ids, *n_union, out);
  else
    oracle_expert_ffn(x, scores, U, D, L, d, E, d_e, NULL, 0, out);
}

/* Whole layer, router included (Eq. 3 -> Sec. 3.3 union -> Eq. 1/2). */
ORACLE_API void oracle_layer_forward(const uint16_t* x, const uint16_t* W_r, const float* gain,
                                     const float* bias, const uint16_t* U, const uint16_t* D,
                                     int L, int d, int E, int d_e, double eps, int union_only,
                                     double* a0, double* scores, uint32_t* tok_mask,
                                     uint32_t* union_mask, int32_t* union_ids, int32_t* n_union,
                                     uint64_t* stats, double* out) {
  oracle_router(x, W_r, gain, bias, L, d, E, eps, a0, scores);
  oracle_token_masks(scores, L, E, tok_mask);
  oracle_chunk_union(tok_mask, L, E, union_mask, union_ids, n_union, stats);
  if (union_only)
    oracle_expert_ffn(x, scores, U, D, L, d, E, d_e, union_ids, *n_union, out);
  else
    oracle_expert_ffn(x, scores, U, D, L, d, E, d_e, NULL, 0, out);
}

/* Residual step of the stacked-decode workload: res += out, and the next
 * layer's input is the bf16 rounding (nearest even) of the f32 value of res.  */
ORACLE_API void oracle_residual_step(double* res, const double* out, int n, uint16_t* x_next) {
  for (int p = 0; p < n; ++p) {
    res[p] += out[p];
    x_next[p] = narrow_to_bf16((float)res[p]);
  }
}

ORACLE_API void oracle_round_to_bf16(const float* src, int n, uint16_t* dst) {
  for (int p = 0; p < n; ++p) dst[p] = narrow_to_bf16(src[p]);
}
