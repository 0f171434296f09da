/*
 * CPU oracle for the MoE-layer hot path: routing, dispatch layout, expert SwiGLU FFN, combine.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, obviously-correct
 * restatement of what the path computes, written to be checked against the paper by eye.
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg may call it.  It shares
 * no code with the CUDA path and the CUDA path never calls it.
 *
 * What it follows (paper: "MoE-Hub", Section II-A, the five steps of a distributed MoE layer):
 *   step 1  routing   : gating scores -> normalisation (softmax) -> top-k selection
 *   step 2  dispatch  : every token row goes to each of its k selected experts
 *   step 3  experts   : two GEMMs with an activation between (here SwiGLU: gate||up, then down)
 *   step 4  combine   : rows return to their token's position
 *   step 5  scaling   : weighted sum of the k expert outputs with the routing scores
 * and Section IV-B (address allocation unit): an expert's rows are densely packed, slot
 * LocalRowID = 0,1,2,... handed out by a self-incrementing row pointer, address =
 * BaseAddr + LocalRowID*RowSize + RowOffset; the source of every row travels with it
 * (Section IV-B, "All-to-All Combine").  The paper packs rows in arrival order, so any order
 * inside one expert's region is correct; the oracle uses the canonical order (token, then k).
 *
 * Precision.  The router logit decides an integer (which experts are picked), so it is computed
 * in the precision of the kernel: one fp32 fused-multiply-add chain per (token, expert), h
 * ascending, starting from 0.  Everything else (softmax weights, FFN, combine) is fp64.
 * bf16 inputs are widened exactly.
 *
 * Diagnostic mode (bf16 storage).  The CUDA path keeps three tensors in bf16: the SwiGLU
 * intermediate, the expert output rows and y.  oracle_expert_ffn_stored and oracle_combine_stored
 * restate steps 3-5 with exactly those three values rounded to bf16 (nearest, ties to even) and
 * every sum still in fp64: the best any implementation with bf16 storage can do.  The distance
 * between this restatement and the exact functions is the rounding a tolerance has to leave room
 * for; the distance between the CUDA path and this restatement is what the kernels add to it.
 *
 * Every function is pinned by tests that do not go through this file (brute force, closed
 * forms, invariants, library routines); see tests/test_oracle_*.py.
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fopenmp -shared -fPIC moe_oracle.c -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_FP32 = 0, ORACLE_BF16 = 1 };

static inline float widen(const void *base, int dtype, int64_t i) {
  if (dtype == ORACLE_FP32) return ((const float *)base)[i];
  uint32_t bits = (uint32_t)((const uint16_t *)base)[i] << 16;
  float f;
  memcpy(&f, &bits, sizeof f);
  return f;
}

static inline size_t elem_bytes(int dtype) { return dtype == ORACLE_FP32 ? 4 : 2; }

/*
 * Nearest bf16 value of a double (ties to even), returned as a double.  bf16 keeps 8 significant
 * bits, a double 53: round away the low 45 bits of the significand.  Finite inputs in bf16's
 * normal range only (everything this file feeds it is); zero stays zero.
 */
double oracle_round_bf16(double v) {
  uint64_t b;
  memcpy(&b, &v, sizeof b);
  const uint64_t lsb = (b >> 45) & 1u;
  b += ((uint64_t)1 << 44) - 1 + lsb;
  b &= ~(((uint64_t)1 << 45) - 1);
  memcpy(&v, &b, sizeof v);
  return v;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/*
 * Step 1a, gating scores: l[t,e] = sum_h x[t,h]*Wr[e,h] (+ bias[e]).
 * One fp32 FMA chain per output, h ascending.  x: [T,H], wr: [E,H], bias: [E] or NULL,
 * logits: [T,E] fp32.
 */
int oracle_logits(int T, int H, int E, int dtype, const void *x, const void *wr, const float *bias,
                  float *logits) {
  if (T < 0 || H <= 0 || E <= 0 || !logits) return -1;
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    for (int e = 0; e < E; ++e) {
      float acc = 0.0f;
      for (int h = 0; h < H; ++h)
        acc = fmaf(widen(x, dtype, (int64_t)t * H + h), widen(wr, dtype, (int64_t)e * H + h), acc);
      logits[(int64_t)t * E + e] = bias ? acc + bias[e] : acc;
    }
  }
  return 0;
}

/*
 * Step 1b, normalisation and top-k selection, from given logits [T,E].
 * Selection: k rounds; each round takes the not-yet-taken expert with the largest logit, the
 * lowest index among equals.  So topk_idx[t,:] is in descending logit order.
 * Weights: softmax over all E experts (fp64, shifted by the largest logit), the selected
 * probabilities; with renormalize != 0 they are divided by their own sum.
 */
int oracle_topk(int T, int E, int K, int renormalize, const float *logits, int32_t *topk_idx,
                float *topk_w) {
  if (T < 0 || E <= 0 || K <= 0 || K > E) return -1;
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    const float *l = logits + (int64_t)t * E;
    int32_t *idx = topk_idx + (int64_t)t * K;
    for (int k = 0; k < K; ++k) {
      int best = -1;
      for (int e = 0; e < E; ++e) {
        int taken = 0;
        for (int j = 0; j < k; ++j) taken |= (idx[j] == e);
        if (taken) continue;
        if (best < 0 || l[e] > l[best]) best = e; /* strict >: the lowest index wins a tie */
      }
      idx[k] = best;
    }
    double m = (double)l[idx[0]];
    double Z = 0.0;
    for (int e = 0; e < E; ++e) Z += exp((double)l[e] - m);
    double sel = 0.0;
    for (int k = 0; k < K; ++k) sel += exp((double)l[idx[k]] - m) / Z;
    for (int k = 0; k < K; ++k) {
      double p = exp((double)l[idx[k]] - m) / Z;
      topk_w[(int64_t)t * K + k] = (float)(renormalize ? p / sel : p);
    }
  }
  return 0;
}

/* Step 1 whole: logits then top-k.  logits_out [T,E] may be NULL. */
int oracle_route(int T, int H, int E, int K, int dtype, int renormalize, const void *x,
                 const void *wr, const float *bias, int32_t *topk_idx, float *topk_w,
                 float *logits_out) {
  if (T < 0 || H <= 0 || E <= 0 || K <= 0 || K > E) return -1;
  float *l = logits_out ? logits_out : (float *)malloc(sizeof(float) * (size_t)(T > 0 ? T : 1) * E);
  if (!l) return -2;
  int rc = oracle_logits(T, H, E, dtype, x, wr, bias, l);
  if (rc == 0) rc = oracle_topk(T, E, K, renormalize, l, topk_idx, topk_w);
  if (!logits_out) free(l);
  return rc;
}

/*
 * Step 2, dispatch layout (the "software mediation": counts, exclusive scan, slot offsets,
 * scatter).  count[E]; offset[E+1] (offset[0]=0, offset[e+1]=offset[e]+count[e]);
 * rank_count[R] = rows received by logical rank r, expert e living on rank e/(E/R);
 * recv [T*K,H] in the input dtype: expert e's rows are offset[e] .. offset[e+1]-1, filled in
 * (t ascending, k ascending) order; src[pos] = t*K+k; slot_of[t*K+k] = pos.
 * recv may be NULL (layout only).
 */
int oracle_dispatch(int T, int H, int E, int R, int K, int dtype, const void *x,
                    const int32_t *topk_idx, int32_t *count, int32_t *offset, int32_t *rank_count,
                    void *recv, int32_t *src, int32_t *slot_of) {
  if (T < 0 || H <= 0 || E <= 0 || R <= 0 || E % R || K <= 0 || K > E) return -1;
  for (int e = 0; e < E; ++e) count[e] = 0;
  for (int64_t a = 0; a < (int64_t)T * K; ++a) {
    int e = topk_idx[a];
    if (e < 0 || e >= E) return -3;
    count[e]++;
  }
  offset[0] = 0;
  for (int e = 0; e < E; ++e) offset[e + 1] = offset[e] + count[e];
  if (rank_count) {
    for (int r = 0; r < R; ++r) rank_count[r] = 0;
    for (int e = 0; e < E; ++e) rank_count[e / (E / R)] += count[e];
  }
  int32_t *fill = (int32_t *)calloc((size_t)E, sizeof(int32_t));
  if (!fill) return -2;
  const size_t row_bytes = (size_t)H * elem_bytes(dtype);
  for (int t = 0; t < T; ++t) {
    for (int k = 0; k < K; ++k) {
      int e = topk_idx[(int64_t)t * K + k];
      int32_t pos = offset[e] + fill[e]++;
      if (recv) memcpy((char *)recv + (size_t)pos * row_bytes, (const char *)x + (size_t)t * row_bytes, row_bytes);
      src[pos] = t * K + k;
      slot_of[(int64_t)t * K + k] = pos;
    }
  }
  free(fill);
  return 0;
}

/*
 * Step 3, expert computation on the dispatched rows (SwiGLU):
 *   g_f = sum_h a_h*Wg[e,f,h],  u_f = sum_h a_h*Wu[e,f,h],  s_f = g_f/(1+exp(-g_f)) * u_f,
 *   o_j = sum_f s_f*Wd[e,j,f].
 * fp64 throughout, no intermediate rounding.  recv: [rows,H] (input dtype), expert e owns rows
 * offset[e]..offset[e+1]-1.  wg/wu/wd are arrays of E pointers to that expert's [F,H], [F,H],
 * [H,F] matrices (an expert without rows may have NULL pointers: its weights are never read).
 * out: [rows,H] fp64.
 */
static int expert_ffn_impl(int H, int F, int E, int dtype, const void *recv, const int32_t *offset,
                           const void *const *wg, const void *const *wu, const void *const *wd,
                           double *out, int stored) {
  if (H <= 0 || F <= 0 || E <= 0) return -1;
  for (int e = 0; e < E; ++e) {
    const int r0 = offset[e], r1 = offset[e + 1];
    if (r1 == r0) continue;
    if (!wg[e] || !wu[e] || !wd[e]) return -4;
#pragma omp parallel
    {
      double *a = (double *)malloc(sizeof(double) * (size_t)H);
      double *s = (double *)malloc(sizeof(double) * (size_t)F);
#pragma omp for schedule(dynamic, 1)
      for (int r = r0; r < r1; ++r) {
        for (int h = 0; h < H; ++h) a[h] = (double)widen(recv, dtype, (int64_t)r * H + h);
        for (int f = 0; f < F; ++f) {
          double g = 0.0, u = 0.0;
          for (int h = 0; h < H; ++h) g += a[h] * (double)widen(wg[e], dtype, (int64_t)f * H + h);
          for (int h = 0; h < H; ++h) u += a[h] * (double)widen(wu[e], dtype, (int64_t)f * H + h);
          s[f] = g / (1.0 + exp(-g)) * u;
          if (stored) s[f] = oracle_round_bf16(s[f]); /* the intermediate is kept in bf16 */
        }
        for (int j = 0; j < H; ++j) {
          double o = 0.0;
          for (int f = 0; f < F; ++f) o += s[f] * (double)widen(wd[e], dtype, (int64_t)j * F + f);
          out[(int64_t)r * H + j] = stored ? oracle_round_bf16(o) : o; /* expert output rows in bf16 */
        }
      }
      free(a);
      free(s);
    }
  }
  return 0;
}

int oracle_expert_ffn(int H, int F, int E, int dtype, const void *recv, const int32_t *offset,
                      const void *const *wg, const void *const *wu, const void *const *wd,
                      double *out) {
  return expert_ffn_impl(H, F, E, dtype, recv, offset, wg, wu, wd, out, 0);
}

/* Diagnostic mode: step 3 with the intermediate and the output rows rounded to bf16 (see the header). */
int oracle_expert_ffn_stored(int H, int F, int E, int dtype, const void *recv, const int32_t *offset,
                             const void *const *wg, const void *const *wu, const void *const *wd,
                             double *out) {
  return expert_ffn_impl(H, F, E, dtype, recv, offset, wg, wu, wd, out, 1);
}

/* Identity experts: o = a (used by the dispatch/combine-only sweep). out: [rows,H] fp64. */
int oracle_identity_ffn(int64_t rows, int H, int dtype, const void *recv, double *out) {
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r)
    for (int h = 0; h < H; ++h) out[r * H + h] = (double)widen(recv, dtype, r * H + h);
  return 0;
}

/*
 * Steps 4+5, combine and scaling: y[t,j] = sum_{k ascending} w[t,k] * rows[slot_of[t,k], j].
 * rows: [*,H] fp64, y: [T,H] fp64.
 */
static int combine_impl(int T, int H, int K, const double *rows, const int32_t *slot_of,
                        const float *topk_w, double *y, int stored) {
  if (T < 0 || H <= 0 || K <= 0) return -1;
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    for (int j = 0; j < H; ++j) {
      double acc = 0.0;
      for (int k = 0; k < K; ++k)
        acc += (double)topk_w[(int64_t)t * K + k] * rows[(int64_t)slot_of[(int64_t)t * K + k] * H + j];
      y[(int64_t)t * H + j] = stored ? oracle_round_bf16(acc) : acc;
    }
  }
  return 0;
}

int oracle_combine(int T, int H, int K, const double *rows, const int32_t *slot_of,
                   const float *topk_w, double *y) {
  return combine_impl(T, H, K, rows, slot_of, topk_w, y, 0);
}

/* Diagnostic mode: steps 4+5 with y rounded to bf16 (see the header). */
int oracle_combine_stored(int T, int H, int K, const double *rows, const int32_t *slot_of,
                          const float *topk_w, double *y) {
  return combine_impl(T, H, K, rows, slot_of, topk_w, y, 1);
}
