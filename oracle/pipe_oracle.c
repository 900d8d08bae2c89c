/*
 * pipe_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, single-pass-per-definition CPU statement of the residual-expanded
 * quantized layer of PIPE (arXiv 2311.15806).  It exists so that the CUDA library can be
 * checked against something written directly from the paper; it shares no code, header,
 * table or helper with the CUDA path and is never linked into or called by it.
 *
 * Every function cites the passage of the paper it follows.  Where the paper leaves a
 * choice open the reading taken is stated in the comment of the function.
 *
 * Arithmetic: the quantizer works in IEEE binary32 (the codes and scales it emits are the
 * object of bit-exact comparison, so the precision is part of the definition): true
 * division, round-half-to-even, one fused multiply-add per residual element.  The
 * contraction is exact integer arithmetic accumulated in int64 and checked to fit int32.
 * Compile with -ffp-contract=off so that no multiply-add is fused except the explicit fmaf.
 *
 * Parity pins (tests/test_oracle_*.py): exponential decrease of the reconstruction error
 * (Lemma B.1 / Sec. 3.1), exact recovery of representable weights, gamma = 1 & M = 1
 * equal to the plain expansion, selection invariants, NumPy integer matmul special case,
 * brute force on tiny inputs in exact rational arithmetic.
 * Parity unpinned: WHICH groups a trained network should keep (the paper gives no
 * criterion for the structured mask; see pipe_oracle_select_groups).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_ERR_ARG 1
#define ORACLE_ERR_NONFINITE 2
#define ORACLE_ERR_ACC_OVERFLOW 3

/* Number of threads the row-parallel loops will use (reported next to timings). */
int pipe_oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Largest code magnitude of a symmetric b-bit quantizer: 2^(b-1) - 1 (the constant of
 * Eq. 5 and Lemma B.1).  b = 2 is the ternary case {-1, 0, +1} named in the introduction. */
static int qmax_of_bits(int bits) { return (1 << (bits - 1)) - 1; }

/* ---------------------------------------------------------------------------------------
 * Sec. 3 "Methodology overview", Eq. 1 with the symmetric per-channel setting of Sec. 4.1:
 * the scale of an output channel comes from the largest magnitude of its row.
 * a[o] = max_i |r[o,i]|.  Returns ORACLE_ERR_NONFINITE if a value is NaN or infinite.
 * ------------------------------------------------------------------------------------- */
int pipe_oracle_row_absmax(const float* r, int64_t O, int64_t I, int64_t ld, float* a) {
  int bad = 0;
#pragma omp parallel for schedule(static) reduction(| : bad)
  for (int64_t o = 0; o < O; ++o) {
    float m = 0.0f;
    for (int64_t i = 0; i < I; ++i) {
      float v = r[o * ld + i];
      if (!isfinite(v)) bad |= 1;
      float av = fabsf(v);
      if (av > m) m = av;
    }
    a[o] = m;
  }
  return bad ? ORACLE_ERR_NONFINITE : ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------
 * Sec. 3.1, masked expansion (the equation with M^K): the structured mask keeps whole
 * output channels ("row-wise zeros"; Sec. 4.1: sparsity is applied to neurons/channels).
 * The paper does not say how the kept channels are chosen.  Reading taken here: channels
 * are grouped g consecutive rows at a time; the score of a group is the largest magnitude
 * of the CURRENT residual over the group's rows (the infinity-norm flavour of Lemma B.2);
 * the n_keep highest-scoring groups are kept, ties going to the lower group index; the
 * kept set is emitted as an ascending list.
 * a: [G*g] row absmax of the current residual.  kept_out: [n_keep].
 * ------------------------------------------------------------------------------------- */
typedef struct {
  float score;
  int32_t index;
} group_score;

static int cmp_score_desc_index_asc(const void* pa, const void* pb) {
  const group_score* x = (const group_score*)pa;
  const group_score* y = (const group_score*)pb;
  if (x->score > y->score) return -1;
  if (x->score < y->score) return 1;
  return (x->index > y->index) - (x->index < y->index);
}

static int cmp_int32_asc(const void* pa, const void* pb) {
  int32_t x = *(const int32_t*)pa, y = *(const int32_t*)pb;
  return (x > y) - (x < y);
}

int pipe_oracle_select_groups(const float* a, int32_t G, int32_t g, int32_t n_keep, int32_t* kept_out) {
  if (G <= 0 || g <= 0 || n_keep < 1 || n_keep > G) return ORACLE_ERR_ARG;
  group_score* gs = (group_score*)malloc(sizeof(group_score) * (size_t)G);
  if (!gs) return ORACLE_ERR_ARG;
  for (int32_t j = 0; j < G; ++j) {
    float m = 0.0f;
    for (int32_t u = 0; u < g; ++u) {
      float v = a[(int64_t)j * g + u];
      if (v > m) m = v;
    }
    gs[j].score = m;
    gs[j].index = j;
  }
  qsort(gs, (size_t)G, sizeof(group_score), cmp_score_desc_index_asc);
  for (int32_t n = 0; n < n_keep; ++n) kept_out[n] = gs[n].index;
  qsort(kept_out, (size_t)n_keep, sizeof(int32_t), cmp_int32_asc);
  free(gs);
  return ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------
 * Sec. 3.1 "Residual Expansion": R^1 = Q^-1(Q(W)), R^K = M^K Q^-1(Q(W - sum_{k<K} R^k)),
 * with Q of Eq. 1 (scale, then round to nearest) applied per output channel.
 *
 * For k = 1..K on the running residual r (r = W at k = 1):
 *   a[o]   = max_i |r[o,i]|
 *   kept_k = all groups for k = 1 (first order is dense in every experiment of the paper)
 *            or when n_keep == G; else the n_keep groups chosen by pipe_oracle_select_groups
 *   for every row o of a kept group, in ascending row order:
 *       s     = a[o] / qmax                         (binary32 division)
 *       q[i]  = clamp(rne(r[o,i] / s), -qmax, qmax) (binary32 division, ties to even)
 *       r[o,i]= fma(-s, q[i], r[o,i])               (one rounding: the exact new residual, rounded)
 *     a row whose scale is zero (all-zero residual, or a/qmax underflowing to zero) emits
 *     zero codes, scale 0 and keeps its residual
 *   rows of pruned groups emit nothing and keep their residual: the sum inside Q at the
 *   next order uses the MASKED R^k, so their error carries over.
 *
 * Outputs (caller-allocated, compacted in kept order, orders back to back):
 *   codes  : int8, one code per byte, [sum_k rows_k, I],  rows_k = kept_count[k]*g
 *   scales : float, [sum_k rows_k]
 *   kept   : int32, [K, G] (first kept_count[k] entries of each row valid, ascending)
 *   kept_count : int32 [K]
 *   residual   : float [O, I] work buffer; holds W - sum_k s_k q_k (as tracked) on return
 *   absmax_trace : optional float [K, O], the a[] seen at each order
 * ------------------------------------------------------------------------------------- */
int pipe_oracle_expand(const float* W, int64_t O, int64_t I, int64_t ldw, int bits, int K, int32_t g,
                       int32_t n_keep, int8_t* codes, float* scales, int32_t* kept, int32_t* kept_count,
                       float* residual, float* absmax_trace) {
  if (O <= 0 || I <= 0 || K < 1 || g < 1 || O % g != 0) return ORACLE_ERR_ARG;
  if (!(bits == 8 || bits == 4 || bits == 2)) return ORACLE_ERR_ARG;
  const int32_t G = (int32_t)(O / g);
  if (n_keep < 1 || n_keep > G) return ORACLE_ERR_ARG;
  const int qmax = qmax_of_bits(bits);
  const float fq = (float)qmax;

  for (int64_t o = 0; o < O; ++o) memcpy(residual + o * I, W + o * ldw, sizeof(float) * (size_t)I);
  float* a = (float*)malloc(sizeof(float) * (size_t)O);
  if (!a) return ORACLE_ERR_ARG;

  int64_t row_base = 0;
  for (int k = 0; k < K; ++k) {
    int rc = pipe_oracle_row_absmax(residual, O, I, I, a);
    if (rc != ORACLE_OK) {
      free(a);
      return rc;
    }
    if (absmax_trace) memcpy(absmax_trace + (int64_t)k * O, a, sizeof(float) * (size_t)O);
    int32_t* kept_k = kept + (int64_t)k * G;
    int32_t count;
    if (k == 0 || n_keep == G) {
      count = G;
      for (int32_t j = 0; j < G; ++j) kept_k[j] = j;
    } else {
      count = n_keep;
      rc = pipe_oracle_select_groups(a, G, g, n_keep, kept_k);
      if (rc != ORACLE_OK) {
        free(a);
        return rc;
      }
    }
    kept_count[k] = count;
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < (int64_t)count * g; ++n) {
      const int64_t o = (int64_t)kept_k[n / g] * g + n % g;
      const float s = a[o] / fq;
      int8_t* q = codes + (row_base + n) * I;
      float* r = residual + o * I;
      scales[row_base + n] = s;
      if (s == 0.0f) {
        for (int64_t i = 0; i < I; ++i) q[i] = 0;
        continue;
      }
      for (int64_t i = 0; i < I; ++i) {
        float v = nearbyintf(r[i] / s); /* default rounding mode: ties to even */
        if (v > fq) v = fq;
        if (v < -fq) v = -fq;
        q[i] = (int8_t)v;
        r[i] = fmaf(-s, v, r[i]);
      }
    }
    row_base += (int64_t)count * g;
  }
  free(a);
  return ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------
 * Storage format of sub-byte codes (the paper stores nothing packed; this is the format
 * the library documents).  Two's complement fields, element e of a row at bit offset e*b
 * of the little-endian bit stream of that row: int4 -> element 2j in bits 0-3 of byte j,
 * element 2j+1 in bits 4-7; ternary -> element 4j+e in bits 2e..2e+1 of byte j
 * (00 = 0, 01 = +1, 11 = -1).  A ragged last byte is padded with zero fields.
 * out: [rows, ceil(I*bits/8)].
 * ------------------------------------------------------------------------------------- */
int pipe_oracle_pack(const int8_t* codes, int64_t rows, int64_t I, int bits, uint8_t* out) {
  if (!(bits == 8 || bits == 4 || bits == 2)) return ORACLE_ERR_ARG;
  const int per = 8 / bits;
  const int64_t nb = (I + per - 1) / per;
  const unsigned mask = (1u << bits) - 1u;
  for (int64_t r = 0; r < rows; ++r) {
    for (int64_t j = 0; j < nb; ++j) {
      unsigned byte = 0;
      for (int e = 0; e < per; ++e) {
        int64_t i = j * per + e;
        if (i < I) byte |= ((unsigned)(int)codes[r * I + i] & mask) << (e * bits);
      }
      out[r * nb + j] = (uint8_t)byte;
    }
  }
  return ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------
 * Appendix B, Eq. 9 (the expanded layer): the input enters as Q(x) with one scale
 * lambda_x for the whole tensor (Sec. 4.1: static, symmetric; activations are int8 here).
 * Reading: lambda_x = max|x| / 127 computed from the tensor itself unless the caller
 * supplies a static scale, in which case values are clamped to +-127.
 * xq[n] = clamp(rne(x[n] / lambda_x), -127, 127); lambda_x == 0 gives all-zero codes.
 * ------------------------------------------------------------------------------------- */
int pipe_oracle_quantize_act(const float* x, int64_t T, int64_t I, int64_t ldx, const float* static_scale,
                             int8_t* xq, int64_t ldxq, float* sx_out) {
  float sx;
  int bad = 0;
  float m = 0.0f;
  for (int64_t t = 0; t < T; ++t)
    for (int64_t i = 0; i < I; ++i) {
      float v = x[t * ldx + i];
      if (!isfinite(v)) bad = 1;
      float av = fabsf(v);
      if (av > m) m = av;
    }
  if (bad) return ORACLE_ERR_NONFINITE;
  if (static_scale) {
    sx = *static_scale;
    if (!(sx >= 0.0f) || !isfinite(sx)) return ORACLE_ERR_ARG;
  } else {
    sx = m / 127.0f;
  }
  *sx_out = sx;
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < T; ++t)
    for (int64_t i = 0; i < I; ++i) {
      if (sx == 0.0f) {
        xq[t * ldxq + i] = 0;
        continue;
      }
      float v = nearbyintf(x[t * ldx + i] / sx);
      if (v > 127.0f) v = 127.0f;
      if (v < -127.0f) v = -127.0f;
      xq[t * ldxq + i] = (int8_t)v;
    }
  return ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------
 * Appendix B, Eq. 9 restricted to one cluster of successive orders (Sec. 3.2; Appendix B:
 * predictor m owns the K_m orders that come right after the clusters of predictors 1..m-1):
 *
 *   acc_k[t, o] = sum_i xq[t,i] * q_k[o,i]                       (exact integers)
 *   y[t, o]     = sum over k = k_begin..k_end-1 ascending, o kept at order k, of
 *                 acc_k[t,o] * lambda_{R^(k)}[o] * lambda_x       (+ b[o] when bias given)
 *
 * Reading of the floating-point order (the paper gives none): the scale product
 * c = s_k[o] * lambda_x is formed first in binary32, each term enters the running sum
 * with one fused multiply-add y = fma((float)acc, c, y) starting from y = 0, the bias is
 * added last.  y64 / yabs (optional) hold the same sum and the sum of term magnitudes
 * evaluated in binary64 from the same integers and scales, for tolerance checks.
 *
 * codes/scales/kept/kept_count are the outputs of pipe_oracle_expand.  partials
 * (optional) is int32 [T, R_total], R_total = sum over ALL K orders of rows_k; order k's
 * columns start at sum_{j<k} rows_j; only the columns of the cluster's orders are written.
 * ------------------------------------------------------------------------------------- */
int pipe_oracle_forward(const int8_t* xq, int64_t T, int64_t I, int64_t ldxq, int64_t O, int K, int32_t g,
                        const int8_t* codes, const float* scales, const int32_t* kept, const int32_t* kept_count,
                        int k_begin, int k_end, float sx, const float* bias, float* y, int64_t ldy,
                        double* y64, double* yabs, int32_t* partials) {
  if (k_begin < 0 || k_end > K || k_begin >= k_end || O % g != 0) return ORACLE_ERR_ARG;
  const int32_t G = (int32_t)(O / g);
  int64_t R_total = 0;
  int64_t row_off[64];
  if (K > 64) return ORACLE_ERR_ARG;
  for (int k = 0; k < K; ++k) {
    row_off[k] = R_total;
    R_total += (int64_t)kept_count[k] * g;
  }
  /* group -> position in the kept list of each order of the cluster, -1 when pruned */
  int32_t* pos = (int32_t*)malloc(sizeof(int32_t) * (size_t)G * (size_t)(k_end - k_begin));
  if (!pos) return ORACLE_ERR_ARG;
  for (int k = k_begin; k < k_end; ++k) {
    int32_t* p = pos + (int64_t)(k - k_begin) * G;
    for (int32_t j = 0; j < G; ++j) p[j] = -1;
    for (int32_t n = 0; n < kept_count[k]; ++n) p[kept[(int64_t)k * G + n]] = n;
  }
  int overflow = 0;
#pragma omp parallel for schedule(static) reduction(| : overflow)
  for (int64_t t = 0; t < T; ++t) {
    const int8_t* xr = xq + t * ldxq;
    for (int64_t o = 0; o < O; ++o) {
      float acc_y = 0.0f;
      double acc64 = 0.0, accabs = 0.0;
      for (int k = k_begin; k < k_end; ++k) {
        const int32_t n = pos[(int64_t)(k - k_begin) * G + o / g];
        if (n < 0) continue; /* row of a pruned group: R^k has a zero row there */
        const int64_t row = row_off[k] + (int64_t)n * g + o % g;
        const int8_t* qr = codes + row * I;
        int64_t acc = 0;
        for (int64_t i = 0; i < I; ++i) acc += (int64_t)xr[i] * (int64_t)qr[i];
        if (acc > INT32_MAX || acc < INT32_MIN) overflow |= 1;
        if (partials) partials[t * R_total + row] = (int32_t)acc;
        const float c = scales[row] * sx;
        acc_y = fmaf((float)(int32_t)acc, c, acc_y);
        const double term = (double)acc * (double)scales[row] * (double)sx;
        acc64 += term;
        accabs += fabs(term);
      }
      if (bias) {
        acc_y = acc_y + bias[o];
        acc64 += (double)bias[o];
        accabs += fabs((double)bias[o]);
      }
      y[t * ldy + o] = acc_y;
      if (y64) y64[t * O + o] = acc64;
      if (yabs) yabs[t * O + o] = accabs;
    }
  }
  free(pos);
  return overflow ? ORACLE_ERR_ACC_OVERFLOW : ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------
 * Sec. 3.2 "Ensembling from Expansion" and Fig. 2: the K orders are cut into M clusters of
 * successive orders [K_1..K_M]; predictor m evaluates only its cluster, on its own input
 * x_m with its own lambda_{x_m}; the bias lives in predictor 1 only; predictor outputs are
 * added after the last layer.  One layer of that scheme:
 *   y_m = forward(cluster m, xq_m, sx_m, bias if m == 1)
 *   if sum_branches: y = ((y_1 + y_2) + ...) + y_M, binary32, ascending m.
 * xq: [M, T, I] (the caller repeats the tensor for a shared input), sx: [M],
 * y: [M, T, O], or [T, O] when sum_branches != 0; partials as in pipe_oracle_forward.
 * ------------------------------------------------------------------------------------- */
int pipe_oracle_ensemble(const int8_t* xq, int64_t T, int64_t I, int64_t O, int K, int32_t g, const int8_t* codes,
                         const float* scales, const int32_t* kept, const int32_t* kept_count, int M,
                         const int32_t* branch_orders, const float* sx, const float* bias, int sum_branches,
                         float* y, int32_t* partials) {
  int total = 0;
  for (int m = 0; m < M; ++m) {
    if (branch_orders[m] < 1) return ORACLE_ERR_ARG;
    total += branch_orders[m];
  }
  if (total != K) return ORACLE_ERR_ARG;
  float* tmp = NULL;
  if (sum_branches) {
    tmp = (float*)malloc(sizeof(float) * (size_t)(T * O));
    if (!tmp) return ORACLE_ERR_ARG;
  }
  int k0 = 0, rc = ORACLE_OK;
  for (int m = 0; m < M; ++m) {
    float* dst = sum_branches ? (m == 0 ? y : tmp) : y + (int64_t)m * T * O;
    int r = pipe_oracle_forward(xq + (int64_t)m * T * I, T, I, I, O, K, g, codes, scales, kept, kept_count, k0,
                                k0 + branch_orders[m], sx[m], m == 0 ? bias : NULL, dst, O, NULL, NULL, partials);
    if (r != ORACLE_OK) rc = r;
    if (sum_branches && m > 0)
      for (int64_t n = 0; n < T * O; ++n) y[n] = y[n] + tmp[n];
    k0 += branch_orders[m];
  }
  free(tmp);
  return rc;
}

/* Sec. 3.2 / Appendix A: the printed splits ([4,4], [3,3,2], [2,2,2,2] for K = 8; [2,2] for
 * K = 4) are all "balanced, remainder to the earliest predictors", and K_1 should be the
 * largest.  K_m = floor(K/M) + (m <= K mod M), m = 1..M. */
int pipe_oracle_balanced_split(int K, int M, int32_t* out) {
  if (K < 1 || M < 1 || M > K) return ORACLE_ERR_ARG;
  for (int m = 0; m < M; ++m) out[m] = K / M + (m < K % M ? 1 : 0);
  return ORACLE_OK;
}

/* Sec. 3.1: "the pruning ratio is given by a sparsity parameter gamma in order to match a
 * total budget of operations": gamma is the KEPT fraction of an order's channel groups
 * (Sec. 4.3 counts a 50 % residue on top of a 4-bit layer as 150 %).  Kept groups per
 * order >= 2: ceil(gamma * G), evaluated in binary64 with a 1e-9 guard against a product
 * that lands a hair above an integer, clamped to [1, G]. */
int32_t pipe_oracle_keep_groups(int32_t G, double gamma) {
  double v = ceil(gamma * (double)G - 1e-9);
  if (v < 1.0) v = 1.0;
  if (v > (double)G) v = (double)G;
  return (int32_t)v;
}
