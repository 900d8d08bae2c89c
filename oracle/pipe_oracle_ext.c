/*
 * pipe_oracle_ext.c -- TEST INFRASTRUCTURE, not product code.
 *
 * The CPU oracle for the variants of the method the paper uses beside its main setting
 * (arXiv 2311.15806): other weight bit-widths (Sec. 4.2: int3, int6), narrower activations
 * (Sec. 4.3: W4/A6, W4/A4), asymmetric activation quantization (Sec. 4.3, the parallelized
 * comparison), a second score for the structured mask and the unstructured mask of Sec. 3.1.
 * Same rules as pipe_oracle.c: plain loops in the paper's order, binary32 quantizer with true
 * division and round-half-to-even, exact integer contraction, nothing shared with the CUDA
 * path.  The functions of pipe_oracle.c are left as they are; these stand beside them.
 *
 * Parity pins (tests/test_oracle_ext_pins.py): half-step residual invariant and exact
 * recovery for every bit-width, NumPy / exact-rational brute force of the activation
 * quantizers, the zero-point identity acc(c - z) = acc(c) - z * rowsum against NumPy integer
 * matmul, the score against math.fsum, the unstructured mask against an independent argsort.
 * Parity unpinned: WHICH weights or groups a trained network should keep (the paper states no
 * criterion for either mask).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_ERR_ARG 1
#define ORACLE_ERR_NONFINITE 2
#define ORACLE_ERR_ACC_OVERFLOW 3

static int bits_ok(int bits) { return bits == 8 || bits == 6 || bits == 4 || bits == 3 || bits == 2; }
/* Largest code magnitude of a symmetric b-bit quantizer (Appendix B, Lemma B.1: 2^(b-1) - 1). */
static int qmax_of(int bits) { return (1 << (bits - 1)) - 1; }

/* ---------------------------------------------------------------------------------------
 * Second score of the structured mask (Sec. 3.1 leaves the criterion open): the squared
 * Euclidean norm of the CURRENT residual over the group's rows.  A sum of squares depends on
 * the order of its additions in the last bits, so the order is part of the definition:
 *   P_l   = sum over i = l, l + 32, l + 64, ... (ascending) of (double) r[o,i]^2,  l = 0..31
 *           (each square is exact in binary64; the additions round)
 *   S[o]  = tree over the 32 partial sums: for off = 16, 8, 4, 2, 1: P_l += P_{l+off} (l < off)
 *   score = sum over the group's rows, ascending, of S[o]       (binary64)
 * ------------------------------------------------------------------------------------- */
static double row_sumsq(const float* r, int64_t I) {
  double P[32];
  for (int l = 0; l < 32; ++l) {
    double s = 0.0;
    for (int64_t i = l; i < I; i += 32) {
      const double v = (double)r[i];
      s = s + v * v;
    }
    P[l] = s;
  }
  for (int off = 16; off >= 1; off >>= 1)
    for (int l = 0; l < off; ++l) P[l] = P[l] + P[l + off];
  return P[0];
}

typedef struct {
  double score;
  int32_t index;
} scored;

static int cmp_scored(const void* pa, const void* pb) {
  const scored* x = (const scored*)pa;
  const scored* y = (const scored*)pb;
  if (x->score > y->score) return -1;
  if (x->score < y->score) return 1;
  return (x->index > y->index) - (x->index < y->index);
}
static int cmp_i32(const void* pa, const void* pb) {
  int32_t x = *(const int32_t*)pa, y = *(const int32_t*)pb;
  return (x > y) - (x < y);
}

/* score_out (optional): double [G].  score_mode 0: max-abs of the group's rows (as in
 * pipe_oracle_select_groups); 1: the squared Euclidean norm defined above.  Ties go to the
 * lower group index, the kept set is returned ascending. */
int pipe_oracle_select_groups_ex(const float* r, int64_t O, int64_t I, int32_t g, int32_t n_keep, int score_mode,
                                 int32_t* kept_out, double* score_out) {
  if (O <= 0 || I <= 0 || g < 1 || O % g != 0 || (score_mode != 0 && score_mode != 1)) return ORACLE_ERR_ARG;
  const int32_t G = (int32_t)(O / g);
  if (n_keep < 1 || n_keep > G) return ORACLE_ERR_ARG;
  scored* gs = (scored*)malloc(sizeof(scored) * (size_t)G);
  if (!gs) return ORACLE_ERR_ARG;
  for (int32_t j = 0; j < G; ++j) {
    double s = 0.0;
    for (int32_t u = 0; u < g; ++u) {
      const float* row = r + ((int64_t)j * g + u) * I;
      if (score_mode == 0) {
        for (int64_t i = 0; i < I; ++i) {
          const double av = fabs((double)row[i]);
          if (av > s) s = av;
        }
      } else {
        s = s + row_sumsq(row, I);
      }
    }
    gs[j].score = s;
    gs[j].index = j;
    if (score_out) score_out[j] = s;
  }
  qsort(gs, (size_t)G, sizeof(scored), cmp_scored);
  for (int32_t n = 0; n < n_keep; ++n) kept_out[n] = gs[n].index;
  qsort(kept_out, (size_t)n_keep, sizeof(int32_t), cmp_i32);
  free(gs);
  return ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------
 * Sec. 3.1 "Residual Expansion" with the general mask M^k, for b in {2, 3, 4, 6, 8}
 * (Sec. 4.2 runs the method at int3, int4, int6 and ternary):
 * the recursion of pipe_oracle_expand, with
 *   - score_mode choosing the score of the structured mask (see above);
 *   - elem_keep > 0: the UNSTRUCTURED mask of Sec. 3.1 on the orders k >= 2 ("a sparse
 *     tensor").  Reading (the paper states the ratio gamma, not the criterion): in every row
 *     the elem_keep entries of the current residual with the largest magnitude are kept, ties
 *     going to the lower index; the others get the code 0 and keep their residual.  The
 *     row's scale is still max|r| / qmax (its largest entry is always among the kept ones).
 *     The structured mask is then not applied (n_keep must equal G): R^k stays a full-height
 *     tensor with zeros in it.
 * Outputs as pipe_oracle_expand (codes one per byte, compacted rows, orders back to back).
 * ------------------------------------------------------------------------------------- */
typedef struct {
  float mag;
  int64_t index;
} elem;

static int cmp_elem(const void* pa, const void* pb) {
  const elem* x = (const elem*)pa;
  const elem* y = (const elem*)pb;
  if (x->mag > y->mag) return -1;
  if (x->mag < y->mag) return 1;
  return (x->index > y->index) - (x->index < y->index);
}

int pipe_oracle_expand_ex(const float* W, int64_t O, int64_t I, int64_t ldw, int bits, int K, int32_t g, int32_t n_keep,
                          int score_mode, int64_t elem_keep, int8_t* codes, float* scales, int32_t* kept,
                          int32_t* kept_count, float* residual) {
  if (O <= 0 || I <= 0 || K < 1 || g < 1 || O % g != 0 || !bits_ok(bits)) return ORACLE_ERR_ARG;
  const int32_t G = (int32_t)(O / g);
  if (n_keep < 1 || n_keep > G || elem_keep < 0 || elem_keep > I) return ORACLE_ERR_ARG;
  if (elem_keep > 0 && n_keep != G) return ORACLE_ERR_ARG;
  const float fq = (float)qmax_of(bits);
  for (int64_t o = 0; o < O; ++o) memcpy(residual + o * I, W + o * ldw, sizeof(float) * (size_t)I);
  for (int64_t n = 0; n < O * I; ++n)
    if (!isfinite(residual[n])) return ORACLE_ERR_NONFINITE;
  elem* order = (elem*)malloc(sizeof(elem) * (size_t)I);
  uint8_t* keep_e = (uint8_t*)malloc((size_t)I);
  if (!order || !keep_e) return ORACLE_ERR_ARG;

  int64_t row_base = 0;
  for (int k = 0; k < K; ++k) {
    int32_t* kept_k = kept + (int64_t)k * G;
    int32_t count = G;
    if (k == 0 || n_keep == G) {
      for (int32_t j = 0; j < G; ++j) kept_k[j] = j;
    } else {
      count = n_keep;
      int rc = pipe_oracle_select_groups_ex(residual, O, I, g, n_keep, score_mode, kept_k, NULL);
      if (rc != ORACLE_OK) return rc;
    }
    kept_count[k] = count;
    for (int64_t n = 0; n < (int64_t)count * g; ++n) {
      const int64_t o = (int64_t)kept_k[n / g] * g + n % g;
      float* r = residual + o * I;
      float a = 0.0f;
      for (int64_t i = 0; i < I; ++i) {
        const float av = fabsf(r[i]);
        if (av > a) a = av;
      }
      const float s = a / fq;
      int8_t* q = codes + (row_base + n) * I;
      scales[row_base + n] = s;
      memset(keep_e, 1, (size_t)I);
      if (elem_keep > 0 && k > 0) {
        for (int64_t i = 0; i < I; ++i) {
          order[i].mag = fabsf(r[i]);
          order[i].index = i;
        }
        qsort(order, (size_t)I, sizeof(elem), cmp_elem);
        memset(keep_e, 0, (size_t)I);
        for (int64_t i = 0; i < elem_keep; ++i) keep_e[order[i].index] = 1;
      }
      for (int64_t i = 0; i < I; ++i) {
        if (s == 0.0f || !keep_e[i]) {
          q[i] = 0;
          continue;
        }
        float v = nearbyintf(r[i] / s);
        if (v > fq) v = fq;
        if (v < -fq) v = -fq;
        q[i] = (int8_t)v;
        r[i] = fmaf(-s, v, r[i]);
      }
    }
    row_base += (int64_t)count * g;
  }
  free(order);
  free(keep_e);
  return ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------
 * Packed form of the codes when b has no storage format of its own: 3-bit codes travel in
 * 4-bit fields and 6-bit codes in bytes (two's complement, the bit order of pipe_oracle_pack);
 * the paper stores nothing packed, so this only fixes what the library is compared against.
 * out: [rows, ceil(I * container / 8)], container = 2, 4, 4, 8, 8 for b = 2, 3, 4, 6, 8.
 * ------------------------------------------------------------------------------------- */
int pipe_oracle_container_bits(int bits) { return bits == 2 ? 2 : (bits <= 4 ? 4 : 8); }

int pipe_oracle_pack_ex(const int8_t* codes, int64_t rows, int64_t I, int bits, uint8_t* out) {
  if (!bits_ok(bits)) return ORACLE_ERR_ARG;
  const int cb = pipe_oracle_container_bits(bits);
  const int per = 8 / cb;
  const int64_t row_bytes = (I + per - 1) / per;
  const unsigned mask = (1u << cb) - 1u;
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t j = 0; j < row_bytes; ++j) {
      unsigned byte = 0;
      for (int e = 0; e < per; ++e) {
        const int64_t i = j * per + e;
        if (i < I) byte |= ((unsigned)(int)codes[r * I + i] & mask) << (e * cb);
      }
      out[r * row_bytes + j] = (uint8_t)byte;
    }
  return ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------
 * Activation quantizers beside the int8 symmetric one (Appendix B, Eq. 9 consumes Q(x) and one
 * scale per tensor; Sec. 4.3 uses A6 and A4, and asymmetric quantization for the parallelized
 * comparison).  Codes are int8 values in every case.
 *   symmetric, b bits:  qx = 2^(b-1) - 1;  lambda = max|x| / qx (or the static scale);
 *                       c = clamp(rne(x / lambda), -qx, qx);  x ~ lambda * c;  zero point 0
 *   asymmetric, b bits: lo = min(x, 0), hi = max(x, 0) over the tensor (zero is representable);
 *                       levels L = 2^b - 1;  lambda = (hi - lo) / L  (binary32: subtraction, division);
 *                       z = clamp(rne(-2^(b-1) - lo / lambda), -2^(b-1), 2^(b-1) - 1)   (binary32)
 *                       c = clamp(rne(x / lambda) + z, -2^(b-1), 2^(b-1) - 1);  x ~ lambda * (c - z)
 *                       (rne(x / lambda) is formed first, the integer z is added to the rounded value)
 *   lambda = 0 (constant-zero tensor) gives all codes equal to z = 0.
 * static_range (optional, asymmetric only): {lo, hi} supplied by the caller instead of the tensor's.
 * ------------------------------------------------------------------------------------- */
int pipe_oracle_quantize_act_ex(const float* x, int64_t T, int64_t I, int64_t ldx, int act_bits, int asymmetric,
                                const float* static_scale, const float* static_range, int8_t* xq, int64_t ldxq,
                                float* sx_out, int32_t* zp_out) {
  if (!(act_bits == 8 || act_bits == 6 || act_bits == 4)) return ORACLE_ERR_ARG;
  float lo = 0.0f, hi = 0.0f, m = 0.0f;
  for (int64_t t = 0; t < T; ++t)
    for (int64_t i = 0; i < I; ++i) {
      const float v = x[t * ldx + i];
      if (!isfinite(v)) return ORACLE_ERR_NONFINITE;
      if (v < lo) lo = v;
      if (v > hi) hi = v;
      if (fabsf(v) > m) m = fabsf(v);
    }
  const float half = (float)(1 << (act_bits - 1)); /* 2^(b-1) */
  float sx, cmin, cmax, z = 0.0f;
  if (!asymmetric) {
    const float qx = half - 1.0f;
    sx = static_scale ? *static_scale : m / qx;
    if (!(sx >= 0.0f) || !isfinite(sx)) return ORACLE_ERR_ARG;
    cmin = -qx;
    cmax = qx;
  } else {
    if (static_range) {
      lo = static_range[0];
      hi = static_range[1];
      if (!(lo <= 0.0f) || !(hi >= 0.0f) || !isfinite(lo) || !isfinite(hi)) return ORACLE_ERR_ARG;
    }
    const float levels = 2.0f * half - 1.0f;
    sx = (hi - lo) / levels;
    cmin = -half;
    cmax = half - 1.0f;
    if (sx != 0.0f) {
      z = nearbyintf(-half - lo / sx);
      if (z < cmin) z = cmin;
      if (z > cmax) z = cmax;
    }
  }
  *sx_out = sx;
  if (zp_out) *zp_out = (int32_t)z;
  for (int64_t t = 0; t < T; ++t)
    for (int64_t i = 0; i < I; ++i) {
      float c = z;
      if (sx != 0.0f) {
        c = nearbyintf(x[t * ldx + i] / sx) + z;
        if (c > cmax) c = cmax;
        if (c < cmin) c = cmin;
      }
      xq[t * ldxq + i] = (int8_t)c;
    }
  return ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------
 * Appendix B, Eq. 9 on asymmetric activation codes: x ~ lambda_x (c - z), so the contraction is
 *     acc_k[t,o] = sum_i (c[t,i] - z) * q_k[o,i]                  (exact integers)
 * and everything after it is pipe_oracle_forward's: c_k = s_k[o] * lambda_x first, one fma per
 * order in ascending order from zero, the bias last.  partials receives acc_k as defined here
 * (zero point already taken out).  rowsum (optional, int64 [R_total]) receives sum_i q_k[o,i]
 * of the cluster's rows, the quantity an implementation folds the zero point into.
 * ------------------------------------------------------------------------------------- */
int pipe_oracle_forward_zp(const int8_t* xq, int64_t T, int64_t I, int64_t ldxq, int64_t O, int K, int32_t g,
                           const int8_t* codes, const float* scales, const int32_t* kept, const int32_t* kept_count,
                           int k_begin, int k_end, float sx, int32_t zero_point, const float* bias, float* y, int64_t ldy,
                           double* y64, double* yabs, int32_t* partials, int64_t* rowsum) {
  if (k_begin < 0 || k_end > K || k_begin >= k_end || O % g != 0 || K > 64) return ORACLE_ERR_ARG;
  const int32_t G = (int32_t)(O / g);
  int64_t R_total = 0;
  int64_t row_off[64];
  for (int k = 0; k < K; ++k) {
    row_off[k] = R_total;
    R_total += (int64_t)kept_count[k] * g;
  }
  int overflow = 0;
  for (int64_t t = 0; t < T; ++t) {
    const int8_t* xr = xq + t * ldxq;
    for (int64_t o = 0; o < O; ++o) {
      float acc_y = 0.0f;
      double acc64 = 0.0, accabs = 0.0;
      for (int k = k_begin; k < k_end; ++k) {
        /* position of the channel's group in the kept list of order k, if it is kept */
        int32_t n = -1;
        for (int32_t u = 0; u < kept_count[k]; ++u)
          if (kept[(int64_t)k * G + u] == (int32_t)(o / g)) n = u;
        if (n < 0) continue;
        const int64_t row = row_off[k] + (int64_t)n * g + o % g;
        const int8_t* qr = codes + row * I;
        int64_t acc = 0, rs = 0;
        for (int64_t i = 0; i < I; ++i) {
          acc += ((int64_t)xr[i] - (int64_t)zero_point) * (int64_t)qr[i];
          rs += (int64_t)qr[i];
        }
        if (acc > INT32_MAX || acc < INT32_MIN) overflow |= 1;
        if (partials) partials[t * R_total + row] = (int32_t)acc;
        if (rowsum) rowsum[row] = rs;
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
  return overflow ? ORACLE_ERR_ACC_OVERFLOW : ORACLE_OK;
}

/* ---------------------------------------------------------------------------------------
 * Sec. 3.2: the activation functions the ensemble approximation is stated for, as an inner
 * layer applies them before the next layer's input quantizer.  Reading of the arithmetic (the
 * paper gives formulas, not roundings): every function is evaluated in binary64 on the
 * binary32 pre-activation and rounded once to binary32.
 *   1 ReLU     max(v, 0)
 *   2 SiLU     v / (1 + exp(-v))
 *   3 GeLU     v * (1 + erf(v / sqrt(2))) / 2
 *   4 sigmoid  1 / (1 + exp(-v))
 *   0 identity
 * ------------------------------------------------------------------------------------- */
int pipe_oracle_activation(const float* v, int64_t n, int kind, float* out) {
  if (kind < 0 || kind > 4) return ORACLE_ERR_ARG;
  for (int64_t i = 0; i < n; ++i) {
    const double x = (double)v[i];
    double r = x;
    if (kind == 1) r = x > 0.0 ? x : 0.0;
    if (kind == 2) r = x / (1.0 + exp(-x));
    if (kind == 3) r = 0.5 * x * (1.0 + erf(x / sqrt(2.0)));
    if (kind == 4) r = 1.0 / (1.0 + exp(-x));
    out[i] = (float)r;
  }
  return ORACLE_OK;
}
