/*
 * CPU oracle for the integer-only Transformer encoder layer of I-BERT.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, obviously-correct
 * restatement of what the paper defines (Sec. 3.1-3.6, Algorithms 1-4,
 * Appendix C.1) with every point the paper leaves open filled in by one
 * explicit reading.  It shares no code, header, table or constant generator
 * with the CUDA path and must never be linked into or imported by it.  Only
 * the tests, the smoke check and the benchmark's CPU-baseline leg call it.
 *
 * Conventions
 *   - every integer value is carried in int64_t; "floor" is toward -inf;
 *   - shifts are written as floor divisions by a power of two;
 *   - constants are derived in IEEE binary64 in exactly the order written
 *     (compile with -ffp-contract=off, no fast-math);
 *   - functions return 0 on success, a negative ORC_ERR_* otherwise.
 *
 * Parity pins (tests/test_oracle_*.py): every function below is pinned to
 * something other than itself -- exact rationals (requant), math.isqrt
 * (I-Sqrt), numpy int64 matmul (linear), float exp / erf-GELU within the
 * paper's error figures (i-exp, i-GELU; Table 1), float softmax and
 * LayerNorm within one output step, fixed-point row-sum bounds.
 * The composed encoder layer is pinned twice: tap by tap to the composition
 * of the separately pinned operators, and to a float64 textbook post-LN
 * encoder layer on the dequantized parameters, every intermediate tensor
 * within quantization noise -- with bounds tight enough that a planted wiring
 * mistake (a dropped residual, K and V swapped, no 1/sqrt(d), heads
 * interleaved, the two LayerNorms exchanged, ...) breaks them.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_OK 0
#define ORC_ERR_ARG (-1)
#define ORC_ERR_SCALE_RANGE (-3)
#define ORC_ERR_VALUE_RANGE (-8)
#define ORC_ERR_NOMEM (-5)

/* ------------------------------------------------------------------ */
/* integer helpers                                                     */
/* ------------------------------------------------------------------ */

/* floor(a / b) for b > 0 */
static int64_t floor_div(int64_t a, int64_t b) {
  int64_t q = a / b;
  if ((a % b) != 0 && a < 0) q -= 1;
  return q;
}

/* floor(v / 2^s): what an arithmetic right shift means */
static int64_t shift_right_floor(int64_t v, int s) {
  return floor_div(v, (int64_t)1 << s);
}

/* number of bits of n >= 0 (0 for n = 0) */
static int bit_length(uint64_t n) {
  int k = 0;
  while (n) { k += 1; n >>= 1; }
  return k;
}

static int64_t clamp_sym(int64_t v, int64_t qmax) {
  if (v > qmax) return qmax;
  if (v < -qmax) return -qmax;
  return v;
}

/* ------------------------------------------------------------------ */
/* Requantization (Appendix C.1: INT32 -> INT8 after every op; the      */
/* dyadic form multiplier b / 2^c follows the cited HAWQ-V3 scheme)     */
/* ------------------------------------------------------------------ */

/* real multiplier m -> (b, c) with m ~= b / 2^c, |b| < 2^31, 0 <= c <= 31 */
int orc_dyadic(double m, int64_t* b, int* c) {
  if (!isfinite(m)) return ORC_ERR_SCALE_RANGE;
  if (m == 0.0) { *b = 0; *c = 0; return ORC_OK; }
  double a = fabs(m);
  int e;
  (void)frexp(a, &e);               /* a = f * 2^e, f in [0.5, 1) */
  int cc = 31 - e;
  if (cc > 31) cc = 31;
  if (cc < 0) return ORC_ERR_SCALE_RANGE;
  double scaled = ldexp(a, cc);      /* exact */
  int64_t bb = (int64_t)floor(scaled + 0.5);
  if (bb == ((int64_t)1 << 31)) { bb = (int64_t)1 << 30; cc -= 1; }
  if (cc < 0) return ORC_ERR_SCALE_RANGE;
  *b = (m < 0.0) ? -bb : bb;
  *c = cc;
  return ORC_OK;
}

/* round-half-up of v / 2^c */
int64_t orc_round_shift(int64_t v, int c) {
  int64_t half = (c > 0) ? ((int64_t)1 << (c - 1)) : 0;
  return shift_right_floor(v + half, c);
}

/* clamp(round(v * b / 2^c), +-qmax) */
int64_t orc_requant(int64_t v, int64_t b, int c, int64_t qmax) {
  return clamp_sym(orc_round_shift(v * b, c), qmax);
}

/* ------------------------------------------------------------------ */
/* Algorithm 4: integer square root                                    */
/* ------------------------------------------------------------------ */

/* returns floor(sqrt(n)); *divisions (optional) counts the integer
   divisions performed, the terminating one included */
int64_t orc_isqrt(int64_t n, int* divisions) {
  int count = 0;
  if (divisions) *divisions = 0;
  if (n <= 0) return 0;
  int bits = bit_length((uint64_t)n);
  int64_t x = (int64_t)1 << ((bits + 1) / 2);    /* 2^ceil(bits/2) */
  for (;;) {
    int64_t x_next = (x + n / x) / 2;
    count += 1;
    if (x_next >= x) {
      if (divisions) *divisions = count;
      return x;
    }
    x = x_next;
  }
}

/* ------------------------------------------------------------------ */
/* Algorithm 1: second-order polynomial a(x+b)^2 + c in integers        */
/* ------------------------------------------------------------------ */

/* q_b = floor(b/S), q_c = floor(c/(a S^2)), S_out = a S^2 (real) */
static void ipoly_consts(double a, double b, double c, double S,
                         int64_t* q_b, int64_t* q_c, double* S_out) {
  double aS2 = (a * S) * S;
  *q_b = (int64_t)floor(b / S);
  *q_c = (int64_t)floor(c / aS2);
  *S_out = aS2;
}

static int64_t ipoly(int64_t q, int64_t q_b, int64_t q_c) {
  return (q + q_b) * (q + q_b) + q_c;
}

/* ------------------------------------------------------------------ */
/* Algorithm 3: i-exp and i-softmax                                    */
/* ------------------------------------------------------------------ */

typedef struct {
  int s_in;          /* static pre-shift of the (non-positive) input */
  int64_t q_ln2;     /* floor(ln2 / S') */
  int64_t q_b;       /* floor(1.353 / S') */
  int64_t q_c;       /* floor(0.344 / (0.3585 S'^2)) */
  int64_t e_top;     /* q_b^2 + q_c, the largest polynomial value */
  int s_out;         /* static post-shift keeping every e below 2^21 */
  double S_e;        /* scale of the returned e */
} orc_exp_consts;

int orc_exp_consts_from_scale(double S, orc_exp_consts* k) {
  const double a = 0.3585, b = 1.353, c = 0.344, ln2 = 0.6931471805599453;
  if (!(S > 0.0) || !isfinite(S)) return ORC_ERR_SCALE_RANGE;
  int s_in = 0;
  while (floor(b / ldexp(S, s_in)) > 32767.0) {
    s_in += 1;
    if (s_in > 62) return ORC_ERR_SCALE_RANGE;
  }
  double Sp = ldexp(S, s_in);
  double S_L;
  k->s_in = s_in;
  k->q_ln2 = (int64_t)floor(ln2 / Sp);
  if (k->q_ln2 < 1) return ORC_ERR_SCALE_RANGE;
  ipoly_consts(a, b, c, Sp, &k->q_b, &k->q_c, &S_L);
  k->e_top = k->q_b * k->q_b + k->q_c;
  int bl = bit_length((uint64_t)k->e_top);
  k->s_out = bl > 21 ? bl - 21 : 0;
  k->S_e = ldexp(S_L, k->s_out);
  return ORC_OK;
}

/* i-exp of one non-positive input q_tilde (scale S): returns e with
   e * S_e ~= exp(q_tilde * S) */
static int64_t iexp_one(int64_t q_tilde, const orc_exp_consts* k) {
  int64_t d = shift_right_floor(-q_tilde, k->s_in);   /* magnitude at scale S' */
  int64_t qt = -d;
  int64_t z = floor_div(-qt, k->q_ln2);
  int64_t q_p = qt + z * k->q_ln2;                     /* in (-q_ln2, 0] */
  int64_t q_L = ipoly(q_p, k->q_b, k->q_c);
  int64_t sh = z + k->s_out;
  if (sh > 31) sh = 31;
  return shift_right_floor(q_L, (int)sh);
}

/* vector i-exp on non-positive inputs */
int orc_iexp(const int64_t* q_tilde, int64_t n, double S, int64_t* e, double* S_e) {
  orc_exp_consts k;
  int rc = orc_exp_consts_from_scale(S, &k);
  if (rc) return rc;
  for (int64_t i = 0; i < n; ++i) {
    if (q_tilde[i] > 0) return ORC_ERR_VALUE_RANGE;
    e[i] = iexp_one(q_tilde[i], &k);
  }
  if (S_e) *S_e = k.S_e;
  return ORC_OK;
}

/* one softmax row; p has L entries in [0, p_max] */
static int softmax_row(const int64_t* q, int L, const orc_exp_consts* k, int64_t p_max,
                       int64_t* e_buf, int64_t* p) {
  int64_t m = q[0];
  for (int j = 1; j < L; ++j) if (q[j] > m) m = q[j];
  int64_t sum = 0;
  for (int j = 0; j < L; ++j) {
    e_buf[j] = iexp_one(q[j] - m, k);
    sum += e_buf[j];
  }
  if (sum <= 0 || sum >= ((int64_t)1 << 31)) return ORC_ERR_VALUE_RANGE;
  for (int j = 0; j < L; ++j) p[j] = floor_div(e_buf[j] * p_max, sum);
  return ORC_OK;
}

int orc_softmax(const int32_t* q, double S, int64_t rows, int L, int p_max,
                uint8_t* out, double* S_ret) {
  orc_exp_consts k;
  if (L < 1 || L > 1024 || rows < 0) return ORC_ERR_ARG;
  if (p_max != 255 && p_max != 127) return ORC_ERR_ARG;
  int rc = orc_exp_consts_from_scale(S, &k);
  if (rc) return rc;
  int err = 0;
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r) {
    int64_t qr[1024], e[1024], p[1024];
    for (int j = 0; j < L; ++j) qr[j] = q[r * L + j];
    int rr = softmax_row(qr, L, &k, p_max, e, p);
    if (rr) { err = rr; continue; }
    for (int j = 0; j < L; ++j) out[r * L + j] = (uint8_t)p[j];
  }
  if (err) return err;
  if (S_ret) *S_ret = 1.0 / (double)p_max;
  return ORC_OK;
}

/* ------------------------------------------------------------------ */
/* Algorithm 2: i-erf and i-GELU                                       */
/* ------------------------------------------------------------------ */

typedef struct {
  int s_in;        /* static pre-shift of the erf argument */
  int64_t q_b;     /* floor(-1.769 / S2), negative */
  int64_t q_c;     /* floor(1 / (-0.2888 S2^2)), negative; equals q_1 = floor(1/S_erf) */
  double S_erf;    /* -0.2888 S2^2 */
  int s_f;         /* static shift keeping q * (q_erf + q_1) inside 32 bits */
  double S_g;      /* scale of g = q * ((q_erf + q_1) >> s_f) */
} orc_gelu_consts;

int orc_gelu_consts_from_scale(double S, orc_gelu_consts* k) {
  const double a = -0.2888, b = -1.769, c = 1.0;
  if (!(S > 0.0) || !isfinite(S)) return ORC_ERR_SCALE_RANGE;
  double S1 = S / sqrt(2.0);
  int s_in = 0;
  while (-floor(b / ldexp(S1, s_in)) > 16384.0) {
    s_in += 1;
    if (s_in > 62) return ORC_ERR_SCALE_RANGE;
  }
  double S2 = ldexp(S1, s_in);
  k->s_in = s_in;
  ipoly_consts(a, b, c, S2, &k->q_b, &k->q_c, &k->S_erf);
  int bl = bit_length((uint64_t)(-2 * k->q_c));
  k->s_f = bl > 16 ? bl - 16 : 0;
  k->S_g = ldexp(S * k->S_erf, k->s_f) / 2.0;
  return ORC_OK;
}

/* i-erf of q at the (pre-shifted) scale S2: sgn(q) * I-Poly(clip(|q|, max = -q_b)) */
static int64_t ierf_one(int64_t q, const orc_gelu_consts* k) {
  int64_t sgn = (q > 0) - (q < 0);
  int64_t mag = q < 0 ? -q : q;
  int64_t u = shift_right_floor(mag, k->s_in);
  if (u > -k->q_b) u = -k->q_b;
  return sgn * ipoly(u, k->q_b, k->q_c);
}

/* g = q * ((q_erf + q_1) >> s_f) with q clamped to +-32767 first */
static int64_t igelu_g_one(int64_t q, const orc_gelu_consts* k) {
  q = clamp_sym(q, 32767);
  int64_t q_erf = ierf_one(q, k);
  int64_t q_1 = k->q_c;
  int64_t f = shift_right_floor(q_erf + q_1, k->s_f);
  return q * f;
}

/* the un-requantized product g (for the approximation-error pins) */
int orc_gelu_raw(const int32_t* q, double S, int64_t n, int64_t* g, double* S_g) {
  orc_gelu_consts k;
  int rc = orc_gelu_consts_from_scale(S, &k);
  if (rc) return rc;
  for (int64_t i = 0; i < n; ++i) {
    g[i] = igelu_g_one(q[i], &k);
    if (g[i] >= ((int64_t)1 << 31) || g[i] <= -((int64_t)1 << 31)) return ORC_ERR_VALUE_RANGE;
  }
  if (S_g) *S_g = k.S_g;
  return ORC_OK;
}

/* i-GELU then requantization to int8 at S_out:
   g2 = round(g / 256) (scale S_g * 256), out = requant(g2; dyadic(S_g2 / S_out)) */
static int gelu_out_multiplier(const orc_gelu_consts* k, double S_out, int64_t* b, int* c) {
  if (!(S_out > 0.0) || !isfinite(S_out)) return ORC_ERR_SCALE_RANGE;
  double S_g2 = k->S_g * 256.0;
  return orc_dyadic(S_g2 / S_out, b, c);
}

static int64_t igelu_int8_one(int64_t q, const orc_gelu_consts* k, int64_t b, int c) {
  int64_t g = igelu_g_one(q, k);
  int64_t g2 = orc_round_shift(g, 8);
  return orc_requant(g2, b, c, 127);
}

int orc_gelu(const int32_t* q, double S, int64_t n, double S_out, int8_t* out, double* S_ret) {
  orc_gelu_consts k;
  int64_t b; int c;
  int rc = orc_gelu_consts_from_scale(S, &k);
  if (rc) return rc;
  rc = gelu_out_multiplier(&k, S_out, &b, &c);
  if (rc) return rc;
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) out[i] = (int8_t)igelu_int8_one(q[i], &k, b, c);
  if (S_ret) *S_ret = S_out;
  return ORC_OK;
}

/* ------------------------------------------------------------------ */
/* Eq. 6: h-GELU(x) = x ReLU6(1.702 x + 3) / 6 -- the hard-sigmoid      */
/* approximation the paper measures i-GELU against (Table 1, Table 3).  */
/* The paper only remarks that it "can be computed with integer         */
/* arithmetic"; the integer form below is this build's reading, kept    */
/* parallel to i-GELU: the same integer q read at scale S_h = 1.702 S   */
/* stands for 1.702 x, so                                               */
/*   q_3 = floor(3 / S_h), q_6 = floor(6 / S_h),                        */
/*   r = clamp(q + q_3, 0, q_6)            (ReLU6 at scale S_h),        */
/*   g = q (r >> s_h)                      (scale S S_h 2^s_h / 6),     */
/* with s_h keeping the product inside 32 bits, then round(g / 256)     */
/* and the dyadic requantization to int8, exactly as for i-GELU.        */
/* ------------------------------------------------------------------ */
int orc_hgelu(const int32_t* q, double S, int64_t n, double S_out, int8_t* out, double* S_ret) {
  if (!(S > 0.0) || !isfinite(S) || !(S_out > 0.0) || !isfinite(S_out) || n < 0) return ORC_ERR_SCALE_RANGE;
  const double S_h = 1.702 * S;
  const double q3d = floor(3.0 / S_h), q6d = floor(6.0 / S_h);
  if (q6d < 1.0 || q6d > 1.0e9) return ORC_ERR_SCALE_RANGE;
  const int64_t q3 = (int64_t)q3d, q6 = (int64_t)q6d;
  const int bl = bit_length((uint64_t)q6);
  const int s_h = bl > 15 ? bl - 15 : 0;
  const double S_g2 = (ldexp(S * S_h, s_h) / 6.0) * 256.0;
  int64_t b; int c;
  int rc = orc_dyadic(S_g2 / S_out, &b, &c);
  if (rc) return rc;
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) {
    const int64_t v = clamp_sym((int64_t)q[i], 32767);
    int64_t r = v + q3;
    if (r < 0) r = 0;
    if (r > q6) r = q6;
    const int64_t g = v * shift_right_floor(r, s_h);
    const int64_t g2 = orc_round_shift(g, 8);
    out[i] = (int8_t)orc_requant(g2, b, c, 127);
  }
  if (S_ret) *S_ret = S_out;
  return ORC_OK;
}

/* ------------------------------------------------------------------ */
/* Sec. 3.6: i-LayerNorm (with the residual add in front of it)        */
/* ------------------------------------------------------------------ */

int orc_layernorm(const int32_t* a, double S, const int8_t* r, double S_r,
                  const double* gamma, const double* beta, int64_t rows, int C,
                  double S_out, int8_t* out, double* S_ret) {
  if (C < 1 || C > 2047 || rows < 0) return ORC_ERR_ARG;
  if (!(S > 0.0) || !isfinite(S) || !(S_out > 0.0) || !isfinite(S_out)) return ORC_ERR_SCALE_RANGE;
  int64_t b_r = 0; int c_r = 0;
  if (r) {
    if (!(S_r > 0.0) || !isfinite(S_r)) return ORC_ERR_SCALE_RANGE;
    int rc = orc_dyadic(S_r / S, &b_r, &c_r);
    if (rc) return rc;
  }
  /* affine + requant folded into one dyadic step per channel */
  double m0 = 1.0 / (S_out * 65536.0);
  double gmax = 0.0;
  for (int i = 0; i < C; ++i) {
    if (!isfinite(gamma[i]) || !isfinite(beta[i])) return ORC_ERR_ARG;
    if (fabs(gamma[i]) > gmax) gmax = fabs(gamma[i]);
  }
  int64_t b_unused; int c;
  int rc = orc_dyadic(gmax * m0, &b_unused, &c);
  if (rc) return rc;
  int64_t* b_i = (int64_t*)malloc(sizeof(int64_t) * (size_t)C);
  int64_t* B_i = (int64_t*)malloc(sizeof(int64_t) * (size_t)C);
  if (!b_i || !B_i) { free(b_i); free(B_i); return ORC_ERR_NOMEM; }
  for (int i = 0; i < C; ++i) {
    int64_t mag = (int64_t)floor(ldexp(fabs(gamma[i]) * m0, c) + 0.5);
    b_i[i] = gamma[i] < 0.0 ? -mag : mag;
    B_i[i] = (int64_t)floor(ldexp(beta[i] / S_out, c) + 0.5);
  }
  int64_t half = (c > 0) ? ((int64_t)1 << (c - 1)) : 0;
  int err = 0;
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < rows; ++t) {
    int64_t q[2047];
    int64_t sum = 0;
    int bad = 0;
    for (int i = 0; i < C; ++i) {
      int64_t v = a[t * C + i];
      if (r) v += orc_round_shift((int64_t)r[t * C + i] * b_r, c_r);
      if (v > ((int64_t)1 << 20) || v < -((int64_t)1 << 20)) bad = 1;
      q[i] = v;
      sum += v;
    }
    if (bad) { err = ORC_ERR_VALUE_RANGE; continue; }
    int64_t mu = floor_div(sum, C);
    int64_t ss = 0;
    for (int i = 0; i < C; ++i) { int64_t y = q[i] - mu; ss += y * y; }
    int64_t var = floor_div(ss, C);
    int64_t sigma = orc_isqrt(var, NULL);
    if (sigma < 1) sigma = 1;
    int64_t rho = floor_div((int64_t)1 << 31, sigma);
    for (int i = 0; i < C; ++i) {
      int64_t y = q[i] - mu;
      int64_t n = shift_right_floor(y * rho, 15);
      int64_t o = shift_right_floor(n * b_i[i] + B_i[i] + half, c);
      out[t * C + i] = (int8_t)clamp_sym(o, 127);
    }
  }
  free(b_i); free(B_i);
  if (err) return err;
  if (S_ret) *S_ret = S_out;
  return ORC_OK;
}

/* ------------------------------------------------------------------ */
/* INT8 MatMul with INT32 accumulation + bias + requantization          */
/* ------------------------------------------------------------------ */

/* out_kind 0: int8 (qmax 127); 1: Q16 held in int32 (qmax 32767);
   2: raw int32 accumulators (no requant). w is [N, K], x is [M, K].
   S_out_cols (optional, N entries) overrides S_out per output column. */
int orc_linear(const int8_t* x, double S_x, const int8_t* w, const double* S_w,
               const int32_t* bias, int64_t M, int N, int K, int out_kind,
               double S_out, const double* S_out_cols, void* out) {
  if (M < 0 || N < 1 || K < 1 || out_kind < 0 || out_kind > 2) return ORC_ERR_ARG;
  if (!(S_x > 0.0) || !isfinite(S_x)) return ORC_ERR_SCALE_RANGE;
  int64_t* b = (int64_t*)malloc(sizeof(int64_t) * (size_t)N);
  int* c = (int*)malloc(sizeof(int) * (size_t)N);
  if (!b || !c) { free(b); free(c); return ORC_ERR_NOMEM; }
  if (out_kind != 2) {
    for (int n = 0; n < N; ++n) {
      double so = S_out_cols ? S_out_cols[n] : S_out;
      if (!(so > 0.0) || !isfinite(so) || !(S_w[n] > 0.0) || !isfinite(S_w[n])) {
        free(b); free(c); return ORC_ERR_SCALE_RANGE;
      }
      int rc = orc_dyadic((S_x * S_w[n]) / so, &b[n], &c[n]);
      if (rc) { free(b); free(c); return rc; }
    }
  }
  int64_t qmax = out_kind == 0 ? 127 : 32767;
  int err = 0;
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m) {
    for (int n = 0; n < N; ++n) {
      int64_t acc = bias ? (int64_t)bias[n] : 0;
      const int8_t* xr = x + m * K;
      const int8_t* wr = w + (int64_t)n * K;
      for (int k = 0; k < K; ++k) acc += (int64_t)xr[k] * (int64_t)wr[k];
      if (acc >= ((int64_t)1 << 31) || acc < -((int64_t)1 << 31)) { err = ORC_ERR_VALUE_RANGE; continue; }
      if (out_kind == 2) ((int32_t*)out)[m * N + n] = (int32_t)acc;
      else {
        int64_t v = orc_requant(acc, b[n], c[n], qmax);
        if (out_kind == 0) ((int8_t*)out)[m * N + n] = (int8_t)v;
        else ((int32_t*)out)[m * N + n] = (int32_t)v;
      }
    }
  }
  free(b); free(c);
  return err;
}

/* ------------------------------------------------------------------ */
/* One attention head group: scores, i-softmax, context                 */
/* ------------------------------------------------------------------ */

/* qkv: [B*L, 3H] int8, columns Q | K | V, head j = columns 64j .. 64j+63
   of each block.  Scores carry the scale S_q S_k / 8 (1/sqrt(64) folded in).
   ctx: [B*L, H] int8 at S_ctx.  probs (optional): [B, heads, L, L] uint8. */
/* Attention of sequences with padding.  The paper does not treat masks; the reading taken here
   is the integer counterpart of the usual additive -inf key mask: sequence b has lens[b] valid
   keys (0 <= lens[b] <= L), keys j >= lens[b] take no part in the row maximum or the row sum and
   get probability 0; every query row (padded ones too) attends to the valid keys.  A sequence
   with no valid key gives context 0.  lens == NULL means every key is valid. */
static int attention_impl(const int8_t* qkv, int B, int L, int H, int heads, const int32_t* lens,
                          double S_q, double S_k, double S_v, double S_ctx, int p_max,
                          int8_t* ctx, uint8_t* probs) {
  if (B < 0 || L < 1 || L > 1024 || heads < 1 || H != heads * 64) return ORC_ERR_ARG;
  if (lens)
    for (int bi = 0; bi < B; ++bi)
      if (lens[bi] < 0 || lens[bi] > L) return ORC_ERR_ARG;
  if (p_max != 255 && p_max != 127) return ORC_ERR_ARG;
  const int d = 64;
  orc_exp_consts k;
  double S_sc = (S_q * S_k) / 8.0;
  int rc = orc_exp_consts_from_scale(S_sc, &k);
  if (rc) return rc;
  int64_t b_c; int c_c;
  if (!(S_ctx > 0.0) || !(S_v > 0.0)) return ORC_ERR_SCALE_RANGE;
  rc = orc_dyadic(((1.0 / (double)p_max) * S_v) / S_ctx, &b_c, &c_c);
  if (rc) return rc;
  int err = 0;
  const int64_t ld = 3 * (int64_t)H;
#pragma omp parallel for collapse(2) schedule(static)
  for (int bi = 0; bi < B; ++bi) {
    for (int h = 0; h < heads; ++h) {
      int64_t s[1024], e[1024], p[1024];
      const int n = lens ? lens[bi] : L;          /* valid keys of this sequence */
      for (int i = 0; i < L; ++i) {
        const int8_t* qi = qkv + ((int64_t)bi * L + i) * ld + h * d;
        for (int j = 0; j < n; ++j) {
          const int8_t* kj = qkv + ((int64_t)bi * L + j) * ld + H + h * d;
          int64_t acc = 0;
          for (int t = 0; t < d; ++t) acc += (int64_t)qi[t] * (int64_t)kj[t];
          s[j] = acc;
        }
        if (n > 0) {
          int rr = softmax_row(s, n, &k, p_max, e, p);
          if (rr) { err = rr; continue; }
        }
        for (int j = n; j < L; ++j) p[j] = 0;
        if (probs)
          for (int j = 0; j < L; ++j)
            probs[(((int64_t)bi * heads + h) * L + i) * L + j] = (uint8_t)p[j];
        for (int t = 0; t < d; ++t) {
          int64_t acc = 0;
          for (int j = 0; j < n; ++j) {
            const int8_t* vj = qkv + ((int64_t)bi * L + j) * ld + 2 * H + h * d;
            acc += p[j] * (int64_t)vj[t];
          }
          ctx[((int64_t)bi * L + i) * H + h * d + t] = (int8_t)orc_requant(acc, b_c, c_c, 127);
        }
      }
    }
  }
  return err;
}

int orc_attention(const int8_t* qkv, int B, int L, int H, int heads,
                  double S_q, double S_k, double S_v, double S_ctx, int p_max,
                  int8_t* ctx, uint8_t* probs) {
  return attention_impl(qkv, B, L, H, heads, NULL, S_q, S_k, S_v, S_ctx, p_max, ctx, probs);
}

int orc_attention_masked(const int8_t* qkv, int B, int L, int H, int heads, const int32_t* lens,
                         double S_q, double S_k, double S_v, double S_ctx, int p_max,
                         int8_t* ctx, uint8_t* probs) {
  return attention_impl(qkv, B, L, H, heads, lens, S_q, S_k, S_v, S_ctx, p_max, ctx, probs);
}

/* ------------------------------------------------------------------ */
/* The encoder layer: attention block, residual + i-LayerNorm, FFN with */
/* i-GELU, residual + i-LayerNorm (post-LN order as in RoBERTa)          */
/* ------------------------------------------------------------------ */

typedef struct {
  int H, heads, F, p_max;
  const int8_t* w_qkv; const double* S_w_qkv; const int32_t* bias_qkv;   /* [3H,H] */
  const int8_t* w_o;   const double* S_w_o;   const int32_t* bias_o;     /* [H,H]  */
  const int8_t* w_f1;  const double* S_w_f1;  const int32_t* bias_f1;    /* [F,H]  */
  const int8_t* w_f2;  const double* S_w_f2;  const int32_t* bias_f2;    /* [H,F]  */
  const double* gamma1; const double* beta1; const double* gamma2; const double* beta2;
  double S_x, S_q, S_k, S_v, S_ctx, S_r1, S_h1, S_gi, S_go, S_r2, S_out;
} orc_layer_desc;

/* Optional taps (any may be NULL): qkv [T,3H] i8, ctx [T,H] i8, r1 [T,H] i32,
   h1 [T,H] i8, g [T,F] i8, r2 [T,H] i32 */
typedef struct {
  int8_t* qkv; int8_t* ctx; int32_t* r1; int8_t* h1; int8_t* g; int32_t* r2;
} orc_layer_taps;

static int encoder_layer_impl(const orc_layer_desc* D, const int8_t* x, int B, int L, const int32_t* lens,
                              int8_t* out, const orc_layer_taps* taps) {
  const int H = D->H, F = D->F;
  const int64_t T = (int64_t)B * L;
  int rc = ORC_OK;
  int8_t* qkv = (int8_t*)malloc((size_t)(T * 3 * H) + 1);
  int8_t* ctx = (int8_t*)malloc((size_t)(T * H) + 1);
  int32_t* r1 = (int32_t*)malloc(sizeof(int32_t) * (size_t)(T * H) + 4);
  int8_t* h1 = (int8_t*)malloc((size_t)(T * H) + 1);
  int32_t* gi = (int32_t*)malloc(sizeof(int32_t) * (size_t)(T * F) + 4);
  int8_t* g = (int8_t*)malloc((size_t)(T * F) + 1);
  int32_t* r2 = (int32_t*)malloc(sizeof(int32_t) * (size_t)(T * H) + 4);
  double* so = (double*)malloc(sizeof(double) * (size_t)(3 * H));
  if (!qkv || !ctx || !r1 || !h1 || !gi || !g || !r2 || !so) { rc = ORC_ERR_NOMEM; goto done; }

  /* a1: Q, K, V projections, each block requantized to its own int8 scale */
  for (int n = 0; n < 3 * H; ++n) so[n] = n < H ? D->S_q : (n < 2 * H ? D->S_k : D->S_v);
  rc = orc_linear(x, D->S_x, D->w_qkv, D->S_w_qkv, D->bias_qkv, T, 3 * H, H, 0, 0.0, so, qkv);
  if (rc) goto done;
  /* a2-a4: scores, i-softmax, context */
  rc = attention_impl(qkv, B, L, H, D->heads, lens, D->S_q, D->S_k, D->S_v, D->S_ctx, D->p_max, ctx, NULL);
  if (rc) goto done;
  /* a5: output projection to Q16 at the residual-sum scale */
  rc = orc_linear(ctx, D->S_ctx, D->w_o, D->S_w_o, D->bias_o, T, H, H, 1, D->S_r1, NULL, r1);
  if (rc) goto done;
  /* a6: residual (x) + i-LayerNorm 1 */
  rc = orc_layernorm(r1, D->S_r1, x, D->S_x, D->gamma1, D->beta1, T, H, D->S_h1, h1, NULL);
  if (rc) goto done;
  /* a7: FFN1 to Q16 at S_gi, then i-GELU to int8 at S_go */
  rc = orc_linear(h1, D->S_h1, D->w_f1, D->S_w_f1, D->bias_f1, T, F, H, 1, D->S_gi, NULL, gi);
  if (rc) goto done;
  rc = orc_gelu(gi, D->S_gi, T * F, D->S_go, g, NULL);
  if (rc) goto done;
  /* a8: FFN2 to Q16 at the second residual-sum scale */
  rc = orc_linear(g, D->S_go, D->w_f2, D->S_w_f2, D->bias_f2, T, H, F, 1, D->S_r2, NULL, r2);
  if (rc) goto done;
  /* a9: residual (h1) + i-LayerNorm 2 */
  rc = orc_layernorm(r2, D->S_r2, h1, D->S_h1, D->gamma2, D->beta2, T, H, D->S_out, out, NULL);
  if (rc) goto done;

  if (taps) {
    if (taps->qkv) memcpy(taps->qkv, qkv, (size_t)(T * 3 * H));
    if (taps->ctx) memcpy(taps->ctx, ctx, (size_t)(T * H));
    if (taps->r1) memcpy(taps->r1, r1, sizeof(int32_t) * (size_t)(T * H));
    if (taps->h1) memcpy(taps->h1, h1, (size_t)(T * H));
    if (taps->g) memcpy(taps->g, g, (size_t)(T * F));
    if (taps->r2) memcpy(taps->r2, r2, sizeof(int32_t) * (size_t)(T * H));
  }
done:
  free(qkv); free(ctx); free(r1); free(h1); free(gi); free(g); free(r2); free(so);
  return rc;
}

int orc_encoder_layer(const orc_layer_desc* D, const int8_t* x, int B, int L,
                      int8_t* out, const orc_layer_taps* taps) {
  return encoder_layer_impl(D, x, B, L, NULL, out, taps);
}

/* the same layer on padded sequences: only the attention sees the lengths (key mask) */
int orc_encoder_layer_masked(const orc_layer_desc* D, const int8_t* x, int B, int L, const int32_t* lens,
                             int8_t* out, const orc_layer_taps* taps) {
  return encoder_layer_impl(D, x, B, L, lens, out, taps);
}

/* ------------------------------------------------------------------ */
/* Around the layers: INT8 embedding + embedding LayerNorm, and a       */
/* classifier on the first token.  The paper only says that the         */
/* Embedding is kept at INT8 (Appendix on implementation); readings:    */
/*  - the word row (int8 at S_word) is the LayerNorm input, the         */
/*    position row (int8 at S_pos) joins it like a residual, i.e.       */
/*    rescaled to S_word by a dyadic multiplier; i-LayerNorm follows    */
/*    (Sec. 3.6);                                                       */
/*  - token t of a [B, L] batch uses position t mod L;                  */
/*  - the head is one integer linear layer on the first token of every  */
/*    sequence, left as raw INT32 accumulators (scale S_x S_w[n]).      */
/* ------------------------------------------------------------------ */

int orc_embedding(const int32_t* ids, int64_t T, int L, const int8_t* word, int64_t V, double S_word,
                  const int8_t* pos, int64_t P, double S_pos, const double* gamma, const double* beta,
                  int H, double S_out, int8_t* out) {
  if (T < 0 || L < 1 || H < 1 || V < 1 || P < L) return ORC_ERR_ARG;
  for (int64_t t = 0; t < T; ++t)
    if (ids[t] < 0 || ids[t] >= V) return ORC_ERR_ARG;
  int32_t* a = (int32_t*)malloc(sizeof(int32_t) * (size_t)(T * H) + 4);
  int8_t* r = (int8_t*)malloc((size_t)(T * H) + 1);
  if (!a || !r) { free(a); free(r); return ORC_ERR_NOMEM; }
  for (int64_t t = 0; t < T; ++t)
    for (int c = 0; c < H; ++c) {
      a[t * H + c] = word[(int64_t)ids[t] * H + c];
      r[t * H + c] = pos[(t % L) * H + c];
    }
  int rc = orc_layernorm(a, S_word, r, S_pos, gamma, beta, T, H, S_out, out, NULL);
  free(a); free(r);
  return rc;
}

int orc_classifier(const int8_t* x, int B, int L, int H, double S_x, const int8_t* w, const double* S_w,
                   const int32_t* bias, int N, int32_t* logits) {
  if (B < 0 || L < 1 || H < 1 || N < 1) return ORC_ERR_ARG;
  int8_t* first = (int8_t*)malloc((size_t)((int64_t)B * H) + 1);
  if (!first) return ORC_ERR_NOMEM;
  for (int b = 0; b < B; ++b) memcpy(first + (int64_t)b * H, x + (int64_t)b * L * H, (size_t)H);
  int rc = orc_linear(first, S_x, w, S_w, bias, B, N, H, 2, 0.0, NULL, logits);
  free(first);
  return rc;
}

/* threads an OpenMP region would use (for reporting the CPU baseline) */
int orc_num_threads(void) {
#ifdef _OPENMP
  extern int omp_get_max_threads(void);
  return omp_get_max_threads();
#else
  return 1;
#endif
}
