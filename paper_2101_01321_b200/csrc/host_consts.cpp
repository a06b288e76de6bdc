// Host-side derivation of the integer constants the kernels consume.
//
// Static quantization (Sec. 3.1): every scale is known before inference, so
// q_b = floor(b/S), q_c = floor(c/(a S^2)) of Algorithm 1, q_ln2 of Algorithm 3,
// q_1 of Algorithm 2 and all dyadic requantization multipliers (Appendix C.1)
// are computed here, once, in IEEE binary64 with the operation order fixed
// below.  Compile without FMA contraction.
#include <cmath>
#include <cstdlib>
#include <cstring>

#include "ibert_internal.h"

namespace ibert {

namespace {

inline bool good_scale(double s) { return std::isfinite(s) && s > 0.0; }

inline int bit_length_u64(uint64_t v) {
  int n = 0;
  while (v) { ++n; v >>= 1; }
  return n;
}

inline int ceil_log2_u32(uint32_t v) {   // smallest l with v <= 2^l
  int l = 0;
  while ((1ull << l) < v) ++l;
  return l;
}

}  // namespace

// m ~= b / 2^c with |b| < 2^31 and 0 <= c <= 31 (Appendix C.1, dyadic requantization)
int dyadic(double m, int32_t* b, int32_t* c) {
  if (!std::isfinite(m)) return IBERT_ERR_SCALE_RANGE;
  if (m == 0.0) { *b = 0; *c = 0; return IBERT_OK; }
  const double mag = std::fabs(m);
  int exponent = 0;
  std::frexp(mag, &exponent);                 // mag = f * 2^exponent, f in [0.5, 1)
  int shift = 31 - exponent;
  if (shift > 31) shift = 31;
  if (shift < 0) return IBERT_ERR_SCALE_RANGE;
  int64_t mult = (int64_t)std::floor(std::ldexp(mag, shift) + 0.5);
  if (mult == (int64_t(1) << 31)) { mult >>= 1; shift -= 1; }
  if (shift < 0) return IBERT_ERR_SCALE_RANGE;
  *b = (int32_t)(m < 0.0 ? -mult : mult);
  *c = shift;
  return IBERT_OK;
}

// Algorithm 3 constants.  The pre-shift s_in keeps q_b within 15 bits so that
// (q_p + q_b)^2 + q_c stays below 2^31; the post-shift s_out keeps every
// exponential below 2^21 so that a row of up to 1024 of them sums in int32.
int make_exp_consts(double S, int p_max, ExpConsts* k) {
  if (!good_scale(S)) return IBERT_ERR_SCALE_RANGE;
  if (p_max != 255 && p_max != 127) return IBERT_ERR_ARG;
  const double coef_a = 0.3585, coef_b = 1.353, coef_c = 0.344;
  const double ln2 = 0.6931471805599453;
  int s_in = 0;
  double Sp = S;
  while (std::floor(coef_b / Sp) > 32767.0) {
    if (++s_in > 62) return IBERT_ERR_SCALE_RANGE;
    Sp = std::ldexp(S, s_in);
  }
  const double q_ln2 = std::floor(ln2 / Sp);
  if (q_ln2 < 1.0) return IBERT_ERR_SCALE_RANGE;
  const double q_b = std::floor(coef_b / Sp);
  const double q_c = std::floor(coef_c / ((coef_a * Sp) * Sp));
  const int64_t e_top = (int64_t)q_b * (int64_t)q_b + (int64_t)q_c;
  if (e_top >= (int64_t(1) << 31)) return IBERT_ERR_SCALE_RANGE;
  const int bl = bit_length_u64((uint64_t)e_top);
  k->s_in = s_in;
  k->q_ln2 = (uint32_t)q_ln2;
  k->d_max = 31u * k->q_ln2;
  if (k->d_max >= (1u << 20)) return IBERT_ERR_SCALE_RANGE;   // cannot happen: q_ln2 <= 16787
  // floor(d / q_ln2) for d <= d_max by multiplication (Granlund-Montgomery): with
  // l = ceil(log2 q_ln2), N = bit length of d_max and m = floor(2^(N+l) / q_ln2) + 1 one has
  // 2^(N+l) < m q_ln2 <= 2^(N+l) + 2^l, which makes floor(d m / 2^(N+l)) exact for d < 2^N.
  // The shift by N+l is split around a 32-bit multiply-high.
  {
    const int l = ceil_log2_u32(k->q_ln2);
    const int N = bit_length_u64(k->d_max);
    const uint64_t m = (uint64_t(1) << (N + l)) / k->q_ln2 + 1;      // < 2^(N+1)
    int pre = 0, post = 0;
    uint64_t mm = m;
    if (N + l >= 32) post = N + l - 32;
    else {
      // move the missing 32 - (N+l) bits into the multiplier, the rest into the operand
      int spare = 0;
      while (spare < 32 - (N + l) && (mm << 1) < (uint64_t(1) << 32)) { mm <<= 1; ++spare; }
      pre = 32 - (N + l) - spare;
    }
    if (mm >= (uint64_t(1) << 32) || N + pre > 32) return IBERT_ERR_SCALE_RANGE;   // cannot happen
    k->div_m = (uint32_t)mm;
    k->div_pre = pre;
    k->div_post = post;
    // 21-bit operands: N + l >= 32 needs l >= 11, else the multiplier takes the slack
    const int N2 = 21;
    uint64_t m2 = (uint64_t(1) << (N2 + l)) / k->q_ln2 + 1;          // < 2^22
    int post2 = N2 + l - 32;
    while (post2 < 0) { m2 <<= 1; ++post2; }                          // m2 < 2^(22 + 11) only if q_ln2 tiny
    if (m2 >= (uint64_t(1) << 32)) { k->wide_m = 0; k->wide_post = -1; }  // not available (q_ln2 <= 2)
    else { k->wide_m = (uint32_t)m2; k->wide_post = post2; }
  }
  k->q_b = (int32_t)q_b;
  k->q_c = (int32_t)q_c;
  k->s_out = bl > 21 ? bl - 21 : 0;
  k->p_max = (uint32_t)p_max;
  k->pow2_k = -1;
  if (s_in == 0 && (k->q_ln2 & (k->q_ln2 - 1)) == 0) {
    int lg = 0;
    while ((1u << lg) < k->q_ln2) ++lg;
    k->pow2_k = lg;
  }
  return IBERT_OK;
}

// Algorithm 2 constants plus the multiplier that takes round(g / 256) to int8 at S_out.
int make_gelu_consts(double S, double S_out, GeluConsts* k) {
  if (!good_scale(S) || !good_scale(S_out)) return IBERT_ERR_SCALE_RANGE;
  const double coef_a = -0.2888, coef_b = -1.769;
  const double S1 = S / std::sqrt(2.0);
  int s_in = 0;
  double S2 = S1;
  while (-std::floor(coef_b / S2) > 16384.0) {
    if (++s_in > 62) return IBERT_ERR_SCALE_RANGE;
    S2 = std::ldexp(S1, s_in);
  }
  const double S_erf = (coef_a * S2) * S2;
  const double q_b = std::floor(coef_b / S2);
  const double q_c = std::floor(1.0 / S_erf);
  if (q_c < -1.0e9) return IBERT_ERR_SCALE_RANGE;              // cannot happen: S2 >= 1.08e-4
  const int bl = bit_length_u64((uint64_t)(-2 * (int64_t)q_c));
  k->s_in = s_in;
  k->nq_b = (int32_t)(-q_b);
  k->q_c = (int32_t)q_c;
  k->s_f = bl > 16 ? bl - 16 : 0;
  const double S_g = std::ldexp(S * S_erf, k->s_f) / 2.0;     // scale of q * ((q_erf + q_1) >> s_f)
  const double S_g2 = S_g * 256.0;                            // after the rounding shift by 8
  int rc = dyadic(S_g2 / S_out, &k->b, &k->c);
  if (rc) return rc;
  std::vector<int32_t> b1(1, k->b), c1(1, k->c);
  k->fast = to_upper_word_form(&b1, c1) ? 1 : 0;
  k->b2 = k->fast ? b1[0] : 0;
  k->add2 = k->fast ? (int64_t(1) << 31) : 0;                 // 2^(c-1) << (32-c)
  k->hard = 0;
  // Bound of the negative results.  For q < 0 the product is a f with a = |q| and
  // f = ceil(t^2 / 2^s_f), t = min(a >> s_in, -q_b) + q_b; f = 0 once a >> s_in reaches -q_b, and
  // below that, with w = (a >> s_in) + 1, a t^2 < 2^s_in w (-q_b + 1 - w)^2 <= 2^s_in (4/27) (-q_b + 1)^3.
  // So g <= 2^s_in (4/27) (-q_b + 1)^3 / 2^s_f + 32767, and the result is at most
  // (g / 256 + 1) |b| / 2^c + 1 in magnitude.
  {
    const double n1 = (double)k->nq_b + 1.0;
    const double g = std::ldexp((4.0 / 27.0) * n1 * n1 * n1, s_in - k->s_f) + 32767.0;
    const double out = std::ldexp((g / 256.0 + 1.0) * std::fabs((double)k->b), -k->c) + 1.0;
    k->low_free = out * 1.001 <= 127.0 ? 1 : 0;
  }
  return IBERT_OK;
}

// Integer h-GELU (Eq. 6): the same integer q read at scale S_h = 1.702 S stands for 1.702 x;
// r = clamp(q + q_3, 0, q_6) is ReLU6(1.702 x + 3) at that scale, g = q (r >> s_h) has scale
// S S_h 2^s_h / 6; round(g / 256) and the dyadic step to S_out follow as for i-GELU.
int make_hgelu_consts(double S, double S_out, GeluConsts* k) {
  if (!good_scale(S) || !good_scale(S_out)) return IBERT_ERR_SCALE_RANGE;
  const double S_h = 1.702 * S;
  const double q3 = std::floor(3.0 / S_h), q6 = std::floor(6.0 / S_h);
  if (q6 < 1.0 || q6 > 1.0e9) return IBERT_ERR_SCALE_RANGE;
  const int bl = bit_length_u64((uint64_t)q6);
  *k = GeluConsts{};
  k->hard = 1;
  k->nq_b = (int32_t)q6;
  k->q_c = (int32_t)q3;
  k->s_f = bl > 15 ? bl - 15 : 0;
  const double S_g2 = (std::ldexp(S * S_h, k->s_f) / 6.0) * 256.0;
  int rc = dyadic(S_g2 / S_out, &k->b, &k->c);
  if (rc) return rc;
  std::vector<int32_t> b1(1, k->b), c1(1, k->c);
  k->fast = to_upper_word_form(&b1, c1) ? 1 : 0;
  k->b2 = k->fast ? b1[0] : 0;
  k->add2 = k->fast ? (int64_t(1) << 31) : 0;
  return IBERT_OK;
}

bool to_upper_word_form(std::vector<int32_t>* b, const std::vector<int32_t>& c) {
  for (size_t n = 0; n < b->size(); ++n) {
    if (c[n] < 1 || c[n] > 31) return false;
    const int64_t shifted = (int64_t)(*b)[n] * (int64_t(1) << (32 - c[n]));
    if (shifted > INT32_MAX || shifted < INT32_MIN) return false;
  }
  for (size_t n = 0; n < b->size(); ++n) (*b)[n] = (int32_t)((int64_t)(*b)[n] * (int64_t(1) << (32 - c[n])));
  return true;
}

// The same for multipliers of 1/2 and more (b 2^(32-c) beyond 32 bits): b <- r, c <- w with
// b 2^(32-c) = w 2^32 + r, r in [-2^31, 2^31).  `max_abs_v` bounds the values that will be
// requantized; the conversion is refused (nothing changed) when v w could leave 32 bits.
bool to_upper_word_wide(std::vector<int32_t>* b, std::vector<int32_t>* c, int64_t max_abs_v) {
  std::vector<int32_t> r(b->size()), w(b->size());
  for (size_t n = 0; n < b->size(); ++n) {
    const int cn = (*c)[n];
    if (cn < 1 || cn > 31) return false;
    const int64_t full = (int64_t)(*b)[n] * (int64_t(1) << (32 - cn));             // |full| < 2^62
    const int64_t wn = (full + (int64_t(1) << 31)) >> 32;                            // nearest multiple of 2^32
    const int64_t rn = full - wn * (int64_t(1) << 32);
    if (rn < INT32_MIN || rn > INT32_MAX || wn < -64 || wn > 64) return false;
    // |v w| + |v r / 2^32| + 1 must stay below 2^31
    if ((double)max_abs_v * ((double)std::llabs(wn) + 0.5) + 2.0 >= 2147483648.0) return false;
    r[n] = (int32_t)rn;
    w[n] = (int32_t)wn;
  }
  *b = r;
  *c = w;
  return true;
}

// LayerNorm affine + requantization folded into one dyadic step per channel: the
// normalized value n ~ y_hat * 2^16, out = (n * b_i + B_i) >> c with a shared c.
int make_ln_tables(const double* gamma, const double* beta, int C, double S_out, LnConsts* k,
                   std::vector<int32_t>* b_i, std::vector<int64_t>* B_i) {
  if (!good_scale(S_out)) return IBERT_ERR_SCALE_RANGE;
  const double m0 = 1.0 / (S_out * 65536.0);
  double g_max = 0.0;
  for (int i = 0; i < C; ++i) {
    if (!std::isfinite(gamma[i]) || !std::isfinite(beta[i])) return IBERT_ERR_ARG;
    g_max = std::fmax(g_max, std::fabs(gamma[i]));
  }
  int32_t b_top = 0, c = 0;
  int rc = dyadic(g_max * m0, &b_top, &c);
  if (rc) return rc;
  b_i->resize(C);
  B_i->resize(C);
  const int64_t half = c > 0 ? (int64_t(1) << (c - 1)) : 0;
  for (int i = 0; i < C; ++i) {
    const int64_t mag = (int64_t)std::floor(std::ldexp(std::fabs(gamma[i]) * m0, c) + 0.5);
    const double add = std::floor(std::ldexp(beta[i] / S_out, c) + 0.5);
    if (std::fabs(add) > 4.0e18) return IBERT_ERR_SCALE_RANGE;
    (*b_i)[i] = (int32_t)(gamma[i] < 0.0 ? -mag : mag);
    (*B_i)[i] = (int64_t)add + half;        // rounding constant folded in
  }
  k->c = c;
  // Upper-word form: the normalized value (|n| < 2^23) is produced pre-shifted by 32 - c, so
  // the shift must stay within 8 bits and the shifted addends within 62 bits.
  k->out_sh = 32 - c;
  k->out_fast = (c >= 24 && c <= 31) ? 1 : 0;
  for (int i = 0; i < C && k->out_fast; ++i)
    if (std::llabs((*B_i)[i]) >= (int64_t(1) << (62 - k->out_sh))) k->out_fast = 0;
  if (k->out_fast)
    for (int i = 0; i < C; ++i) (*B_i)[i] *= (int64_t(1) << k->out_sh);
  return IBERT_OK;
}

// dyadic(S_r / S) for the residual in front of LayerNorm, plus its upper-word form
int make_ln_residual(double S_r, double S, LnConsts* k) {
  if (!good_scale(S_r) || !good_scale(S)) return IBERT_ERR_SCALE_RANGE;
  int rc = dyadic(S_r / S, &k->b_r, &k->c_r);
  if (rc) return rc;
  // |r| <= 127 leaves 24 bits of headroom: r << (32 - c_r) fits int32 for c_r >= 8
  k->res_fast = (k->c_r >= 8 && k->c_r <= 31) ? 1 : 0;
  k->res_sh = 32 - k->c_r;
  // narrow form: drop seven bits of the 31-bit multiplier (|r| <= 128 then keeps the product inside int32) and
  // keep it only if every int8 value gives the exact form's result.  For a candidate multiplier nb the
  // addend may be any value that puts all 256 results on the right side of their floors: each r bounds it
  // to an interval, and the candidate serves if the intervals intersect.
  k->res_narrow = 0;
  k->res_nb = k->res_nc = k->res_nhalf = 0;
  if (k->c_r >= 8 && k->c_r <= 31) {
    const int nc = k->c_r - 7;
    const int64_t base = (int64_t)k->b_r >> 7;
    static const int kTry[4] = {0, 1, -1, 2};
    for (int t = 0; t < 4 && !k->res_narrow; ++t) {
      const int64_t nb = base + kTry[t];
      if (nb <= 0 || nb >= (int64_t(1) << 24)) continue;
      int64_t lo = INT64_MIN, hi = INT64_MAX;
      for (int r = -128; r <= 127; ++r) {
        const int64_t exact = ((int64_t)r * k->b_r + (int64_t(1) << (k->c_r - 1))) >> k->c_r;
        lo = std::max(lo, exact * (int64_t(1) << nc) - (int64_t)r * nb);
        hi = std::min(hi, (exact + 1) * (int64_t(1) << nc) - 1 - (int64_t)r * nb);
      }
      if (lo > hi) continue;
      const int64_t nhalf = std::min(std::max(int64_t(1) << (nc - 1), lo), hi);   // the usual half where it serves
      bool same = true;
      for (int r = -128; r <= 127 && same; ++r) {
        const int64_t exact = ((int64_t)r * k->b_r + (int64_t(1) << (k->c_r - 1))) >> k->c_r;
        const int64_t narrow = ((int64_t)r * nb + nhalf) >> nc;
        same = exact == narrow && std::llabs((int64_t)r * nb + nhalf) < (int64_t(1) << 31);
      }
      if (same) { k->res_narrow = 1; k->res_nb = (int32_t)nb; k->res_nc = nc; k->res_nhalf = (int32_t)nhalf; }
    }
  }
  return IBERT_OK;
}

int make_linear_tables(double S_x, const double* S_w, int N, const double* S_out_cols, double S_out,
                       std::vector<int32_t>* b, std::vector<int32_t>* c) {
  if (!good_scale(S_x)) return IBERT_ERR_SCALE_RANGE;
  b->resize(N);
  c->resize(N);
  for (int n = 0; n < N; ++n) {
    const double so = S_out_cols ? S_out_cols[n] : S_out;
    if (!good_scale(so) || !good_scale(S_w[n])) return IBERT_ERR_SCALE_RANGE;
    int rc = dyadic((S_x * S_w[n]) / so, &(*b)[n], &(*c)[n]);
    if (rc) return rc;
  }
  return IBERT_OK;
}

}  // namespace ibert
