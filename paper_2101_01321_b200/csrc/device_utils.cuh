// Device-side integer building blocks shared by the kernels: dyadic requantization,
// the i-GELU element function, the i-exp element function and exact integer division
// helpers.  Everything here is integer arithmetic; no floating-point instruction is used.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "ibert_internal.h"

namespace ibert {

// clamp((v * b + add) >> c, +-qmax); `add` carries the rounding constant 2^(c-1)
// (and, in GEMM epilogues, bias * b).  64-bit product, arithmetic shift, 0 <= c <= 31.
__device__ __forceinline__ int32_t requant_add(int32_t v, int32_t b, int64_t add, int c, int32_t qmax) {
  int64_t p = (int64_t)v * (int64_t)b + add;
  p >>= c;
  p = p > (int64_t)qmax ? (int64_t)qmax : p;
  p = p < -(int64_t)qmax ? -(int64_t)qmax : p;
  return (int32_t)p;
}

// The same requantization when the host could pre-shift the multiplier (b2 = b << (32 - c)):
// (v * b2 + 2^31) >> 32, not yet clamped.  Written as a 32x32->64 multiply whose upper word is
// corrected by bit 31 of the lower word: a multiply-add with a 64-bit addend issues at less than
// half the rate of this form on the integer pipes.
__device__ __forceinline__ int32_t requant_upper(int32_t v, int32_t b2) {
  const int64_t t = (int64_t)v * (int64_t)b2;
  return (int32_t)(t >> 32) + (int32_t)((uint32_t)t >> 31);
}

// The upper-word requantization for multipliers of 1/2 and more: b 2^(32-c) no longer fits 32 bits,
// so it is split into w 2^32 + r with r in [-2^31, 2^31) and the product into v w + (v r >> 32).
// Exact like the others; the host checks that v w cannot overflow.
__device__ __forceinline__ int32_t requant_upper_wide(int32_t v, int32_t r, int32_t w) {
  const int64_t t = (int64_t)v * (int64_t)r;
  return v * w + (int32_t)(t >> 32) + (int32_t)((uint32_t)t >> 31);
}

// (v * b2 + add) >> 32 for a general 64-bit addend, the carry of the lower words propagated by hand
__device__ __forceinline__ int32_t requant_upper_add(int32_t v, int32_t b2, int64_t add) {
  const int64_t t = (int64_t)v * (int64_t)b2;
  int32_t hi;
  asm("{\n\t.reg .u32 s;\n\t"
      "add.cc.u32 s, %1, %3;\n\t"
      "addc.s32 %0, %2, %4;\n\t}"
      : "=r"(hi)
      : "r"((uint32_t)t), "r"((int32_t)(t >> 32)), "r"((uint32_t)add), "r"((int32_t)(add >> 32)));
  return hi;
}

// four int32 -> four int8 lanes of one word, each saturated to [-128, 127]
__device__ __forceinline__ uint32_t pack4_sat_s8(int32_t v0, int32_t v1, int32_t v2, int32_t v3) {
  uint32_t hi, r;
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(v3), "r"(v2), "r"(0));
  asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(v1), "r"(v0), "r"(hi));
  return r;
}

// byte k of a word as a sign-extended int32 in one permute (`prmt`: a selector nibble with bit 3
// set replicates the sign of the byte it selects)
__device__ __forceinline__ int32_t sext_byte(uint32_t w, int k) {
  int32_t r;
  asm("prmt.b32 %0, %1, 0, %2;" : "=r"(r) : "r"(w), "r"(0x8880 + k * 0x1111));
  return r;
}

// 16-bit half h of a word as a sign-extended int32, likewise in one permute
__device__ __forceinline__ int32_t sext_half(uint32_t w, int h) {
  int32_t r;
  asm("prmt.b32 %0, %1, 0, %2;" : "=r"(r) : "r"(w), "r"(h ? 0xBB32 : 0x9910));
  return r;
}

__device__ __forceinline__ int64_t rounding_half(int c) { return c > 0 ? (int64_t(1) << (c - 1)) : 0; }

__device__ __forceinline__ int32_t clamp_sym(int32_t v, int32_t qmax) { return max(-qmax, min(v, qmax)); }

// i-GELU of one Q16 value (Algorithm 2): i-erf = sgn(q) * [(min(|q| >> s_in, -q_b) + q_b)^2 + q_c],
// g = q * ((i-erf + q_1) >> s_f), then round(g / 256) and the dyadic requantization to int8.
__device__ __forceinline__ int32_t igelu_q16_to_int8(int32_t q, const GeluConsts& k, int64_t half) {
  const int32_t mag = abs(q);
  const int32_t t = min(mag >> k.s_in, k.nq_b) - k.nq_b;    // clip(|q|, max = -q_b) + q_b, in [q_b, 0]
  const int32_t poly = t * t + k.q_c;                        // I-Poly; negative
  const int32_t f = k.q_c + (q < 0 ? -poly : poly);          // q_erf + q_1 (value for q = 0 is unused: g = 0)
  const int32_t g = q * (f >> k.s_f);
  const int32_t g2 = (g + 128) >> 8;
  return requant_add(g2, k.b, half, k.c, 127);
}

// Same function, written for the integer pipes: sign applied by a select, the final
// requantization in upper-word form; the result still needs the upper clamp (pack4_sat_s8).
__device__ __forceinline__ int32_t igelu_q16_upper(int32_t q, const GeluConsts& k) {
  const int32_t t = min(abs(q) >> k.s_in, k.nq_b) - k.nq_b;
  const int32_t tt = t * t;
  // q_erf + q_1 = sgn(q) (t^2 + q_c) + q_c: -t^2 for q < 0, t^2 + 2 q_c otherwise (unused for q = 0)
  const int32_t f = q < 0 ? -tt : tt + 2 * k.q_c;
  const int32_t g2 = (q * (f >> k.s_f) + 128) >> 8;
  return max(requant_upper(g2, k.b2), -127);
}

// Magnitude form of the same function, taking the Q16 value BEFORE its clamp (x; q = clamp(x)):
// with a = |q| = min(|x|, 32767) and t as above,
//   q >= 0:  g = q ((t^2 + 2 q_c) >> s_f)                    = a ((t^2 + 2 q_c) >> s_f)
//   q <  0:  g = q ((-t^2) >> s_f) = q (-ceil(t^2 / 2^s_f))   = a ((t^2 + 2^s_f - 1) >> s_f)
// so one select of the addend replaces the two-sided clamp, the negation and the select of f.
// `rnd_f` = 2^s_f - 1.  The result still needs both clamps to +-127.
__device__ __forceinline__ int32_t igelu_magnitude_upper(int32_t x, const GeluConsts& k, int32_t rnd_f) {
  const int32_t a = (int32_t)min((uint32_t)abs(x), 32767u);    // unsigned: |INT32_MIN| stays 2^31
  const int32_t t = min(a >> k.s_in, k.nq_b) - k.nq_b;
  const int32_t f = (t * t + (x >= 0 ? 2 * k.q_c : rnd_f)) >> k.s_f;
  const int32_t g2 = (a * f + 128) >> 8;
  return requant_upper(g2, k.b2);
}

// Integer h-GELU (Eq. 6) of one Q16 value before its clamp: r = clamp(q + q_3, 0, q_6) >> s_h,
// g = q r, round(g / 256), dyadic requantization (GeluConsts with hard != 0).
__device__ __forceinline__ int32_t ihgelu_upper(int32_t x, const GeluConsts& k) {
  const int32_t v = clamp_sym(x, 32767);
  const int32_t r = min(max(v + k.q_c, 0), k.nq_b) >> k.s_f;
  return requant_upper((v * r + 128) >> 8, k.b2);
}
__device__ __forceinline__ int32_t ihgelu_to_int8(int32_t q, const GeluConsts& k, int64_t half) {
  const int32_t r = min(max(q + k.q_c, 0), k.nq_b) >> k.s_f;
  return requant_add((q * r + 128) >> 8, k.b, half, k.c, 127);
}

__device__ __forceinline__ uint32_t shr_clamped(uint32_t v, uint32_t n) {
  uint32_t r;
  asm("shr.u32 %0, %1, %2;" : "=r"(r) : "r"(v), "r"(n));   // shift counts above 31 give 0
  return r;
}

// i-exp of one non-negative distance d = max - q (Algorithm 3): z = floor(d'/q_ln2),
// r = d' - z q_ln2, e = ((q_b - r)^2 + q_c) >> min(z + s_out, 31); d' = min(d >> s_in, 31 q_ln2).
// The polynomial is below 2^31, so a shift by more than 31 equals the shift by 31 (both give 0).
// DIV: 0 = multiply-high alone gives z, 1 = followed by a shift, 2 = operand pre-shifted as well.
template <int DIV>
__device__ __forceinline__ uint32_t iexp_dist(uint32_t d, const ExpConsts& k) {
  const uint32_t dp = min(d >> k.s_in, k.d_max);
  uint32_t z;
  if (DIV == 0) z = __umulhi(dp, k.div_m);
  else if (DIV == 1) z = __umulhi(dp, k.div_m) >> k.div_post;
  else z = __umulhi(dp << k.div_pre, k.div_m) >> k.div_post;
  const int32_t t = (int32_t)(z * k.q_ln2) + (k.q_b - (int32_t)dp);      // q_b - r
  const uint32_t poly = (uint32_t)(t * t + k.q_c);
  return shr_clamped(poly, z + (uint32_t)k.s_out);
}
// i-exp for distances below 2^21 (attention scores): no clamp of the distance -- a quotient above
// 31 just shifts the polynomial out completely, exactly like the clamped form.
__device__ __forceinline__ uint32_t iexp_dist_wide(uint32_t d, const ExpConsts& k) {
  const uint32_t dp = d >> k.s_in;
  const uint32_t z = __umulhi(dp, k.wide_m) >> k.wide_post;
  const int32_t t = (int32_t)(z * k.q_ln2) + (k.q_b - (int32_t)dp);      // q_b - r
  const uint32_t poly = (uint32_t)(t * t + k.q_c);
  return shr_clamped(poly, z + (uint32_t)k.s_out);
}
// i-exp when q_ln2 = 2^k (and no pre-shift): z and r are a shift and a mask of the distance.
// `dk` = distance + s_out 2^k, so that dk >> k = z + s_out is the final shift count directly.
__device__ __forceinline__ uint32_t iexp_dist_pow2(uint32_t dk, int32_t q_b, int32_t q_c, uint32_t k, uint32_t mask) {
  const int32_t t = q_b - (int32_t)(dk & mask);                          // q_b - r
  return shr_clamped((uint32_t)(t * t + q_c), dk >> k);
}
__host__ __device__ __forceinline__ int exp_div_mode(const ExpConsts& k) {
  return k.div_pre != 0 ? 2 : (k.div_post != 0 ? 1 : 0);
}

// Per-row divisor for p = floor(e * p_max / sum) with e < 2^21 and e <= sum < 2^31:
// with l = bit length of sum, K = 21 + l and m = ceil(p_max 2^K / sum) (< 2^30),
// floor(e m / 2^K) is exact: the excess e (m sum - p_max 2^K) / (sum 2^K) stays below 2^-l < 1/sum.
// Evaluated as umulhi(e << pre, m) >> post with post - pre = K - 32.
struct RowDivisor {
  uint32_t m;
  int pre, post;
};

__device__ __forceinline__ RowDivisor make_row_divisor(uint32_t sum, uint32_t p_max) {
  RowDivisor r;
  const int l = 32 - __clz(sum);
  const int K = 21 + l;
  const uint64_t num = ((uint64_t)p_max << K) + (uint64_t)(sum - 1u);
  r.m = (uint32_t)(num / (uint64_t)sum);
  r.pre = K < 32 ? 32 - K : 0;
  r.post = K < 32 ? 0 : K - 32;
  return r;
}

__device__ __forceinline__ uint32_t softmax_quotient(uint32_t e, const RowDivisor& r) {
  return __umulhi(e << r.pre, r.m) >> r.post;
}
// the common case pre == 0 (row sum >= 2^10)
__device__ __forceinline__ uint32_t softmax_quotient_nopre(uint32_t e, const RowDivisor& r) {
  return __umulhi(e, r.m) >> r.post;
}

}  // namespace ibert
