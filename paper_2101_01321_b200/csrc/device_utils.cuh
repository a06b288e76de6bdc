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

// i-exp of one non-negative distance d = max - q (Algorithm 3): z = floor(d'/q_ln2),
// r = d' - z q_ln2, e = ((q_b - r)^2 + q_c) >> min(z + s_out, 31); d' = min(d >> s_in, 31 q_ln2).
__device__ __forceinline__ uint32_t iexp_dist(uint32_t d, const ExpConsts& k) {
  const uint32_t dp = min(d >> k.s_in, k.d_max);
  const uint32_t z = __umulhi(dp << 12, k.div_m) >> k.div_l;
  const int32_t t = k.q_b - (int32_t)(dp - z * k.q_ln2);
  const uint32_t poly = (uint32_t)(t * t + k.q_c);
  return poly >> min(z + (uint32_t)k.s_out, 31u);
}

// Per-row reciprocal for p = floor(e * p_max / sum), exact for e * p_max < 2^29:
// with l = bit length of sum and m = floor(2^(29+l) / sum) + 1,
// floor(n / sum) = umulhi(n << 3, m) >> l for every n < 2^29.
struct RowDivisor {
  uint32_t m;
  int l;
};

__device__ __forceinline__ RowDivisor make_row_divisor(uint32_t sum) {
  RowDivisor r;
  r.l = 32 - __clz(sum);
  r.m = (uint32_t)((uint64_t(1) << (29 + r.l)) / sum) + 1u;
  return r;
}

__device__ __forceinline__ uint32_t softmax_quotient(uint32_t e, uint32_t pm8, const RowDivisor& r) {
  return __umulhi(e * pm8, r.m) >> r.l;
}

// floor(sqrt(n)) by the Newton iteration of Algorithm 4 (x0 = 2^ceil(bits/2), stop when the
// iterate no longer decreases), on 64-bit n.
__device__ __forceinline__ uint32_t isqrt_newton(uint64_t n) {
  if (n == 0) return 0;
  const int bits = 64 - __clzll((long long)n);
  uint64_t x = uint64_t(1) << ((bits + 1) >> 1);
  for (int it = 0; it < 64; ++it) {
    const uint64_t y = (x + n / x) >> 1;
    if (y >= x) break;
    x = y;
  }
  return (uint32_t)x;
}

}  // namespace ibert
