// Standalone integer non-linearities: i-GELU (Algorithm 2), i-softmax (Algorithm 3) and
// residual + i-LayerNorm (Sec. 3.6, Algorithm 4).  All three are HBM-streaming kernels:
// 128-bit coalesced loads of the int32 inputs, all arithmetic in registers, packed int8
// stores.  Rows are owned by one warp and reduced with warp shuffles.
#include <algorithm>

#include "device_utils.cuh"
#include "sm100_ptx.cuh"

namespace ibert {

namespace {

constexpr int kThreads = 256;

// ----------------------------------------------------------------------------- i-GELU
// Each thread converts 4 int4 vectors (16 values); vector j of a thread sits 32 vectors
// after vector j-1 so that every load and store instruction of a warp is contiguous.
__global__ void __launch_bounds__(kThreads) gelu_kernel(const int32_t* __restrict__ q, int64_t n,
                                                        GeluConsts k, int8_t* __restrict__ out) {
  const int64_t half = rounding_half(k.c);
  const int64_t n_vec = n >> 2;
  const int32_t rnd_f = (1 << k.s_f) - 1;
  const int lane = threadIdx.x & 31;
  const int64_t warp_global = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
  const int64_t warp_count = ((int64_t)gridDim.x * kThreads) >> 5;
  const int4* q4 = reinterpret_cast<const int4*>(q);
  uint32_t* o4 = reinterpret_cast<uint32_t*>(out);
  for (int64_t base = warp_global * 128; base < n_vec; base += warp_count * 128) {
    int4 v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int64_t idx = base + j * 32 + lane;
      v[j] = idx < n_vec ? __ldcs(q4 + idx) : make_int4(0, 0, 0, 0);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int64_t idx = base + j * 32 + lane;
      if (idx < n_vec) {
        int32_t a, b, c, d;
        if (k.hard) {
          a = k.fast ? max(ihgelu_upper(v[j].x, k), -127) : ihgelu_to_int8(clamp_sym(v[j].x, 32767), k, half);
          b = k.fast ? max(ihgelu_upper(v[j].y, k), -127) : ihgelu_to_int8(clamp_sym(v[j].y, 32767), k, half);
          c = k.fast ? max(ihgelu_upper(v[j].z, k), -127) : ihgelu_to_int8(clamp_sym(v[j].z, 32767), k, half);
          d = k.fast ? max(ihgelu_upper(v[j].w, k), -127) : ihgelu_to_int8(clamp_sym(v[j].w, 32767), k, half);
        } else if (k.fast) {
          a = max(igelu_magnitude_upper(v[j].x, k, rnd_f), -127);
          b = max(igelu_magnitude_upper(v[j].y, k, rnd_f), -127);
          c = max(igelu_magnitude_upper(v[j].z, k, rnd_f), -127);
          d = max(igelu_magnitude_upper(v[j].w, k, rnd_f), -127);
        } else {
          a = igelu_q16_to_int8(clamp_sym(v[j].x, 32767), k, half);
          b = igelu_q16_to_int8(clamp_sym(v[j].y, 32767), k, half);
          c = igelu_q16_to_int8(clamp_sym(v[j].z, 32767), k, half);
          d = igelu_q16_to_int8(clamp_sym(v[j].w, 32767), k, half);
        }
        __stcs(o4 + idx, pack4_sat_s8(a, b, c, d));
      }
    }
  }
  // ragged tail (n not a multiple of 4)
  const int64_t tid = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  const int64_t tail = n_vec << 2;
  if (tid < n - tail)
    out[tail + tid] = (int8_t)(k.hard ? ihgelu_to_int8(clamp_sym(q[tail + tid], 32767), k, half)
                                      : igelu_q16_to_int8(clamp_sym(q[tail + tid], 32767), k, half));
}

// ----------------------------------------------------------------------------- table look-up GELU
// The alternative the paper argues against: a 65535-entry table of the int8 result for every Q16
// input, built by running the i-GELU kernel once over the ramp -32767 .. 32767 (so its bits are the
// integer function's), then one load per element.
__global__ void __launch_bounds__(kThreads) ramp_q16_kernel(int32_t* __restrict__ q) {
  const int i = blockIdx.x * kThreads + threadIdx.x;
  if (i < 65535) q[i] = i - 32767;
}

__global__ void __launch_bounds__(kThreads) gelu_lut_kernel(const int32_t* __restrict__ q, int64_t n,
                                                            const int8_t* __restrict__ table,
                                                            int8_t* __restrict__ out) {
  const int64_t n_vec = n >> 2;
  const int4* q4 = reinterpret_cast<const int4*>(q);
  uint32_t* o4 = reinterpret_cast<uint32_t*>(out);
  const int64_t stride = (int64_t)gridDim.x * kThreads;
  for (int64_t idx = (int64_t)blockIdx.x * kThreads + threadIdx.x; idx < n_vec; idx += stride) {
    const int4 v = __ldcs(q4 + idx);
    const uint32_t a = (uint8_t)__ldg(table + clamp_sym(v.x, 32767) + 32767);
    const uint32_t b = (uint8_t)__ldg(table + clamp_sym(v.y, 32767) + 32767);
    const uint32_t c = (uint8_t)__ldg(table + clamp_sym(v.z, 32767) + 32767);
    const uint32_t d = (uint8_t)__ldg(table + clamp_sym(v.w, 32767) + 32767);
    __stcs(o4 + idx, a | (b << 8) | (c << 16) | (d << 24));
  }
  const int64_t tid = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  const int64_t tail = n_vec << 2;
  if (tid < n - tail) out[tail + tid] = __ldg(table + clamp_sym(q[tail + tid], 32767) + 32767);
}

// ----------------------------------------------------------------------------- i-softmax
// One warp per row; a lane keeps VPL int4 vectors (4*VPL scores) in registers.
// VEC: rows are 16-byte aligned (L % 4 == 0) and loaded/stored as vectors.
// DIV 0..2: how i-exp divides by q_ln2; DIV 3: i-exp read from `table` (comparison variant).
constexpr int kExpByTable = 3;

// table[i] = i-exp of the pre-shifted distance i, for i = 0 .. d_max
__global__ void __launch_bounds__(kThreads) exp_table_kernel(ExpConsts k, uint32_t* __restrict__ table) {
  const uint32_t i = blockIdx.x * kThreads + threadIdx.x;
  if (i > k.d_max) return;
  const uint32_t d = i << k.s_in;
  const int mode = exp_div_mode(k);
  table[i] = mode == 0 ? iexp_dist<0>(d, k) : (mode == 1 ? iexp_dist<1>(d, k) : iexp_dist<2>(d, k));
}

template <int VPL, bool VEC, int DIV>
__global__ void __launch_bounds__(kThreads) softmax_kernel(const int32_t* __restrict__ q, int64_t rows,
                                                           int L, ExpConsts k, uint8_t* __restrict__ out,
                                                           const uint32_t* __restrict__ table) {
  const int lane = threadIdx.x & 31;
  const int64_t warp_global = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
  const int64_t warp_count = ((int64_t)gridDim.x * kThreads) >> 5;
  for (int64_t row = warp_global; row < rows; row += warp_count) {
    const int32_t* qr = q + row * L;
    uint8_t* orow = out + row * L;
    int32_t v[VPL][4];
    int32_t mx = INT32_MIN;
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
      const int col = 4 * (j * 32 + lane);
      if (VEC) {
        if (col < L) {
          const int4 t = __ldcs(reinterpret_cast<const int4*>(qr + col));
          v[j][0] = t.x; v[j][1] = t.y; v[j][2] = t.z; v[j][3] = t.w;
        } else {
          v[j][0] = v[j][1] = v[j][2] = v[j][3] = INT32_MIN;
        }
      } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) v[j][i] = (col + i < L) ? qr[col + i] : INT32_MIN;
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) mx = max(mx, v[j][i]);
    }
    mx = __reduce_max_sync(0xffffffffu, mx);
    uint32_t sum = 0;
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
      const int col = 4 * (j * 32 + lane);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t dist = (uint32_t)mx - (uint32_t)v[j][i];
        uint32_t e = 0u;
        if (col + i < L) {
          if constexpr (DIV == kExpByTable) e = __ldg(table + min(dist >> k.s_in, k.d_max));
          else e = iexp_dist<DIV>(dist, k);
        }
        v[j][i] = (int32_t)e;
        sum += e;
      }
    }
    sum = __reduce_add_sync(0xffffffffu, sum);
    const RowDivisor rd = make_row_divisor(sum, k.p_max);
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
      const int col = 4 * (j * 32 + lane);
      uint32_t p[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) p[i] = softmax_quotient((uint32_t)v[j][i], rd);
      if (VEC) {
        if (col < L)
          __stcs(reinterpret_cast<uint32_t*>(orow + col), p[0] | (p[1] << 8) | (p[2] << 16) | (p[3] << 24));
      } else {
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (col + i < L) orow[col + i] = (uint8_t)p[i];
      }
    }
  }
}

// ----------------------------------------------------------------------------- i-LayerNorm
// floor(sqrt(floor(ss / C))), i.e. the largest s with s*s*C <= ss -- the value Algorithm 4
// returns for n = floor(ss / C).  A 64-bit integer division costs on the order of a hundred
// instructions here, so instead of iterating x <- (x + n/x)/2 the warp finds the same integer by
// a radix-32 search: in each of five rounds the 32 lanes test 32 candidates with one multiply
// each.  Needs s < 2^25 and ss < 2^61 / C.
__device__ __forceinline__ uint32_t warp_isqrt_of_quotient(uint64_t ss, uint32_t C, int lane) {
  uint32_t base = 0;
  // ss / C < 2^bits bounds the result below 2^ceil(bits / 2): rounds above that cannot set a digit
  const int bits = 64 - __clzll((long long)(ss | 1ull)) - (31 - __clz((int)C));
  const int top = 5 * ((min(max((bits + 1) >> 1, 1), 25) + 4) / 5 - 1);
  for (int shift = top; shift >= 0; shift -= 5) {
    const uint32_t cand = base + ((uint32_t)lane << shift);
    const uint64_t sq = (uint64_t)cand * (uint64_t)cand;
    const bool le = sq * (uint64_t)C <= ss;                       // true for a prefix of the lanes
    const uint32_t cnt = __popc(__ballot_sync(0xffffffffu, le));  // >= 1: lane 0 tests `base` itself
    base += (cnt - 1u) << shift;
  }
  return base;
}

// Four consecutive Q16 values of a row, from an int32 or an int16 container (16 / 8 bytes)
template <typename QT>
__device__ __forceinline__ void load_q4(const QT* p, int32_t (&v)[4], bool streaming) {
  if constexpr (sizeof(QT) == 4) {
    const int4 t = streaming ? __ldcs(reinterpret_cast<const int4*>(p)) : *reinterpret_cast<const int4*>(p);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  } else {
    const uint2 t = streaming ? __ldcs(reinterpret_cast<const uint2*>(p)) : *reinterpret_cast<const uint2*>(p);
    // sign-extending halves of a word: one byte permute each
    v[0] = sext_half(t.x, 0); v[1] = sext_half(t.x, 1);
    v[2] = sext_half(t.y, 0); v[3] = sext_half(t.y, 1);
  }
}

// One warp per row, the whole row in registers (VPL int4 vectors per lane).
// FAST: residual rescale and output requantization are in upper-word form (one multiply-add each).
// Resident CTAs per SM the register budget is tuned for: the kernel is latency-bound on the row
// loads, so short rows trade registers for more warps in flight.
constexpr int ln_min_blocks(int vpl) { return vpl <= 4 ? 4 : (vpl <= 6 ? 3 : (vpl <= 8 ? 2 : 1)); }

template <int VPL, bool VEC, bool FAST, typename QT>
__global__ void __launch_bounds__(kThreads, ln_min_blocks(VPL)) layernorm_kernel(const QT* __restrict__ q,
                                                             const int8_t* __restrict__ r, int64_t rows,
                                                             LnConsts k, const int32_t* __restrict__ b_i,
                                                             const int64_t* __restrict__ B_i,
                                                             int8_t* __restrict__ out) {
  const int lane = threadIdx.x & 31;
  const int C = k.C;
  const int64_t warp_global = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
  const int64_t warp_count = ((int64_t)gridDim.x * kThreads) >> 5;
  const int64_t half_r = rounding_half(k.c_r);
  for (int64_t row = warp_global; row < rows; row += warp_count) {
    const QT* qr = q + row * C;
    const int8_t* rr = r + row * C;
    int8_t* orow = out + row * C;
    int32_t v[VPL][4];
    int32_t sum = 0;
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
      const int col = 4 * (j * 32 + lane);
      if (VEC) {
        if (col < C) {
          load_q4(qr + col, v[j], true);
          if (k.has_res) {
            const uint32_t rw = __ldcs(reinterpret_cast<const uint32_t*>(rr + col));
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int32_t rv = (int32_t)(int8_t)(rw >> (8 * i));
              if (FAST) v[j][i] += requant_upper(rv << k.res_sh, k.b_r);
              else v[j][i] += (int32_t)(((int64_t)rv * k.b_r + half_r) >> k.c_r);
            }
          }
        } else {
          v[j][0] = v[j][1] = v[j][2] = v[j][3] = 0;
        }
      } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          int32_t t = 0;
          if (col + i < C) {
            t = (int32_t)qr[col + i];
            if (k.has_res) t += (int32_t)(((int64_t)rr[col + i] * k.b_r + half_r) >> k.c_r);
          }
          v[j][i] = t;
        }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) sum += v[j][i];
    }
    sum = __reduce_add_sync(0xffffffffu, sum);
    // mu = floor(sum / C)
    int32_t mu = sum / C;
    if (sum - mu * C < 0) mu -= 1;
    uint64_t ss = 0;
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
      const int col = 4 * (j * 32 + lane);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int32_t y = (col + i < C) ? v[j][i] - mu : 0;
        v[j][i] = y;
        ss += (uint64_t)((int64_t)y * (int64_t)y);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    uint32_t sigma = warp_isqrt_of_quotient(ss, (uint32_t)C, lane);   // I-Sqrt(floor(ss / C))
    sigma = sigma < 1u ? 1u : sigma;
    const int64_t rho64 = (int64_t)(0x80000000u / sigma);            // floor(2^31 / sigma)
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
      const int col = 4 * (j * 32 + lane);
      int32_t o[4] = {0, 0, 0, 0};
      if (FAST) {
        if (col < C) {
          const int4 bb = __ldg(reinterpret_cast<const int4*>(b_i + col));
          const longlong2 B01 = __ldg(reinterpret_cast<const longlong2*>(B_i + col));
          const longlong2 B23 = __ldg(reinterpret_cast<const longlong2*>(B_i + col + 2));
          const int32_t bv[4] = {bb.x, bb.y, bb.z, bb.w};
          const int64_t Bv[4] = {B01.x, B01.y, B23.x, B23.y};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            // normalized value floor(y * rho / 2^15), then pre-shifted by out_sh (|.| < 2^31)
            const int32_t nrm = (int32_t)(((int64_t)v[j][i] * rho64) >> 15) << k.out_sh;
            o[i] = max(requant_upper_add(nrm, bv[i], Bv[i]), -127);
          }
        }
      } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          if (col + i < C) {
            const int32_t nrm = (int32_t)(((int64_t)v[j][i] * rho64) >> 15);
            int64_t t;
            if (k.out_fast) {   // the addend table is pre-shifted: undo it on this path
              t = ((int64_t)nrm * ((int64_t)__ldg(b_i + col + i) << k.out_sh) + __ldg(B_i + col + i)) >> 32;
            } else {
              t = ((int64_t)nrm * (int64_t)__ldg(b_i + col + i) + __ldg(B_i + col + i)) >> k.c;
            }
            t = t > 127 ? 127 : t;
            t = t < -127 ? -127 : t;
            o[i] = (int32_t)t;
          }
        }
      }
      if (VEC) {
        if (col < C) __stcs(reinterpret_cast<uint32_t*>(orow + col), pack4_sat_s8(o[0], o[1], o[2], o[3]));
      } else {
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (col + i < C) orow[col + i] = (int8_t)o[i];
      }
    }
  }
}

// Same row computation, fed by bulk async copies: every warp streams its rows (Q16 row and int8
// residual row) through a private ring of DEPTH shared-memory slots, so the loads of the next
// rows are in flight while the current row is reduced -- the row loop no longer waits on HBM.
// Requires C % 16 == 0 (16-byte aligned rows), upper-word constants, and a residual.
// FULL: C == 128 VPL, no lane ever runs past the row.
template <int VPL, int DEPTH, typename QT, bool FULL>
__global__ void __launch_bounds__(kThreads, DEPTH == 2 ? 3 : 2) layernorm_pipe_kernel(const QT* __restrict__ q,
                                                                     const int8_t* __restrict__ r, int64_t rows,
                                                                     LnConsts k, const int32_t* __restrict__ b_i,
                                                                     const int64_t* __restrict__ B_i,
                                                                     int8_t* __restrict__ out, int32_t* status) {
  extern __shared__ __align__(128) uint8_t ln_smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int C = k.C;
  const uint32_t q_bytes = (uint32_t)C * (uint32_t)sizeof(QT), r_bytes = (uint32_t)C;
  const uint32_t slot_bytes = q_bytes + r_bytes;                 // multiple of 16
  uint8_t* ring = ln_smem + (size_t)warp * DEPTH * slot_bytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(ln_smem + (size_t)(kThreads / 32) * DEPTH * slot_bytes) + warp * DEPTH;
  // the per-channel tables, copied once per CTA: every row reads all of them
  int64_t* s_B = reinterpret_cast<int64_t*>(ln_smem + (size_t)(kThreads / 32) * DEPTH * slot_bytes + (kThreads / 32) * DEPTH * 8);
  int32_t* s_b = reinterpret_cast<int32_t*>(s_B + C);
  const int64_t warp_global = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
  const int64_t warp_count = ((int64_t)gridDim.x * kThreads) >> 5;
  for (int i = threadIdx.x; i < C; i += kThreads) {        // constants, not outputs of the previous kernel
    s_b[i] = __ldg(b_i + i);
    s_B[i] = __ldg(B_i + i);
  }
  __syncthreads();

  ptx::grid_dep_launch();
  ptx::grid_dep_wait();              // the kernel that produced q (and r) has completed
  auto issue = [&](int64_t row, int slot) {
    const uint32_t bar = ptx::smem_addr(bars + slot);
    const uint32_t dst = ptx::smem_addr(ring + (size_t)slot * slot_bytes);
    ptx::mbar_arrive_expect_tx(bar, slot_bytes);
    ptx::bulk_load_1d(dst, q + row * C, q_bytes, bar);
    ptx::bulk_load_1d(dst + q_bytes, r + row * C, r_bytes, bar);
  };
  if (lane == 0) {
    for (int s = 0; s < DEPTH; ++s) ptx::mbar_init(ptx::smem_addr(bars + s), 1);
    ptx::fence_mbar_init();
    for (int s = 0; s < DEPTH; ++s) {
      const int64_t row = warp_global + (int64_t)s * warp_count;
      if (row < rows) issue(row, s);
    }
  }
  __syncwarp();

  int slot = 0;
  uint32_t phase = 0;
  for (int64_t row = warp_global; row < rows; row += warp_count) {
    const bool ok = __all_sync(0xffffffffu, ptx::mbar_wait(ptx::smem_addr(bars + slot), phase));
    if (!ok) {
      if (lane == 0) atomicCAS(status, 0, IBERT_ERR_TIMEOUT);
      // the copies already issued into the other slots must land (or run out of time as well)
      // before this CTA's shared memory is given up
      for (int j = 1; j < DEPTH; ++j) {
        int s2 = slot + j;
        uint32_t ph2 = phase;
        if (s2 >= DEPTH) { s2 -= DEPTH; ph2 ^= 1; }
        if (row + (int64_t)j * warp_count < rows) ptx::mbar_wait(ptx::smem_addr(bars + s2), ph2);
      }
      break;
    }
    const uint8_t* sq = ring + (size_t)slot * slot_bytes;
    int32_t v[VPL][4];
    uint32_t rw[VPL];
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
      const int col = 4 * (j * 32 + lane);
      if (FULL || col < C) {
        load_q4(reinterpret_cast<const QT*>(sq) + col, v[j], false);
        rw[j] = *reinterpret_cast<const uint32_t*>(sq + q_bytes + col);
      } else {
        v[j][0] = v[j][1] = v[j][2] = v[j][3] = 0;
        rw[j] = 0;
      }
    }
    __syncwarp();                                    // every lane has its copy: the slot can be refilled
    if (lane == 0) {
      const int64_t next = row + (int64_t)DEPTH * warp_count;
      if (next < rows) issue(next, slot);
    }
    if (++slot == DEPTH) { slot = 0; phase ^= 1; }

    // one pass over the row: sum v and sum v^2 (columns past C hold zeros); the centred sum of squares
    // follows exactly in integers: sum (v - mu)^2 = sum v^2 - 2 mu sum v + C mu^2
    int32_t sum = 0;
    uint64_t s2 = 0;
#pragma unroll
    for (int j = 0; j < VPL; ++j)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        v[j][i] += (sext_byte(rw[j], i) * k.res_nb + k.res_nhalf) >> k.res_nc;   // the residual, rescaled (narrow form)
        sum += v[j][i];
        s2 += (uint64_t)((int64_t)v[j][i] * (int64_t)v[j][i]);
      }
    sum = __reduce_add_sync(0xffffffffu, sum);
    // a lane's share is below 2^50 (|v| <= 2^21, at most 64 values): two 25-bit halves reduce as 32-bit sums
    s2 = (uint64_t)__reduce_add_sync(0xffffffffu, (uint32_t)s2 & 0x1ffffffu) +
         ((uint64_t)__reduce_add_sync(0xffffffffu, (uint32_t)(s2 >> 25)) << 25);
    int32_t mu = sum / C;                            // mu = floor(sum / C)
    if (sum - mu * C < 0) mu -= 1;
    const uint64_t ss = (uint64_t)((int64_t)s2 - 2 * (int64_t)mu * (int64_t)sum + (int64_t)C * (int64_t)mu * (int64_t)mu);
    uint32_t sigma = warp_isqrt_of_quotient(ss, (uint32_t)C, lane);   // I-Sqrt(floor(ss / C))
    sigma = sigma < 1u ? 1u : sigma;
    // floor(2^31 / sigma) as a positive int32 multiplier: for sigma = 1 use 2^30 and shift one less
    const int32_t rho = sigma == 1u ? (1 << 30) : (int32_t)(0x80000000u / sigma);
    const int nsh = sigma == 1u ? 14 : 15;
    int8_t* orow = out + row * C;
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
      const int col = 4 * (j * 32 + lane);
      if (FULL || col < C) {
        const int4 bb = *reinterpret_cast<const int4*>(s_b + col);
        const longlong2 B01 = *reinterpret_cast<const longlong2*>(s_B + col);
        const longlong2 B23 = *reinterpret_cast<const longlong2*>(s_B + col + 2);
        const int32_t bv[4] = {bb.x, bb.y, bb.z, bb.w};
        const int64_t Bv[4] = {B01.x, B01.y, B23.x, B23.y};
        int32_t o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int64_t pr = (int64_t)(v[j][i] - mu) * (int64_t)rho;
          // floor(pr / 2^nsh) fits 32 bits: the low word of the 64-bit shift is a funnel shift
          const int32_t nrm = (int32_t)__funnelshift_r((uint32_t)pr, (uint32_t)(pr >> 32), (uint32_t)nsh) << k.out_sh;
          o[i] = max(requant_upper_add(nrm, bv[i], Bv[i]), -127);
        }
        __stcs(reinterpret_cast<uint32_t*>(orow + col), pack4_sat_s8(o[0], o[1], o[2], o[3]));
      }
    }
  }
}

// ----------------------------------------------------------------------------- embedding gather
// One warp per token: 16 bytes of the word row and of the position row per lane and step.
// Packed batches (cu != nullptr: [B + 1] first rows of the sequences): the position of token t is
// its distance from the first row of its sequence, found by bisection; a position beyond the
// position table (a sequence longer than the stated maximum) records IBERT_ERR_VALUE_RANGE.
__global__ void __launch_bounds__(kThreads) embed_gather_kernel(const int32_t* __restrict__ ids, int64_t T, int L,
                                                                const int8_t* __restrict__ word, int64_t V,
                                                                const int8_t* __restrict__ pos, int H,
                                                                int32_t* __restrict__ q, int8_t* __restrict__ r,
                                                                int32_t* status, const int32_t* __restrict__ cu, int B) {
  const int lane = threadIdx.x & 31;
  const int64_t warp_global = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
  const int64_t warp_count = ((int64_t)gridDim.x * kThreads) >> 5;
  for (int64_t t = warp_global; t < T; t += warp_count) {
    int64_t id = __ldg(ids + t);
    if (id < 0 || id >= V) {
      if (lane == 0) atomicCAS(status, 0, IBERT_ERR_VALUE_RANGE);
      id = 0;
    }
    int64_t p = t % L;
    if (cu) {
      int lo = 0, hi = B;                    // the last sequence whose first row is <= t
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if ((int64_t)__ldg(cu + mid) <= t) lo = mid; else hi = mid;
      }
      p = t - (int64_t)__ldg(cu + lo);
      if (p >= L) {
        if (lane == 0) atomicCAS(status, 0, IBERT_ERR_VALUE_RANGE);
        p = L - 1;
      }
    }
    const int8_t* wrow = word + id * H;
    const int8_t* prow = pos + p * H;
    for (int c = lane * 16; c < H; c += 512) {
      const uint4 wv = __ldg(reinterpret_cast<const uint4*>(wrow + c));
      const uint4 pv = __ldg(reinterpret_cast<const uint4*>(prow + c));
      const uint32_t ww[4] = {wv.x, wv.y, wv.z, wv.w};
      int32_t o[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) o[i] = (int32_t)(int8_t)(ww[i >> 2] >> (8 * (i & 3)));
      int4* qd = reinterpret_cast<int4*>(q + t * H + c);
#pragma unroll
      for (int i = 0; i < 4; ++i) qd[i] = make_int4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
      *reinterpret_cast<uint4*>(r + t * H + c) = pv;
    }
  }
}

// ----------------------------------------------------------------------------- wait self-test
// Two warps wait on an mbarrier nobody arrives on, with a short limit: one by the polling form of the
// bounded wait (mbar_wait_ns), one by the parked form the GEMM feeder threads use (mbar_wait_parked_ns).
// When BOTH limits have run out the kernel records IBERT_ERR_TIMEOUT like every kernel of the library
// does, and returns normally.
__global__ void __launch_bounds__(64) wait_timeout_kernel(uint64_t limit_ns, int32_t* status) {
  __shared__ uint64_t bar;
  __shared__ int expired;
  if (threadIdx.x == 0) {
    ptx::mbar_init(ptx::smem_addr(&bar), 1);
    ptx::fence_mbar_init();
    expired = 0;
  }
  __syncthreads();
  const bool ok = (threadIdx.x < 32) ? __all_sync(0xffffffffu, ptx::mbar_wait_ns(ptx::smem_addr(&bar), 0, limit_ns))
                                     : __all_sync(0xffffffffu, ptx::mbar_wait_parked_ns(ptx::smem_addr(&bar), 0, limit_ns));
  if (!ok && (threadIdx.x & 31) == 0) atomicAdd(&expired, 1);
  __syncthreads();
  if (threadIdx.x == 0 && expired == 2) atomicCAS(status, 0, IBERT_ERR_TIMEOUT);
}

// Row cu[b] of x (the first token of sequence b of a packed batch) -> row b of out; one warp per row.
__global__ void __launch_bounds__(kThreads) gather_first_rows_kernel(const int8_t* __restrict__ x, const int32_t* __restrict__ cu,
                                                                     int B, int H, int8_t* __restrict__ out) {
  const int lane = threadIdx.x & 31;
  const int b = (int)(((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5);
  if (b >= B) return;
  const int8_t* src = x + (int64_t)__ldg(cu + b) * H;
  for (int c = lane * 16; c < H; c += 512)
    *reinterpret_cast<uint4*>(out + (int64_t)b * H + c) = __ldg(reinterpret_cast<const uint4*>(src + c));
}

// Short rows (L <= 128, a multiple of 4: one 16-byte vector per lane): a warp takes R rows at a time.  The one
// true division a row needs (Algorithm 3's quotient by the row sum, made a multiplication for its elements)
// costs about as much as the rest of a 128-element row; lane r performs it for row r, so one division
// instruction stream serves R rows, and the R loads of a lane are in flight together.
template <int R, int DIV>
__global__ void __launch_bounds__(kThreads, 4) softmax_short_kernel(const int32_t* __restrict__ q, int64_t rows,
                                                                 int L, ExpConsts k, uint8_t* __restrict__ out,
                                                                 const uint32_t* __restrict__ table) {
  const int lane = threadIdx.x & 31;
  const int64_t warp_global = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
  const int64_t warp_count = ((int64_t)gridDim.x * kThreads) >> 5;
  const int col = 4 * lane;
  const bool in_row = col < L;
  for (int64_t row0 = warp_global * R; row0 < rows; row0 += warp_count * R) {
    int32_t v[R][4];
    uint32_t sums[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      if (in_row && row0 + r < rows) {
        const int4 t = __ldcs(reinterpret_cast<const int4*>(q + (row0 + r) * L + col));
        v[r][0] = t.x; v[r][1] = t.y; v[r][2] = t.z; v[r][3] = t.w;
      } else {
        v[r][0] = v[r][1] = v[r][2] = v[r][3] = INT32_MIN;
      }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      int32_t mx = max(max(v[r][0], v[r][1]), max(v[r][2], v[r][3]));
      mx = __reduce_max_sync(0xffffffffu, mx);
      uint32_t sum = 0;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t dist = (uint32_t)mx - (uint32_t)v[r][i];
        uint32_t e = 0u;
        if (in_row && row0 + r < rows) {
          if constexpr (DIV == kExpByTable) e = __ldg(table + min(dist >> k.s_in, k.d_max));
          else e = iexp_dist<DIV>(dist, k);
        }
        v[r][i] = (int32_t)e;
        sum += e;
      }
      sums[r] = max(__reduce_add_sync(0xffffffffu, sum), 1u);     // (0 only for a row past the end)
    }
    uint32_t my_sum = sums[0];
#pragma unroll
    for (int r = 1; r < R; ++r) my_sum = lane == r ? sums[r] : my_sum;
    const uint32_t my_m = make_row_divisor(my_sum, k.p_max).m;
#pragma unroll
    for (int r = 0; r < R; ++r) {
      RowDivisor rd;
      rd.m = __shfl_sync(0xffffffffu, my_m, r);
      const int K = 21 + 32 - __clz(sums[r]);
      rd.pre = K < 32 ? 32 - K : 0;
      rd.post = K < 32 ? 0 : K - 32;
      uint32_t p[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) p[i] = softmax_quotient((uint32_t)v[r][i], rd);
      if (in_row && row0 + r < rows)
        __stcs(reinterpret_cast<uint32_t*>(out + (row0 + r) * L + col), p[0] | (p[1] << 8) | (p[2] << 16) | (p[3] << 24));
    }
  }
}

int grid_for(ibert_ctx* ctx, int64_t work_warps, int max_ctas_per_sm) {
  const int64_t ctas = (work_warps + (kThreads / 32) - 1) / (kThreads / 32);
  const int64_t cap = (int64_t)ctx->num_sms * max_ctas_per_sm;
  return (int)(ctas < 1 ? 1 : (ctas > cap ? cap : ctas));
}

// grid of at most one wave of resident CTAs of `kernel` (its registers decide how many an SM holds: a larger
// grid of grid-stride CTAs runs as a full wave plus a partial one)
template <typename Kernel>
int wave_grid(ibert_ctx* ctx, Kernel kernel, int64_t work_warps) {
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreads, 0) != cudaSuccess || per_sm < 1) per_sm = 1;
  return grid_for(ctx, work_warps, std::min(per_sm, 8));
}

int check_launch() { return cudaGetLastError() == cudaSuccess ? IBERT_OK : IBERT_ERR_CUDA; }

}  // namespace

int launch_wait_timeout(ibert_ctx* ctx, uint64_t limit_ns) {
  wait_timeout_kernel<<<1, 64, 0, ctx->stream>>>(limit_ns, ctx->d_status);
  return check_launch();
}

int launch_embed_gather(ibert_ctx* ctx, const int32_t* ids, int64_t T, int L, const int8_t* word, int64_t V,
                        const int8_t* pos, int H, int32_t* q, int8_t* r, const int32_t* cu_seqlens, int B) {
  if (T == 0) return IBERT_OK;
  embed_gather_kernel<<<grid_for(ctx, T, 8), kThreads, 0, ctx->stream>>>(ids, T, L, word, V, pos, H, q, r,
                                                                          ctx->d_status, cu_seqlens, B);
  return check_launch();
}

int launch_gather_first_rows(ibert_ctx* ctx, const int8_t* x, const int32_t* cu_seqlens, int B, int H, int8_t* out) {
  if (B == 0) return IBERT_OK;
  gather_first_rows_kernel<<<(B + kThreads / 32 - 1) / (kThreads / 32), kThreads, 0, ctx->stream>>>(x, cu_seqlens, B, H, out);
  return check_launch();
}

int launch_gelu_table(ibert_ctx* ctx, const GeluConsts& k, int32_t* ramp_scratch, int8_t* table) {
  ramp_q16_kernel<<<(65535 + kThreads - 1) / kThreads, kThreads, 0, ctx->stream>>>(ramp_scratch);
  if (int rc = check_launch()) return rc;
  return launch_gelu(ctx, ramp_scratch, 65535, k, table);
}

int launch_gelu_lut(ibert_ctx* ctx, const int32_t* q, int64_t n, const int8_t* table, int8_t* out) {
  if (n == 0) return IBERT_OK;
  const int64_t warps = ((n >> 2) + 31) / 32 / 8 + 1;          // ~8 vectors per thread
  gelu_lut_kernel<<<wave_grid(ctx, gelu_lut_kernel, warps), kThreads, 0, ctx->stream>>>(q, n, table, out);
  return check_launch();
}

int launch_gelu(ibert_ctx* ctx, const int32_t* q, int64_t n, const GeluConsts& k, int8_t* out) {
  if (n == 0) return IBERT_OK;
  const int64_t warps = ((n >> 2) + 127) / 128 + 1;
  gelu_kernel<<<wave_grid(ctx, gelu_kernel, warps), kThreads, 0, ctx->stream>>>(q, n, k, out);
  return check_launch();
}

int launch_exp_table(ibert_ctx* ctx, const ExpConsts& k, uint32_t* table) {
  exp_table_kernel<<<(int)((k.d_max + kThreads) / kThreads), kThreads, 0, ctx->stream>>>(k, table);
  return check_launch();
}

int launch_softmax(ibert_ctx* ctx, const int32_t* q, int64_t rows, int L, const ExpConsts& k, uint8_t* out,
                   const uint32_t* exp_table) {
  if (rows == 0) return IBERT_OK;
  const bool vec = (L % 4) == 0;
  const int vpl = (L + 127) / 128;   // vectors per lane
  const int div = exp_table ? kExpByTable : exp_div_mode(k);
#define IBERT_SM2(V, D)                                                                                       \
  do {                                                                                                        \
    if (vec) softmax_kernel<V, true, D><<<wave_grid(ctx, softmax_kernel<V, true, D>, rows), kThreads, 0, ctx->stream>>>(q, rows, L, k, out, exp_table);   \
    else softmax_kernel<V, false, D><<<wave_grid(ctx, softmax_kernel<V, false, D>, rows), kThreads, 0, ctx->stream>>>(q, rows, L, k, out, exp_table);      \
  } while (0)
#define IBERT_SM(V)                 \
  do {                              \
    if (div == 0) IBERT_SM2(V, 0);  \
    else if (div == 1) IBERT_SM2(V, 1); \
    else if (div == 2) IBERT_SM2(V, 2); \
    else IBERT_SM2(V, kExpByTable);     \
  } while (0)
  if (vpl <= 1 && vec) {
    constexpr int R = 4;
    const int sgrid = grid_for(ctx, (rows + R - 1) / R, 4);      // (one wave: four CTAs are resident per SM)
    if (div == 0) softmax_short_kernel<R, 0><<<sgrid, kThreads, 0, ctx->stream>>>(q, rows, L, k, out, exp_table);
    else if (div == 1) softmax_short_kernel<R, 1><<<sgrid, kThreads, 0, ctx->stream>>>(q, rows, L, k, out, exp_table);
    else if (div == 2) softmax_short_kernel<R, 2><<<sgrid, kThreads, 0, ctx->stream>>>(q, rows, L, k, out, exp_table);
    else softmax_short_kernel<R, kExpByTable><<<sgrid, kThreads, 0, ctx->stream>>>(q, rows, L, k, out, exp_table);
  }
  else if (vpl <= 1) IBERT_SM(1);
  else if (vpl <= 2) IBERT_SM(2);
  else if (vpl <= 4) IBERT_SM(4);
  else IBERT_SM(8);
#undef IBERT_SM
#undef IBERT_SM2
  return check_launch();
}

template <typename QT>
static int launch_layernorm_t(ibert_ctx* ctx, const QT* q, const int8_t* r, int64_t rows, const LnConsts& k,
                              const int32_t* d_b, const int64_t* d_B, int8_t* out) {
  if (rows == 0) return IBERT_OK;
  const bool vec = (k.C % 4) == 0;
  const int vpl = (k.C + 127) / 128;
  const bool fast = vec && k.out_fast && (!k.has_res || k.res_fast);
  if (fast && k.has_res && k.res_narrow && k.C % 16 == 0 && k.C <= 1024) {
    // streaming variant: per-warp ring of row slots filled by bulk async copies
    const int depth = 2;
    const size_t smem = (size_t)(kThreads / 32) * depth * (size_t)k.C * (sizeof(QT) + 1) + (kThreads / 32) * depth * 8 +
                        (size_t)k.C * 12;                  // rows in flight, barriers, the two tables
    // one wave of resident CTAs: three per SM by registers, fewer when the row slots take more shared memory
    // (C = 1024 with int32 input: two -- a grid of three per SM ran as a wave and a half)
    const int per_sm = (int)std::min<size_t>(3, (size_t)(227 * 1024) / (smem + 1024));
    const int pgrid = (int)std::min<int64_t>((rows + 7) / 8, (int64_t)ctx->num_sms * std::max(per_sm, 1));
#define IBERT_LNP2(V, D, F)                                                                                 \
  do {                                                                                                      \
    static bool attr_dev[kMaxDevices] = {false};                                                            \
    bool& attr = attr_dev[ctx->device % kMaxDevices];                                                       \
    if (!attr) {                                                                                            \
      if (cudaFuncSetAttribute(layernorm_pipe_kernel<V, D, QT, F>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                               100 * 1024) != cudaSuccess) return IBERT_ERR_CUDA;                           \
      attr = true;                                                                                          \
    }                                                                                                       \
    if (int rc_ = launch_pdl(layernorm_pipe_kernel<V, D, QT, F>, dim3(pgrid), dim3(kThreads), smem, ctx->stream, 1, q, r, \
                             rows, k, d_b, d_B, out, ctx->d_status))                                        \
      return rc_;                                                                                           \
  } while (0)
#define IBERT_LNP(V, D)                       \
  do {                                        \
    if (k.C == 128 * V) IBERT_LNP2(V, D, true); \
    else IBERT_LNP2(V, D, false);             \
  } while (0)
    if (k.C <= 256) IBERT_LNP(2, 2);
    else if (k.C <= 512) IBERT_LNP(4, 2);
    else if (k.C <= 768) IBERT_LNP(6, 2);
    else IBERT_LNP(8, 2);
#undef IBERT_LNP
#undef IBERT_LNP2
    return check_launch();
  }
#define IBERT_LN(V)                                                                                              \
  do {                                                                                                           \
    if (fast) layernorm_kernel<V, true, true, QT><<<wave_grid(ctx, layernorm_kernel<V, true, true, QT>, rows), kThreads, 0, ctx->stream>>>(q, r, rows, k, d_b, d_B, out);  \
    else if (vec) layernorm_kernel<V, true, false, QT><<<wave_grid(ctx, layernorm_kernel<V, true, false, QT>, rows), kThreads, 0, ctx->stream>>>(q, r, rows, k, d_b, d_B, out); \
    else layernorm_kernel<V, false, false, QT><<<wave_grid(ctx, layernorm_kernel<V, false, false, QT>, rows), kThreads, 0, ctx->stream>>>(q, r, rows, k, d_b, d_B, out);     \
  } while (0)
  if (vpl <= 2) IBERT_LN(2);
  else if (vpl <= 4) IBERT_LN(4);
  else if (vpl <= 6) IBERT_LN(6);
  else if (vpl <= 8) IBERT_LN(8);
  else IBERT_LN(16);
#undef IBERT_LN
  return check_launch();
}

int launch_layernorm(ibert_ctx* ctx, const int32_t* q, const int8_t* r, int64_t rows, const LnConsts& k,
                     const int32_t* d_b, const int64_t* d_B, int8_t* out) {
  return launch_layernorm_t<int32_t>(ctx, q, r, rows, k, d_b, d_B, out);
}

int launch_layernorm_i16(ibert_ctx* ctx, const int16_t* q, const int8_t* r, int64_t rows, const LnConsts& k,
                         const int32_t* d_b, const int64_t* d_B, int8_t* out) {
  return launch_layernorm_t<int16_t>(ctx, q, r, rows, k, d_b, d_B, out);
}

}  // namespace ibert
