// Fused integer-only attention for one (batch, head, 128-query tile) per CTA:
//   S = Q K^T (tcgen05 kind::i8, int32 accumulators in TMEM; scale S_q S_k / 8)
//   P = i-softmax(S) (Algorithm 3: row max, i-exp, int32 row sum, fixed-point quotient) -> u8
//   ctx = requant(P V) (u8 x s8 tcgen05 MMA, accumulator reuses the score columns)
// Scores never leave the SM: they live in TMEM, the exponentials overwrite them in place,
// and the probabilities go to shared memory in the layout the second MMA reads.
#include <cuda.h>

#include "device_utils.cuh"
#include "sm100_ptx.cuh"

namespace ibert {

namespace {

constexpr int kAttnThreads = 128;   // thread t owns query row t (= TMEM lane t)
constexpr int kHeadDim = 64;

struct AttnArgs {
  int B, L, H, heads;
  int Lp;            // L rounded up to a multiple of 32 (MMA N / K granularity)
  int n_slabs;       // ceil(L / 128)
  uint32_t tmem_cols;
  AttnConsts k;
  int8_t* out;
  int32_t* status;
};

// byte offset of element (row, col) in a K-major operand tile made of 128-byte-wide K blocks
// with the 128-byte swizzle: 16-byte chunk c of row r sits at chunk c ^ (r & 7).
__device__ __forceinline__ uint32_t sw128_offset(uint32_t row, uint32_t col, uint32_t rows_per_block) {
  const uint32_t kb = col >> 7, cc = (col >> 4) & 7, by = col & 15;
  return kb * (rows_per_block * 128u) + row * 128u + (((cc ^ (row & 7u)) << 4) | by);
}

// i-softmax (Algorithm 3) of one score row held in TMEM lane `t_row`, columns [0, L):
// pass 1 row maximum, pass 2 i-exp + int32 row sum (exponentials written back over the scores),
// pass 3 fixed-point quotient -> u8 probabilities into the swizzled operand tile `sP`, row `row`.
// Columns [L, Lp) are padding: excluded from max and sum, written as probability 0.
template <int DIV>
__device__ __forceinline__ void softmax_row(uint32_t t_row, int L, int Lp, const ExpConsts& ek, uint8_t* sP,
                                            uint32_t row) {
  const int full = L & ~31;             // columns covered by whole 32-column chunks
  int32_t mx = INT32_MIN;
  for (int c0 = 0; c0 < Lp; c0 += 32) {
    uint32_t v[32];
    ptx::tmem_ld32(t_row + c0, v);
    ptx::tmem_wait_ld();
    if (c0 < full) {
#pragma unroll
      for (int i = 0; i < 32; ++i) mx = max(mx, (int32_t)v[i]);
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i)
        if (c0 + i < L) mx = max(mx, (int32_t)v[i]);
    }
  }
  uint32_t sum = 0;
  for (int c0 = 0; c0 < Lp; c0 += 32) {
    uint32_t v[32];
    ptx::tmem_ld32(t_row + c0, v);
    ptx::tmem_wait_ld();
    if (c0 < full) {
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        v[i] = iexp_dist<DIV>((uint32_t)mx - v[i], ek);
        sum += v[i];
      }
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        v[i] = (c0 + i < L) ? iexp_dist<DIV>((uint32_t)mx - v[i], ek) : 0u;
        sum += v[i];
      }
    }
    ptx::tmem_st32(t_row + c0, v);
  }
  ptx::tmem_wait_st();
  const RowDivisor rd = make_row_divisor(sum, ek.p_max);
  for (int c0 = 0; c0 < Lp; c0 += 32) {
    uint32_t v[32];
    ptx::tmem_ld32(t_row + c0, v);
    ptx::tmem_wait_ld();
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      uint32_t w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int j = h * 16 + i * 4;
        w[i] = softmax_quotient(v[j], rd) | (softmax_quotient(v[j + 1], rd) << 8) |
               (softmax_quotient(v[j + 2], rd) << 16) | (softmax_quotient(v[j + 3], rd) << 24);
      }
      *reinterpret_cast<uint4*>(sP + sw128_offset(row, (uint32_t)(c0 + h * 16), 128)) =
          make_uint4(w[0], w[1], w[2], w[3]);
    }
  }
}

__global__ void __launch_bounds__(kAttnThreads)
attention_kernel(const __grid_constant__ CUtensorMap map_qk, const __grid_constant__ CUtensorMap map_v,
                 const AttnArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int slab_bytes = 128 * kHeadDim;                       // 8 KB
  uint8_t* sQ = smem;
  uint8_t* sK = sQ + slab_bytes;
  uint8_t* sVt = sK + a.n_slabs * slab_bytes;                   // [n_slabs][64 rows][128 B], swizzled
  uint8_t* sP = sVt + a.n_slabs * slab_bytes;                   // [n_slabs][128 rows][128 B], swizzled
  uint8_t* sVs = sP;                                            // V staging [L][64], aliases P (used before it)
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(sP + a.n_slabs * 128 * 128);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_bar + 2);
  const uint32_t bar_load = ptx::smem_addr(s_bar);
  const uint32_t bar_mma = bar_load + 8;

  const int tid = threadIdx.x, warp = tid >> 5;
  const int q0 = blockIdx.x * 128, head = blockIdx.y, batch = blockIdx.z;
  const int L = a.L, Lp = a.Lp;

  if (tid == 0) {
    ptx::mbar_init(bar_load, 1);
    ptx::mbar_init(bar_mma, 1);
    ptx::fence_mbar_init();
    ptx::tma_prefetch_desc(&map_qk);
    ptx::tma_prefetch_desc(&map_v);
  }
  if (warp == 0) {
    ptx::tmem_alloc(ptx::smem_addr(s_tmem), a.tmem_cols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *s_tmem;

  // ---- loads: Q tile, all K rows (64-byte swizzle, MMA operand layout), all V rows (plain)
  if (tid == 0) {
    ptx::mbar_arrive_expect_tx(bar_load, (uint32_t)((1 + 2 * a.n_slabs) * slab_bytes));
    ptx::tma_load_3d(ptx::smem_addr(sQ), &map_qk, bar_load, head * kHeadDim, q0, batch);
    for (int s = 0; s < a.n_slabs; ++s) {
      ptx::tma_load_3d(ptx::smem_addr(sK + s * slab_bytes), &map_qk, bar_load, a.H + head * kHeadDim, s * 128, batch);
      ptx::tma_load_3d(ptx::smem_addr(sVs + s * slab_bytes), &map_v, bar_load, 2 * a.H + head * kHeadDim, s * 128, batch);
    }
  }
  bool ok = __all_sync(0xffffffffu, ptx::mbar_wait(bar_load, 0));

  // ---- S = Q K^T: K = 64 bytes = two MMA K-steps; N in chunks of at most 256 columns
  if (ok && tid == 0) {
    ptx::tc_fence_after_sync();
    const uint64_t dq = ptx::make_kmajor_desc(ptx::smem_addr(sQ), 512, ptx::kSwizzle64);
    for (int n0 = 0; n0 < Lp; n0 += 256) {
      const int nn = min(256, Lp - n0);
      const uint32_t idesc = ptx::make_idesc_i8(128, nn, true, true);
      const uint64_t dk = ptx::make_kmajor_desc(ptx::smem_addr(sK + n0 * kHeadDim), 512, ptx::kSwizzle64);
      ptx::mma_i8_ss(tmem_base + n0, dq, dk, idesc, 0u);
      ptx::mma_i8_ss(tmem_base + n0, dq + 2, dk + 2, idesc, 1u);
    }
    ptx::mma_commit(bar_mma);
  }

  // ---- meanwhile: transpose V [j][d] -> Vt [d][j] into the swizzled K-major operand layout
  if (ok) {
    for (int j = tid; j < a.n_slabs * 128; j += kAttnThreads) {
      const uint4* src = reinterpret_cast<const uint4*>(sVs + j * kHeadDim);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const uint4 v = src[c];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const uint32_t d = c * 16 + i;
          sVt[sw128_offset(d, (uint32_t)j, 64)] = (uint8_t)(w[i >> 2] >> (8 * (i & 3)));
        }
      }
    }
  }
  __syncthreads();                                            // staging is dead: P may overwrite it
  if (ok) ok = __all_sync(0xffffffffu, ptx::mbar_wait(bar_mma, 0));

  // ---- i-softmax on the row this thread owns
  const uint32_t t_row = tmem_base + ((uint32_t)(warp * 32) << 16);
  if (ok) {
    ptx::tc_fence_after_sync();
    switch (exp_div_mode(a.k.e)) {
      case 0: softmax_row<0>(t_row, L, Lp, a.k.e, sP, (uint32_t)tid); break;
      case 1: softmax_row<1>(t_row, L, Lp, a.k.e, sP, (uint32_t)tid); break;
      default: softmax_row<2>(t_row, L, Lp, a.k.e, sP, (uint32_t)tid); break;
    }
    ptx::fence_proxy_async_smem();          // P and Vt were written by ordinary stores; the MMA reads them
  }
  ptx::tc_fence_before_sync();
  __syncthreads();

  // ---- ctx = P V: K = Lp in steps of 32, accumulator in columns 0..63 (scores are dead)
  if (ok && tid == 0) {
    ptx::tc_fence_after_sync();
    const uint32_t idesc = ptx::make_idesc_i8(128, kHeadDim, false, true);   // u8 x s8
    for (int kk = 0; kk < Lp / 32; ++kk) {
      const int kb = kk >> 2, ks = kk & 3;
      const uint64_t dp = ptx::make_kmajor_desc(ptx::smem_addr(sP + kb * 128 * 128), 1024, ptx::kSwizzle128);
      const uint64_t dv = ptx::make_kmajor_desc(ptx::smem_addr(sVt + kb * 64 * 128), 1024, ptx::kSwizzle128);
      ptx::mma_i8_ss(tmem_base, dp + 2 * ks, dv + 2 * ks, idesc, kk != 0 ? 1u : 0u);
    }
    ptx::mma_commit(bar_mma);
  }
  if (ok) ok = __all_sync(0xffffffffu, ptx::mbar_wait(bar_mma, 1));

  // ---- epilogue: requantize the 64 context values of this row to int8
  if (ok) {
    ptx::tc_fence_after_sync();
    const int64_t half = rounding_half(a.k.c);
    const int q_row = q0 + tid;
    int8_t* orow = a.out + ((int64_t)batch * L + q_row) * a.H + head * kHeadDim;
#pragma unroll
    for (int c0 = 0; c0 < kHeadDim; c0 += 32) {
      uint32_t v[32];
      ptx::tmem_ld32(t_row + c0, v);
      ptx::tmem_wait_ld();
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint32_t pk = 0;
#pragma unroll
          for (int e = 0; e < 4; ++e)
            pk |= (uint32_t)(requant_add((int32_t)v[h * 16 + i * 4 + e], a.k.b, half, a.k.c, 127) & 0xff) << (8 * e);
          w[i] = pk;
        }
        if (q_row < L) *reinterpret_cast<uint4*>(orow + c0 + h * 16) = make_uint4(w[0], w[1], w[2], w[3]);
      }
    }
  }
  if (!ok) atomicCAS(a.status, 0, IBERT_ERR_TIMEOUT);
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, a.tmem_cols);
  }
}

}  // namespace

int launch_attention(ibert_ctx* ctx, const int8_t* qkv, int B, int L, int H, int heads,
                     const AttnConsts& k, int8_t* out) {
  if (B == 0) return IBERT_OK;
  AttnArgs a{};
  a.B = B; a.L = L; a.H = H; a.heads = heads;
  a.Lp = (L + 31) & ~31;
  a.n_slabs = (L + 127) / 128;
  uint32_t cols = 64;
  while ((int)cols < a.Lp) cols <<= 1;
  a.tmem_cols = cols;
  a.k = k;
  a.out = out;
  a.status = ctx->d_status;
  CUtensorMap mqk, mv;
  const uint64_t dims[3] = {(uint64_t)3 * H, (uint64_t)L, (uint64_t)B};
  const uint64_t str[2] = {(uint64_t)3 * H, (uint64_t)3 * H * L};
  const uint32_t box[3] = {kHeadDim, 128, 1};
  int rc = encode_tensor_map(&mqk, qkv, 3, dims, str, box, 64);
  if (rc) return rc;
  rc = encode_tensor_map(&mv, qkv, 3, dims, str, box, 0);
  if (rc) return rc;
  const int smem = (1 + 2 * a.n_slabs) * 128 * kHeadDim + a.n_slabs * 128 * 128 + 64 + 1024;
  static int smem_set = 0;
  if (smem > smem_set) {
    if (cudaFuncSetAttribute(attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
      return IBERT_ERR_CUDA;
    smem_set = smem;
  }
  dim3 grid((L + 127) / 128, heads, B);
  attention_kernel<<<grid, kAttnThreads, smem, ctx->stream>>>(mqk, mv, a);
  return cudaGetLastError() == cudaSuccess ? IBERT_OK : IBERT_ERR_CUDA;
}

}  // namespace ibert
