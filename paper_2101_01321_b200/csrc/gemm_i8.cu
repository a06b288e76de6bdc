// INT8 x INT8 -> INT32 GEMM on the 5th-generation tensor cores (tcgen05.mma kind::i8,
// accumulators in TMEM, operands staged by TMA) with the integer epilogue fused:
// bias add + dyadic requantization to int8 or Q16, raw accumulators, or requantization
// to Q16 followed by i-GELU (Algorithm 2) and a second requantization to int8.
//
// out[m, n] = epilogue( sum_k x[m, k] * w[n, k] + bias[n] )      x: [M, K], w: [N, K]
//
// One persistent CTA per SM walks 128 x BN output tiles.  Warp 0 is the TMA producer,
// warp 1 issues the MMAs, warps 2.. run the epilogue; two TMEM accumulator stages let
// the (integer-ALU heavy) epilogue of tile i overlap the MMAs of tile i+1.
#include <cuda.h>

#include <mutex>

#include "device_utils.cuh"
#include "sm100_ptx.cuh"

namespace ibert {

// --------------------------------------------------------------------------------------
// tensor-map encoding through the driver entry point
// --------------------------------------------------------------------------------------
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
    else
      cudaGetLastError();
  });
  return fn;
}

}  // namespace

int encode_tensor_map(CUtensorMap* map, const void* base, int rank, const uint64_t* dims,
                      const uint64_t* strides_bytes, const uint32_t* box, int swizzle_bytes) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return IBERT_ERR_CUDA;
  cuuint64_t gdim[5];
  cuuint64_t gstr[5];
  cuuint32_t bdim[5];
  cuuint32_t estr[5];
  for (int i = 0; i < rank; ++i) {
    gdim[i] = dims[i];
    bdim[i] = box[i];
    estr[i] = 1;
    if (i + 1 < rank) gstr[i] = strides_bytes[i];
  }
  const CUtensorMapSwizzle sw = swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                : swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                                      : CU_TENSOR_MAP_SWIZZLE_NONE;
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, (cuuint32_t)rank, const_cast<void*>(base), gdim, gstr,
                  bdim, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? IBERT_OK : IBERT_ERR_CUDA;
}

// --------------------------------------------------------------------------------------
// kernel
// --------------------------------------------------------------------------------------
namespace {

constexpr int BM = 128;           // rows per tile = TMEM lanes
constexpr int BK = 128;           // K bytes per pipeline stage = one 128-byte swizzle span
constexpr int UMMA_K = 32;        // K per tcgen05.mma kind::i8
// Epilogue warps: every warp handles two 32-column chunks of the 32 rows (TMEM lanes) its
// position in the warp quartet gives it access to, so a tile of BN columns takes BN / 16 warps.
// The integer epilogue is what bounds these GEMMs at K <= 1024, hence the many warps.
__host__ __device__ constexpr int epi_warps(int bn) { return bn / 16; }
__host__ __device__ constexpr int gemm_threads(int bn) { return 64 + 32 * epi_warps(bn); }   // + producer warp, MMA warp

template <int BN>
struct GemmSmem {
  static constexpr int kStages = BN >= 256 ? 3 : 5;
  static constexpr int kABytes = BM * BK;
  static constexpr int kBBytes = BN * BK;
  static constexpr int kStageBytes = kABytes + kBBytes;
  // operand stages | output staging (one 4 KB tile per epilogue warp) | per-column epilogue
  // parameters (int4 per column) | barriers
  static constexpr int kOutOff = kStages * kStageBytes;
  static constexpr int kOutTileBytes = 32 * 128;
  static constexpr int kParamOff = kOutOff + epi_warps(BN) * kOutTileBytes;
  static constexpr int kBarOff = kParamOff + BN * 16;
  static constexpr int kBytes = kBarOff + 256;
  static constexpr int kAlloc = kBytes + 1024;   // slack to align the operand area to 1024 bytes
};

struct GemmArgs {
  int64_t M;
  int N, K;
  const int32_t* b;
  const int32_t* c;
  const int32_t* bias;
  GeluConsts gelu;
  int32_t* status;
};

// One 32-column chunk of one accumulator row: registers -> epilogue -> the warp's staging tile
// (32 rows x ROW_BYTES, 16-byte pieces XOR-swizzled the way the TMA store expects).
// `piece0` is the index of the first 16-byte piece this chunk occupies in the staging row.
// FAST: every column's requantization is in upper-word form (one 64-bit multiply-add).
template <int ROW_BYTES>
__device__ __forceinline__ uint32_t staging_piece_offset(uint32_t row, uint32_t piece) {
  if constexpr (ROW_BYTES == 128) return row * 128u + ((piece ^ (row & 7u)) << 4);
  else return row * 64u + ((piece ^ ((row >> 1) & 3u)) << 4);
}

template <int KIND, bool FAST, int ROW_BYTES>
__device__ __forceinline__ void epilogue_chunk(const uint32_t (&v)[32], const int4* __restrict__ prm,
                                               const GeluConsts& gk, int64_t gelu_half, uint8_t* stage,
                                               uint32_t row, uint32_t piece0) {
  if constexpr (KIND == EPI_RAW || KIND == EPI_Q16) {
#pragma unroll
    for (int g = 0; g < 8; ++g) {
      int32_t o[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int4 p = prm[g * 4 + i];
        const int32_t a = (int32_t)v[g * 4 + i];
        const int64_t add = (int64_t)(((uint64_t)(uint32_t)p.w << 32) | (uint32_t)p.z);
        if constexpr (KIND == EPI_RAW) o[i] = a + p.x;
        else if constexpr (FAST) o[i] = clamp_sym(requant_upper(a, p.x, add), 32767);
        else o[i] = requant_add(a, p.x, add, p.y, 32767);
      }
      *reinterpret_cast<int4*>(stage + staging_piece_offset<ROW_BYTES>(row, piece0 + g)) =
          make_int4(o[0], o[1], o[2], o[3]);
    }
  } else {
#pragma unroll
    for (int g = 0; g < 2; ++g) {
      uint32_t w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        int32_t o[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int idx = g * 16 + i * 4 + e;
          const int4 p = prm[idx];
          const int32_t a = (int32_t)v[idx];
          const int64_t add = (int64_t)(((uint64_t)(uint32_t)p.w << 32) | (uint32_t)p.z);
          if constexpr (KIND == EPI_INT8) {
            if constexpr (FAST) o[e] = max(requant_upper(a, p.x, add), -127);
            else o[e] = requant_add(a, p.x, add, p.y, 127);
          } else {
            if constexpr (FAST) {
              const int32_t q16 = clamp_sym(requant_upper(a, p.x, add), 32767);
              o[e] = igelu_q16_upper(q16, gk);
            } else {
              const int32_t q16 = requant_add(a, p.x, add, p.y, 32767);
              o[e] = igelu_q16_to_int8(q16, gk, gelu_half);
            }
          }
        }
        w[i] = pack4_sat_s8(o[0], o[1], o[2], o[3]);    // upper clamp (+127) happens here
      }
      *reinterpret_cast<uint4*>(stage + staging_piece_offset<ROW_BYTES>(row, piece0 + g)) =
          make_uint4(w[0], w[1], w[2], w[3]);
    }
  }
}

template <int BN, int KIND, bool FAST>
__global__ void __launch_bounds__(gemm_threads(BN), 1)
gemm_i8_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_out, const GemmArgs args) {
  using SM = GemmSmem<BN>;
  constexpr int kStages = SM::kStages;
  constexpr int kEpiThreads = 32 * epi_warps(BN);
  constexpr uint32_t kTmemCols = 2 * BN;          // two accumulator stages (power of two >= 32)
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = ptx::smem_addr(smem);
  int4* s_param = reinterpret_cast<int4*>(smem + SM::kParamOff);
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(smem + SM::kBarOff);
  // barrier slots: full[kStages], empty[kStages], acc_full[2], acc_empty[2], then the TMEM base word
  const uint32_t bar_full = ptx::smem_addr(s_bar);
  const uint32_t bar_empty = bar_full + 8 * kStages;
  const uint32_t bar_acc_full = bar_empty + 8 * kStages;
  const uint32_t bar_acc_empty = bar_acc_full + 16;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_bar + 2 * kStages + 4);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int n_tiles = (args.N + BN - 1) / BN;
  const int64_t m_tiles = (args.M + BM - 1) / BM;
  const int64_t total_tiles = m_tiles * n_tiles;
  const int k_blocks = (args.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(bar_full + 8 * s, 1);
      ptx::mbar_init(bar_empty + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(bar_acc_full + 8 * a, 1);
      ptx::mbar_init(bar_acc_empty + 8 * a, kEpiThreads);
    }
    ptx::fence_mbar_init();
    ptx::tma_prefetch_desc(&map_a);
    ptx::tma_prefetch_desc(&map_b);
    ptx::tma_prefetch_desc(&map_out);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_addr(s_tmem), kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *s_tmem;
  bool ok = true;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      for (int64_t tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const int m0 = (int)(tile / n_tiles) * BM;
        const int n0 = (int)(tile % n_tiles) * BN;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!ptx::mbar_wait(bar_empty + 8 * stage, phase ^ 1)) { ok = false; break; }
          const uint32_t sa = smem_base + stage * SM::kStageBytes;
          ptx::mbar_arrive_expect_tx(bar_full + 8 * stage, SM::kStageBytes);
          ptx::tma_load_2d(sa, &map_a, bar_full + 8 * stage, kb * BK, m0);
          ptx::tma_load_2d(sa + SM::kABytes, &map_b, bar_full + 8 * stage, kb * BK, n0);
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::make_idesc_i8(BM, BN, true, true);
      uint32_t stage = 0, phase = 0;
      uint32_t acc = 0, acc_phase = 0;
      for (int64_t tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        if (!ptx::mbar_wait(bar_acc_empty + 8 * acc, acc_phase ^ 1)) { ok = false; break; }
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!ptx::mbar_wait(bar_full + 8 * stage, phase)) { ok = false; break; }
          ptx::tc_fence_after_sync();
          const uint32_t sa = smem_base + stage * SM::kStageBytes;
          const uint64_t da = ptx::make_kmajor_desc(sa, 1024, ptx::kSwizzle128);
          const uint64_t db = ptx::make_kmajor_desc(sa + SM::kABytes, 1024, ptx::kSwizzle128);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // advancing K inside the swizzle span: +32 bytes = +2 in the encoded start address
            ptx::mma_i8_ss(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          ptx::mma_commit(bar_empty + 8 * stage);     // frees the stage once these MMAs have read it
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        ptx::mma_commit(bar_acc_full + 8 * acc);      // accumulator complete
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1;
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..)
    // Warp w owns TMEM lanes 32*(w%4)..+31 (rows) and, of those rows, 64 of the tile's
    // columns.  Results go through a swizzled staging tile in shared memory and leave with a TMA
    // store (full-line writes; rows / columns beyond M / N are clipped by the tensor map).
    constexpr bool kOut32 = (KIND == EPI_RAW || KIND == EPI_Q16);
    constexpr int kChunks = 2;                         // 32-column chunks per warp and tile
    constexpr int kRowBytes = kOut32 ? 128 : 64;       // staging row: one chunk of int32 or both chunks of int8
    const int quarter = warp & 3;
    const int part = (warp - 2) >> 2;                  // which 64-column part of the tile
    const int et = threadIdx.x - 64;                   // 0..kEpiThreads-1
    uint8_t* stage = smem + SM::kOutOff + (warp - 2) * SM::kOutTileBytes;
    const GeluConsts gk = args.gelu;
    const int64_t gelu_half = rounding_half(gk.c);
    uint32_t acc = 0, acc_phase = 0;
    for (int64_t tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
      const int64_t m0 = (tile / n_tiles) * BM;
      const int n0 = (int)(tile % n_tiles) * BN;
      // per-column parameters of this tile.  generic: {b, c, (bias*b + 2^(c-1)) lo, hi};
      // fast: {b << (32-c), -, (bias*(b << (32-c)) + 2^31) lo, hi};  raw: {bias, 0, 0, 0}
      asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");   // previous tile's readers are done
      for (int j = et; j < BN; j += kEpiThreads) {
        const int n = n0 + j;
        int4 p = make_int4(0, 0, 0, 0);
        if (n < args.N) {
          const int32_t bias = args.bias ? __ldg(args.bias + n) : 0;
          if constexpr (KIND == EPI_RAW) {
            p.x = bias;
          } else {
            const int32_t b = __ldg(args.b + n), c = __ldg(args.c + n);
            const int64_t add = (int64_t)bias * b + (FAST ? (int64_t(1) << 31) : rounding_half(c));
            p = make_int4(b, c, (int32_t)(uint32_t)(uint64_t)add, (int32_t)(add >> 32));
          }
        }
        s_param[j] = p;
      }
      asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");

      // After a failed wait the loop keeps running (the named barriers above must still be
      // reached by every epilogue thread) but touches neither TMEM nor memory.
      if (ok) ok = ptx::mbar_wait(bar_acc_full + 8 * acc, acc_phase);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) continue;
      ptx::tc_fence_after_sync();
      const int out_row0 = (int)m0 + quarter * 32;
      const uint32_t t_row = tmem_base + acc * BN + ((uint32_t)(quarter * 32) << 16);
#pragma unroll 1
      for (int ci = 0; ci < kChunks; ++ci) {
        const int ch = part * kChunks + ci;
        uint32_t v[32];
        ptx::tmem_ld32(t_row + ch * 32, v);
        ptx::tmem_wait_ld();
        if (kOut32 || ci == 0) {
          // the previous store from this staging tile must have finished reading it
          if (lane == 0) ptx::bulk_wait_read<0>();
          __syncwarp();
        }
        epilogue_chunk<KIND, FAST, kRowBytes>(v, s_param + ch * 32, gk, gelu_half, stage, (uint32_t)lane,
                                              kOut32 ? 0u : (uint32_t)(ci * 2));
        if (kOut32 || ci == kChunks - 1) {
          ptx::fence_proxy_async_smem();               // staging writes -> visible to the TMA engine
          __syncwarp();
          if (lane == 0) {
            const int x_bytes = kOut32 ? (n0 + ch * 32) * 4 : n0 + part * 64;
            ptx::tma_store_2d(&map_out, ptx::smem_addr(stage), x_bytes, out_row0);
            ptx::bulk_commit();
          }
        }
      }
      ptx::tc_fence_before_sync();
      ptx::mbar_arrive(bar_acc_empty + 8 * acc);
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1;
    }
    if (lane == 0) ptx::bulk_wait<0>();                // all of this warp's stores have landed
  }

  if (!ok) atomicCAS(args.status, 0, IBERT_ERR_TIMEOUT);
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

template <int BN, int KIND, bool FAST>
int launch_inst(ibert_ctx* ctx, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mo,
                const GemmArgs& args) {
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(gemm_i8_kernel<BN, KIND, FAST>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             GemmSmem<BN>::kAlloc) != cudaSuccess)
      return IBERT_ERR_CUDA;
    attr_set = true;
  }
  const int64_t tiles = ((args.M + BM - 1) / BM) * ((args.N + BN - 1) / BN);
  const int grid = (int)(tiles < ctx->num_sms ? tiles : ctx->num_sms);
  gemm_i8_kernel<BN, KIND, FAST><<<grid, gemm_threads(BN), GemmSmem<BN>::kAlloc, ctx->stream>>>(ma, mb, mo, args);
  return cudaGetLastError() == cudaSuccess ? IBERT_OK : IBERT_ERR_CUDA;
}

template <int BN>
int launch_bn(ibert_ctx* ctx, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mo, const GemmArgs& a,
              int kind, bool fast) {
  switch (kind) {
    case EPI_INT8: return fast ? launch_inst<BN, EPI_INT8, true>(ctx, ma, mb, mo, a) : launch_inst<BN, EPI_INT8, false>(ctx, ma, mb, mo, a);
    case EPI_Q16: return fast ? launch_inst<BN, EPI_Q16, true>(ctx, ma, mb, mo, a) : launch_inst<BN, EPI_Q16, false>(ctx, ma, mb, mo, a);
    case EPI_GELU: return fast ? launch_inst<BN, EPI_GELU, true>(ctx, ma, mb, mo, a) : launch_inst<BN, EPI_GELU, false>(ctx, ma, mb, mo, a);
    default: return launch_inst<BN, EPI_RAW, false>(ctx, ma, mb, mo, a);
  }
}

}  // namespace

int launch_gemm_i8(ibert_ctx* ctx, const int8_t* x, const int8_t* w, int64_t M, int N, int K,
                   const GemmEpilogue& epi, void* out) {
  if (M == 0) return IBERT_OK;
  // tile width: 256 when it divides the work well, else 128
  const int64_t m_tiles = (M + BM - 1) / BM;
  const bool wide = (N % 256 == 0) && m_tiles * (N / 256) >= ctx->num_sms;
  const int BN = wide ? 256 : 128;
  CUtensorMap ma, mb;
  {
    const uint64_t dims[2] = {(uint64_t)K, (uint64_t)M};
    const uint64_t str[1] = {(uint64_t)K};
    const uint32_t box[2] = {BK, BM};
    int rc = encode_tensor_map(&ma, x, 2, dims, str, box, 128);
    if (rc) return rc;
  }
  {
    const uint64_t dims[2] = {(uint64_t)K, (uint64_t)N};
    const uint64_t str[1] = {(uint64_t)K};
    const uint32_t box[2] = {BK, (uint32_t)BN};
    int rc = encode_tensor_map(&mb, w, 2, dims, str, box, 128);
    if (rc) return rc;
  }
  CUtensorMap mo;
  {
    // the output as a byte matrix [M, N * element size]; one box = one warp's staging tile
    const bool out32 = epi.kind == EPI_RAW || epi.kind == EPI_Q16;
    const uint64_t row_bytes = (uint64_t)N * (out32 ? 4 : 1);
    const uint32_t box_bytes = out32 ? 128u : 64u;
    const uint64_t dims[2] = {row_bytes, (uint64_t)M};
    const uint64_t str[1] = {row_bytes};
    const uint32_t box[2] = {box_bytes, 32};
    int rc = encode_tensor_map(&mo, out, 2, dims, str, box, (int)box_bytes);
    if (rc) return rc;
  }
  GemmArgs a{};
  a.M = M; a.N = N; a.K = K;
  a.b = epi.d_b; a.c = epi.d_c; a.bias = epi.d_bias; a.gelu = epi.gelu;
  a.status = ctx->d_status;
  // upper-word epilogue needs both the per-column multipliers and (for GELU) the final one in that form
  const bool fast = epi.fast != 0 && (epi.kind != EPI_GELU || epi.gelu.fast != 0);
  return wide ? launch_bn<256>(ctx, ma, mb, mo, a, epi.kind, fast) : launch_bn<128>(ctx, ma, mb, mo, a, epi.kind, fast);
}

}  // namespace ibert
