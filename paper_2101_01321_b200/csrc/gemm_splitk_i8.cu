// Split-K INT8 GEMM for problems with fewer output tiles than SMs (small batches): the same
// integer-only linear layer as gemm_i8.cu -- INT8 x INT8 -> INT32 accumulation followed by the
// dyadic requantization (Sec. 3.2 integer-only pipeline, Fig. 1) and, for FFN1, i-GELU
// (Algorithm 2) -- but one 128-channel x 128-token output tile is computed by a cluster of S
// CTAs, each reducing its own 1/S of K.
//
// With one tile per SM a CTA walks all K / 128 operand blocks one after the other at the
// bandwidth a single SM gets from L2; at T = 128 and K = 3072 that serial walk is the whole
// kernel.  Here every CTA of the cluster
//   1. runs the TMA -> tcgen05.mma pipeline over its K range into its own TMEM accumulator,
//   2. writes the raw INT32 partial sums into its shared memory (the operand ring, free by then),
//   3. after a cluster barrier sums, for its own 1/S of the tile's tokens, the partial sums of all
//      S CTAs through distributed shared memory, applies the epilogue and stores the result,
// so both the K walk and the epilogue are split S ways.  Integer addition is associative: the
// result is bit-identical to the unsplit kernel's.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <type_traits>

#include "device_utils.cuh"
#include "ibert_internal.h"
#include "sm100_ptx.cuh"

namespace ibert {
namespace {

constexpr int kCh = 128;          // output channels per tile = TMEM lanes
constexpr int kTok = 128;         // tokens per tile = TMEM columns
constexpr int kBK = 128;          // K bytes per pipeline stage = one 128-byte swizzle span
constexpr int kUmmaK = 32;        // K per tcgen05.mma kind::i8
constexpr int kStages = 6;
constexpr int kWBytes = kCh * kBK;
constexpr int kStageBytes = (kCh + kTok) * kBK;          // 32 KB
constexpr int kRingBytes = kStages * kStageBytes;        // 192 KB
constexpr int kEpiWarps = 8;                             // (TMEM lane quadrant) x (token half)
constexpr int kThreads = 64 + 32 * kEpiWarps;            // + producer warp, MMA warp
constexpr int kBarOff = kRingBytes;
constexpr int kAlloc = kRingBytes + 256 + 1024;          // barriers, slack to align to 1024 bytes
static_assert(kCh * kTok * 4 <= kRingBytes, "the partial sums are staged in the operand ring");

struct SplitArgs {
  int64_t T;       // tokens
  int N, K;        // output channels, reduction length
  int split;       // CTAs per tile (cluster width): 2 or 4
  const int32_t* b;
  const int32_t* c;
  const int32_t* bias;
  GeluConsts gelu;
  void* out;       // [T, N] int8 or int32
  int32_t* status;
};

__device__ __forceinline__ int32_t ld_cluster_s32(uint32_t cluster_addr) {
  int32_t v;
  asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(v) : "r"(cluster_addr) : "memory");
  return v;
}

// one output value from one complete accumulator
template <int KIND, bool FAST>
__device__ __forceinline__ int32_t epilogue_value(int32_t a, int32_t bias, int32_t pb, int32_t pc, int64_t padd,
                                                  const GeluConsts& gk, int64_t gelu_half, int32_t gelu_rnd) {
  if constexpr (KIND == EPI_RAW) return a + bias;
  else if constexpr (KIND == EPI_Q16 || KIND == EPI_Q16H) {
    if constexpr (FAST) return clamp_sym(requant_upper(a + bias, pb), 32767);
    else return requant_add(a, pb, padd, pc, 32767);
  } else if constexpr (KIND == EPI_INT8) {
    if constexpr (FAST) return clamp_sym(requant_upper(a + bias, pb), 127);
    else return requant_add(a, pb, padd, pc, 127);
  } else if constexpr (KIND == EPI_HGELU) {
    if constexpr (FAST) return clamp_sym(ihgelu_upper(requant_upper(a + bias, pb), gk), 127);
    else return ihgelu_to_int8(requant_add(a, pb, padd, pc, 32767), gk, gelu_half);
  } else {
    if constexpr (FAST) return clamp_sym(igelu_magnitude_upper(requant_upper(a + bias, pb), gk, gelu_rnd), 127);
    else return igelu_q16_to_int8(requant_add(a, pb, padd, pc, 32767), gk, gelu_half);
  }
}

template <int KIND, bool FAST>
__global__ void __launch_bounds__(kThreads, 1)
gemm_splitk_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
                   const SplitArgs args) {
  constexpr bool kOut32 = (KIND == EPI_RAW || KIND == EPI_Q16);
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = ptx::smem_addr(smem);
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(smem + kBarOff);
  const uint32_t bar_full = ptx::smem_addr(s_bar);         // full[kStages], empty[kStages], acc_full
  const uint32_t bar_empty = bar_full + 8 * kStages;
  const uint32_t bar_acc_full = bar_empty + 8 * kStages;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_bar + 2 * kStages + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int S = args.split;
  const int rank = (int)ptx::cluster_ctarank();
  const int tile = (int)blockIdx.x / S;
  const int c_tiles = (args.N + kCh - 1) / kCh;
  const int c0 = (tile % c_tiles) * kCh;
  const int t0 = (tile / c_tiles) * kTok;
  // this CTA's share of the K blocks (may be empty when S does not divide their number)
  const int k_blocks = (args.K + kBK - 1) / kBK;
  const int per = (k_blocks + S - 1) / S;
  const int kb0 = min(rank * per, k_blocks), kb1 = min(kb0 + per, k_blocks);
  const bool has_k = kb1 > kb0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(bar_full + 8 * s, 1);
      ptx::mbar_init(bar_empty + 8 * s, 1);
    }
    ptx::mbar_init(bar_acc_full, 1);
    ptx::fence_mbar_init();
    ptx::tma_prefetch_desc(&map_w);
    ptx::tma_prefetch_desc(&map_x);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_addr(s_tmem), kTok);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *s_tmem;
  bool ok = true;
  // set-up done: the next kernel may be scheduled; the previous one must be complete before
  // any operand is read or any output written
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!ptx::mbar_wait(bar_empty + 8 * stage, phase ^ 1)) { ok = false; break; }
        const uint32_t sw = smem_base + stage * kStageBytes;
        ptx::mbar_arrive_expect_tx(bar_full + 8 * stage, kStageBytes);
        ptx::tma_load_2d(sw, &map_w, bar_full + 8 * stage, kb * kBK, c0);
        ptx::tma_load_2d(sw + kWBytes, &map_x, bar_full + 8 * stage, kb * kBK, t0);
        if (++stage == kStages) { stage = 0; phase ^= 1; }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0 && has_k) {
      constexpr uint32_t idesc = ptx::make_idesc_i8(kCh, kTok, true, true);
      uint32_t stage = 0, phase = 0;
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!ptx::mbar_wait(bar_full + 8 * stage, phase)) { ok = false; break; }
        ptx::tc_fence_after_sync();
        const uint32_t sw = smem_base + stage * kStageBytes;
        const uint64_t dw = ptx::make_kmajor_desc(sw, 1024, ptx::kSwizzle128);
        const uint64_t dx = ptx::make_kmajor_desc(sw + kWBytes, 1024, ptx::kSwizzle128);
#pragma unroll
        for (int k = 0; k < kBK / kUmmaK; ++k)   // +32 bytes inside the swizzle span = +2 in the encoded address
          ptx::mma_i8_ss(tmem_base, dw + 2 * k, dx + 2 * k, idesc, (kb > kb0 || k != 0) ? 1u : 0u);
        ptx::mma_commit(bar_empty + 8 * stage);
        if (++stage == kStages) { stage = 0; phase ^= 1; }
      }
      ptx::mma_commit(bar_acc_full);             // arrives once every MMA above has completed
    }
    __syncwarp();
  }

  // ---------------------------------------------------------------- partial sums -> shared memory
  // Epilogue warp w reads TMEM lane quadrant w & 3 (the only lanes it may address) and the token
  // half (w - 2) >> 2.  Staging layout: red[token][channel] (channel fastest), so that the 32 lanes
  // of a warp touch 32 consecutive words both here and in the reduction below.
  const int quarter = warp & 3;
  const int half = (warp - 2) >> 2;
  const int row = quarter * 32 + lane;                   // channel within the tile
  if (warp >= 2) {
    if (has_k) {
      ok = ptx::mbar_wait(bar_acc_full, 0);              // every MMA done: TMEM complete, operand ring free
      ok = __all_sync(0xffffffffu, ok);
      ptx::tc_fence_after_sync();
    }
    int32_t* red = reinterpret_cast<int32_t*>(smem);
#pragma unroll 1
    for (int ci = 0; ci < 2; ++ci) {
      const int col = half * 64 + ci * 32;
      uint32_t v[32];
      if (has_k && ok) {
        ptx::tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + col, v);
        ptx::tmem_wait_ld();
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = 0u;          // no K block of its own: contributes nothing
      }
#pragma unroll
      for (int i = 0; i < 32; ++i) red[(col + i) * kCh + row] = (int32_t)v[i];
    }
  }
  if (!ok) atomicCAS(args.status, 0, IBERT_ERR_TIMEOUT);
  ptx::tc_fence_before_sync();
  ptx::cluster_sync();                                   // all S staging areas are complete and visible

  // ---------------------------------------------------------------- reduction + epilogue of 1/S of the tokens
  if (warp >= 2) {
    const int n = c0 + row;
    int32_t pb = 0, pc = 0, bias = 0;
    int64_t padd = 0;
    if (n < args.N) {
      bias = args.bias ? __ldg(args.bias + n) : 0;
      if constexpr (KIND != EPI_RAW) {
        pb = __ldg(args.b + n);
        pc = __ldg(args.c + n);
        padd = (int64_t)bias * pb + rounding_half(pc);
      }
    }
    const GeluConsts gk = args.gelu;
    const int64_t gelu_half = rounding_half(gk.c);
    const int32_t gelu_rnd = (1 << gk.s_f) - 1;
    auto reduce_and_store = [&](auto width) {
      constexpr int W = decltype(width)::value;            // cluster width, compile-time here
      constexpr int per_warp = kTok / W / 2;               // tokens this thread finishes
      const int col0 = rank * (kTok / W) + half * per_warp;
      uint32_t peer[W];
#pragma unroll
      for (int r = 0; r < W; ++r) peer[r] = ptx::map_to_cta(smem_base, (uint32_t)r);
      // every remote load is issued before the first use: one round trip through the cluster
      // network instead of one per token
      int32_t part[per_warp][W];
#pragma unroll
      for (int j = 0; j < per_warp; ++j) {
        const uint32_t off = (uint32_t)(((col0 + j) * kCh + row) * 4);
#pragma unroll
        for (int r = 0; r < W; ++r) part[j][r] = ld_cluster_s32(peer[r] + off);
      }
#pragma unroll
      for (int j = 0; j < per_warp; ++j) {
        int32_t a = part[j][0];
#pragma unroll
        for (int r = 1; r < W; ++r) a += part[j][r];
        const int32_t o = epilogue_value<KIND, FAST>(a, bias, pb, pc, padd, gk, gelu_half, gelu_rnd);
        const int64_t t = (int64_t)t0 + col0 + j;
        if (t < args.T && n < args.N) {
          if constexpr (kOut32) static_cast<int32_t*>(args.out)[t * args.N + n] = o;
          else if constexpr (KIND == EPI_Q16H) static_cast<int16_t*>(args.out)[t * args.N + n] = (int16_t)o;
          else static_cast<int8_t*>(args.out)[t * args.N + n] = (int8_t)o;
        }
      }
    };
    if (S == 4) reduce_and_store(std::integral_constant<int, 4>{});
    else reduce_and_store(std::integral_constant<int, 2>{});
  }
  ptx::cluster_sync();                                   // nobody's staging area goes away while it is read
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, kTok);
  }
}

template <int KIND, bool FAST>
int launch_inst(ibert_ctx* ctx, const CUtensorMap& mw, const CUtensorMap& mx, const SplitArgs& a, int tiles) {
  static bool attr_set_dev[kMaxDevices] = {false};
  bool& attr_set = attr_set_dev[ctx->device % kMaxDevices];
  if (!attr_set) {
    if (cudaFuncSetAttribute(gemm_splitk_kernel<KIND, FAST>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAlloc) !=
        cudaSuccess)
      return IBERT_ERR_CUDA;
    attr_set = true;
  }
  return launch_pdl(gemm_splitk_kernel<KIND, FAST>, dim3(tiles * a.split), dim3(kThreads), (size_t)kAlloc, ctx->stream,
                    a.split, mw, mx, a);
}

}  // namespace

int gemm_splitk_width(const ibert_ctx* ctx, int64_t M, int N, int K) {
  // Worth it only for a long K walk: the cluster barrier and the exchange of the partial sums cost
  // about as much as four K blocks of a single CTA.
  const int64_t tiles = ((M + kTok - 1) / kTok) * ((N + kCh - 1) / kCh);
  const int k_blocks = (K + kBK - 1) / kBK;
  if (k_blocks < 12 || tiles * 2 > ctx->num_sms) return 1;
  return tiles * 4 <= ctx->num_sms ? 4 : 2;
}

int launch_gemm_splitk_i8(ibert_ctx* ctx, const int8_t* x, const int8_t* w, int64_t M, int N, int K,
                          const GemmEpilogue& epi, void* out, int split) {
  if (M == 0) return IBERT_OK;
  if (split != 2 && split != 4) return IBERT_ERR_ARG;
  CUtensorMap mw, mx;
  {
    const uint64_t dims[2] = {(uint64_t)K, (uint64_t)N};
    const uint64_t str[1] = {(uint64_t)K};
    const uint32_t box[2] = {kBK, kCh};
    int rc = encode_tensor_map(&mw, w, 2, dims, str, box, 128);
    if (rc) return rc;
  }
  {
    const uint64_t dims[2] = {(uint64_t)K, (uint64_t)M};
    const uint64_t str[1] = {(uint64_t)K};
    const uint32_t box[2] = {kBK, kTok};
    int rc = encode_tensor_map(&mx, x, 2, dims, str, box, 128);
    if (rc) return rc;
  }
  SplitArgs a{};
  a.T = M; a.N = N; a.K = K; a.split = split;
  a.b = epi.d_b; a.c = epi.d_c; a.bias = epi.d_bias; a.gelu = epi.gelu;
  a.out = out; a.status = ctx->d_status;
  const int tiles = (int)(((M + kTok - 1) / kTok) * ((N + kCh - 1) / kCh));
  const bool fast = epi.fast != 0 && ((epi.kind != EPI_GELU && epi.kind != EPI_HGELU) || epi.gelu.fast != 0);
  switch (epi.kind) {
    case EPI_INT8: return fast ? launch_inst<EPI_INT8, true>(ctx, mw, mx, a, tiles) : launch_inst<EPI_INT8, false>(ctx, mw, mx, a, tiles);
    case EPI_Q16: return fast ? launch_inst<EPI_Q16, true>(ctx, mw, mx, a, tiles) : launch_inst<EPI_Q16, false>(ctx, mw, mx, a, tiles);
    case EPI_Q16H: return fast ? launch_inst<EPI_Q16H, true>(ctx, mw, mx, a, tiles) : launch_inst<EPI_Q16H, false>(ctx, mw, mx, a, tiles);
    case EPI_GELU: return fast ? launch_inst<EPI_GELU, true>(ctx, mw, mx, a, tiles) : launch_inst<EPI_GELU, false>(ctx, mw, mx, a, tiles);
    case EPI_HGELU: return fast ? launch_inst<EPI_HGELU, true>(ctx, mw, mx, a, tiles) : launch_inst<EPI_HGELU, false>(ctx, mw, mx, a, tiles);
    default: return launch_inst<EPI_RAW, false>(ctx, mw, mx, a, tiles);
  }
}

}  // namespace ibert
