// INT8 x INT8 -> INT32 GEMM on the 5th-generation tensor cores (tcgen05.mma kind::i8,
// accumulators in TMEM, operands staged by TMA) with the integer epilogue fused:
// bias add + dyadic requantization to int8 or Q16, raw accumulators, or requantization
// to Q16 followed by i-GELU (Algorithm 2) and a second requantization to int8.
//
// out[t, n] = epilogue( sum_k x[t, k] * w[n, k] + bias[n] )      x: [T, K], w: [N, K]
//
// The MMA computes the transposed tile D[n, t] = W X^T: output channels n sit on the 128
// TMEM lanes, tokens t on the columns.  An epilogue thread therefore owns ONE channel and keeps
// that channel's requantization constants in registers -- per-column constants would have to be
// re-read from shared memory for every element, and that broadcast traffic, not the tensor
// pipe, bounded the first version of this kernel.  Results are transposed back for free on the
// way out: each warp writes its 32-token x 32-channel block into a small staging tile and a TMA
// store moves it to out[t, n].
//
// Persistent CTAs walk the output tiles.  Warp 0 is the TMA producer, warp 1 issues the MMAs,
// warps 2.. run the epilogue; two TMEM accumulator stages let the (integer-ALU heavy) epilogue of
// tile i overlap the MMAs of tile i+1.  With PAIR a cluster of two CTAs shares one
// 256-channel x 256-token tile (tcgen05.mma.cta_group::2): each CTA loads only its own 128
// weight rows and 128 of the 256 token rows, which cuts the operand bytes an SM must pull per
// MMA by a third.  No TMA multicast is used anywhere.
#include <cuda.h>

#include <algorithm>
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
                                : swizzle_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B
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

constexpr int BC = 128;           // output channels per CTA = TMEM lanes
constexpr int BK = 128;           // K bytes per pipeline stage = one 128-byte swizzle span
constexpr int UMMA_K = 32;        // K per tcgen05.mma kind::i8

// i-GELU epilogue whose results provably stay above -127 (GeluConsts::low_free): no lower clamp.
// A kind of its own, internal to this file, so that the choice costs no instruction in the loop.
constexpr int kEpiGeluLowFree = 16;
// The same two i-GELU epilogues with per-channel multipliers of 1/2 and more (requant_upper_wide)
constexpr int kEpiGeluWide = 17, kEpiGeluLowFreeWide = 18;
// i-GELU and its requantization read from a table of all 65535 Q16 inputs held in shared memory:
// the epilogue is bound by the integer ALU pipe, the load/store pipe idles, and the table (filled by
// the i-GELU kernel itself) returns the same bits.  Costs 64 KB, i.e. two of six operand stages.
constexpr int kEpiGeluTable = 19, kEpiGeluTableWide = 20;
constexpr int kGeluTableBytes = 65536;
// int8 results (upper-word requantization) written as the transposed tensor out[n][t]
constexpr int kEpiInt8T = 24;
// the table kinds with the transposed result (FFN1 feeding the cluster kernel, which reads it as an MN-major operand)
constexpr int kEpiGeluTableT = 25, kEpiGeluTableWideT = 26;
__host__ __device__ constexpr bool epi_transposed(int kind) { return kind == kEpiInt8T || kind == kEpiGeluTableT || kind == kEpiGeluTableWideT; }

template <int TOK, bool PAIR, int KIND>
struct Cfg {
  static constexpr bool kOut32 = (KIND == EPI_RAW || KIND == EPI_Q16 || KIND == EPI_Q16H);   // light epilogue, wide output
  static constexpr int kOutElem = (KIND == EPI_RAW || KIND == EPI_Q16) ? 4 : (KIND == EPI_Q16H ? 2 : 1);   // bytes per output value
  static constexpr int kChunks = TOK / 32;                       // 32-token chunks of a tile
  // the int8 epilogues are ALU-bound: one warp per 64 tokens; the int32 ones per 128 tokens
  static constexpr int kEpiWarps = kOut32 ? TOK / 32 : TOK / 16;
  static constexpr int kParts = kEpiWarps / 4;                   // token ranges (4 warps cover the 128 lanes)
  static constexpr int kChunksPerWarp = kChunks / kParts;
  static constexpr int kThreads = 64 + 32 * kEpiWarps;           // + producer warp, MMA warp
  static constexpr int kXRows = PAIR ? TOK / 2 : TOK;            // token rows this CTA loads per K block
  static constexpr int kWBytes = BC * BK;
  static constexpr int kStageBytes = kWBytes + kXRows * BK;
  static constexpr int kOutTileBytes = 32 * 32 * kOutElem;            // 32 tokens x 32 channels
  static constexpr int kOutBytes = kEpiWarps * 2 * kOutTileBytes;     // double-buffered per warp
  static constexpr bool kTable = (KIND == kEpiGeluTable || KIND == kEpiGeluTableWide || KIND == kEpiGeluTableT || KIND == kEpiGeluTableWideT);
  static constexpr int kTableBytes = kTable ? kGeluTableBytes : 0;
  static constexpr int kBudget = 227 * 1024 - 1024 - 512 - kOutBytes - kTableBytes;
  static constexpr int kStages = kBudget / kStageBytes > 8 ? 8 : kBudget / kStageBytes;
  static constexpr int kOutOff = kStages * kStageBytes;
  static constexpr int kTableOff = kOutOff + kOutBytes;
  static constexpr int kBarOff = kTableOff + kTableBytes;
  static constexpr int kAlloc = kBarOff + 512 + 1024;            // + slack to align to 1024 bytes
  static constexpr bool kValid = kEpiWarps % 4 == 0 && kChunks % kParts == 0 && kStages >= 3;
};

struct GemmArgs {
  int64_t T;       // tokens (rows of x and of out)
  int N, K;        // output channels, reduction length
  const int32_t* b;
  const int32_t* c;
  const int32_t* bias;
  GeluConsts gelu;
  int32_t* status;
  const int8_t* gelu_table;   // kEpiGeluTable kinds only
};

template <int TOK, bool PAIR, int KIND, bool FAST>
__global__ void __launch_bounds__(Cfg<TOK, PAIR, KIND>::kThreads, 1)
gemm_i8_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
               const __grid_constant__ CUtensorMap map_out, const GemmArgs args) {
  using C = Cfg<TOK, PAIR, KIND>;
  static_assert(C::kValid, "tile configuration");
  constexpr int kStages = C::kStages;
  constexpr uint32_t kTmemCols = 2 * TOK;          // two accumulator stages
  constexpr int kTileChannels = PAIR ? 2 * BC : BC;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = ptx::smem_addr(smem);
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(smem + C::kBarOff);
  // full[kStages] (PAIR: the leader's only), empty[kStages], acc_full[2], acc_empty[2] (leader's), TMEM base
  const uint32_t bar_full = ptx::smem_addr(s_bar);
  const uint32_t bar_empty = bar_full + 8 * kStages;
  const uint32_t bar_acc_full = bar_empty + 8 * kStages;
  const uint32_t bar_acc_empty = bar_acc_full + 16;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_bar + 2 * kStages + 4);
  const uint32_t bar_table = bar_acc_empty + 24;   // (after the TMEM base word)

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = PAIR ? ptx::cluster_ctarank() : 0u;   // 0 = leader: issues the MMAs
  const int worker = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int num_workers = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  const int c_tiles = (args.N + kTileChannels - 1) / kTileChannels;
  const int64_t t_tiles = (args.T + TOK - 1) / TOK;
  const int64_t total_tiles = t_tiles * c_tiles;
  const int k_blocks = (args.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(bar_full + 8 * s, 1);
      ptx::mbar_init(bar_empty + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(bar_acc_full + 8 * a, 1);
      ptx::mbar_init(bar_acc_empty + 8 * a, (PAIR ? 2 : 1) * C::kEpiWarps);   // one lane per epilogue warp
    }
    if constexpr (C::kTable) ptx::mbar_init(bar_table, 1);
    ptx::fence_mbar_init();
    ptx::tma_prefetch_desc(&map_w);
    ptx::tma_prefetch_desc(&map_x);
    ptx::tma_prefetch_desc(&map_out);
  }
  if (warp == 1) {
    if constexpr (PAIR) { ptx::tmem_alloc_pair(ptx::smem_addr(s_tmem), kTmemCols); ptx::tmem_relinquish_pair(); }
    else { ptx::tmem_alloc(ptx::smem_addr(s_tmem), kTmemCols); ptx::tmem_relinquish(); }
  }
  ptx::tc_fence_before_sync();
  if constexpr (PAIR) ptx::cluster_sync(); else __syncthreads();   // barriers (of both CTAs) are initialised
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
      if constexpr (C::kTable) {
        // the table may have been written by the kernel before this one: fetched after the dependency wait
        ptx::mbar_arrive_expect_tx(bar_table, kGeluTableBytes);
        ptx::bulk_load_1d(smem_base + C::kTableOff, args.gelu_table, kGeluTableBytes, bar_table);
      }
      uint32_t stage = 0, phase = 0;
      const uint32_t full_leader0 = PAIR ? ptx::map_to_cta(bar_full, 0) : bar_full;
      for (int64_t tile = worker; tile < total_tiles && ok; tile += num_workers) {
        const int c0 = (int)(tile % c_tiles) * kTileChannels + (int)rank * BC;
        const int t0 = (int)(tile / c_tiles) * TOK + (int)rank * C::kXRows;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!ptx::mbar_wait_parked(bar_empty + 8 * stage, phase ^ 1)) { ok = false; break; }
          const uint32_t sw = smem_base + stage * C::kStageBytes;
          if constexpr (PAIR) {
            // both CTAs' copies complete on the leader's barrier, which expects the bytes of both
            const uint32_t full_leader = full_leader0 + 8 * stage;
            if (rank == 0) ptx::mbar_arrive_expect_tx(bar_full + 8 * stage, 2 * C::kStageBytes);
            ptx::tma_load_2d_pair(sw, &map_w, full_leader, kb * BK, c0);
            ptx::tma_load_2d_pair(sw + C::kWBytes, &map_x, full_leader, kb * BK, t0);
          } else {
            ptx::mbar_arrive_expect_tx(bar_full + 8 * stage, C::kStageBytes);
            ptx::tma_load_2d(sw, &map_w, bar_full + 8 * stage, kb * BK, c0);
            ptx::tma_load_2d(sw + C::kWBytes, &map_x, bar_full + 8 * stage, kb * BK, t0);
          }
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
      }
      if constexpr (C::kTable) {
        if (!ptx::mbar_wait(bar_table, 0)) ok = false;     // nobody leaves with the copy in flight
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (PAIR: leader CTA only)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = ptx::make_idesc_i8(kTileChannels, TOK, true, true);
      uint32_t stage = 0, phase = 0;
      uint32_t acc = 0, acc_phase = 0;
      const uint64_t dw0 = ptx::make_kmajor_desc(smem_base, 1024, ptx::kSwizzle128);
      const uint64_t dx0 = ptx::make_kmajor_desc(smem_base + C::kWBytes, 1024, ptx::kSwizzle128);
      for (int64_t tile = worker; tile < total_tiles && ok; tile += num_workers) {
        if (!ptx::mbar_wait_parked(bar_acc_empty + 8 * acc, acc_phase ^ 1)) { ok = false; break; }
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * TOK;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!ptx::mbar_wait_parked(bar_full + 8 * stage, phase)) { ok = false; break; }
          ptx::tc_fence_after_sync();
          // (descriptor start addresses count 16-byte units; a stage is a multiple of 1024 bytes)
          const uint64_t dw = dw0 + (uint64_t)(stage * (C::kStageBytes >> 4)), dx = dx0 + (uint64_t)(stage * (C::kStageBytes >> 4));
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // advancing K inside the swizzle span: +32 bytes = +2 in the encoded start address
            if constexpr (PAIR) ptx::mma_i8_ss_pair(d_tmem, dw + 2 * k, dx + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
            else ptx::mma_i8_ss(d_tmem, dw + 2 * k, dx + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          // frees the stage (in both CTAs) once these MMAs have read it
          if constexpr (PAIR) ptx::mma_commit_pair(bar_empty + 8 * stage, 3); else ptx::mma_commit(bar_empty + 8 * stage);
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        if constexpr (PAIR) ptx::mma_commit_pair(bar_acc_full + 8 * acc, 3); else ptx::mma_commit(bar_acc_full + 8 * acc);
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1;
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..)
    // Warp w reads TMEM lanes 32*(w%4)..+31: thread = one output channel, registers = 32 tokens.
    constexpr bool kOut32 = C::kOut32;
    const int quarter = warp & 3;
    const int part = (warp - 2) >> 2;                  // which token range of the tile
    uint8_t* stage0 = smem + C::kOutOff + (warp - 2) * 2 * C::kOutTileBytes;
    uint32_t buf = 0;
    const GeluConsts gk = args.gelu;
    const int64_t gelu_half = rounding_half(gk.c);
    const int32_t gelu_rnd = (1 << gk.s_f) - 1;
    uint32_t acc_empty_addr = bar_acc_empty;
    if constexpr (PAIR) acc_empty_addr = ptx::map_to_cta(bar_acc_empty, 0);
    uint32_t acc = 0, acc_phase = 0;
    // this thread's channel constants for a tile.  generic: b, c, bias*b + 2^(c-1);
    // fast: b << (32-c) (the bias is added to the accumulator first);  raw: bias
    int32_t pb = 0, pc = 0, bias = 0;
    int64_t padd = 0;
    auto load_constants = [&](int64_t tile) {
      const int n = (int)(tile % c_tiles) * kTileChannels + (int)rank * BC + quarter * 32 + lane;
      pb = 0; pc = 0; bias = 0; padd = 0;
      if (tile < total_tiles && n < args.N) {
        bias = args.bias ? __ldg(args.bias + n) : 0;
        if constexpr (KIND != EPI_RAW) {
          pb = __ldg(args.b + n);
          pc = __ldg(args.c + n);
          padd = (int64_t)bias * pb + rounding_half(pc);
        }
      }
    };
    load_constants(worker);
    // table kinds: shared-memory address of the entry of Q16 value 0, and of the two ends
    const int32_t table_mid = (int32_t)smem_base + C::kTableOff + 32767;
    const int32_t table_lo = table_mid - 32767, table_hi = table_mid + 32767;
    if constexpr (C::kTable) ok = ptx::mbar_wait(bar_table, 0);
    for (int64_t tile = worker; tile < total_tiles; tile += num_workers) {
      const int ch0 = (int)(tile % c_tiles) * kTileChannels + (int)rank * BC + quarter * 32;   // this warp's channels
      const int t0 = (int)(tile / c_tiles) * TOK + part * (C::kChunksPerWarp * 32);
      const int32_t cur_pb = pb, cur_pc = pc, cur_bias = bias;
      const int64_t cur_padd = padd;
      load_constants(tile + num_workers);              // the next tile's, ahead of its accumulator
      if (ok) ok = ptx::mbar_wait(bar_acc_full + 8 * acc, acc_phase);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) continue;                               // keep walking the tiles, touch nothing
      ptx::tc_fence_after_sync();
      const uint32_t t_row = tmem_base + acc * TOK + ((uint32_t)(quarter * 32) << 16);
      // (a warp whose token range lies past the last row -- the ragged last tile of a token count that is
      // not a multiple of the tile -- has nothing to read or store: the tile then costs its main loop only)
#pragma unroll 1
      for (int ci = 0; ci < ((int64_t)t0 < args.T ? C::kChunksPerWarp : 0); ++ci) {
        const int col = (part * C::kChunksPerWarp + ci) * 32;
        uint32_t v[32];
        ptx::tmem_ld32(t_row + col, v);
        ptx::tmem_wait_ld();
        // GELU kinds: the warp's two 1 KB tiles form one 64-token block that leaves with a single
        // store per output tile (one proxy fence and one TMA issue less; -1.6 us on FFN1).  The
        // light int8 epilogue keeps two stores: it would catch up with its own previous store
        // (+2 us on the QKV GEMM).  Otherwise a tile is reused two chunks later.  Either way the
        // store that last read this staging tile must have finished reading it.
        constexpr bool kOneStore = !kOut32 && C::kChunksPerWarp == 2 && KIND != EPI_INT8 && !epi_transposed(KIND);
        // the same for the transposed GELU kinds: the warp's 32 channels x 64 tokens leave as one 2 KB block
        constexpr bool kOneStoreT = C::kChunksPerWarp == 2 && (KIND == kEpiGeluTableT || KIND == kEpiGeluTableWideT);
        if (!(kOneStore || kOneStoreT) || ci == 0) {
          if (lane == 0) { if constexpr (kOneStore || kOneStoreT) ptx::bulk_wait_read<0>(); else ptx::bulk_wait_read<1>(); }
          __syncwarp();
        }
        uint8_t* stage = stage0 + (kOneStore ? ci : (int)buf) * C::kOutTileBytes;
        // (all results first, then the stores: a table load may not pass an earlier store to shared
        // memory, so element-by-element order would put the load latency between any two stores)
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int32_t a = (int32_t)v[i];
          int32_t o;
          if constexpr (KIND == EPI_RAW) o = a + cur_bias;
          else if constexpr (KIND == EPI_Q16) {
            if constexpr (FAST) o = clamp_sym(requant_upper(a + cur_bias, cur_pb), 32767);
            else o = requant_add(a, cur_pb, cur_padd, cur_pc, 32767);
          } else if constexpr (KIND == EPI_Q16H) {
            if constexpr (FAST) o = clamp_sym(requant_upper(a + cur_bias, cur_pb), 32767);
            else o = requant_add(a, cur_pb, cur_padd, cur_pc, 32767);
          } else if constexpr (KIND == kEpiInt8T) {
            o = max(requant_upper(a + cur_bias, cur_pb), -127);      // the pack below saturates the upper side
          } else if constexpr (KIND == EPI_INT8) {
            if constexpr (FAST) o = clamp_sym(requant_upper(a + cur_bias, cur_pb), 127);
            else o = requant_add(a, cur_pb, cur_padd, cur_pc, 127);
          } else {
            if constexpr (KIND == EPI_HGELU) {
              if constexpr (FAST) o = clamp_sym(ihgelu_upper(requant_upper(a + cur_bias, cur_pb), gk), 127);
              else o = ihgelu_to_int8(requant_add(a, cur_pb, cur_padd, cur_pc, 32767), gk, gelu_half);
            } else if constexpr (KIND == kEpiGeluTable || KIND == kEpiGeluTableT) {
              // |requantized value| < 2^30 (upper word of a product of two int32): the sum cannot wrap
              const int32_t at = max(__viaddmin_s32(requant_upper(a + cur_bias, cur_pb), table_mid, table_hi), table_lo);
              asm volatile("ld.shared.u8 %0, [%1];" : "=r"(o) : "r"(at));
            } else if constexpr (KIND == kEpiGeluTableWide || KIND == kEpiGeluTableWideT) {
              const int32_t at = clamp_sym(requant_upper_wide(a + cur_bias, cur_pb, cur_pc), 32767) + table_mid;
              asm volatile("ld.shared.u8 %0, [%1];" : "=r"(o) : "r"(at));
            } else if constexpr (KIND == kEpiGeluLowFree) {
              o = min(igelu_magnitude_upper(requant_upper(a + cur_bias, cur_pb), gk, gelu_rnd), 127);
            } else if constexpr (KIND == kEpiGeluLowFreeWide) {
              o = min(igelu_magnitude_upper(requant_upper_wide(a + cur_bias, cur_pb, cur_pc), gk, gelu_rnd), 127);
            } else if constexpr (KIND == kEpiGeluWide) {
              o = clamp_sym(igelu_magnitude_upper(requant_upper_wide(a + cur_bias, cur_pb, cur_pc), gk, gelu_rnd), 127);
            } else {
              if constexpr (FAST) o = clamp_sym(igelu_magnitude_upper(requant_upper(a + cur_bias, cur_pb), gk, gelu_rnd), 127);
              else o = igelu_q16_to_int8(requant_add(a, cur_pb, cur_padd, cur_pc, 32767), gk, gelu_half);
            }
          }
          v[i] = (uint32_t)o;
        }
        if constexpr (epi_transposed(KIND)) {
          // staging tile of the transposed output: row = this lane's channel, 32 tokens = 32 bytes, written as
          // two 16-byte chunks placed by the 32-byte swizzle of the store's tensor map (chunk index XOR bit 2
          // of the row): a quarter-warp's stores cover all banks once -- 8 wavefronts per block instead of 32
          uint32_t w[8];
#pragma unroll
          for (int j = 0; j < 8; ++j)
            w[j] = KIND == kEpiInt8T
                       ? pack4_sat_s8((int32_t)v[4 * j], (int32_t)v[4 * j + 1], (int32_t)v[4 * j + 2], (int32_t)v[4 * j + 3])
                       : __byte_perm(__byte_perm(v[4 * j], v[4 * j + 1], 0x0040), __byte_perm(v[4 * j + 2], v[4 * j + 3], 0x0040), 0x5410);   // table bytes
          if constexpr (kOneStoreT) {
            // rows of 64 tokens = four 16-byte chunks, placed by the 64-byte swizzle (chunk index XOR bits 1..2
            // of the row); this 32-token chunk fills chunks 2 ci and 2 ci + 1
            const uint32_t sw = ((uint32_t)lane >> 1) & 3u, c0 = 2u * (uint32_t)ci;
            *reinterpret_cast<uint4*>(stage0 + lane * 64 + ((c0 ^ sw) * 16u)) = make_uint4(w[0], w[1], w[2], w[3]);
            *reinterpret_cast<uint4*>(stage0 + lane * 64 + (((c0 + 1u) ^ sw) * 16u)) = make_uint4(w[4], w[5], w[6], w[7]);
          } else {
          const uint32_t sw = ((uint32_t)lane >> 2) & 1u;
          *reinterpret_cast<uint4*>(stage + lane * 32 + sw * 16u) = make_uint4(w[0], w[1], w[2], w[3]);
          *reinterpret_cast<uint4*>(stage + lane * 32 + (sw ^ 1u) * 16u) = make_uint4(w[4], w[5], w[6], w[7]);
          }
        } else
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int32_t o = (int32_t)v[i];
          // staging tile: row = token i, column = this lane's channel
          if constexpr (C::kOutElem == 4) reinterpret_cast<int32_t*>(stage)[i * 32 + lane] = o;
          else if constexpr (C::kOutElem == 2)
            asm volatile("st.shared.u16 [%0], %1;" ::"r"(ptx::smem_addr(stage) + (i * 32 + lane) * 2), "h"((uint16_t)o) : "memory");
          else  // low byte of the register, stored without a narrowing conversion
            asm volatile("st.shared.u8 [%0], %1;" ::"r"(ptx::smem_addr(stage) + i * 32 + lane), "r"(o) : "memory");
        }
        if (!(kOneStore || kOneStoreT) || ci == 1) {
          ptx::fence_proxy_async_smem();               // staging writes -> visible to the TMA engine
          __syncwarp();
          if (lane == 0) {
            if constexpr (kOneStoreT) ptx::tma_store_2d(&map_out, ptx::smem_addr(stage0), t0, ch0);
            else if constexpr (kOneStore) ptx::tma_store_2d(&map_out, ptx::smem_addr(stage0), ch0, t0);
            else if constexpr (epi_transposed(KIND)) ptx::tma_store_2d(&map_out, ptx::smem_addr(stage), t0 + ci * 32, ch0);
            else ptx::tma_store_2d(&map_out, ptx::smem_addr(stage), ch0 * C::kOutElem, t0 + ci * 32);
            ptx::bulk_commit();
          }
        }
        buf ^= 1;
      }
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) {                                 // this warp is done with the accumulator stage
        if (PAIR && rank != 0) ptx::mbar_arrive_remote(acc_empty_addr + 8 * acc);
        else ptx::mbar_arrive(bar_acc_empty + 8 * acc);
      }
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1;
    }
    if (lane == 0) ptx::bulk_wait<0>();                // all of this warp's stores have landed
  }

  if (!ok) atomicCAS(args.status, 0, IBERT_ERR_TIMEOUT);
  ptx::tc_fence_before_sync();
  if constexpr (PAIR) ptx::cluster_sync(); else __syncthreads();   // nobody leaves while a peer may use its memory
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    if constexpr (PAIR) ptx::tmem_dealloc_pair(tmem_base, kTmemCols); else ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

template <int TOK, bool PAIR, int KIND, bool FAST>
int launch_inst(ibert_ctx* ctx, const CUtensorMap& mw, const CUtensorMap& mx, const CUtensorMap& mo,
                const GemmArgs& args) {
  using C = Cfg<TOK, PAIR, KIND>;
  static bool attr_set_dev[kMaxDevices] = {false};
  bool& attr_set = attr_set_dev[ctx->device % kMaxDevices];
  if (!attr_set) {
    if (cudaFuncSetAttribute(gemm_i8_kernel<TOK, PAIR, KIND, FAST>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             C::kAlloc) != cudaSuccess)
      return IBERT_ERR_CUDA;
    attr_set = true;
  }
  const int64_t tiles = ((args.T + TOK - 1) / TOK) * ((args.N + (PAIR ? 255 : 127)) / (PAIR ? 256 : 128));
  const int workers = (int)std::min<int64_t>(tiles, PAIR ? ctx->num_sms / 2 : ctx->num_sms);
  return launch_pdl(gemm_i8_kernel<TOK, PAIR, KIND, FAST>, dim3(PAIR ? 2 * workers : workers), dim3(C::kThreads),
                    (size_t)C::kAlloc, ctx->stream, PAIR ? 2 : 1, mw, mx, mo, args);
}

template <int TOK, bool PAIR>
int launch_shape(ibert_ctx* ctx, const CUtensorMap& mw, const CUtensorMap& mx, const CUtensorMap& mo, const GemmArgs& a,
                 int kind, bool fast, bool wide_form, bool transposed) {
  if (transposed) {
    if (kind == EPI_INT8) return launch_inst<TOK, PAIR, kEpiInt8T, true>(ctx, mw, mx, mo, a);
    if constexpr (Cfg<TOK, PAIR, kEpiGeluTable>::kValid) {
      if (kind == EPI_GELU && fast && a.gelu_table)
        return wide_form ? launch_inst<TOK, PAIR, kEpiGeluTableWideT, true>(ctx, mw, mx, mo, a)
                         : launch_inst<TOK, PAIR, kEpiGeluTableT, true>(ctx, mw, mx, mo, a);
    }
    return IBERT_ERR_ARG;
  }
  if (kind == EPI_GELU && fast && a.gelu_table) {
    if constexpr (Cfg<TOK, PAIR, kEpiGeluTable>::kValid)          // (256 tokens on one CTA: no room for the table)
      return wide_form ? launch_inst<TOK, PAIR, kEpiGeluTableWide, true>(ctx, mw, mx, mo, a)
                       : launch_inst<TOK, PAIR, kEpiGeluTable, true>(ctx, mw, mx, mo, a);
  }
  if (kind == EPI_GELU && fast && wide_form)
    return a.gelu.low_free ? launch_inst<TOK, PAIR, kEpiGeluLowFreeWide, true>(ctx, mw, mx, mo, a)
                           : launch_inst<TOK, PAIR, kEpiGeluWide, true>(ctx, mw, mx, mo, a);
  switch (kind) {
    case EPI_INT8: return fast ? launch_inst<TOK, PAIR, EPI_INT8, true>(ctx, mw, mx, mo, a) : launch_inst<TOK, PAIR, EPI_INT8, false>(ctx, mw, mx, mo, a);
    case EPI_Q16: return fast ? launch_inst<TOK, PAIR, EPI_Q16, true>(ctx, mw, mx, mo, a) : launch_inst<TOK, PAIR, EPI_Q16, false>(ctx, mw, mx, mo, a);
    case EPI_Q16H: return fast ? launch_inst<TOK, PAIR, EPI_Q16H, true>(ctx, mw, mx, mo, a) : launch_inst<TOK, PAIR, EPI_Q16H, false>(ctx, mw, mx, mo, a);
    case EPI_GELU:
      if (fast && a.gelu.low_free) return launch_inst<TOK, PAIR, kEpiGeluLowFree, true>(ctx, mw, mx, mo, a);
      return fast ? launch_inst<TOK, PAIR, EPI_GELU, true>(ctx, mw, mx, mo, a) : launch_inst<TOK, PAIR, EPI_GELU, false>(ctx, mw, mx, mo, a);
    case EPI_HGELU: return fast ? launch_inst<TOK, PAIR, EPI_HGELU, true>(ctx, mw, mx, mo, a) : launch_inst<TOK, PAIR, EPI_HGELU, false>(ctx, mw, mx, mo, a);
    default: return launch_inst<TOK, PAIR, EPI_RAW, false>(ctx, mw, mx, mo, a);
  }
}

// tile shape: 256 channels x 256 tokens on a CTA pair when that fills every pair, else one CTA
// per 128 channels x 256 (or 128) tokens
void tile_shape(const ibert_ctx* ctx, int64_t M, int N, bool* pair, bool* wide) {
  const int64_t t256 = (M + 255) / 256;
  *pair = ctx->num_sms >= 2 && t256 * ((N + 255) / 256) >= ctx->num_sms / 2;
  *wide = *pair || t256 * ((N + 127) / 128) >= ctx->num_sms;
}

}  // namespace

bool gemm_gelu_takes_transposed(const ibert_ctx* ctx, int64_t M, int N) {
  bool pair, wide;
  tile_shape(ctx, M, N, &pair, &wide);
  return M % 16 == 0 && (pair || !wide);     // (256 tokens on one CTA leave no room for the table)
}

int launch_gemm_i8(ibert_ctx* ctx, const int8_t* x, const int8_t* w, int64_t M, int N, int K,
                   const GemmEpilogue& epi, void* out) {
  if (M == 0) return IBERT_OK;
  {
    // few output tiles (small batches): split K over a cluster instead of leaving most SMs idle
    if (epi.out_transposed) {
      const bool int8_ok = epi.kind == EPI_INT8 && epi.fast == 1;
      const bool gelu_ok = epi.kind == EPI_GELU && epi.fast != 0 && epi.gelu.fast != 0 && epi.gelu_table && ctx->gelu_table_mode == 0;
      if ((!int8_ok && !gelu_ok) || M % 16 != 0) return IBERT_ERR_ARG;
    }
    int split = (ctx->splitk_mode == 1 || epi.fast == 2 || epi.out_transposed) ? 1 : gemm_splitk_width(ctx, M, N, K);
    if ((ctx->splitk_mode == 2 || ctx->splitk_mode == 4) && K > 128 && epi.fast != 2 && !epi.out_transposed &&
        ((M + 127) / 128) * ((N + 127) / 128) * ctx->splitk_mode <= 65535)
      split = ctx->splitk_mode;
    if (split > 1) return launch_gemm_splitk_i8(ctx, x, w, M, N, K, epi, out, split);
  }
  bool pair, wide;
  tile_shape(ctx, M, N, &pair, &wide);
  const int TOK = wide ? 256 : 128;
  const uint32_t out_elem = (epi.kind == EPI_RAW || epi.kind == EPI_Q16) ? 4u : (epi.kind == EPI_Q16H ? 2u : 1u);
  CUtensorMap mw, mx, mo;
  {
    const uint64_t dims[2] = {(uint64_t)K, (uint64_t)N};
    const uint64_t str[1] = {(uint64_t)K};
    const uint32_t box[2] = {BK, BC};
    int rc = encode_tensor_map(&mw, w, 2, dims, str, box, 128);
    if (rc) return rc;
  }
  {
    const uint64_t dims[2] = {(uint64_t)K, (uint64_t)M};
    const uint64_t str[1] = {(uint64_t)K};
    const uint32_t box[2] = {BK, (uint32_t)(pair ? TOK / 2 : TOK)};   // a pair's CTA loads half of the token rows
    int rc = encode_tensor_map(&mx, x, 2, dims, str, box, 128);
    if (rc) return rc;
  }
  {
    // the output as a byte matrix [T, N * element size]; one box = one warp's 32-token x 32-channel block
    const uint64_t row_bytes = (uint64_t)N * out_elem;
    const uint64_t dims[2] = {row_bytes, (uint64_t)M};
    const uint64_t str[1] = {row_bytes};
    // (the GELU epilogues store a warp's 64 tokens at once)
    const bool gelu_kind = epi.kind == EPI_GELU || epi.kind == EPI_HGELU;   // (with or without the table)
    const uint32_t box[2] = {32u * out_elem, gelu_kind ? 64u : 32u};
    int rc = encode_tensor_map(&mo, out, 2, dims, str, box, 0);
    if (rc) return rc;
    if (epi.out_transposed) {
      // out^T [N][M]: one box = 32 channels x 32 tokens, rows of 32 bytes, 32-byte swizzle
      const uint64_t tdims[2] = {(uint64_t)M, (uint64_t)N};
      const uint64_t tstr[1] = {(uint64_t)M};
      // (the GELU kinds store a warp's 64 tokens at once: rows of 64 bytes, 64-byte swizzle)
      const uint32_t tbox[2] = {gelu_kind ? 64u : 32u, 32u};
      if ((rc = encode_tensor_map(&mo, out, 2, tdims, tstr, tbox, gelu_kind ? 64 : 32))) return rc;
    }
  }
  GemmArgs a{};
  a.T = M; a.N = N; a.K = K;
  a.b = epi.d_b; a.c = epi.d_c; a.bias = epi.d_bias; a.gelu = epi.gelu;
  a.status = ctx->d_status;
  a.gelu_table = ctx->gelu_table_mode == 1 ? nullptr : epi.gelu_table;
  // upper-word epilogue needs both the per-channel multipliers and (for GELU) the final one in that form
  const bool fast = epi.fast != 0 && ((epi.kind != EPI_GELU && epi.kind != EPI_HGELU) || epi.gelu.fast != 0);
  const bool wide_form = epi.fast == 2;
  if (wide_form && (epi.kind != EPI_GELU || !fast)) return IBERT_ERR_ARG;      // tables in a form nothing else reads
  if (pair) return launch_shape<256, true>(ctx, mw, mx, mo, a, epi.kind, fast, wide_form, epi.out_transposed);
  return wide ? launch_shape<256, false>(ctx, mw, mx, mo, a, epi.kind, fast, wide_form, epi.out_transposed)
              : launch_shape<128, false>(ctx, mw, mx, mo, a, epi.kind, fast, wide_form, epi.out_transposed);
}

}  // namespace ibert
