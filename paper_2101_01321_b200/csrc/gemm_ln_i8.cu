// INT8 GEMM with the whole tail of a Transformer sub-block fused into its epilogue:
//   out[t, :] = i-LayerNorm( requant_Q16(x[t, :] W^T + bias) + rescale(res[t, :]) )      (Sec. 3.6, Eq. 16)
// i.e. the output projection or FFN2, the residual addition and the integer LayerNorm in ONE
// kernel: the Q16 tensor never goes to HBM and two launches per layer disappear.
//
// LayerNorm needs statistics over all H channels of a token, so a thread-block CLUSTER of
// H / 256 CTAs owns a 128-token tile: CTA r computes D[t, n] = X W^T for its 256 channels
// (tcgen05.mma kind::i8, M = 128 tokens on the TMEM lanes, N = 256 channels on the columns).
// With tokens on the lanes an epilogue thread owns ONE token, so the row sums are plain
// per-thread accumulations; only 2 numbers per token cross the cluster (distributed shared
// memory `red`), between the two passes of the epilogue:
//   pass A  v = clamp(requant(acc + bias)) + rescale(res);  sum v, sum v^2;  v written back to TMEM
//   exchange  per-token (sum, sum of squares) added into every CTA of the cluster
//   pass B  mu, sigma = I-Sqrt(var) (exact, Algorithm 4's value), y = v - mu, affine + requant -> int8
// sum (v - mu)^2 = sum v^2 - 2 mu sum v + C mu^2 holds exactly in integers, so one pass over the
// accumulators yields the variance numerator.  Per-channel constants are read from shared memory
// (broadcast loads; the load/store pipe is otherwise idle in this ALU-bound epilogue).
//
// Warp roles as in the plain GEMM: warp 0 TMA producer, warp 1 MMA issuer, warps 2..17 epilogue
// (warp w: TMEM lane quadrant w & 3, channel quarter (w - 2) >> 2); two TMEM accumulator stages.
// Every wait is bounded; no TMA multicast is used.
#include <cuda.h>

#include <algorithm>
#include <cmath>

#include "device_utils.cuh"
#include "sm100_ptx.cuh"

namespace ibert {

namespace {

constexpr int kTok = 128;           // tokens per tile = TMEM lanes = MMA M
constexpr int kCh = 256;            // channels per CTA = MMA N = TMEM columns per accumulator stage
constexpr int kBK = 128;            // K bytes per pipeline stage (one 128-byte swizzle span)
constexpr int kMaxStages = 4;       // barrier slots; a kernel instance uses 3 (48 KB stages) or 4 (32 KB, CTA pairs)
constexpr int kEpiWarps = 16;
constexpr int kEpiThreads = 32 * kEpiWarps;
constexpr int kThreads = 64 + kEpiThreads;
constexpr int kXBytes = kTok * kBK;              // 16 KB
constexpr int kOperandBytes = 3 * (kXBytes + kCh * kBK);   // 144 KB of operand stages either way
constexpr int kMaxCta = 4;                       // cluster width the statistics buffers are sized for (H <= 1024)
constexpr int kOutOff = kOperandBytes;            // per epilogue warp: [32 tokens][32 B] output staging
constexpr int kOutTile = 32 * 32;
constexpr int kOutBytes = kEpiWarps * kOutTile;
constexpr int kResOff = kOutOff + kOutBytes;     // per epilogue warp: 2 x [32 tokens][32 B] of the residual
constexpr int kCbOff = kResOff + 2 * kOutBytes;  // int2 {multiplier, bias} per channel
constexpr int kLnOff = kCbOff + kCh * 8;         // int4 {b_i, 0, B_i lo, B_i hi} per channel
// statistics of a tile: a block of 128 uint64 sums of squares followed by 128 int32 sums
constexpr int kStatBytes = kTok * 12;
constexpr int kLocOff = kLnOff + kCh * 16;       // [3]: this CTA's partial sums, by tile index mod 3
constexpr int kGatOff = kLocOff + 3 * kStatBytes;   // [2][kMaxCta]: every CTA's partial sums, by tile parity
constexpr int kParOff = kGatOff + 2 * kMaxCta * kStatBytes;   // [2][128] int4 {mu, floor(2^31 / sigma), shift, -}
constexpr int kBarOff = kParOff + 2 * kTok * 16;
constexpr int kAlloc = kBarOff + 512 + 1024;     // + slack to align the base to 1024 bytes
static_assert(kAlloc <= 227 * 1024, "shared memory budget");

struct GemmLnArgs {
  int64_t T;
  int K, H;
  const int32_t* pb;       // per channel: requantization multiplier in upper-word form
  const int32_t* bias;     // per channel: int32 bias at the accumulator scale
  const int32_t* b_i;      // per channel: LayerNorm output multiplier (upper-word form)
  const int64_t* B_i;      // per channel: LayerNorm output addend
  LnConsts ln;
  int32_t* status;
};

// floor(sqrt(floor(ss / C))) = the largest s with s^2 C <= ss, one thread per value, bit by bit.
// ss / C < 2^(bits(ss) - floor(log2 C)) bounds the highest bit that can be set, so the loop runs
// about half the bit length of the variance.  Needs s < 2^24 and C < 2^12 (then s^2 C < 2^60).
__device__ __forceinline__ uint32_t isqrt_of_quotient(uint64_t ss, uint32_t C) {
  const int bits = 64 - __clzll((long long)(ss | 1ull)) - (31 - __clz((int)C));   // ss / C < 2^bits
  uint32_t s = 0;
  for (int bit = min(max((bits + 1) >> 1, 1), 24) - 1; bit >= 0; --bit) {
    const uint32_t cand = s | (1u << bit);
    const uint64_t sq = (uint64_t)cand * (uint64_t)cand;
    if (sq * (uint64_t)C <= ss) s = cand;
  }
  return s;
}

// PAIR: two CTAs (same 256 channels, adjacent 128-token tiles) share every MMA through
// tcgen05.mma.cta_group::2 -- each loads its own token rows and half of the weight rows, which cuts
// the bytes an SM pulls from L2 per MMA by a third (L2 bandwidth bounds the K = 3072 main loop).
// XT: x is given transposed, x^T [K][T] (token index contiguous), as the FFN1 GEMM writes it without a
// transposing store: a stage's token tile is then [128 K rows][128 tokens], an MN-major A operand
// (instruction-descriptor bit 15; 1 KB from one group of eight K rows to the next).
template <bool PAIR, bool XT = false>
__global__ void __launch_bounds__(kThreads, 1)
gemm_ln_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
               const __grid_constant__ CUtensorMap map_res, const __grid_constant__ CUtensorMap map_out,
               const GemmLnArgs args) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = ptx::smem_addr(smem);
  int2* s_cb = reinterpret_cast<int2*>(smem + kCbOff);
  int4* s_ln = reinterpret_cast<int4*>(smem + kLnOff);
  uint8_t* s_loc = smem + kLocOff;
  const uint8_t* s_gat = smem + kGatOff;
  int4* s_par = reinterpret_cast<int4*>(smem + kParOff);
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(smem + kBarOff);
  constexpr int kStages = PAIR ? 4 : 3;
  constexpr int kWBytes = (PAIR ? kCh / 2 : kCh) * kBK;    // weight rows this CTA loads per K block
  constexpr int kStageBytes = kXBytes + kWBytes;
  // full[4], empty[4], acc_full[2], acc_empty[2], stats[2], TMEM base, res[16 warps][2], decision flags
  const uint32_t bar_full = ptx::smem_addr(s_bar);
  const uint32_t bar_empty = bar_full + 8 * kMaxStages;
  const uint32_t bar_acc_full = bar_empty + 8 * kMaxStages;
  const uint32_t bar_acc_empty = bar_acc_full + 16;
  const uint32_t bar_stats = bar_acc_empty + 16;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_bar + 20);
  const uint32_t bar_res = bar_full + 192;                 // two per epilogue warp
  volatile int* s_flag = reinterpret_cast<volatile int*>(s_bar + 60);   // the epilogue's next-step decision

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();
  const int n_slices = args.H / kCh;                       // CTAs that share a token tile
  const int cl = PAIR ? 2 * n_slices : n_slices;           // cluster width
  const int slice = PAIR ? (int)(rank >> 1) : (int)rank;   // which 256 channels
  const int half = PAIR ? (int)(rank & 1u) : 0;            // which of the pair's two token tiles
  const uint32_t leader = PAIR ? (rank & ~1u) : rank;      // the CTA of the pair that issues the MMAs
  const int cluster_id = (int)blockIdx.x / cl;
  const int num_clusters = (int)gridDim.x / cl;
  const int64_t t_tiles = (args.T + kTok - 1) / kTok;
  const int64_t n_units = PAIR ? (t_tiles + 1) / 2 : t_tiles;   // tiles (pairs of tiles) a cluster steps through
  const int k_blocks = (args.K + kBK - 1) / kBK;
  const int n0 = slice * kCh;                              // this CTA's first channel
  // unit / token tile of this CTA at step `it` of its cluster (a tile past T reads zeros, stores nothing)
  auto unit_of = [&](uint32_t it) { return (int64_t)cluster_id + (int64_t)it * num_clusters; };
  auto tile_of = [&](uint32_t it) { return PAIR ? 2 * unit_of(it) + half : unit_of(it); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(bar_full + 8 * s, 1);
      ptx::mbar_init(bar_empty + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(bar_acc_full + 8 * a, 1);
      ptx::mbar_init(bar_acc_empty + 8 * a, (PAIR ? 2 : 1) * kEpiWarps);   // the leader's is the one in use
      ptx::mbar_init(bar_stats + 8 * a, 1);                    // armed with the expected bytes by this CTA
    }
    for (int i = 0; i < 2 * kEpiWarps; ++i) ptx::mbar_init(bar_res + 8 * i, 1);
    ptx::fence_mbar_init();
    ptx::tma_prefetch_desc(&map_res);
    ptx::tma_prefetch_desc(&map_x);
    ptx::tma_prefetch_desc(&map_w);
    ptx::tma_prefetch_desc(&map_out);
  }
  if (warp == 1) {
    if constexpr (PAIR) { ptx::tmem_alloc_pair(ptx::smem_addr(s_tmem), 2 * kCh); ptx::tmem_relinquish_pair(); }
    else { ptx::tmem_alloc(ptx::smem_addr(s_tmem), 2 * kCh); ptx::tmem_relinquish(); }
  }
  // statistics start at zero; the per-channel constants are weights, not outputs of the previous
  // kernel, so they may be read before the grid dependency is resolved
  for (int i = threadIdx.x; i < 3 * kStatBytes / 4; i += kThreads) reinterpret_cast<uint32_t*>(s_loc)[i] = 0;
  for (int i = threadIdx.x; i < kCh; i += kThreads) {
    s_cb[i] = make_int2(__ldg(args.pb + n0 + i), args.bias ? __ldg(args.bias + n0 + i) : 0);
    const int64_t B = __ldg(args.B_i + n0 + i);
    s_ln[i] = make_int4(__ldg(args.b_i + n0 + i), 0, (int32_t)(uint32_t)B, (int32_t)(B >> 32));
  }
  ptx::tc_fence_before_sync();
  ptx::cluster_sync();                 // barriers and statistics of every CTA are initialised
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *s_tmem;
  bool ok = true;
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();                // x and res come from the previous kernels

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      for (uint32_t it = 0; unit_of(it) < n_units && ok; ++it) {
        const int t0 = (int)tile_of(it) * kTok;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!ptx::mbar_wait_parked(bar_empty + 8 * stage, phase ^ 1)) { ok = false; break; }
          const uint32_t sx = smem_base + stage * kStageBytes;
          if constexpr (PAIR) {
            // both CTAs' copies complete on the leader's barrier, which expects the bytes of both
            const uint32_t full_leader = ptx::map_to_cta(bar_full + 8 * stage, leader);
            if (half == 0) ptx::mbar_arrive_expect_tx(bar_full + 8 * stage, 2 * kStageBytes);
            if constexpr (XT) ptx::tma_load_2d_pair(sx, &map_x, full_leader, t0, kb * kBK);
            else ptx::tma_load_2d_pair(sx, &map_x, full_leader, kb * kBK, t0);
            ptx::tma_load_2d_pair(sx + kXBytes, &map_w, full_leader, kb * kBK, n0 + half * (kCh / 2));
          } else {
            ptx::mbar_arrive_expect_tx(bar_full + 8 * stage, kStageBytes);
            if constexpr (XT) ptx::tma_load_2d(sx, &map_x, bar_full + 8 * stage, t0, kb * kBK);
            else ptx::tma_load_2d(sx, &map_x, bar_full + 8 * stage, kb * kBK, t0);
            ptx::tma_load_2d(sx + kXBytes, &map_w, bar_full + 8 * stage, kb * kBK, n0);
          }
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (PAIR: the pair's leader only)
    if (lane == 0 && half == 0) {
      constexpr uint32_t idesc = ptx::make_idesc_i8(PAIR ? 2 * kTok : kTok, kCh, true, true) | (XT ? (1u << 15) : 0u);
      const uint16_t pair_mask = (uint16_t)(3u << leader);
      uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
      for (uint32_t it = 0; unit_of(it) < n_units && ok; ++it) {
        if (!ptx::mbar_wait_parked(bar_acc_empty + 8 * acc, acc_phase ^ 1)) { ok = false; break; }
        ptx::tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * kCh;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!ptx::mbar_wait_parked(bar_full + 8 * stage, phase)) { ok = false; break; }
          ptx::tc_fence_after_sync();
          const uint32_t sx = smem_base + stage * kStageBytes;
          const uint64_t dx = ptx::make_kmajor_desc(sx, 1024, ptx::kSwizzle128);
          const uint64_t dw = ptx::make_kmajor_desc(sx + kXBytes, 1024, ptx::kSwizzle128);
          // (MN-major X tile: the same fields -- 1 KB between groups of eight K rows -- and a K step of 32 rows
          // is four groups = 4 KB further on; K-major: 32 bytes further inside the swizzle span)
          constexpr uint64_t x_step = XT ? (4096 >> 4) : 2;
#pragma unroll
          for (int k = 0; k < kBK / 32; ++k) {
            if constexpr (PAIR) ptx::mma_i8_ss_pair(d_tmem, dx + x_step * k, dw + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
            else ptx::mma_i8_ss(d_tmem, dx + x_step * k, dw + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          // frees the stage (in both CTAs of a pair) once these MMAs have read it
          if constexpr (PAIR) ptx::mma_commit_pair(bar_empty + 8 * stage, pair_mask);
          else ptx::mma_commit(bar_empty + 8 * stage);
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        if constexpr (PAIR) ptx::mma_commit_pair(bar_acc_full + 8 * acc, pair_mask);
        else ptx::mma_commit(bar_acc_full + 8 * acc);
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1;
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..17)
    // All 16 warps work on the same tile: warp w takes TMEM lane quadrant w & 3 (32 tokens) and
    // channel quarter (w - 2) >> 2 (64 channels, two 32-column chunks).  Tiles are handled greedily:
    // when the next tile's accumulator is already complete, its pass A runs before this tile's
    // pass B, so the statistics exchange of one tile hides behind arithmetic of the other.
    const int ew = warp - 2;                           // 0..15
    const int quad = warp & 3;
    const int part = ew >> 2;
    const int tok = quad * 32 + lane;                  // this thread's token inside the tile
    const int e_tid = threadIdx.x - 64;                // 0..511
    uint8_t* stage0 = smem + kOutOff + ew * kOutTile;
    const uint8_t* res0 = smem + kResOff + ew * 2 * kOutTile;
    const uint32_t my_res = bar_res + 16 * ew;
    const LnConsts ln = args.ln;
    const int C = ln.C;
    const uint32_t t_lane = tmem_base + ((uint32_t)(quad * 32) << 16);

    // residual block of this warp for tile `it` (32 tokens x 64 channels) into its two private
    // buffers; rows past T read as zero.  Called by lane 0 once both buffers have been consumed.
    auto issue_res = [&](uint32_t it) {
      const int t0 = (int)tile_of(it) * kTok;
      for (int b = 0; b < 2; ++b) {
        ptx::mbar_arrive_expect_tx(my_res + 8 * b, kOutTile);
        ptx::tma_load_2d(ptx::smem_addr(res0 + b * kOutTile), &map_res, my_res + 8 * b, n0 + part * 64 + b * 32,
                         t0 + quad * 32);
      }
    };
    // pass A of tile `it`: v = clamp(requant(acc + bias)) + rescale(res) written back to TMEM,
    // this thread's sums added to the CTA's partial sums
    auto pass_a = [&](uint32_t it) {
      const uint32_t par = it & 1u, phase = (it >> 1) & 1u;
      if (ok) ok = ptx::mbar_wait(bar_acc_full + 8 * par, phase);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        ptx::tc_fence_after_sync();
        int32_t s1 = 0;
        uint64_t s2 = 0;
#pragma unroll 1
        for (int ci = 0; ci < 2; ++ci) {
          const int col = part * 64 + ci * 32;
          uint32_t v[32];
          ptx::tmem_ld32(t_lane + par * kCh + col, v);
          const bool got = __all_sync(0xffffffffu, ptx::mbar_wait(my_res + 8 * ci, it & 1u));   // one fill per tile
          const uint8_t* rsrc = res0 + ci * kOutTile + lane * 32;
          const uint4 ra = *reinterpret_cast<const uint4*>(rsrc), rb = *reinterpret_cast<const uint4*>(rsrc + 16);
          const uint32_t rw[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w};
          ptx::tmem_wait_ld();
          if (!got) ok = false;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int2 cb = s_cb[col + i];
            const int32_t q16 = clamp_sym(requant_upper((int32_t)v[i] + cb.y, cb.x), 32767);
            const int32_t rv = sext_byte(rw[i >> 2], i & 3);
            const int32_t val = q16 + ((rv * ln.res_nb + ln.res_nhalf) >> ln.res_nc);   // the residual, rescaled (narrow form)
            v[i] = (uint32_t)val;
            s1 += val;
            s2 += (uint64_t)((int64_t)val * (int64_t)val);
          }
          ptx::tmem_st32(t_lane + par * kCh + col, v);
        }
        ptx::tmem_wait_st();
        uint8_t* loc = s_loc + (it % 3u) * kStatBytes;
        atomicAdd(reinterpret_cast<unsigned long long*>(loc) + tok, (unsigned long long)s2);
        atomicAdd(reinterpret_cast<int32_t*>(loc + kTok * 8) + tok, s1);
      }
      ptx::fence_proxy_async_smem();
      __syncwarp();                                    // both residual buffers are consumed
      if (lane == 0 && ok && unit_of(it + 1) < n_units) issue_res(it + 1);
    };
    // sends the CTA's partial sums of tile `it` to every CTA of the cluster: one bulk copy of the
    // 1.5 KB block per destination, credited to the destination's statistics barrier (one thread;
    // needs a barrier after pass A, and -- so that the receivers have read the block of tile
    // it - 2 -- comes after this CTA has seen the blocks of tile it - 1 complete)
    auto exchange = [&](uint32_t it) {
      if (e_tid != 0 || !ok) return;
      const uint32_t par = it & 1u;
      ptx::fence_proxy_async_smem();                   // the sums were written by ordinary atomics
      ptx::mbar_arrive_expect_tx(bar_stats + 8 * par, (uint32_t)n_slices * kStatBytes);
      const uint32_t src = ptx::smem_addr(s_loc + (it % 3u) * kStatBytes);
      const uint32_t dst = ptx::smem_addr(s_gat + (par * kMaxCta + slice) * kStatBytes);
      for (int sl = 0; sl < n_slices; ++sl) {            // the CTAs that hold the other channels of this token tile
        const uint32_t r = PAIR ? (uint32_t)(2 * sl + half) : (uint32_t)sl;
        ptx::bulk_copy_to_cta(ptx::map_to_cta(dst, r), src, kStatBytes, ptx::map_to_cta(bar_stats + 8 * par, r));
      }
    };
    // mean and inverse standard deviation of the tokens of tile `it` (warps 4..7, one token per
    // thread); a barrier of all epilogue warps must follow before pass B reads them
    auto params = [&](uint32_t it) {
      const uint32_t par = it & 1u, phase = (it >> 1) & 1u;
      if (ew >= 4 && ew < 8) {
        const int tk = e_tid - 128;
        const int i = par * kTok + tk;
        if (ok) ok = ptx::mbar_wait_cluster(bar_stats + 8 * par, phase);
        ok = __all_sync(0xffffffffu, ok);
        int32_t mu = 0, rho = 1 << 30, nsh = 14;
        if (ok) {
          int32_t sum = 0;
          uint64_t sumsq = 0;
          for (int r = 0; r < n_slices; ++r) {
            const uint8_t* blk = s_gat + (par * kMaxCta + r) * kStatBytes;
            sumsq += reinterpret_cast<const unsigned long long*>(blk)[tk];
            sum += reinterpret_cast<const int32_t*>(blk + kTok * 8)[tk];
          }
          // every CTA has this tile's blocks, so each has read the blocks of the tile before:
          // that tile's own partial sums can be cleared for their next use three tiles on
          if (it > 0) {
            uint8_t* old = s_loc + ((it - 1) % 3u) * kStatBytes;
            reinterpret_cast<unsigned long long*>(old)[tk] = 0;
            reinterpret_cast<int32_t*>(old + kTok * 8)[tk] = 0;
          }
          mu = sum / C;                                // floor(sum / C)
          if (sum - mu * C < 0) mu -= 1;
          const int64_t ss = (int64_t)sumsq - 2 * (int64_t)mu * (int64_t)sum + (int64_t)C * (int64_t)mu * (int64_t)mu;
          const uint32_t sigma = isqrt_of_quotient((uint64_t)ss, (uint32_t)C);
          if (sigma > 1u) { rho = (int32_t)(0x80000000u / sigma); nsh = 15; }   // floor(2^31 / sigma); sigma <= 1: 2^30, one shift less
        }
        s_par[i] = make_int4(mu, rho, nsh, 0);
      }
    };
    // pass B of tile `it`: normalize, affine + requantize to int8, store; frees the accumulator stage
    auto pass_b = [&](uint32_t it) {
      const uint32_t par = it & 1u;
      const int t0 = (int)tile_of(it) * kTok;
      if (ok) {
        const int4 mr = s_par[par * kTok + tok];
        const int32_t mu = mr.x, rho = mr.y;
        const uint32_t nsh = (uint32_t)mr.z;
#pragma unroll 1
        for (int ci = 0; ci < 2; ++ci) {
          const int col = part * 64 + ci * 32;
          uint32_t v[32];
          ptx::tmem_ld32(t_lane + par * kCh + col, v);
          ptx::tmem_wait_ld();
          if (lane == 0) ptx::bulk_wait_read<0>();     // the previous store has read the staging tile
          __syncwarp();
          uint8_t* stage = stage0;
          uint32_t w[8];
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            int32_t o[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int4 lc = s_ln[col + i + j];
              const int32_t y = (int32_t)v[i + j] - mu;
              const int64_t pr = (int64_t)y * (int64_t)rho;
              // floor(pr / 2^nsh) fits 32 bits: the low word of the 64-bit shift is a funnel shift
              const int32_t nrm = (int32_t)__funnelshift_r((uint32_t)pr, (uint32_t)(pr >> 32), nsh) << ln.out_sh;
              const int64_t Bv = (int64_t)(((uint64_t)(uint32_t)lc.w << 32) | (uint32_t)lc.z);
              o[j] = max(requant_upper_add(nrm, lc.x, Bv), -127);
            }
            w[i >> 2] = pack4_sat_s8(o[0], o[1], o[2], o[3]);
          }
          *reinterpret_cast<uint4*>(stage + lane * 32) = make_uint4(w[0], w[1], w[2], w[3]);
          *reinterpret_cast<uint4*>(stage + lane * 32 + 16) = make_uint4(w[4], w[5], w[6], w[7]);
          ptx::fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            ptx::tma_store_2d(&map_out, ptx::smem_addr(stage), n0 + col, t0 + quad * 32);
            ptx::bulk_commit();
          }
        }
      }
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) {
        if (PAIR && half != 0) ptx::mbar_arrive_remote(ptx::map_to_cta(bar_acc_empty + 8 * par, leader));
        else ptx::mbar_arrive(bar_acc_empty + 8 * par);
      }
    };

    // decision taken by the last epilogue thread right after its pass A of tile `it`: run pass A of
    // tile it + 1 before pass B of tile it?  Only if that accumulator is complete already.
    auto decide = [&](uint32_t it) {
      if (e_tid == kEpiThreads - 1)
        s_flag[it & 1u] = (unit_of(it + 1) < n_units &&
                           ptx::mbar_test_now(bar_acc_full + 8 * ((it + 1) & 1u), ((it + 1) >> 1) & 1u)) ? 1 : 0;
    };
    // One loop body for every schedule (so pass A and pass B are instantiated once -- the
    // instruction cache matters here).  Iteration `it` finishes tile `it`; its two steps are
    //   step 0: statistics of tile it, [pass A of tile it + 1 if it may run early], pass B of tile it
    //   step 1: pass A of tile it + 1 if it did not run early
    // and iteration -1 only runs pass A of tile 0.  After every pass A: decision for that tile,
    // barrier (sums complete, decision and statistics visible), exchange.
    if (unit_of(0) < n_units) {
      if (lane == 0) issue_res(0);
      for (int it = -1;; ++it) {
        const bool has_next = unit_of((uint32_t)(it + 1)) < n_units;
        const bool early = it >= 0 && s_flag[it & 1] != 0;
#pragma unroll 1
        for (int step = 0; step < 2; ++step) {
          const bool finish = step == 0 && it >= 0;
          const bool do_a = step == 0 ? early : (!early && has_next);
          if (finish) params((uint32_t)it);
          if (do_a) {
            pass_a((uint32_t)(it + 1));
            decide((uint32_t)(it + 1));
          }
          if (finish || do_a) ptx::named_bar_sync(1, kEpiThreads);
          if (do_a) exchange((uint32_t)(it + 1));
          if (finish) pass_b((uint32_t)it);
        }
        if (!has_next) break;
      }
    }
    if (lane == 0) ptx::bulk_wait<0>();
  }

  if (!ok) atomicCAS(args.status, 0, IBERT_ERR_TIMEOUT);
  ptx::tc_fence_before_sync();
  ptx::cluster_sync();                 // nobody leaves while a peer may still add into its shared memory
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    if constexpr (PAIR) ptx::tmem_dealloc_pair(tmem_base, 2 * kCh); else ptx::tmem_dealloc(tmem_base, 2 * kCh);
  }
}

}  // namespace

bool gemm_ln_supported(int H, int K, const GemmEpilogue& epi, const LnConsts& ln) {
  if (H % kCh != 0 || H / kCh > kMaxCta || K % 16 != 0) return false;    // cluster of H / 256 CTAs, at most 4
  if (!epi.fast || epi.kind != EPI_Q16) return false;
  if (!ln.has_res || !ln.res_fast || !ln.res_narrow || !ln.out_fast || ln.C != H) return false;
  // |v| = |Q16 value + rescaled residual| must stay below 2^18: sums over H <= 2048 channels then fit
  // int32, sums of squares 2^47, and sigma 2^24
  const double res_max = 127.0 * std::ldexp((double)ln.b_r, ln.res_sh - 32);
  return res_max < 200000.0;
}

int launch_gemm_ln_i8(ibert_ctx* ctx, const int8_t* x, const int8_t* w, int64_t T, int H, int K,
                      const GemmEpilogue& epi, const int8_t* res, const LnConsts& ln, const int32_t* d_b_i,
                      const int64_t* d_B_i, int8_t* out, bool x_transposed) {
  if (T == 0) return IBERT_OK;
  if (!gemm_ln_supported(H, K, epi, ln)) return IBERT_ERR_SHAPE;
  if (x_transposed && T % 16 != 0) return IBERT_ERR_ARG;
  CUtensorMap mx, mw, mr, mo;
  int rc;
  {
    const uint64_t dims[2] = {(uint64_t)K, (uint64_t)T};
    const uint64_t str[1] = {(uint64_t)K};
    const uint32_t box[2] = {kBK, kTok};
    if ((rc = encode_tensor_map(&mx, x, 2, dims, str, box, 128))) return rc;
    if (x_transposed) {
      // x^T [K][T]: a stage's tile is 128 K rows x 128 tokens
      const uint64_t tdims[2] = {(uint64_t)T, (uint64_t)K};
      const uint64_t tstr[1] = {(uint64_t)T};
      const uint32_t tbox[2] = {kTok, kBK};
      if ((rc = encode_tensor_map(&mx, x, 2, tdims, tstr, tbox, 128))) return rc;
    }
  }
  {
    const uint64_t dims[2] = {(uint64_t)K, (uint64_t)H};
    const uint64_t str[1] = {(uint64_t)K};
    const uint32_t box[2] = {kBK, kCh};
    if ((rc = encode_tensor_map(&mw, w, 2, dims, str, box, 128))) return rc;
  }
  {
    const uint64_t dims[2] = {(uint64_t)H, (uint64_t)T};
    const uint64_t str[1] = {(uint64_t)H};
    const uint32_t obox[2] = {32, 32};
    if ((rc = encode_tensor_map(&mr, res, 2, dims, str, obox, 0))) return rc;
    if ((rc = encode_tensor_map(&mo, out, 2, dims, str, obox, 0))) return rc;
  }
  GemmLnArgs a{};
  a.T = T; a.K = K; a.H = H;
  a.pb = epi.d_b; a.bias = epi.d_bias; a.b_i = d_b_i; a.B_i = d_B_i;
  a.ln = ln;
  a.status = ctx->d_status;
  const int n_slices = H / kCh;
  const int64_t t_tiles = (T + kTok - 1) / kTok;
  // CTA pairs (two token tiles per cluster step) when the cluster stays within 6 CTAs and there are
  // tiles for both halves; resident clusters from the occupancy query, cached
  static int max_clusters[kMaxDevices][2][9] = {{{0}}};
  auto resident = [&](bool pair, int cl) {
    int& slot = max_clusters[ctx->device % kMaxDevices][pair ? 1 : 0][cl];
    if (slot == 0) {
      const void* fn = pair ? (const void*)gemm_ln_kernel<true> : (const void*)gemm_ln_kernel<false>;
      const void* fnt = pair ? (const void*)gemm_ln_kernel<true, true> : (const void*)gemm_ln_kernel<false, true>;
      if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, kAlloc) != cudaSuccess ||
          cudaFuncSetAttribute(fnt, cudaFuncAttributeMaxDynamicSharedMemorySize, kAlloc) != cudaSuccess) {
        cudaGetLastError();
        slot = -1;
        return slot;
      }
      cudaLaunchConfig_t cfg{};
      cfg.gridDim = dim3(cl * ctx->num_sms);
      cfg.blockDim = dim3(kThreads);
      cfg.dynamicSmemBytes = kAlloc;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = cl; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr; cfg.numAttrs = 1;
      int n = 0;
      const cudaError_t e = pair ? cudaOccupancyMaxActiveClusters(&n, gemm_ln_kernel<true>, &cfg)
                                 : cudaOccupancyMaxActiveClusters(&n, gemm_ln_kernel<false>, &cfg);
      if (e != cudaSuccess) { cudaGetLastError(); n = 0; }
      slot = n >= 1 ? n : -1;
    }
    return slot;
  };
  // (clusters of 8 fit only 16 times on the 148 SMs and measured slower than clusters of 4 single CTAs)
  const bool want_pair = 2 * n_slices <= 6 && t_tiles >= 2;
  if (want_pair && resident(true, 2 * n_slices) > 0) {
    const int cl = 2 * n_slices;
    CUtensorMap mw2;
    const uint64_t dims[2] = {(uint64_t)K, (uint64_t)H};
    const uint64_t str[1] = {(uint64_t)K};
    const uint32_t box[2] = {kBK, kCh / 2};            // each CTA of a pair loads half of the weight rows
    if ((rc = encode_tensor_map(&mw2, w, 2, dims, str, box, 128))) return rc;
    const int clusters = (int)std::min<int64_t>((t_tiles + 1) / 2, resident(true, cl));
    if (x_transposed)
      return launch_pdl(gemm_ln_kernel<true, true>, dim3(clusters * cl), dim3(kThreads), (size_t)kAlloc, ctx->stream, cl,
                        mx, mw2, mr, mo, a);
    return launch_pdl(gemm_ln_kernel<true>, dim3(clusters * cl), dim3(kThreads), (size_t)kAlloc, ctx->stream, cl,
                      mx, mw2, mr, mo, a);
  }
  if (resident(false, n_slices) <= 0) return IBERT_ERR_CUDA;
  const int clusters = (int)std::min<int64_t>(t_tiles, resident(false, n_slices));
  if (x_transposed)
    return launch_pdl(gemm_ln_kernel<false, true>, dim3(clusters * n_slices), dim3(kThreads), (size_t)kAlloc, ctx->stream,
                      n_slices, mx, mw, mr, mo, a);
  return launch_pdl(gemm_ln_kernel<false>, dim3(clusters * n_slices), dim3(kThreads), (size_t)kAlloc, ctx->stream,
                    n_slices, mx, mw, mr, mo, a);
}

}  // namespace ibert
