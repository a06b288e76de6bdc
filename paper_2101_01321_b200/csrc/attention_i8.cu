// Fused integer-only attention, per (batch, head) and 128-query tile:
//   S = Q K^T (tcgen05 kind::i8, int32 accumulators in TMEM; scale S_q S_k / 8)
//   P = i-softmax(S) (Algorithm 3: row max, i-exp, int32 row sum, fixed-point quotient) -> u8
//   ctx = requant(P V) (u8 x s8 tcgen05 MMA, accumulator reuses the score columns)
// Scores never leave the SM: they live in TMEM, the exponentials overwrite them in place,
// and the probabilities go to shared memory in the layout the second MMA reads.
// Two kernels: `attention_kernel` (the one every realistic scale takes) and
// `attention_coarse_kernel` for score scales so coarse that the i-exp quotient needs its clamp.
#include <cuda.h>

#include <algorithm>

#include "device_utils.cuh"
#include "sm100_ptx.cuh"

namespace ibert {

namespace {

constexpr int kAttnThreads = 128;   // thread t owns query row t (= TMEM lane t)
constexpr int kHeadDim = 64;

struct CoarseArgs {
  int B, L, H, heads;
  int Lp;            // L rounded up to a multiple of 32 (MMA N / K granularity)
  int n_slabs;       // ceil(L / 128)
  uint32_t tmem_cols;
  int stages;        // operand stages in shared memory: 2 (next item prefetched) or 1
  AttnConsts k;
  const int32_t* lens;   // [B] valid keys per sequence, or nullptr: all L
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
// DIV: the division form of iexp_dist (distance clamped to 31 q_ln2).

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
      for (int i = 0; i < 32; i += 2) mx = __vimax3_s32(mx, (int32_t)v[i], (int32_t)v[i + 1]);
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
  const RowDivisor rd = make_row_divisor(max(sum, 1u), ek.p_max);   // sum = 0 only without valid keys
  const bool nopre = __all_sync(0xffffffffu, rd.pre == 0);      // usual case: every row sum >= 2^10
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
        uint32_t p0, p1, p2, p3;
        if (nopre) {
          p0 = softmax_quotient_nopre(v[j], rd); p1 = softmax_quotient_nopre(v[j + 1], rd);
          p2 = softmax_quotient_nopre(v[j + 2], rd); p3 = softmax_quotient_nopre(v[j + 3], rd);
        } else {
          p0 = softmax_quotient(v[j], rd); p1 = softmax_quotient(v[j + 1], rd);
          p2 = softmax_quotient(v[j + 2], rd); p3 = softmax_quotient(v[j + 3], rd);
        }
        w[i] = ((p3 * 256u + p2) * 256u + p1) * 256u + p0;      // multiply-adds: off the shift/logic pipe
      }
      *reinterpret_cast<uint4*>(sP + sw128_offset(row, (uint32_t)(c0 + h * 16), 128)) =
          make_uint4(w[0], w[1], w[2], w[3]);
    }
  }
}

// Transposes V [j][64] (plain rows in `sVs`) into Vt [64][j] in the swizzled K-major operand
// layout of `sVt`.  A thread takes 4 consecutive keys x 16 head dims, transposes the four 4x4 byte
// blocks with byte permutes and writes 16 words (4 keys of one head dim each).
__device__ __forceinline__ void transpose_v(const uint8_t* sVs, uint8_t* sVt, int n_keys, int tid,
                                            int n_threads = kAttnThreads) {
  for (int item = tid; item < (n_keys / 4) * 4; item += n_threads) {
    // consecutive lanes take the four 16-byte chunks of one key row, then the next key quad: a
    // quarter-warp reads 128 contiguous bytes per load (no bank conflict; the 16 stores per thread
    // then collide four ways, which costs less than the eight-way conflicts of the loads did)
    const int dc = item & 3, jq = item >> 2;                          // 16-dim chunk, key quad
    uint32_t r[4][4];
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      const uint4 t = *reinterpret_cast<const uint4*>(sVs + (jq * 4 + jj) * kHeadDim + dc * 16);
      r[jj][0] = t.x; r[jj][1] = t.y; r[jj][2] = t.z; r[jj][3] = t.w;
    }
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      // rows r[0..3][w] hold dims d0..d0+3 of keys j..j+3; output word i = dim d0+i of the 4 keys
      const uint32_t a01 = __byte_perm(r[0][w], r[1][w], 0x5140);   // k0d0 k1d0 k0d1 k1d1
      const uint32_t b01 = __byte_perm(r[0][w], r[1][w], 0x7362);   // k0d2 k1d2 k0d3 k1d3
      const uint32_t a23 = __byte_perm(r[2][w], r[3][w], 0x5140);
      const uint32_t b23 = __byte_perm(r[2][w], r[3][w], 0x7362);
      const uint32_t o[4] = {__byte_perm(a01, a23, 0x5410), __byte_perm(a01, a23, 0x7632),
                             __byte_perm(b01, b23, 0x5410), __byte_perm(b01, b23, 0x7632)};
#pragma unroll
      for (int i = 0; i < 4; ++i)
        *reinterpret_cast<uint32_t*>(sVt + sw128_offset((uint32_t)(dc * 16 + w * 4 + i), (uint32_t)(jq * 4), 64)) = o[i];
    }
  }
}

// Fallback for coarse score scales (q_ln2 <= 2, where the unclamped quotient of iexp_dist_wide is
// not available).  Persistent CTA of 128 threads, thread = query row: walks (batch, head, query
// tile) work items; while one item is computed the TMA loads of the next one land in the other
// operand stage (when `a.stages` == 2).
__global__ void __launch_bounds__(kAttnThreads, 3)
attention_coarse_kernel(const __grid_constant__ CUtensorMap map_qk, const __grid_constant__ CUtensorMap map_v,
                        const CoarseArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int slab_bytes = 128 * kHeadDim;                       // 8 KB
  const int stage_bytes = (1 + 2 * a.n_slabs) * slab_bytes;     // Q | K slabs | V slabs (plain rows)
  uint8_t* sStage = smem;
  uint8_t* sVt = smem + a.stages * stage_bytes;                 // [n_slabs][64 rows][128 B], swizzled
  uint8_t* sP = sVt + a.n_slabs * slab_bytes;                   // [n_slabs][128 rows][128 B], swizzled
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(sP + a.n_slabs * 128 * 128);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_bar + 3);
  const uint32_t bar_load0 = ptx::smem_addr(s_bar);             // one per stage
  const uint32_t bar_mma = bar_load0 + 16;

  const int tid = threadIdx.x, warp = tid >> 5;
  const int L = a.L, Lp = a.Lp;
  const int q_tiles = a.n_slabs;
  const int total = a.B * a.heads * q_tiles;

  if (tid == 0) {
    ptx::mbar_init(bar_load0, 1);
    ptx::mbar_init(bar_load0 + 8, 1);
    ptx::mbar_init(bar_mma, 1);
    ptx::fence_mbar_init();
    ptx::tma_prefetch_desc(&map_qk);
  }
  if (warp == 0) {
    ptx::tmem_alloc(ptx::smem_addr(s_tmem), a.tmem_cols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *s_tmem;
  const uint32_t t_row = tmem_base + ((uint32_t)(warp * 32) << 16);
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();              // the kernel that wrote qkv has completed

  // loads of one work item: Q tile, all K rows (64-byte swizzle, MMA operand layout), all V rows
  auto issue_loads = [&](int item, int stage) {
    const int qt = item % q_tiles, head = (item / q_tiles) % a.heads, batch = item / (q_tiles * a.heads);
    const uint32_t bar = bar_load0 + 8 * stage;
    uint8_t* base = sStage + stage * stage_bytes;
    ptx::mbar_arrive_expect_tx(bar, (uint32_t)stage_bytes);
    ptx::tma_load_3d(ptx::smem_addr(base), &map_qk, bar, head * kHeadDim, qt * 128, batch);
    for (int s = 0; s < a.n_slabs; ++s) {
      ptx::tma_load_3d(ptx::smem_addr(base + (1 + s) * slab_bytes), &map_qk, bar, a.H + head * kHeadDim, s * 128, batch);
      ptx::tma_load_3d(ptx::smem_addr(base + (1 + a.n_slabs + s) * slab_bytes), &map_v, bar,
                       2 * a.H + head * kHeadDim, s * 128, batch);
    }
  };

  int stage = 0;
  uint32_t load_phase[2] = {0, 0};
  uint32_t mma_phase = 0;
  bool ok = true;
  if (tid == 0 && (int)blockIdx.x < total) issue_loads(blockIdx.x, 0);

  for (int item = blockIdx.x; item < total; item += gridDim.x) {
    const int qt = item % q_tiles, head = (item / q_tiles) % a.heads, batch = item / (q_tiles * a.heads);
    const int q0 = qt * 128;
    uint8_t* sQ = sStage + stage * stage_bytes;
    uint8_t* sK = sQ + slab_bytes;
    uint8_t* sVs = sK + a.n_slabs * slab_bytes;
    const int next = item + gridDim.x;
    ok = __all_sync(0xffffffffu, ptx::mbar_wait(bar_load0 + 8 * stage, load_phase[stage]));
    load_phase[stage] ^= 1;

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
    // two stages: the other one was released by the barrier that ended the previous item, so the
    // next item's loads go out now, behind the MMAs and off this item's critical path
    // (one stage: nothing to overlap, they are issued at the end of this item)
    if (tid == 0 && next < total && a.stages == 2) issue_loads(next, stage ^ 1);
    // ---- meanwhile: V [j][d] -> Vt [d][j] in the swizzled K-major operand layout
    if (ok) transpose_v(sVs, sVt, a.n_slabs * 128, tid);
    if (ok) ok = __all_sync(0xffffffffu, ptx::mbar_wait(bar_mma, mma_phase));
    mma_phase ^= 1;

    // ---- i-softmax on the row this thread owns
    if (ok) {
      ptx::tc_fence_after_sync();
      // keys beyond the sequence's length are masked like the padding columns
      const int n_keys = a.lens ? min(max(__ldg(a.lens + batch), 0), L) : L;
      switch (exp_div_mode(a.k.e)) {
        case 0: softmax_row<0>(t_row, n_keys, Lp, a.k.e, sP, (uint32_t)tid); break;
        case 1: softmax_row<1>(t_row, n_keys, Lp, a.k.e, sP, (uint32_t)tid); break;
        default: softmax_row<2>(t_row, n_keys, Lp, a.k.e, sP, (uint32_t)tid); break;
      }
      ptx::fence_proxy_async_smem();        // P and Vt were written by ordinary stores; the MMA reads them
    }
    ptx::tc_fence_before_sync();
    ok = __syncthreads_and(ok);             // P, Vt complete; every row's scores have been consumed
    if (!ok) break;

    // ---- ctx = P V: K = Lp in steps of 32, accumulator in columns 0..63 (scores are dead)
    if (tid == 0) {
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
    ok = __all_sync(0xffffffffu, ptx::mbar_wait(bar_mma, mma_phase));
    mma_phase ^= 1;

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
            const int j = h * 16 + i * 4;
            if (a.k.fast) {
              w[i] = pack4_sat_s8(max(requant_upper((int32_t)v[j], a.k.b2), -127),
                                  max(requant_upper((int32_t)v[j + 1], a.k.b2), -127),
                                  max(requant_upper((int32_t)v[j + 2], a.k.b2), -127),
                                  max(requant_upper((int32_t)v[j + 3], a.k.b2), -127));
            } else {
              w[i] = pack4_sat_s8(requant_add((int32_t)v[j], a.k.b, half, a.k.c, 127),
                                  requant_add((int32_t)v[j + 1], a.k.b, half, a.k.c, 127),
                                  requant_add((int32_t)v[j + 2], a.k.b, half, a.k.c, 127),
                                  requant_add((int32_t)v[j + 3], a.k.b, half, a.k.c, 127));
            }
          }
          if (q_row < L) *reinterpret_cast<uint4*>(orow + c0 + h * 16) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
    }
    ptx::tc_fence_before_sync();
    ok = __syncthreads_and(ok);             // TMEM columns, Vt, P and this operand stage are free again
    if (!ok) break;
    if (a.stages == 2) stage ^= 1;
    else if (tid == 0 && next < total) issue_loads(next, 0);
  }
  if (!ok) atomicCAS(a.status, 0, IBERT_ERR_TIMEOUT);
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, a.tmem_cols);
  }
}

// ---------------------------------------------------------------------------------------------
// The main kernel.  A persistent CTA owns one (batch, head) pair at a time and walks its 128-query
// tiles, so K and V are loaded once per pair.  V is the B operand of the second MMA exactly as TMA
// delivers it ([key][head dim], 64-byte swizzle): head dim contiguous is the MN-major operand form
// (instruction-descriptor bit 16), one descriptor per 32 keys -- no transposed copy.  The CTA has 128 G threads,
// G >= ceil(L / 128) column groups: warp w works on TMEM lane quadrant w & 3 (the only lanes a warp
// may address) and on the 32-column chunks of group w >> 2, so a score row is shared by G threads
// that exchange their partial maximum and partial sum through shared memory.  Up to 128 keys and
// with many pairs that is one thread per row and four CTAs per SM; at 512 keys one CTA of 16 warps
// fills the SM's TMEM; with fewer pairs than SMs the launcher raises G to shorten the lone CTA's softmax.
// Every operand buffer is refilled as soon as its last reader is done (K and a lone Q after the
// score MMAs, V after the P V MMAs), so the next pair's loads hide behind the softmax and the epilogue.
// Requires the unclamped i-exp form (ExpConsts::wide_post >= 0).
// ---------------------------------------------------------------------------------------------
constexpr int kMaxThreads = 512;
// MN-major operand tiles [64 dims][128 tokens]: 8 KB from one 128-token tile to the next, 1 KB from one
// group of eight dims to the next
constexpr uint32_t kMnLbo = 8192, kMnSbo = 1024;

struct AttnArgs {
  int B, L, H, heads;
  int Lp, n_slabs, groups;
  int q_bufs;        // 2 when a pair has several query tiles (next tile's Q prefetched), else 1
  uint32_t tmem_cols;
  AttnConsts k;
  // padded batches: [B] valid keys per sequence, or nullptr: all L.  Packed batches (the PACKED
  // instantiation of the kernel): [B + 1] first rows of the sequences in a [total tokens, 3H] tensor
  // without padding -- sequence b = rows lens[b] .. lens[b+1]-1, at most L of them.  (One field for
  // both: the size of this argument block is part of what the compiler's schedule hangs on.)
  const int32_t* lens;
  int8_t* out;
  int32_t* status;
};

// PACKED: a.lens holds first-row offsets (a separate instantiation: the padded path compiles as without it)
// QT: the input is the TRANSPOSED tensor qkv^T [3H][tokens] (token index contiguous), as the QKV GEMM
// writes it without a transposing store: Q^T and K^T tiles [64 dims][128 tokens] are MN-major
// operands of the score MMA (instruction-descriptor bits 15 and 16), V^T [64 dims][128 keys] is the
// K-major B operand of the second MMA.  Padded batches with L a multiple of 16 only.
constexpr int kMaxSorted = 256;    // packed batches up to this many sequences are walked longest first

template <bool PACKED, bool QT = false>
__global__ void __launch_bounds__(kMaxThreads, 1)
attention_kernel(const __grid_constant__ CUtensorMap map_qk, const AttnArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int slab_bytes = 128 * kHeadDim;                       // 8 KB
  uint8_t* sQ = smem;                                          // [q_bufs][128 rows][64 B], 64-byte swizzle
  uint8_t* sK = sQ + a.q_bufs * slab_bytes;                    // [n_slabs][128][64 B], 64-byte swizzle
  uint8_t* sVs = sK + a.n_slabs * slab_bytes;                  // [n_slabs][128][64 B], 64-byte swizzle
  uint8_t* sP = sVs + a.n_slabs * slab_bytes;                  // [n_slabs][128 rows][128 B], swizzled
  int32_t* s_max = reinterpret_cast<int32_t*>(sP + a.n_slabs * 128 * 128);   // [4][128]
  uint32_t* s_sum = reinterpret_cast<uint32_t*>(s_max + 4 * 128);            // [4][128]
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(s_sum + 4 * 128);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_bar + 5);
  const uint32_t bar_q0 = ptx::smem_addr(s_bar);               // two Q buffers
  const uint32_t bar_k = bar_q0 + 16, bar_v = bar_q0 + 24, bar_mma = bar_q0 + 32;

  // score columns per tensor-memory load of the softmax passes: 32; 16 for packed batches, whose rows end
  // anywhere (finer skipping of columns past a sequence's end, half the masked tail; measured -5 % there
  // and +3 % on padded batches)
  constexpr int kW = PACKED ? 16 : 32;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_threads = blockDim.x;
  const int quad = warp & 3, grp = warp >> 2, G = a.groups;
  const int row = quad * 32 + lane;                            // query row inside the tile = TMEM lane
  const int L = a.L, q_tiles_padded = a.n_slabs;
  const int total = a.B * a.heads;

  if (tid == 0) {
    ptx::mbar_init(bar_q0, 1);
    ptx::mbar_init(bar_q0 + 8, 1);
    ptx::mbar_init(bar_k, 1);
    ptx::mbar_init(bar_v, 1);
    ptx::mbar_init(bar_mma, 1);
    ptx::fence_mbar_init();
    ptx::tma_prefetch_desc(&map_qk);
  }
  // Packed batches of up to 256 sequences are walked longest first: with work items of unequal length the
  // order decides how evenly the CTAs finish (the sentence mix: -6 % per launch).  Every CTA ranks the
  // sequences by length itself (the offsets are an input of the call, not a product of the kernel before
  // this one, so this runs ahead of the dependency wait): s_order[rank] = sequence.
  uint16_t* s_order = reinterpret_cast<uint16_t*>(s_tmem + 4);
  const bool sorted = PACKED && a.B <= kMaxSorted;
  if constexpr (PACKED) {
    if (sorted) {
      for (int i = tid; i < a.B; i += n_threads) {
        const int len_i = __ldg(a.lens + i + 1) - __ldg(a.lens + i);
        int rank = 0, prev = __ldg(a.lens);
        for (int j = 0; j < a.B; ++j) {
          const int cur = __ldg(a.lens + j + 1), len_j = cur - prev;
          prev = cur;
          rank += (len_j > len_i || (len_j == len_i && j < i)) ? 1 : 0;
        }
        s_order[rank] = (uint16_t)i;
      }
    }
  }
  if (warp == 0) {
    ptx::tmem_alloc(ptx::smem_addr(s_tmem), a.tmem_cols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *s_tmem;
  const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16);
  ptx::grid_dep_launch();
  ptx::grid_dep_wait();              // the kernel that wrote qkv has completed
  // sequence of a work item (items of one sequence are consecutive: its heads)
  auto seq_of = [&](int item) {
    const int s0 = item / a.heads;
    if constexpr (PACKED) return sorted ? (int)s_order[s0] : s0;
    else return s0;
  };

  // (packed: the tensor maps see one "batch" of all rows; a sequence starts at row cu[batch], and
  // rows loaded past its end -- the next sequence's, or zero fill past the last row -- are masked)
  auto load_q = [&](int item, int qt, int buf) {
    const int head = item % a.heads, batch = seq_of(item);
    const int row0 = PACKED ? __ldg(a.lens + batch) : 0, zb = PACKED ? 0 : batch;
    ptx::mbar_arrive_expect_tx(bar_q0 + 8 * buf, (uint32_t)slab_bytes);
    if constexpr (QT) ptx::tma_load_2d(ptx::smem_addr(sQ + buf * slab_bytes), &map_qk, bar_q0 + 8 * buf, batch * a.L + qt * 128, head * kHeadDim);
    else
    ptx::tma_load_3d(ptx::smem_addr(sQ + buf * slab_bytes), &map_qk, bar_q0 + 8 * buf, head * kHeadDim, row0 + qt * 128, zb);
  };
  auto load_k = [&](int item) {
    const int head = item % a.heads, batch = seq_of(item);
    const int row0 = PACKED ? __ldg(a.lens + batch) : 0, zb = PACKED ? 0 : batch;
    ptx::mbar_arrive_expect_tx(bar_k, (uint32_t)(a.n_slabs * slab_bytes));
    for (int s = 0; s < a.n_slabs; ++s) {
      if constexpr (QT) ptx::tma_load_2d(ptx::smem_addr(sK + s * slab_bytes), &map_qk, bar_k, batch * a.L + s * 128, a.H + head * kHeadDim);
      else
      ptx::tma_load_3d(ptx::smem_addr(sK + s * slab_bytes), &map_qk, bar_k, a.H + head * kHeadDim, row0 + s * 128, zb);
    }
  };
  auto load_v = [&](int item) {
    const int head = item % a.heads, batch = seq_of(item);
    const int row0 = PACKED ? __ldg(a.lens + batch) : 0, zb = PACKED ? 0 : batch;
    ptx::mbar_arrive_expect_tx(bar_v, (uint32_t)(a.n_slabs * slab_bytes));
    for (int s = 0; s < a.n_slabs; ++s) {
      if constexpr (QT) ptx::tma_load_2d(ptx::smem_addr(sVs + s * slab_bytes), &map_qk, bar_v, batch * a.L + s * 128, 2 * a.H + head * kHeadDim);
      else
      ptx::tma_load_3d(ptx::smem_addr(sVs + s * slab_bytes), &map_qk, bar_v, 2 * a.H + head * kHeadDim, row0 + s * 128, zb);
    }
  };

  uint32_t q_phase[2] = {0, 0};
  uint32_t kv_phase = 0, mma_phase = 0;
  int qbuf = 0;
  bool ok = true;
  if (tid == 0 && (int)blockIdx.x < total) {
    load_q(blockIdx.x, 0, 0);
    load_k(blockIdx.x);
    load_v(blockIdx.x);
  }

  // Packed batches: sequences differ in length, so after its first (batch, head) pair a CTA draws the
  // following ones from a counter in global memory instead of a fixed stride -- a CTA that got short
  // sequences takes more pairs.  The pair after the current one is drawn at the top of an iteration
  // (its loads are issued during the current pair) and handed to the other threads through shared
  // memory, two slots alternating.  Words 4 and 5 of the status block: the counter, and the number of
  // CTAs that are done; the last CTA to finish zeroes both for the next launch.
  int* s_next = reinterpret_cast<int*>(s_tmem + 1);
  int32_t* draw = a.status + 4;
  int next = 0;
  for (int item = blockIdx.x, iter = 0; item < total && ok; item = next, ++iter) {
    const int head = item % a.heads, batch = seq_of(item);
    if constexpr (PACKED) {
      if (tid == 0) s_next[iter & 1] = (int)gridDim.x + atomicAdd(draw, 1);
    } else {
      next = item + gridDim.x;
    }
    // valid keys of this sequence (key-padding mask): keys >= n take no part in max or sum and get
    // probability 0; the MMAs and the softmax only cover the 32-column chunks that hold valid keys
    // (at least one chunk, so that a sequence without valid keys yields P = 0 and context 0)
    const int row0 = PACKED ? __ldg(a.lens + batch) : 0;           // packed: first row of this sequence
    const int len = PACKED ? __ldg(a.lens + batch + 1) - row0 : 0;
    if (PACKED && len > L && tid == 0) atomicCAS(a.status, 0, IBERT_ERR_VALUE_RANGE);   // longer than the stated maximum
    const int n = PACKED ? min(max(len, 0), L) : (a.lens ? min(max(__ldg(a.lens + batch), 0), L) : L);
    // query rows: all L of a padded sequence, only the existing ones of a packed one
    const int q_tiles = PACKED ? max((n + 127) >> 7, 1) : q_tiles_padded;
    const int Lp = max((n + 31) & ~31, 32);
    const int n_chunks = Lp >> 5, per_grp = (n_chunks + G - 1) / G;
    const int c_begin = min(grp * per_grp, n_chunks) * 32, c_end = min((grp + 1) * per_grp, n_chunks) * 32;

    if constexpr (PACKED) {
      ok = __syncthreads_and(ok);             // the draw of the next pair is visible
      if (!ok) break;
      next = s_next[iter & 1];
    }
    ok = __all_sync(0xffffffffu, ptx::mbar_wait(bar_k, kv_phase));
    kv_phase ^= 1;

    for (int qt = 0; qt < q_tiles; ++qt) {
      const bool last_tile = qt == q_tiles - 1;
      if (ok) ok = __all_sync(0xffffffffu, ptx::mbar_wait(bar_q0 + 8 * qbuf, q_phase[qbuf]));
      q_phase[qbuf] ^= 1;

      // ---- S = Q K^T: K = 64 bytes = two MMA K-steps; N in chunks of at most 256 columns
      if (ok && tid == 0) {
        ptx::tc_fence_after_sync();
        if constexpr (QT) {
          // MN-major operands: [64 dims][128 tokens] tiles, 128-byte swizzle; eight dims form a 1 KB group,
          // a K step of 32 dims is four groups (4 KB); a second 128 keys of N is the next 8 KB tile
          auto mn_desc = [](uint32_t addr) {
            return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(kMnLbo >> 4) << 16) | ((uint64_t)(kMnSbo >> 4) << 32) |
                   ((uint64_t)1 << 46) | ((uint64_t)ptx::kSwizzle128 << 61);
          };
          const uint64_t dq = mn_desc(ptx::smem_addr(sQ + qbuf * slab_bytes));
          for (int n0 = 0; n0 < Lp; n0 += 256) {
            const int nn = min(256, Lp - n0);
            const uint32_t idesc = ptx::make_idesc_i8(128, nn, true, true) | (1u << 15) | (1u << 16);
            const uint64_t dk = mn_desc(ptx::smem_addr(sK + (n0 >> 7) * slab_bytes));
            ptx::mma_i8_ss(tmem_base + n0, dq, dk, idesc, 0u);
            ptx::mma_i8_ss(tmem_base + n0, dq + (4096 >> 4), dk + (4096 >> 4), idesc, 1u);
          }
        } else {
        const uint64_t dq = ptx::make_kmajor_desc(ptx::smem_addr(sQ + qbuf * slab_bytes), 512, ptx::kSwizzle64);
        for (int n0 = 0; n0 < Lp; n0 += 256) {
          const int nn = min(256, Lp - n0);
          const uint32_t idesc = ptx::make_idesc_i8(128, nn, true, true);
          const uint64_t dk = ptx::make_kmajor_desc(ptx::smem_addr(sK + n0 * kHeadDim), 512, ptx::kSwizzle64);
          ptx::mma_i8_ss(tmem_base + n0, dq, dk, idesc, 0u);
          ptx::mma_i8_ss(tmem_base + n0, dq + 2, dk + 2, idesc, 1u);
        }
        }
        ptx::mma_commit(bar_mma);
        // the other Q buffer was read by the previous tile's score MMAs, which have completed
        if (a.q_bufs == 2) {
          if (!last_tile) load_q(item, qt + 1, qbuf ^ 1);
          else if (next < total) load_q(next, 0, qbuf ^ 1);
        }
      }
      if (ok) ok = __all_sync(0xffffffffu, ptx::mbar_wait(bar_mma, mma_phase));
      mma_phase ^= 1;
      // K is no longer read once the last tile's scores exist: fetch the next pair's K behind the softmax
      if (ok && tid == 0 && last_tile && next < total) {
        load_k(next);
        if (a.q_bufs == 1) load_q(next, 0, 0);      // single tile per pair: Q is as dead as K by now
      }

      // packed: a warp whose 32 query rows all lie past the sequence's end computes nothing (its rows of P
      // keep stale bytes; the context rows the second MMA makes of them are never stored)
      const bool live = !PACKED || qt * 128 + quad * 32 < max(n, 1);
      // ---- i-softmax, pass 1: maximum of this thread's columns, then of the row
      int32_t mx = INT32_MIN;
      if (ok && live) {
        ptx::tc_fence_after_sync();
        for (int c0 = c_begin; c0 < c_end; c0 += kW) {
          uint32_t v[kW];
          ptx::tmem_ld(t_row + c0, v);
          ptx::tmem_wait_ld();
          if (c0 + kW <= n) {
#pragma unroll
            for (int i = 0; i < kW; i += 2) mx = __vimax3_s32(mx, (int32_t)v[i], (int32_t)v[i + 1]);
          } else {
#pragma unroll
            for (int i = 0; i < kW; ++i)
              if (c0 + i < n) mx = max(mx, (int32_t)v[i]);
          }
        }
        s_max[grp * 128 + row] = mx;
      }
      if (G > 1) __syncthreads();                  // one thread per row: nothing to exchange
      // ---- pass 2: i-exp written back over the scores, partial sums
      uint32_t sum = 0;
      if (ok && live) {
        for (int g = 0; g < G; ++g) mx = max(mx, s_max[g * 128 + row]);
        if (a.k.e.pow2_k >= 0) {
          // score scale exactly ln2 / 2^k: quotient and remainder by shift and mask
          const uint32_t k2 = (uint32_t)a.k.e.pow2_k, mask = (1u << k2) - 1u;
          const uint32_t mxk = (uint32_t)mx + ((uint32_t)a.k.e.s_out << k2);
          const int32_t q_b = a.k.e.q_b, q_c = a.k.e.q_c;
          for (int c0 = c_begin; c0 < c_end; c0 += kW) {
            uint32_t v[kW];
            ptx::tmem_ld(t_row + c0, v);
            ptx::tmem_wait_ld();
            if (c0 + kW <= n) {
#pragma unroll
              for (int i = 0; i < kW; ++i) {
                v[i] = iexp_dist_pow2(mxk - v[i], q_b, q_c, k2, mask);
                sum += v[i];
              }
            } else {
#pragma unroll
              for (int i = 0; i < kW; ++i) {
                v[i] = (c0 + i < n) ? iexp_dist_pow2(mxk - v[i], q_b, q_c, k2, mask) : 0u;
                sum += v[i];
              }
            }
            ptx::tmem_st(t_row + c0, v);
          }
        } else {
          for (int c0 = c_begin; c0 < c_end; c0 += kW) {
            uint32_t v[kW];
            ptx::tmem_ld(t_row + c0, v);
            ptx::tmem_wait_ld();
            if (c0 + kW <= n) {
#pragma unroll
              for (int i = 0; i < kW; ++i) {
                v[i] = iexp_dist_wide((uint32_t)mx - v[i], a.k.e);
                sum += v[i];
              }
            } else {
#pragma unroll
              for (int i = 0; i < kW; ++i) {
                v[i] = (c0 + i < n) ? iexp_dist_wide((uint32_t)mx - v[i], a.k.e) : 0u;
                sum += v[i];
              }
            }
            ptx::tmem_st(t_row + c0, v);
          }
        }
        ptx::tmem_wait_st();
        s_sum[grp * 128 + row] = sum;
      }
      if (G > 1) __syncthreads();
      // ---- pass 3: u8 probabilities into the operand tile of the second MMA
      if (ok && live) {
        sum = 0;
        for (int g = 0; g < G; ++g) sum += s_sum[g * 128 + row];
        const RowDivisor rd = make_row_divisor(max(sum, 1u), a.k.e.p_max);   // sum = 0 only without valid keys
        const bool nopre = __all_sync(0xffffffffu, rd.pre == 0);
        for (int c0 = c_begin; c0 < c_end; c0 += kW) {
          uint32_t v[kW];
          ptx::tmem_ld(t_row + c0, v);
          ptx::tmem_wait_ld();
#pragma unroll
          for (int h = 0; h < kW / 16; ++h) {
            uint32_t w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int j = h * 16 + i * 4;
              uint32_t p0, p1, p2, p3;
              if (nopre) {
                p0 = softmax_quotient_nopre(v[j], rd); p1 = softmax_quotient_nopre(v[j + 1], rd);
                p2 = softmax_quotient_nopre(v[j + 2], rd); p3 = softmax_quotient_nopre(v[j + 3], rd);
              } else {
                p0 = softmax_quotient(v[j], rd); p1 = softmax_quotient(v[j + 1], rd);
                p2 = softmax_quotient(v[j + 2], rd); p3 = softmax_quotient(v[j + 3], rd);
              }
              w[i] = ((p3 * 256u + p2) * 256u + p1) * 256u + p0;
            }
            *reinterpret_cast<uint4*>(sP + sw128_offset((uint32_t)row, (uint32_t)(c0 + h * 16), 128)) =
                make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
        ptx::fence_proxy_async_smem();
      }
      // V of this pair (requested while the previous pair's epilogue ran) is needed from here on
      if (qt == 0 && ok) ok = __all_sync(0xffffffffu, ptx::mbar_wait(bar_v, kv_phase ^ 1));
      ptx::tc_fence_before_sync();
      ok = __syncthreads_and(ok);             // P complete; every row's exponentials have been consumed
      if (!ok) break;

      // ---- ctx = P V: K = Lp in steps of 32, accumulator in columns 0..63 (scores are dead)
      if (tid == 0) {
        ptx::tc_fence_after_sync();
        // B = V as loaded ([key][head dim], head dim contiguous): the MN-major operand form (bit 16)
        const uint32_t idesc = ptx::make_idesc_i8(128, kHeadDim, false, true) | (QT ? 0u : (1u << 16));   // u8 x s8
        for (int kk = 0; kk < Lp / 32; ++kk) {
          const int kb = kk >> 2, ks = kk & 3;
          const uint64_t dp = ptx::make_kmajor_desc(ptx::smem_addr(sP + kb * 128 * 128), 1024, ptx::kSwizzle128);
          if constexpr (QT) {
            // V^T [64 dims][128 keys]: the plain K-major operand
            const uint64_t dvt = ptx::make_kmajor_desc(ptx::smem_addr(sVs + kb * slab_bytes), 1024, ptx::kSwizzle128);
            ptx::mma_i8_ss(tmem_base, dp + 2 * ks, dvt + 2 * ks, idesc, kk != 0 ? 1u : 0u);
            continue;
          }
          const uint32_t va = ptx::smem_addr(sVs + kk * 32 * kHeadDim);
          const uint64_t dv = (uint64_t)((va & 0x3FFFFu) >> 4) | ((uint64_t)(512 >> 4) << 16) | ((uint64_t)(512 >> 4) << 32) |
                              ((uint64_t)1 << 46) | ((uint64_t)ptx::kSwizzle64 << 61);
          ptx::mma_i8_ss(tmem_base, dp + 2 * ks, dv, idesc, kk != 0 ? 1u : 0u);
        }
        ptx::mma_commit(bar_mma);
      }
      ok = __all_sync(0xffffffffu, ptx::mbar_wait(bar_mma, mma_phase));
      mma_phase ^= 1;
      if (ok && tid == 0 && last_tile && next < total) load_v(next);   // V was read by the MMAs that just completed

      // ---- epilogue: the 64 context values of a row in two halves, taken by column groups 0 and 1
      // (by group 0 alone when there is only one)
      if (ok && grp < 2 && live) {
        ptx::tc_fence_after_sync();
        const int64_t half = rounding_half(a.k.c);
        const int q_row = qt * 128 + row;
        for (int part = grp; part < 2; part += G) {
          int8_t* orow = a.out + (PACKED ? (int64_t)row0 + q_row : (int64_t)batch * L + q_row) * a.H + head * kHeadDim + part * 32;
          uint32_t v[32];
          ptx::tmem_ld32(t_row + part * 32, v);
          ptx::tmem_wait_ld();
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            uint32_t w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int j = h * 16 + i * 4;
              if (a.k.fast) {
                w[i] = pack4_sat_s8(max(requant_upper((int32_t)v[j], a.k.b2), -127),
                                    max(requant_upper((int32_t)v[j + 1], a.k.b2), -127),
                                    max(requant_upper((int32_t)v[j + 2], a.k.b2), -127),
                                    max(requant_upper((int32_t)v[j + 3], a.k.b2), -127));
              } else {
                w[i] = pack4_sat_s8(requant_add((int32_t)v[j], a.k.b, half, a.k.c, 127),
                                    requant_add((int32_t)v[j + 1], a.k.b, half, a.k.c, 127),
                                    requant_add((int32_t)v[j + 2], a.k.b, half, a.k.c, 127),
                                    requant_add((int32_t)v[j + 3], a.k.b, half, a.k.c, 127));
              }
            }
            if (q_row < (PACKED ? n : L)) *reinterpret_cast<uint4*>(orow + h * 16) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
      ptx::tc_fence_before_sync();
      ok = __syncthreads_and(ok);             // TMEM columns and P are free for the next tile
      if (!ok) break;
      if (a.q_bufs == 2) qbuf ^= 1;
    }
  }
  if (!ok) atomicCAS(a.status, 0, IBERT_ERR_TIMEOUT);
  if constexpr (PACKED) {
    if (tid == 0 && atomicAdd(draw + 1, 1) == (int)gridDim.x - 1) {   // every CTA has drawn its last pair
      draw[0] = 0;
      draw[1] = 0;
    }
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, a.tmem_cols);
  }
}

}  // namespace

bool attention_takes_transposed(int B, int L, const AttnConsts& k) {
  // token offsets b L are the innermost TMA coordinate (16-byte aligned), B L the row pitch
  return L % 16 == 0 && ((int64_t)B * L) % 16 == 0 && k.e.wide_post >= 0;
}

int launch_attention(ibert_ctx* ctx, const int8_t* qkv, int B, int L, int H, int heads,
                     const AttnConsts& k, const int32_t* lens, int8_t* out, const int32_t* cu_seqlens,
                     int64_t total_rows, bool qkv_t) {
  if (B == 0) return IBERT_OK;
  if (qkv_t && (cu_seqlens || !attention_takes_transposed(B, L, k))) return IBERT_ERR_ARG;
  if (cu_seqlens && k.e.wide_post < 0) return IBERT_ERR_SCALE_RANGE;   // packed batches: main kernel only
  const int Lp = (L + 31) & ~31, n_slabs = (L + 127) / 128;
  uint32_t cols = 64;
  while ((int)cols < Lp) cols <<= 1;
  CUtensorMap mqk, mv;
  // padded: [B][L][3H]; packed: one "batch" of all rows
  const uint64_t n_rows = cu_seqlens ? (uint64_t)total_rows : (uint64_t)L;
  const uint64_t dims[3] = {(uint64_t)3 * H, n_rows, cu_seqlens ? (uint64_t)1 : (uint64_t)B};
  const uint64_t str[2] = {(uint64_t)3 * H, (uint64_t)3 * H * n_rows};
  const uint32_t box[3] = {kHeadDim, 128, 1};
  int rc = encode_tensor_map(&mqk, qkv, 3, dims, str, box, 64);
  if (rc) return rc;
  if (qkv_t) {
    // qkv^T [3H][B L]: a tile is 64 dims x 128 tokens, rows of 128 bytes, 128-byte swizzle
    const uint64_t tdims[2] = {(uint64_t)B * L, (uint64_t)3 * H};
    const uint64_t tstr[1] = {(uint64_t)B * L};
    const uint32_t tbox[2] = {128, kHeadDim};
    if ((rc = encode_tensor_map(&mqk, qkv, 2, tdims, tstr, tbox, 128))) return rc;
  }
  rc = encode_tensor_map(&mv, qkv, 3, dims, str, box, 0);
  if (rc) return rc;
  const int slab = 128 * kHeadDim;

  if (k.e.wide_post >= 0) {
    AttnArgs a{};
    a.B = B; a.L = L; a.H = H; a.heads = heads;
    a.Lp = Lp; a.n_slabs = n_slabs; a.groups = n_slabs;
    {
      // few pairs: a score row is shared by more threads than its slabs ask for, as many as still
      // keep every pair resident at once (the softmax of a lone CTA per SM is latency-bound)
      const int64_t items = (int64_t)B * heads;
      const int g = items <= ctx->num_sms ? 4 : (items <= 2 * (int64_t)ctx->num_sms ? 2 : 1);
      a.groups = std::min(std::max(n_slabs, g), std::max(Lp / 32, n_slabs));
    }
    a.q_bufs = n_slabs > 1 ? 2 : 1;
    a.tmem_cols = cols; a.k = k; a.lens = cu_seqlens ? cu_seqlens : lens; a.out = out; a.status = ctx->d_status;
    const int smem = a.q_bufs * slab + 2 * n_slabs * slab + n_slabs * 128 * 128 + 2 * 4 * 128 * 4 + 64 + 1024 +
                     (cu_seqlens ? 2 * kMaxSorted : 0);      // (packed: the sequence order)
    // resident CTAs per SM: bounded by the register file (128 G threads of at most 128 registers),
    // by the 512 TMEM columns and by shared memory.  The bound must not exceed what TMEM allows:
    // a CTA that cannot get its columns would wait for a resident one to finish.
    int per_sm = std::min(std::min(4 / a.groups, (int)(512 / cols)), (227 * 1024) / (smem + 1024));
    if (per_sm < 1) per_sm = 1;
    const int grid = std::min(B * heads, ctx->num_sms * per_sm);
    static int smem_set_dev[kMaxDevices] = {0};
    int& smem_set = smem_set_dev[ctx->device % kMaxDevices];
    if (smem > smem_set) {
      if (cudaFuncSetAttribute(attention_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
          cudaFuncSetAttribute(attention_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
          cudaFuncSetAttribute(attention_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
        return IBERT_ERR_CUDA;
      smem_set = smem;
    }
    if (qkv_t) {
      if (int rc2 = launch_pdl(attention_kernel<false, true>, dim3(grid), dim3(128 * a.groups), (size_t)smem, ctx->stream, 1, mqk, a)) return rc2;
      return cudaGetLastError() == cudaSuccess ? IBERT_OK : IBERT_ERR_CUDA;
    }
    if (int rc2 = cu_seqlens ? launch_pdl(attention_kernel<true>, dim3(grid), dim3(128 * a.groups), (size_t)smem, ctx->stream, 1, mqk, a)
                             : launch_pdl(attention_kernel<false>, dim3(grid), dim3(128 * a.groups), (size_t)smem, ctx->stream, 1, mqk, a))
      return rc2;
    return cudaGetLastError() == cudaSuccess ? IBERT_OK : IBERT_ERR_CUDA;
  }

  // scales too coarse for the unclamped division (q_ln2 <= 2): the plain one-tile-per-item kernel
  CoarseArgs a{};
  a.B = B; a.L = L; a.H = H; a.heads = heads;
  a.Lp = Lp; a.n_slabs = n_slabs;
  a.tmem_cols = cols; a.k = k; a.lens = lens; a.out = out; a.status = ctx->d_status;
  const int stage_bytes = (1 + 2 * n_slabs) * slab;
  const int fixed_bytes = n_slabs * slab + n_slabs * 128 * 128 + 64 + 1024;
  a.stages = (2 * stage_bytes + fixed_bytes <= 112 * 1024) ? 2 : 1;     // keep at least 2 CTAs per SM
  const int smem = a.stages * stage_bytes + fixed_bytes;
  static int smem_set_dev[kMaxDevices] = {0};
  int& smem_set = smem_set_dev[ctx->device % kMaxDevices];
  if (smem > smem_set) {
    if (cudaFuncSetAttribute(attention_coarse_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
      return IBERT_ERR_CUDA;
    smem_set = smem;
  }
  const int total = B * heads * n_slabs;
  int per_sm = std::min(3, std::min((int)(512 / cols), (227 * 1024) / (smem + 1024)));
  if (per_sm < 1) per_sm = 1;
  const int grid = std::min(total, ctx->num_sms * per_sm);
  if (int rc2 = launch_pdl(attention_coarse_kernel, dim3(grid), dim3(kAttnThreads), (size_t)smem, ctx->stream, 1,
                           mqk, mv, a)) return rc2;
  return cudaGetLastError() == cudaSuccess ? IBERT_OK : IBERT_ERR_CUDA;
}

}  // namespace ibert
