// Probe: the rate at which tcgen05.mma kind::i8 can be issued on all 148 SMs -- MMAs alone on
// operands already in shared memory, and fed by TMA tile loads through an mbarrier ring -- for
// single-CTA 128 x N tiles and CTA-pair 256 x 256 tiles.  The "MMA only" figure is the INT8 dense
// peak the GEMM kernels are measured against.  Every wait is bounded.
#include <cstdio>
#include <cstdlib>
#include <cuda.h>
#include <cuda_runtime.h>
#include "../ibert_internal.h"
#include "../sm100_ptx.cuh"
using namespace ibert;

// the probe builds its own tensor maps (driver entry point looked up at run time)
static int probe_tensor_map(CUtensorMap* map, const void* base, const uint64_t* dims, uint64_t pitch, const uint32_t* box) {
  typedef CUresult (*Fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                         const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                         CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  void* p = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || !p) return -1;
  const cuuint64_t gd[2] = {dims[0], dims[1]}, gs[1] = {pitch};
  const cuuint32_t bd[2] = {box[0], box[1]}, es[2] = {1, 1};
  return reinterpret_cast<Fn>(p)(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), gd, gs, bd, es,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS ? 0 : -1;
}

// MODE 0: MMA only; 1: TMA fills + MMA.  PAIR: cta_group::2 (cluster of 2).  BN: tile N (per MMA)
template <int BN, bool PAIR, int MODE, int STAGES>
__global__ void __launch_bounds__(128, 1) probe(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                                                int kblocks, int* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  constexpr int A_BYTES = 128 * 128;
  constexpr int B_ROWS = PAIR ? BN / 2 : BN;
  constexpr int B_BYTES = B_ROWS * 128;
  constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  const uint32_t sbase = ptx::smem_addr(smem);
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);
  const uint32_t bar_full = ptx::smem_addr(s_bar), bar_empty = bar_full + 8 * STAGES, bar_done = bar_empty + 8 * STAGES;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_bar + 2 * STAGES + 2);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = PAIR ? ptx::cluster_ctarank() : 0;
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(bar_full + 8 * s, 1); ptx::mbar_init(bar_empty + 8 * s, 1); }
    ptx::mbar_init(bar_done, 1);
    ptx::fence_mbar_init();
  }
  if (warp == 1) { if (PAIR) { ptx::tmem_alloc_pair(ptx::smem_addr(s_tmem), 256); ptx::tmem_relinquish_pair(); } else { ptx::tmem_alloc(ptx::smem_addr(s_tmem), 256); ptx::tmem_relinquish(); } }
  ptx::tc_fence_before_sync();
  if (PAIR) ptx::cluster_sync(); else __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem = *s_tmem;
  bool ok = true;
  if (warp == 0 && lane == 0 && MODE == 1) {
    uint32_t stage = 0, phase = 0;
    for (int kb = 0; kb < kblocks && ok; ++kb) {
      if (!ptx::mbar_wait(bar_empty + 8 * stage, phase ^ 1)) { ok = false; break; }
      const uint32_t sa = sbase + stage * STAGE_BYTES;
      const int row = ((blockIdx.x * 7 + kb) % 64) * 128;   // spread over a 8192-row operand
      const int kc = (kb % 8) * 128;
      if (PAIR) {
        const uint32_t fl = ptx::map_to_cta(bar_full + 8 * stage, 0);
        if (rank == 0) ptx::mbar_arrive_expect_tx(bar_full + 8 * stage, 2 * STAGE_BYTES);
        ptx::tma_load_2d_pair(sa, &map_a, fl, kc, row);
        ptx::tma_load_2d_pair(sa + A_BYTES, &map_b, fl, kc, row);
      } else {
        ptx::mbar_arrive_expect_tx(bar_full + 8 * stage, STAGE_BYTES);
        ptx::tma_load_2d(sa, &map_a, bar_full + 8 * stage, kc, row);
        ptx::tma_load_2d(sa + A_BYTES, &map_b, bar_full + 8 * stage, kc, row);
      }
      if (++stage == STAGES) { stage = 0; phase ^= 1; }
    }
  } else if (warp == 1 && lane == 0 && rank == 0) {
    const uint32_t idesc = ptx::make_idesc_i8(PAIR ? 256 : 128, BN, true, true);
    uint32_t stage = 0, phase = 0;
    for (int kb = 0; kb < kblocks && ok; ++kb) {
      if (MODE == 1) { if (!ptx::mbar_wait(bar_full + 8 * stage, phase)) { ok = false; break; } ptx::tc_fence_after_sync(); }
      const uint32_t sa = sbase + stage * STAGE_BYTES;
      const uint64_t da = ptx::make_kmajor_desc(sa, 1024, ptx::kSwizzle128);
      const uint64_t db = ptx::make_kmajor_desc(sa + A_BYTES, 1024, ptx::kSwizzle128);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (PAIR) ptx::mma_i8_ss_pair(tmem, da + 2 * k, db + 2 * k, idesc, 1u);
        else ptx::mma_i8_ss(tmem, da + 2 * k, db + 2 * k, idesc, 1u);
      }
      if (MODE == 1) { if (PAIR) ptx::mma_commit_pair(bar_empty + 8 * stage, 3); else ptx::mma_commit(bar_empty + 8 * stage); }
      if (++stage == STAGES) { stage = 0; phase ^= 1; }
    }
    if (PAIR) ptx::mma_commit_pair(bar_done, 3); else ptx::mma_commit(bar_done);
  }
  if (PAIR || true) { if (!ptx::mbar_wait(bar_done, 0)) ok = false; }
  if (!ok) atomicCAS(status, 0, -7);
  ptx::tc_fence_before_sync();
  if (PAIR) ptx::cluster_sync(); else __syncthreads();
  if (warp == 1) { ptx::tc_fence_after_sync(); if (PAIR) ptx::tmem_dealloc_pair(tmem, 256); else ptx::tmem_dealloc(tmem, 256); }
}

template <int BN, bool PAIR, int MODE, int STAGES>
void run(const char* name, const int8_t* buf, int* status) {
  constexpr int B_ROWS = PAIR ? BN / 2 : BN;
  CUtensorMap ma, mb;
  const uint64_t dims[2] = {1024, 8192}; const uint64_t str[1] = {1024};
  const uint32_t boxa[2] = {128, 128}, boxb[2] = {128, (uint32_t)B_ROWS};
  if (probe_tensor_map(&ma, buf, dims, str[0], boxa) || probe_tensor_map(&mb, buf + (8 << 20), dims, str[0], boxb)) {
    printf("%-34s tensor map encoding failed\n", name);
    return;
  }
  const int smem = STAGES * (128 * 128 + B_ROWS * 128) + 256 + 1024;
  cudaFuncSetAttribute(probe<BN, PAIR, MODE, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  const int kblocks = 4096;
  cudaLaunchConfig_t cfg{}; cfg.gridDim = dim3(148); cfg.blockDim = dim3(128); cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr[1]; attr[0].id = cudaLaunchAttributeClusterDimension; attr[0].val.clusterDim.x = PAIR ? 2 : 1; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  cudaEvent_t a, b; cudaEventCreate(&a); cudaEventCreate(&b);
  float best = 1e9;
  for (int i = 0; i < 3; ++i) {
    cudaEventRecord(a);
    cudaLaunchKernelEx(&cfg, probe<BN, PAIR, MODE, STAGES>, ma, mb, kblocks, status);
    cudaEventRecord(b); cudaEventSynchronize(b);
    float ms; cudaEventElapsedTime(&ms, a, b); if (ms < best) best = ms;
  }
  int st = 0; cudaMemcpy(&st, status, 4, cudaMemcpyDeviceToHost);
  const double ops = 148.0 * kblocks * 4 * 2.0 * 128 * BN * 32;     // per CTA: 128 rows x BN cols x 32 deep per MMA
  printf("%-34s %8.1f us  %7.0f TOP/s  status %d  %s\n", name, best * 1e3, ops / (best * 1e-3) / 1e12, st, cudaGetErrorString(cudaGetLastError()));
}

int main() {
  int8_t* buf; cudaMalloc(&buf, 16 << 20); cudaMemset(buf, 1, 16 << 20);
  int* status; cudaMalloc(&status, 4); cudaMemset(status, 0, 4);
  run<256, false, 0, 3>("1cta N256 mma-only", buf, status);
  run<128, false, 0, 3>("1cta N128 mma-only", buf, status);
  run<256, true, 0, 3>("pair N256 mma-only", buf, status);
  run<256, false, 1, 3>("1cta N256 tma 3 stages", buf, status);
  run<256, false, 1, 4>("1cta N256 tma 4 stages", buf, status);
  run<128, false, 1, 6>("1cta N128 tma 6 stages", buf, status);
  run<256, true, 1, 4>("pair N256 tma 4 stages", buf, status);
  run<256, true, 1, 6>("pair N256 tma 6 stages", buf, status);
  return 0;
}
