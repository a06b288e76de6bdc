// Probe: the rates of the three data paths a GEMM epilogue thread uses besides the integer pipes --
// tcgen05.ld (TMEM -> registers, 32 lanes x 32 columns per instruction), byte stores into a shared
// staging tile (32 lanes -> 32 consecutive bytes), and byte loads from a 64 KB shared-memory table at
// scattered addresses -- each alone, for 4, 8 and 16 warps per SM on all 148 SMs.  Reported as warp
// instructions per 1000 SM cycles and as bytes per cycle and SM.  Every wait is bounded.
#include <cstdio>
#include <cstdlib>
#include <cuda_runtime.h>
#include "../ibert_internal.h"
#include "../sm100_ptx.cuh"
using namespace ibert;

// MODE 0: tcgen05.ld x32 + wait per instruction; 1: two loads per wait; 2: 32 st.shared.u8 per round;
// 3: 32 ld.shared.u8 per round at pseudo-random table addresses; 4: 8 st.shared.b32 per round
template <int MODE>
__global__ void __launch_bounds__(512, 1) probe(int rounds, long long* cycles, uint32_t* sink) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint32_t s_tmem;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp == 0) { ptx::tmem_alloc(ptx::smem_addr(&s_tmem), 512); ptx::tmem_relinquish(); }
  for (int i = threadIdx.x; i < 65536 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem)[i] = i * 2654435761u;
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t t_row = s_tmem + ((uint32_t)((warp & 3) * 32) << 16);
  const uint32_t table = ptx::smem_addr(smem);
  const uint32_t stage = ptx::smem_addr(smem) + 65536 + warp * 2048;
  uint32_t acc = lane * 40503u + warp;
  __syncthreads();
  const long long t0 = clock64();
  for (int r = 0; r < rounds; ++r) {
    if (MODE == 0) {
      uint32_t v[32];
      ptx::tmem_ld32(t_row + ((r * 32) & 511), v);
      ptx::tmem_wait_ld();
      acc ^= v[0] ^ v[17] ^ v[31];
    } else if (MODE == 1) {
      uint32_t v[32], w[32];
      ptx::tmem_ld32(t_row + ((r * 64) & 511), v);
      ptx::tmem_ld32(t_row + ((r * 64 + 32) & 511), w);
      ptx::tmem_wait_ld();
      acc ^= v[0] ^ v[17] ^ w[3] ^ w[31];
    } else if (MODE == 2) {
#pragma unroll
      for (int i = 0; i < 32; ++i)
        asm volatile("st.shared.u8 [%0], %1;" ::"r"(stage + ((r & 1) * 1024) + i * 32 + lane), "r"(acc + i) : "memory");
    } else if (MODE == 3) {
      uint32_t o[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const uint32_t at = table + (((acc + r) * 2246822519u + i * 3266489917u) >> 16);
        asm volatile("ld.shared.u8 %0, [%1];" : "=r"(o[i]) : "r"(at));
      }
#pragma unroll
      for (int i = 0; i < 32; ++i) acc += o[i];
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i)
        asm volatile("st.shared.b32 [%0], %1;" ::"r"(stage + ((r & 1) * 1024) + (i * 32 + lane) * 4), "r"(acc + i) : "memory");
    }
  }
  const long long t1 = clock64();
  if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
  if (acc == 0x12345678u) sink[0] = acc;
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) { ptx::tc_fence_after_sync(); ptx::tmem_dealloc(s_tmem, 512); }
}

template <int MODE>
void run(const char* name, int warps, double instr_per_round, double bytes_per_round, long long* d_cycles, uint32_t* sink) {
  const int rounds = 2000;
  const int smem = 65536 + 16 * 2048 + 1024;
  cudaFuncSetAttribute(probe<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  for (int i = 0; i < 2; ++i) probe<MODE><<<148, warps * 32, smem>>>(rounds, d_cycles, sink);
  if (cudaDeviceSynchronize() != cudaSuccess) { printf("%-40s %s\n", name, cudaGetErrorString(cudaGetLastError())); return; }
  long long h[148];
  cudaMemcpy(h, d_cycles, sizeof(h), cudaMemcpyDeviceToHost);
  double mean = 0;
  for (long long c : h) mean += (double)c / 148.0;
  const double instr = instr_per_round * rounds * warps;
  printf("%-40s %2d warps  %8.0f cycles  %7.1f warp instr / 1000 cycles  %7.1f bytes / cycle / SM\n", name, warps, mean,
         instr / mean * 1000.0, bytes_per_round * rounds * warps / mean);
}

int main() {
  long long* d_cycles; cudaMalloc(&d_cycles, 148 * sizeof(long long));
  uint32_t* sink; cudaMalloc(&sink, 4);
  for (int warps : {4, 8, 16}) {
    run<0>("tcgen05.ld 32x32b.x32, wait each", warps, 1, 4096, d_cycles, sink);
    run<1>("tcgen05.ld 32x32b.x32, two per wait", warps, 2, 8192, d_cycles, sink);
    run<2>("st.shared.u8, 32 consecutive bytes", warps, 32, 32 * 32, d_cycles, sink);
    run<4>("st.shared.b32, 128 consecutive bytes", warps, 8, 8 * 128, d_cycles, sink);
    run<3>("ld.shared.u8, scattered in 64 KB", warps, 32, 32 * 32, d_cycles, sink);
  }
  return 0;
}
