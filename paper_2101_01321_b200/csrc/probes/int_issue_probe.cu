// Probe: per-SM issue rate of the 32-bit integer instructions the epilogues and i-softmax use, in
// lane-operations per clock and SM (148 CTAs of 512 threads, 8 independent chains per thread), and
// of mixes of an ALU-pipe and a multiply-add-pipe instruction -- the mixes show whether the two
// pipes add up or share one issue port.  Prints one line per instruction; no library code involved.
#include <cstdio>
#include <cuda_runtime.h>
#include <stdint.h>
enum { OP_IADD, OP_IMNMX, OP_SHF, OP_LOP, OP_IMAD, OP_IMADWIDE, OP_IMADHI, OP_MAX3, OP_PRMT, OP_STSU8, OP_STS32, OP_ABS, OP_CVTPACK, OP_SHR64, OP_REQ, OP_REQHI, OP_MULWIDE, OP_REQ2, OP_MIX_ADD_MAD, OP_MIX_ADD2_MAD, OP_MIX_ADD_WIDE, OP_ADDMIN, OP_MIX_ADD_FFMA, OP_FFMA };
template <int OP>
__global__ void __launch_bounds__(512) k(int iters, int seed, int* out, long long* clk) {
  __shared__ uint32_t sm[2048];
  int a[8]; long long w[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) { a[j] = seed + threadIdx.x * 7 + j; w[j] = a[j]; }
  int b = seed * 3 + 1, c = seed ^ 0x55;
  __syncthreads();
  long long t0 = clock64();
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        if (OP == OP_IADD) asm volatile("add.s32 %0, %0, %1;" : "+r"(a[j]) : "r"(b));
        if (OP == OP_IMNMX) asm volatile("max.s32 %0, %0, %1;" : "+r"(a[j]) : "r"(b));
        if (OP == OP_SHF) asm volatile("shr.s32 %0, %0, %1;" : "+r"(a[j]) : "r"(c & 3));
        if (OP == OP_LOP) asm volatile("xor.b32 %0, %0, %1;" : "+r"(a[j]) : "r"(b));
        if (OP == OP_IMAD) asm volatile("mad.lo.s32 %0, %0, %1, %2;" : "+r"(a[j]) : "r"(b), "r"(c));
        if (OP == OP_IMADWIDE) asm volatile("mad.wide.s32 %0, %1, %2, %0;" : "+l"(w[j]) : "r"(a[j]), "r"(b));
        if (OP == OP_IMADHI) asm volatile("mul.hi.s32 %0, %0, %1;" : "+r"(a[j]) : "r"(b));
        if (OP == OP_MAX3) a[j] = __vimax3_s32(a[j], b, c - j);
        if (OP == OP_PRMT) a[j] = __byte_perm(a[j], b, 0x5140);
        if (OP == OP_ABS) a[j] = abs(a[j]) - b;
        if (OP == OP_STSU8) ((volatile uint8_t*)sm)[(j * 4 + r) * 32 + (threadIdx.x & 31) + (threadIdx.x >> 5) * 128 * 0] = (uint8_t)a[j];
        if (OP == OP_STS32) ((volatile uint32_t*)sm)[((j * 4 + r) * 32 + (threadIdx.x & 31)) & 2047] = a[j];
        if (OP == OP_CVTPACK) { uint32_t d; asm volatile("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a[j]), "r"(b), "r"(c)); a[j] = d; }
        if (OP == OP_SHR64) w[j] = (w[j] >> 7) + b;
        if (OP == OP_REQ) a[j] = (int)(((long long)a[j] * (long long)b + w[j]) >> 32) + j;
        if (OP == OP_REQHI) a[j] = __mulhi(a[j], b) + j;
        if (OP == OP_MULWIDE) { long long t = (long long)a[j] * (long long)b; a[j] = (int)(t >> 32) + (int)((unsigned)t >> 31); }
        if (OP == OP_MIX_ADD_MAD) { asm volatile("add.s32 %0, %0, %1;" : "+r"(a[j]) : "r"(b)); asm volatile("mad.lo.s32 %0, %0, %1, %2;" : "+r"(a[j]) : "r"(b), "r"(c)); }
        if (OP == OP_MIX_ADD2_MAD) { asm volatile("add.s32 %0, %0, %1;" : "+r"(a[j]) : "r"(b)); asm volatile("max.s32 %0, %0, %1;" : "+r"(a[j]) : "r"(c)); asm volatile("mad.lo.s32 %0, %0, %1, %2;" : "+r"(a[j]) : "r"(b), "r"(c)); }
        if (OP == OP_MIX_ADD_WIDE) { asm volatile("add.s32 %0, %0, %1;" : "+r"(a[j]) : "r"(b)); asm volatile("mad.wide.s32 %0, %1, %2, %0;" : "+l"(w[j]) : "r"(a[j]), "r"(b)); }
        if (OP == OP_ADDMIN) a[j] = __viaddmin_s32(a[j], b, c);
        if (OP == OP_FFMA) { float f = __int_as_float(a[j]); asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(f) : "f"(1.0001f), "f"(0.5f)); a[j] = __float_as_int(f); }
        if (OP == OP_MIX_ADD_FFMA) { asm volatile("add.s32 %0, %0, %1;" : "+r"(a[j]) : "r"(b)); float f = __int_as_float((int)w[j]); asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(f) : "f"(1.0001f), "f"(0.5f)); w[j] = __float_as_int(f); }
        if (OP == OP_REQ2) { a[j] = max(-127, min(127, (int)(((long long)a[j] * (long long)b + w[j]) >> 32))) + c; }
      }
    }
  }
  long long t1 = clock64();
  int s = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) s += a[j] + (int)w[j];
  if (s == 123456) out[0] = s;
  if (threadIdx.x == 0 && blockIdx.x == 0) clk[0] = t1 - t0;
}
template <int OP> void run(const char* name, int per_step = 1) {
  int* out; long long* clk; cudaMalloc(&out, 4); cudaMalloc(&clk, 8);
  const int iters = 2000;
  k<OP><<<148, 512>>>(iters, 12345, out, clk); cudaDeviceSynchronize();
  k<OP><<<148, 512>>>(iters, 12345, out, clk); cudaDeviceSynchronize();
  long long h; cudaMemcpy(&h, clk, 8, cudaMemcpyDeviceToHost);
  const double ops = 512.0 * iters * 32 * per_step;
  printf("%-22s %8.1f lane-ops/clk/SM   (%s)\n", name, ops / (double)h, cudaGetErrorString(cudaGetLastError()));
}
int main() {
  run<OP_IADD>("IADD"); run<OP_IMNMX>("IMNMX"); run<OP_SHF>("SHF.R"); run<OP_LOP>("LOP3"); run<OP_IMAD>("IMAD"); run<OP_IMADWIDE>("IMAD.WIDE");
  run<OP_IMADHI>("IMAD.HI"); run<OP_MAX3>("VIMNMX3"); run<OP_PRMT>("PRMT"); run<OP_ABS>("IABS+sub"); run<OP_STSU8>("STS.U8"); run<OP_STS32>("STS.32"); run<OP_CVTPACK>("CVT.PACK"); run<OP_SHR64>("SHR64+add"); run<OP_REQ>("requant_upper+add"); run<OP_REQHI>("mulhi+add"); run<OP_MULWIDE>("mulwide+round"); run<OP_REQ2>("requant+clamp+add");
  run<OP_ADDMIN>("VIADDMNMX");
  run<OP_FFMA>("FFMA");
  run<OP_MIX_ADD_MAD>("IADD + IMAD", 2); run<OP_MIX_ADD2_MAD>("IADD + IMNMX + IMAD", 3); run<OP_MIX_ADD_WIDE>("IADD + IMAD.WIDE", 2);
  run<OP_MIX_ADD_FFMA>("IADD + FFMA", 2);
  return 0;
}
