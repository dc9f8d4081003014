// Pipe-rate microbenchmark for one B200: lane-operations per clock per SM of FFMA, packed FFMA2, MUFU.EX2, SHFL and a
// dependent LDS chain, alone and in the mixes the scan kernels use, at 128..1024 threads per SM (one CTA per SM).
// The benchmark's ALU roofline takes its MUFU and FP32 rates from this program's output.
// A second table mixes two instruction kinds with independent operands and prints the cycles one scheduler spends per
// warp on a group of them: it shows which pipes overlap (FP32 with MUFU, shared-memory loads, shuffles) and which share
// the dispatch path (FP32 with the integer/logic pipe: LOP3 and IMAD each cost two cycles that FFMA cannot hide).
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -o pipe_rates pipe_rates.cu && ./pipe_rates
#include <cstdio>
#include <cuda_runtime.h>
#include <cstdint>
#define ITERS 4096
template <int MODE>
__global__ void k(float* out, long long* cyc, float a, float b) {
  float x[8];
  unsigned long long p[8];
  __shared__ float sm[4096];
  for (int i = 0; i < 8; ++i) { x[i] = threadIdx.x * 0.001f + i; p[i] = (unsigned long long)__float_as_uint(x[i]) | ((unsigned long long)__float_as_uint(x[i]+1.f) << 32); }
  for (int i = threadIdx.x; i < 4096; i += blockDim.x) sm[i] = i;
  unsigned long long aa = (unsigned long long)__float_as_uint(a) | ((unsigned long long)__float_as_uint(a) << 32);
  unsigned long long bb = (unsigned long long)__float_as_uint(b) | ((unsigned long long)__float_as_uint(b) << 32);
  __syncthreads();
  long long t0 = clock64();
  for (int it = 0; it < ITERS; ++it) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (MODE == 0) x[i] = fmaf(x[i], a, b);
      if (MODE == 1) asm volatile("fma.rn.f32x2 %0, %0, %1, %2;" : "+l"(p[i]) : "l"(aa), "l"(bb));
      if (MODE == 2) asm volatile("ex2.approx.ftz.f32 %0, %0;" : "+f"(x[i]));
      if (MODE == 3) x[i] = __shfl_xor_sync(0xffffffffu, x[i], 1 + (i & 15));
      if (MODE == 4) { x[i] = fmaf(x[i], a, b); if ((i & 7) == 0) asm volatile("ex2.approx.ftz.f32 %0, %0;" : "+f"(x[i])); }
      if (MODE == 5) x[i] = sm[(threadIdx.x + (int)x[i]) & 4095];
      if (MODE == 6) { asm volatile("fma.rn.f32x2 %0, %0, %1, %2;" : "+l"(p[i]) : "l"(aa), "l"(bb)); if ((i & 3) == 0) asm volatile("ex2.approx.ftz.f32 %0, %0;" : "+f"(x[i])); }
      if (MODE == 7) { asm volatile("fma.rn.f32x2 %0, %0, %1, %2;" : "+l"(p[i]) : "l"(aa), "l"(bb)); if ((i & 3) == 0) x[i] = __shfl_xor_sync(0xffffffffu, x[i], 1); }
      if (MODE == 8) { x[i] = fmaf(x[i], a, b); if ((i & 3) == 0) x[(i+1)&7] = __shfl_xor_sync(0xffffffffu, x[(i+1)&7], 1); }
      if (MODE == 9) { x[i] = fmaf(x[i], a, b); if ((i & 3) == 0) asm volatile("ex2.approx.ftz.f32 %0, %0;" : "+f"(x[(i+1)&7])); }
    }
  }
  long long t1 = clock64();
  float s = 0; for (int i = 0; i < 8; ++i) s += x[i] + (float)(p[i] & 0xff);
  out[blockIdx.x * blockDim.x + threadIdx.x] = s;
  if (threadIdx.x == 0) cyc[blockIdx.x] = t1 - t0;
}
template <int MODE> void run(const char* name, double ops_per_iter_per_thread, int threads) {
  float* out; long long* cyc; cudaMalloc(&out, 148 * 1024 * 4); cudaMalloc(&cyc, 148 * 8);
  k<MODE><<<148, threads>>>(out, cyc, 0.999f, 0.001f); cudaDeviceSynchronize();
  k<MODE><<<148, threads>>>(out, cyc, 0.999f, 0.001f); cudaDeviceSynchronize();
  long long h[148]; cudaMemcpy(h, cyc, sizeof(h), cudaMemcpyDeviceToHost);
  double c = 0; for (int i = 0; i < 148; ++i) c += h[i]; c /= 148;
  printf("%-28s threads/SM %4d: %7.2f lane-ops/clk/SM (%.0f cycles)\n", name, threads, ops_per_iter_per_thread * ITERS * threads / c, c);
  cudaFree(out); cudaFree(cyc);
}

// ---- mixes: NA operations of kind KA interleaved with NB of kind KB, all on independent registers ----
// kinds: 0 FFMA, 1 FFMA2, 2 LOP3, 3 EX2, 5 SHFL, 6 IMAD
template <int K> __device__ __forceinline__ void op(float& x, unsigned long long& p, int& q, float& e, float a, float b,
                                                    unsigned long long aa, unsigned long long bb, int ia) {
  if (K == 0) x = fmaf(x, a, b);
  if (K == 1) asm volatile("fma.rn.f32x2 %0, %0, %1, %2;" : "+l"(p) : "l"(aa), "l"(bb));
  if (K == 2) asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(q) : "r"(ia), "r"(ia));
  if (K == 3) asm volatile("ex2.approx.ftz.f32 %0, %0;" : "+f"(e));
  if (K == 5) e = __shfl_xor_sync(0xffffffffu, e, 1);
  if (K == 6) asm volatile("mad.lo.s32 %0, %0, %1, %2;" : "+r"(q) : "r"(ia), "r"(ia));
}
template <int KA, int NA, int KB, int NB>
__global__ void mixk(float* out, long long* cyc, float a, float b, int ia) {
  float x[16]; unsigned long long p[16]; int q[16]; float e[16];
  for (int i = 0; i < 16; ++i) { x[i] = threadIdx.x * 0.001f + i; q[i] = threadIdx.x + i; e[i] = -0.001f * threadIdx.x - i;
    p[i] = (unsigned long long)__float_as_uint(x[i]) | ((unsigned long long)__float_as_uint(x[i] + 1.f) << 32); }
  unsigned long long aa = (unsigned long long)__float_as_uint(a) | ((unsigned long long)__float_as_uint(a) << 32);
  unsigned long long bb = (unsigned long long)__float_as_uint(b) | ((unsigned long long)__float_as_uint(b) << 32);
  __syncthreads();
  long long t0 = clock64();
  for (int it = 0; it < ITERS; ++it) {
    constexpr int N = NA > NB ? NA : NB;
#pragma unroll
    for (int i = 0; i < N; ++i) {
      if (i < NA) op<KA>(x[i & 15], p[i & 15], q[i & 15], e[i & 15], a, b, aa, bb, ia);
      if (i < NB) op<KB>(x[(i + 8) & 15], p[(i + 8) & 15], q[(i + 8) & 15], e[(i + 8) & 15], a, b, aa, bb, ia);
    }
  }
  long long t1 = clock64();
  float s = 0; for (int i = 0; i < 16; ++i) s += x[i] + (float)(p[i] & 0xff) + q[i] + e[i];
  out[blockIdx.x * blockDim.x + threadIdx.x] = s;
  if (threadIdx.x == 0) cyc[blockIdx.x] = t1 - t0;
}
template <int KA, int NA, int KB, int NB> void runmix(const char* name, int threads) {
  float* out; long long* cyc; cudaMalloc(&out, 148 * 1024 * 4); cudaMalloc(&cyc, 148 * 8);
  for (int r = 0; r < 2; ++r) { mixk<KA, NA, KB, NB><<<148, threads>>>(out, cyc, 0.999f, 0.001f, 12345); cudaDeviceSynchronize(); }
  long long h[148]; cudaMemcpy(h, cyc, sizeof(h), cudaMemcpyDeviceToHost);
  double c = 0; for (int i = 0; i < 148; ++i) c += h[i]; c /= 148;
  printf("%-28s threads/SM %4d: %6.2f cycles per warp and group on one scheduler\n", name, threads, c / ITERS / (threads / 128.0));
  cudaFree(out); cudaFree(cyc);
}
int main() {
  for (int th : {128, 256, 512, 1024}) {
    run<0>("FFMA", 8, th);
    run<1>("FFMA2 (counted as 2 fma)", 16, th);
    run<2>("MUFU.EX2", 8, th);
    run<3>("SHFL", 8, th);
    run<5>("LDS.32", 8, th);
    run<4>("FFMA + 1/8 EX2 (fma count)", 8, th);
    run<9>("FFMA + 1/4 EX2 indep (fma)", 8, th);
    run<6>("FFMA2 + 1/4 EX2 (fma count)", 16, th);
    run<7>("FFMA2 + 1/4 SHFL (fma count)", 16, th);
    run<8>("FFMA + 1/4 SHFL (fma count)", 8, th);
  }
  for (int th : {384, 1024}) {
    runmix<0, 8, 0, 8>("16 FFMA", th);
    runmix<1, 8, 1, 8>("16 FFMA2", th);
    runmix<2, 8, 2, 8>("16 LOP3", th);
    runmix<6, 8, 6, 8>("16 IMAD", th);
    runmix<3, 4, 3, 4>("8 EX2", th);
    runmix<0, 16, 3, 2>("16 FFMA + 2 EX2", th);
    runmix<0, 16, 3, 4>("16 FFMA + 4 EX2", th);
    runmix<1, 16, 3, 4>("16 FFMA2 + 4 EX2", th);
    runmix<1, 16, 5, 8>("16 FFMA2 + 8 SHFL", th);
    runmix<0, 16, 2, 16>("16 FFMA + 16 LOP3", th);
    runmix<1, 16, 2, 16>("16 FFMA2 + 16 LOP3", th);
    runmix<0, 16, 6, 16>("16 FFMA + 16 IMAD", th);
    runmix<1, 16, 6, 16>("16 FFMA2 + 16 IMAD", th);
    runmix<1, 16, 0, 16>("16 FFMA2 + 16 FFMA", th);
  }
  return 0;
}
