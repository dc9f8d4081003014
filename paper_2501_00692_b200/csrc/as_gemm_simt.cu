// FP32-pipe tiled GEMM with generic operand strides.  This is the contraction path for fp32 I/O,
// where the 1e-4 parity bar rules out TF32/bf16 tensor-core inputs, and the general fallback shape
// handler for the small [16 x P] blocks.
#include "as_internal.cuh"

namespace as {

namespace {
constexpr int BM = 64, BN = 64, BK = 16, TM = 4, TN = 4, NT = 256;

__device__ __forceinline__ float ld_elem(const void* p, int bf16, int64_t idx) {
  return bf16 ? __bfloat162float(__ldg(reinterpret_cast<const __nv_bfloat16*>(p) + idx))
              : __ldg(reinterpret_cast<const float*>(p) + idx);
}

__device__ __forceinline__ float softplus_f(float u) {
  return fmaxf(u, 0.f) + log1pf(expf(-fabsf(u)));
}

__global__ void __launch_bounds__(NT) gemm_simt_kernel(GemmArgs g) {
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int tid = threadIdx.x;
  const int64_t m0 = (int64_t)blockIdx.x * BM;
  const int n0 = blockIdx.y * BN;
  // K range of this split
  const int64_t kchunk = ((g.K + g.splitk - 1) / g.splitk + BK - 1) / BK * BK;
  const int64_t kbeg = (int64_t)blockIdx.z * kchunk;
  const int64_t kend = min(g.K, kbeg + kchunk);
  if (kbeg >= kend) return;

  const int tx = tid % 16, ty = tid / 16;  // thread's 4x4 micro-tile: rows ty*4.., cols tx*4..
  float acc[TM][TN];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

  const bool a_kmajor = (g.a_sk == 1);
  const bool b_kmajor = (g.b_sk == 1);

  for (int64_t k0 = kbeg; k0 < kend; k0 += BK) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int mm, kk;
      if (a_kmajor) { kk = tid % BK; mm = tid / BK + i * (NT / BK); }
      else { mm = tid % BM; kk = tid / BM + i * (NT / BM); }
      int64_t m = m0 + mm, k = k0 + kk;
      As[kk][mm] = (m < g.M && k < kend) ? ld_elem(g.A, g.a_bf16, m * g.a_sm + k * g.a_sk) : 0.f;
      int nn;
      if (b_kmajor) { kk = tid % BK; nn = tid / BK + i * (NT / BK); }
      else { nn = tid % BN; kk = tid / BN + i * (NT / BN); }
      int64_t n = n0 + nn;
      k = k0 + kk;
      Bs[kk][nn] = (n < g.N && k < kend) ? ld_elem(g.Bm, g.b_bf16, n * g.b_sn + k * g.b_sk) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[TM], b[TN];
      const float4 av = *reinterpret_cast<const float4*>(&As[kk][ty * TM]);
      const float4 bv = *reinterpret_cast<const float4*>(&Bs[kk][tx * TN]);
      a[0] = av.x; a[1] = av.y; a[2] = av.z; a[3] = av.w;
      b[0] = bv.x; b[1] = bv.y; b[2] = bv.z; b[3] = bv.w;
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }

#pragma unroll
  for (int i = 0; i < TM; ++i) {
    const int64_t m = m0 + ty * TM + i;
    if (m >= g.M) continue;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      const int n = n0 + tx * TN + j;
      if (n >= g.N) continue;
      float* dst = g.C + m * g.ldc + g.coff + n;
      float v = acc[i][j];
      switch (g.epi) {
        case EPI_STORE: *dst = v; break;
        case EPI_SOFTPLUS_BIAS: *dst = softplus_f(v + __ldg(g.bias + n)); break;
        case EPI_ATOMIC: atomicAdd(dst, v); break;
        default: *dst += v; break;
      }
    }
  }
}
}  // namespace

int launch_gemm_simt(const GemmArgs& g, cudaStream_t st) {
  if (g.M <= 0 || g.N <= 0 || g.K <= 0) return 0;
  GemmArgs a = g;
  if (a.splitk < 1) a.splitk = 1;
  dim3 grid((unsigned)((a.M + BM - 1) / BM), (unsigned)((a.N + BN - 1) / BN), (unsigned)a.splitk);
  gemm_simt_kernel<<<grid, NT, 0, st>>>(a);
  count_launch();
  return (int)cudaGetLastError();
}

}  // namespace as
