// Residual-stack glue: gain-free RMSNorm over d_model (forward and VJP) and the residual add.
// One warp per token; fp32 arithmetic; I/O in the activation dtype.
#include "as_internal.cuh"

namespace as {
namespace {
__device__ __forceinline__ float wsum(float v) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

template <typename IO>
__global__ void rmsnorm_fwd_kernel(int64_t rows, int P, const IO* __restrict__ y, IO* __restrict__ yhat, float eps) {
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  const IO* yr = y + row * P;
  float ss = 0.f;
  for (int i = lane; i < P; i += 32) { const float v = ld_io<IO>(yr + i); ss = fmaf(v, v, ss); }
  ss = wsum(ss);
  const float rinv = 1.f / sqrtf(ss / (float)P + eps);
  for (int i = lane; i < P; i += 32) st_io<IO>(yhat + row * P + i, ld_io<IO>(yr + i) * rinv);
}

template <typename IO>
__global__ void rmsnorm_bwd_add_kernel(int64_t rows, int P, const IO* __restrict__ y, const IO* __restrict__ dyhat,
                                       IO* __restrict__ G, float eps) {
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  const IO* yr = y + row * P;
  const IO* dr = dyhat + row * P;
  float ss = 0.f, dot = 0.f;
  for (int i = lane; i < P; i += 32) {
    const float v = ld_io<IO>(yr + i);
    ss = fmaf(v, v, ss);
    dot = fmaf(v, ld_io<IO>(dr + i), dot);
  }
  ss = wsum(ss); dot = wsum(dot);
  const float rinv = 1.f / sqrtf(ss / (float)P + eps);
  const float m = dot * rinv / (float)P;  // mean_p(dyhat * yhat)
  for (int i = lane; i < P; i += 32) {
    const float yh = ld_io<IO>(yr + i) * rinv;
    const float gi = (float)G[row * P + i];
    st_io<IO>(G + row * P + i, gi + (ld_io<IO>(dr + i) - yh * m) * rinv);
  }
}

template <typename IO>
__global__ void residual_add_kernel(int64_t n, const IO* __restrict__ a, const IO* __restrict__ b, IO* __restrict__ out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) st_io<IO>(out + i, ld_io<IO>(a + i) + ld_io<IO>(b + i));
}
}  // namespace

int launch_rmsnorm_fwd(const as_shape_t* sh, const void* y, void* yhat, float eps, cudaStream_t st) {
  const int64_t rows = (int64_t)sh->batch * sh->seqlen;
  const unsigned blocks = (unsigned)((rows + 7) / 8);
  if (sh->io == AS_BF16)
    rmsnorm_fwd_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(rows, sh->d_model, (const __nv_bfloat16*)y, (__nv_bfloat16*)yhat, eps);
  else
    rmsnorm_fwd_kernel<float><<<blocks, 256, 0, st>>>(rows, sh->d_model, (const float*)y, (float*)yhat, eps);
  count_launch();
  return (int)cudaGetLastError();
}

int launch_rmsnorm_bwd_add(const as_shape_t* sh, const void* y, const void* dyhat, void* G, float eps, cudaStream_t st) {
  const int64_t rows = (int64_t)sh->batch * sh->seqlen;
  const unsigned blocks = (unsigned)((rows + 7) / 8);
  if (sh->io == AS_BF16)
    rmsnorm_bwd_add_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(rows, sh->d_model, (const __nv_bfloat16*)y,
                                                                 (const __nv_bfloat16*)dyhat, (__nv_bfloat16*)G, eps);
  else
    rmsnorm_bwd_add_kernel<float><<<blocks, 256, 0, st>>>(rows, sh->d_model, (const float*)y, (const float*)dyhat, (float*)G, eps);
  count_launch();
  return (int)cudaGetLastError();
}

int launch_residual_add(const as_shape_t* sh, const void* a, const void* b, void* out, cudaStream_t st) {
  const int64_t n = (int64_t)sh->batch * sh->seqlen * sh->d_model;
  const unsigned blocks = (unsigned)((n + 255) / 256);
  if (sh->io == AS_BF16)
    residual_add_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(n, (const __nv_bfloat16*)a, (const __nv_bfloat16*)b, (__nv_bfloat16*)out);
  else
    residual_add_kernel<float><<<blocks, 256, 0, st>>>(n, (const float*)a, (const float*)b, (float*)out);
  count_launch();
  return (int)cudaGetLastError();
}

// One launch clears every buffer a gradient call accumulates into (status block, the [dB|dC] accumulator and, unless
// the caller accumulates, the five parameter gradients): seven separate memsets cost more in launch gaps than in
// bytes.  All regions are 16-byte aligned and a multiple of 16 bytes long.
namespace {
__global__ void zero_regions_kernel(ZeroList z) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int r = 0; r < z.n; ++r) {
    uint4* p = reinterpret_cast<uint4*>(z.ptr[r]);
    const int64_t n16 = (int64_t)(z.bytes[r] / 16);
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += stride) p[i] = make_uint4(0u, 0u, 0u, 0u);
  }
}
}  // namespace

int launch_zero_regions(const ZeroList& z, cudaStream_t st) {
  size_t total = 0;
  for (int r = 0; r < z.n; ++r) total += z.bytes[r];
  int64_t blocks = (int64_t)((total / 16 + 255) / 256);
  const int64_t cap = (int64_t)sm_count() * 8;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  zero_regions_kernel<<<(unsigned)blocks, 256, 0, st>>>(z);
  count_launch();
  return (int)cudaGetLastError();
}

}  // namespace as
