// Plain backpropagation through time for the same layer: the comparator for the adjoint path.
// Deliberately simple and coded separately from the scan kernels: one thread per channel walks the
// whole sequence, forward once to drop a state snapshot every 64 tokens, then backward chunk by chunk
// (rebuilding the chunk's states in local memory) carrying dL/dh.
#include "as_internal.cuh"

namespace as {
namespace {
constexpr int BCK = 64;

template <typename IO>
__global__ void bptt_forward_kernel(Plan pl, const IO* __restrict__ x, const float* __restrict__ A_log,
                                    char* __restrict__ ws) {
  const int p = blockIdx.x * blockDim.x + threadIdx.x;
  const int b = blockIdx.y;
  if (p >= pl.P) return;
  const float* delta = reinterpret_cast<const float*>(ws + pl.off_delta);
  const float* bc = reinterpret_cast<const float*>(ws + pl.off_bc);
  float* snap = reinterpret_cast<float*>(ws + pl.off_bptt_ckpt);
  const int64_t nck = (pl.T + BCK - 1) / BCK;
  float A[NS], h[NS];
  for (int n = 0; n < NS; ++n) { A[n] = -expf(pl.scalar ? A_log[p] : A_log[(int64_t)p * NS + n]); h[n] = 0.f; }
  for (int64_t t = 0; t < pl.T; ++t) {
    if (t % BCK == 0)
      for (int n = 0; n < NS; ++n) snap[(((int64_t)b * nck + t / BCK) * pl.P + p) * NS + n] = h[n];
    const int64_t row = (int64_t)b * pl.T + t;
    const float d = delta[row * pl.P + p];
    const float xv = ld_io<IO>(x + row * pl.P + p);
    for (int n = 0; n < NS; ++n) h[n] = expf(d * A[n]) * h[n] + d * xv * bc[row * NBC + n];
  }
}

__device__ __forceinline__ float warp_sum(float v) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

template <typename IO>
__global__ void __launch_bounds__(32) bptt_reverse_kernel(Plan pl, const IO* __restrict__ x, const IO* __restrict__ dy,
                                                          const float* __restrict__ A_log, char* __restrict__ ws,
                                                          float* __restrict__ dA_log, float* __restrict__ db_delta) {
  const int pp = blockIdx.x * 32 + threadIdx.x;
  const int b = blockIdx.y;
  const bool active = pp < pl.P;
  const int p = active ? pp : pl.P - 1;
  const float* delta = reinterpret_cast<const float*>(ws + pl.off_delta);
  const float* bc = reinterpret_cast<const float*>(ws + pl.off_bc);
  const float* snap = reinterpret_cast<const float*>(ws + pl.off_bptt_ckpt);
  IO* du = reinterpret_cast<IO*>(ws + pl.off_du);
  IO* dxdir = reinterpret_cast<IO*>(ws + pl.off_dxdir);
  float* dbc = reinterpret_cast<float*>(ws + pl.off_dbc);
  const int64_t nck = (pl.T + BCK - 1) / BCK;
  float A[NS], dh[NS], dA[NS];
  for (int n = 0; n < NS; ++n) { A[n] = -expf(pl.scalar ? A_log[p] : A_log[(int64_t)p * NS + n]); dh[n] = 0.f; dA[n] = 0.f; }
  float dbias = 0.f;
  float H[BCK + 1][NS];  // H[k] = state before token (chunk start + k)
  for (int64_t c = nck - 1; c >= 0; --c) {
    const int64_t tc = c * BCK;
    const int nt = (int)min((int64_t)BCK, pl.T - tc);
    for (int n = 0; n < NS; ++n) H[0][n] = snap[(((int64_t)b * nck + c) * pl.P + p) * NS + n];
    for (int k = 0; k < nt; ++k) {
      const int64_t row = (int64_t)b * pl.T + tc + k;
      const float d = delta[row * pl.P + p];
      const float xv = ld_io<IO>(x + row * pl.P + p);
      for (int n = 0; n < NS; ++n) H[k + 1][n] = expf(d * A[n]) * H[k][n] + d * xv * bc[row * NBC + n];
    }
    for (int k = nt - 1; k >= 0; --k) {
      const int64_t row = (int64_t)b * pl.T + tc + k;
      const float d = delta[row * pl.P + p];
      const float xv = ld_io<IO>(x + row * pl.P + p);
      const float g = active ? ld_io<IO>(dy + row * pl.P + p) : 0.f;
      float d_delta = 0.f, sB = 0.f;
      for (int n = 0; n < NS; ++n) {
        const float Bn = bc[row * NBC + n], Cn = bc[row * NBC + NS + n];
        dh[n] += g * Cn;                                   // y_t = C_t h_t
        const float dCn = warp_sum(g * H[k + 1][n]);
        const float a = expf(d * A[n]);
        const float d_e = dh[n] * H[k][n] * a;             // through abar = exp(delta A)
        d_delta += d_e * A[n];
        dA[n] += d_e * d;
        sB += dh[n] * Bn;                                  // through bbar = delta B x
        const float dBn = warp_sum(dh[n] * d * xv);
        if (threadIdx.x == 0) {
          atomicAdd(dbc + row * NBC + n, dBn);
          atomicAdd(dbc + row * NBC + NS + n, dCn);
        }
        dh[n] *= a;
      }
      d_delta += xv * sB;
      const float sig = 1.f / (1.f + expf(-logf(expm1f(d))));  // u = softplus^{-1}(delta)
      const float duv = d_delta * sig;
      if (active) {
        st_io<IO>(du + row * pl.du_ld + p, duv);
        st_io<IO>(dxdir + row * pl.P + p, d * sB);
        dbias += duv;
      }
    }
  }
  if (active) {
    if (pl.scalar) {
      float tot = 0.f;
      for (int n = 0; n < NS; ++n) tot += dA[n] * A[n];
      atomicAdd(dA_log + p, tot);
    } else {
      for (int n = 0; n < NS; ++n) atomicAdd(dA_log + (int64_t)p * NS + n, dA[n] * A[n]);
    }
    atomicAdd(db_delta + p, dbias);
  }
}
}  // namespace

int launch_bptt(const Plan& pl, const ScanPtrs& sp, float* dA_log, float* db_delta, cudaStream_t st) {
  dim3 gf((pl.P + 63) / 64, pl.B), gr((pl.P + 31) / 32, pl.B);
  if (pl.io == AS_BF16) {
    bptt_forward_kernel<__nv_bfloat16><<<gf, 64, 0, st>>>(pl, (const __nv_bfloat16*)sp.x, sp.A_log, sp.ws);
    bptt_reverse_kernel<__nv_bfloat16><<<gr, 32, 0, st>>>(pl, (const __nv_bfloat16*)sp.x, (const __nv_bfloat16*)sp.dy,
                                                          sp.A_log, sp.ws, dA_log, db_delta);
  } else {
    bptt_forward_kernel<float><<<gf, 64, 0, st>>>(pl, (const float*)sp.x, sp.A_log, sp.ws);
    bptt_reverse_kernel<float><<<gr, 32, 0, st>>>(pl, (const float*)sp.x, (const float*)sp.dy, sp.A_log, sp.ws,
                                                  dA_log, db_delta);
  }
  count_launch(2);
  return (int)cudaGetLastError();
}
}  // namespace as
