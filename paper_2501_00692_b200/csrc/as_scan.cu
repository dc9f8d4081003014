// Time-segmented scan kernels: forward state recurrence, summed adjoint cotangent (reverse
// recurrence with exact window exit) and the per-token vector-Jacobian products.
//
// Thread mapping: one thread per channel p holding the 16 states of that channel in registers;
// a CTA owns CH channels of one batch element over one time segment.  B_t, C_t are warp-uniform.
#include "as_internal.cuh"

namespace as {

// ------------------------------------------------------------------------------------------------
// plan
// ------------------------------------------------------------------------------------------------
static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

int make_plan(const as_shape_t* sh, int64_t tbar, Plan* pl) {
  Plan p{};
  p.B = sh->batch; p.P = sh->d_model; p.T = sh->seqlen; p.io = sh->io;
  p.tc = (sh->io == AS_BF16 && sh->d_model % 32 == 0) ? 1 : 0;
  p.du_ld = p.tc ? p.P + NBC : p.P;
  p.full = tbar >= p.T;
  p.tbar = p.full ? p.T : tbar;
  const int64_t tiles = (int64_t)((p.P + CH - 1) / CH) * p.B;
  const int64_t target = 148 * 2 * 4;
  int64_t s_target = (target + tiles - 1) / tiles;
  int64_t L = (p.T + s_target - 1) / s_target;
  L = (L + CK - 1) / CK * CK;
  if (L < 64) L = 64;
  if (L > 2048) L = 2048;
  p.L = (int)L;
  p.S = (int)((p.T + L - 1) / L);
  p.NC = (p.T + CK - 1) / CK;
  p.m = (int)(p.tbar / L);
  p.r = (int)(p.tbar % L);
  const size_t e = sh->io == AS_BF16 ? 2 : 4;
  const size_t BTP = (size_t)p.B * p.T * p.P;
  const size_t BT = (size_t)p.B * p.T;
  const size_t BSPN = (size_t)p.B * p.S * p.P * NS;
  const size_t BSP = (size_t)p.B * p.S * p.P;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
  p.off_status = take(256);
  p.off_delta = take(BTP * 4);
  p.off_bc = take(BT * NBC * 4);
  p.off_hend = take(BSPN * 4);
  p.off_segd = take(BSP * 4);
  p.off_hstart = take(BSPN * 4);
  p.off_wcat = take((size_t)(p.P + NBC) * p.P * 2);
  p.total_fwd = o;
  p.off_ckpt = take((size_t)p.B * p.NC * p.P * NS * 4);
  p.off_cs = take((size_t)p.B * p.NC * p.P * 4);
  p.off_muloc = take(BSPN * 4);
  p.off_mupart = take(BSPN * 4);
  p.off_partd = take(BSP * 4);
  p.off_firstd = take(BSP * 4);
  p.off_carry = take(BSPN * 4);
  p.off_swin = take(BSP * 8);
  p.off_du = take(BT * (size_t)p.du_ld * e);
  p.off_dxdir = take(BTP * e);
  p.off_dbc = take(BT * NBC * 4);
  p.off_dxacc = take(BTP * 4);
  p.off_bptt_ckpt = take((size_t)p.B * ((p.T + 63) / 64) * p.P * NS * 4);
  p.total_grad = o;
  *pl = p;
  return AS_OK;
}

namespace {

// index of state group q (0..3) of channel p in a [.., 4, P, 4] array, in float4 units
__device__ __forceinline__ int64_t q4(int64_t base_pn, int P, int q, int p) {
  return base_pn / 4 + (int64_t)q * P + p;
}

__device__ __forceinline__ void load16(const float* arr, int64_t base_pn, int P, int p, float (&v)[NS]) {
  const float4* a4 = reinterpret_cast<const float4*>(arr);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    float4 t = __ldg(a4 + q4(base_pn, P, q, p));
    v[4 * q] = t.x; v[4 * q + 1] = t.y; v[4 * q + 2] = t.z; v[4 * q + 3] = t.w;
  }
}
__device__ __forceinline__ void store16(float* arr, int64_t base_pn, int P, int p, const float (&v)[NS]) {
  float4* a4 = reinterpret_cast<float4*>(arr);
#pragma unroll
  for (int q = 0; q < 4; ++q)
    a4[q4(base_pn, P, q, p)] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
}

__device__ __forceinline__ void load_bc(const float* bc_row, float (&Bt)[NS], float (&Ct)[NS]) {
  const float4* r4 = reinterpret_cast<const float4*>(bc_row);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    float4 t = __ldg(r4 + q);
    Bt[4 * q] = t.x; Bt[4 * q + 1] = t.y; Bt[4 * q + 2] = t.z; Bt[4 * q + 3] = t.w;
    float4 c = __ldg(r4 + 4 + q);
    Ct[4 * q] = c.x; Ct[4 * q + 1] = c.y; Ct[4 * q + 2] = c.z; Ct[4 * q + 3] = c.w;
  }
}

// ------------------------------------------------------------------------------------------------
// pre-pass: ascending local scan of one segment from h = 0.
//   writes: state at the start of every CK-token chunk (relative to a zero segment start) and the
//   local exclusive cumulative Delta there; the segment's end state and Delta sum; and, for the
//   reverse recurrence, the segment-local cotangent sum referenced to the segment's first token
//   mu_loc = sum_t gC_t prod_{j=start+1..t} abar_j, plus its snapshot after the first r tokens.
// ------------------------------------------------------------------------------------------------
template <typename IO, bool WITH_MU, bool WITH_CKPT>
__global__ void __launch_bounds__(CH) prepass_kernel(Plan pl, const IO* __restrict__ x, const IO* __restrict__ dy,
                                                     const float* __restrict__ A_log, char* __restrict__ ws) {
  const int p = blockIdx.x * CH + threadIdx.x;
  const int s = blockIdx.y, b = blockIdx.z;
  const int P = pl.P;
  if (p >= P) return;
  const float* delta = reinterpret_cast<const float*>(ws + pl.off_delta);
  const float* bc = reinterpret_cast<const float*>(ws + pl.off_bc);
  float* ckpt = reinterpret_cast<float*>(ws + pl.off_ckpt);
  float* cs = reinterpret_cast<float*>(ws + pl.off_cs);

  float A2[NS], h[NS], Pr[NS], acc[NS], snap[NS];
#pragma unroll
  for (int n = 0; n < NS; ++n) {
    A2[n] = -__expf(__ldg(A_log + (int64_t)p * NS + n)) * LOG2E;
    h[n] = 0.f; Pr[n] = 1.f; acc[n] = 0.f; snap[n] = 0.f;
  }
  const int64_t t0 = (int64_t)s * pl.L;
  const int64_t t1 = min(pl.T, t0 + pl.L);
  float cum = 0.f, partd = 0.f, firstd = 0.f;
  for (int64_t t = t0; t < t1; ++t) {
    const int64_t row = (int64_t)b * pl.T + t;
    if (WITH_CKPT && ((t - t0) % CK) == 0) {
      const int64_t c = (int64_t)b * pl.NC + t / CK;
      store16(ckpt, c * P * NS, P, p, h);
      cs[c * P + p] = cum;
    }
    const float dv = __ldg(delta + row * P + p);
    const float xv = ld_io<IO>(x + row * P + p);
    float Bt[NS], Ct[NS];
    load_bc(bc + row * NBC, Bt, Ct);
    const float dx = dv * xv;
    float gv = 0.f;
    if (WITH_MU) gv = ld_io<IO>(dy + row * P + p);
#pragma unroll
    for (int n = 0; n < NS; ++n) {
      const float a = ex2_approx(dv * A2[n]);
      h[n] = fmaf(a, h[n], dx * Bt[n]);
      if (WITH_MU) {
        if (t > t0) Pr[n] *= a;
        acc[n] = fmaf(gv * Ct[n], Pr[n], acc[n]);
      }
    }
    if (t == t0) firstd = dv;
    cum += dv;
    if (WITH_MU && (t - t0 + 1) == pl.r) {
      partd = cum;
#pragma unroll
      for (int n = 0; n < NS; ++n) snap[n] = acc[n];
    }
  }
  if (WITH_MU && (t1 - t0) < pl.r) {   // ragged last segment shorter than r tokens: the snapshot is the whole segment
    partd = cum;
#pragma unroll
    for (int n = 0; n < NS; ++n) snap[n] = acc[n];
  }
  const int64_t sb = (int64_t)b * pl.S + s;
  store16(reinterpret_cast<float*>(ws + pl.off_hend), sb * P * NS, P, p, h);
  reinterpret_cast<float*>(ws + pl.off_segd)[sb * P + p] = cum;
  if (WITH_MU) {
    store16(reinterpret_cast<float*>(ws + pl.off_muloc), sb * P * NS, P, p, acc);
    store16(reinterpret_cast<float*>(ws + pl.off_mupart), sb * P * NS, P, p, snap);
    reinterpret_cast<float*>(ws + pl.off_partd)[sb * P + p] = partd;
    reinterpret_cast<float*>(ws + pl.off_firstd)[sb * P + p] = firstd;
  }
}

// ------------------------------------------------------------------------------------------------
// carries across segments: one thread per (batch, channel, state).
//   hstart[s]  true state entering segment s.
//   carry[s]   abar_{e+1} * mu_{e+1} for e the last token of segment s, i.e. what the reverse
//              recurrence inside segment s starts from (mu_{e+1} is the window sum that starts on
//              the first token of segment s+1: m whole segments plus r tokens).
//   swin[s]    sum of Delta over the Tbar tokens after e (fp64), for the window-exit factor.
// ------------------------------------------------------------------------------------------------
__global__ void fixup_kernel(Plan pl, const float* __restrict__ A_log, char* __restrict__ ws, int with_mu) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int P = pl.P, S = pl.S;
  if (idx >= (int64_t)pl.B * P * NS) return;
  const int n = (int)(idx % NS);
  const int p = (int)((idx / NS) % P);
  const int b = (int)(idx / ((int64_t)NS * P));
  const float A2 = -__expf(__ldg(A_log + (int64_t)p * NS + n)) * LOG2E;
  auto at = [&](int s) -> int64_t {  // float index of (b,s,p,n) in a [B,S,4,P,4] array
    return (((int64_t)b * S + s) * 4 + n / 4) * (int64_t)P * 4 + (int64_t)p * 4 + (n % 4);
  };
  const float* hend = reinterpret_cast<const float*>(ws + pl.off_hend);
  const float* segd = reinterpret_cast<const float*>(ws + pl.off_segd);
  float* hstart = reinterpret_cast<float*>(ws + pl.off_hstart);
  float hs = 0.f;
  for (int s = 0; s < S; ++s) {
    hstart[at(s)] = hs;
    hs = fmaf(ex2_approx(A2 * segd[((int64_t)b * S + s) * P + p]), hs, hend[at(s)]);
  }
  if (!with_mu) return;
  const float* muloc = reinterpret_cast<const float*>(ws + pl.off_muloc);
  const float* mupart = reinterpret_cast<const float*>(ws + pl.off_mupart);
  const float* partd = reinterpret_cast<const float*>(ws + pl.off_partd);
  const float* firstd = reinterpret_cast<const float*>(ws + pl.off_firstd);
  float* carry = reinterpret_cast<float*>(ws + pl.off_carry);
  double* swin = reinterpret_cast<double*>(ws + pl.off_swin);
  auto sp = [&](int s) -> int64_t { return ((int64_t)b * S + s) * P + p; };
  // decay over (start(s), start(s+1)]
  auto dsh = [&](int s) -> float {
    const float nxt = (s + 1 < S) ? firstd[sp(s + 1)] : 0.f;
    return ex2_approx(A2 * (segd[sp(s)] - firstd[sp(s)] + nxt));
  };
  if (pl.full) {
    float mstart = 0.f;  // mu at the first token of segment s+1
    for (int s = S - 1; s >= 0; --s) {
      carry[at(s)] = (s + 1 < S) ? ex2_approx(A2 * firstd[sp(s + 1)]) * mstart : 0.f;
      mstart = fmaf(dsh(s), mstart, muloc[at(s)]);
    }
  } else {
    for (int s = 0; s < S; ++s) {
      const int s1 = s + 1;
      float val = 0.f;
      if (s1 < S) {
        const int sp_ = s1 + pl.m;  // partial segment
        val = (sp_ < S) ? mupart[at(sp_)] : 0.f;
        for (int k = pl.m - 1; k >= 0; --k) {
          const int sg = s1 + k;
          val = (sg < S) ? fmaf(dsh(sg), val, muloc[at(sg)]) : 0.f;
        }
        val *= ex2_approx(A2 * firstd[sp(s1)]);
      }
      carry[at(s)] = val;
      if (n == 0) {
        double sw = 0.0;
        for (int k = 1; k <= pl.m; ++k)
          if (s + k < S) sw += (double)segd[sp(s + k)];
        if (s + pl.m + 1 < S) sw += (double)partd[sp(s + pl.m + 1)];
        swin[sp(s)] = sw;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// forward output pass: h from the true segment start, y_t = sum_n C_t[n] h_t[n].
// ------------------------------------------------------------------------------------------------
template <typename IO>
__global__ void __launch_bounds__(CH) forward_y_kernel(Plan pl, const IO* __restrict__ x, const float* __restrict__ A_log,
                                                       const char* __restrict__ ws, IO* __restrict__ y) {
  const int p = blockIdx.x * CH + threadIdx.x;
  const int s = blockIdx.y, b = blockIdx.z;
  const int P = pl.P;
  if (p >= P) return;
  const float* delta = reinterpret_cast<const float*>(ws + pl.off_delta);
  const float* bc = reinterpret_cast<const float*>(ws + pl.off_bc);
  float A2[NS], h[NS];
#pragma unroll
  for (int n = 0; n < NS; ++n) A2[n] = -__expf(__ldg(A_log + (int64_t)p * NS + n)) * LOG2E;
  load16(reinterpret_cast<const float*>(ws + pl.off_hstart), ((int64_t)b * pl.S + s) * P * NS, P, p, h);
  const int64_t t0 = (int64_t)s * pl.L;
  const int64_t t1 = min(pl.T, t0 + pl.L);
  for (int64_t t = t0; t < t1; ++t) {
    const int64_t row = (int64_t)b * pl.T + t;
    const float dv = __ldg(delta + row * P + p);
    const float dx = dv * ld_io<IO>(x + row * P + p);
    float Bt[NS], Ct[NS];
    load_bc(bc + row * NBC, Bt, Ct);
    float yv = 0.f;
#pragma unroll
    for (int n = 0; n < NS; ++n) {
      h[n] = fmaf(ex2_approx(dv * A2[n]), h[n], dx * Bt[n]);
      yv = fmaf(Ct[n], h[n], yv);
    }
    st_io<IO>(y + row * P + p, yv);
  }
}

// ------------------------------------------------------------------------------------------------
// main adjoint kernel: descending over the CK-token chunks of one segment.
//   per chunk: rebuild h for the chunk from its checkpoint, then walk it backwards updating the summed
//   cotangent mu_i = gC_i + abar_{i+1} mu_{i+1} - W_i gC_{i+Tbar} and evaluating the per-token VJPs.
// ------------------------------------------------------------------------------------------------
template <typename IO, bool FULL>
__global__ void __launch_bounds__(CH, 2)
adjoint_main_kernel(Plan pl, const IO* __restrict__ x, const IO* __restrict__ dy, const float* __restrict__ A_log,
                    char* __restrict__ ws, float* __restrict__ dA_log, float* __restrict__ db_delta) {
  __shared__ float red[CH / 32][CK][NBC];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int pp = blockIdx.x * CH + tid;
  const int s = blockIdx.y, b = blockIdx.z;
  const int P = pl.P;
  const bool active = pp < P;
  const int p = active ? pp : P - 1;   // inactive threads shadow a valid channel and contribute zeros

  const float* delta = reinterpret_cast<const float*>(ws + pl.off_delta);
  const float* bc = reinterpret_cast<const float*>(ws + pl.off_bc);
  const float* ckpt = reinterpret_cast<const float*>(ws + pl.off_ckpt);
  const float* cs = reinterpret_cast<const float*>(ws + pl.off_cs);
  IO* du = reinterpret_cast<IO*>(ws + pl.off_du);
  IO* dxdir = reinterpret_cast<IO*>(ws + pl.off_dxdir);
  float* dbc = reinterpret_cast<float*>(ws + pl.off_dbc);

  float A2[NS], mu[NS], dAacc[NS];
  const int64_t sb = (int64_t)b * pl.S + s;
#pragma unroll
  for (int n = 0; n < NS; ++n) {
    A2[n] = -__expf(__ldg(A_log + (int64_t)p * NS + n)) * LOG2E;
    dAacc[n] = 0.f;
  }
  load16(reinterpret_cast<const float*>(ws + pl.off_carry), sb * P * NS, P, p, mu);
  if (!active) {
#pragma unroll
    for (int n = 0; n < NS; ++n) mu[n] = 0.f;
  }
  float A2max = A2[0];  // least negative exponent scale: the slowest-decaying state
#pragma unroll
  for (int n = 1; n < NS; ++n) A2max = fmaxf(A2max, A2[n]);
  double sw = 0.0;
  if (!FULL) sw = reinterpret_cast<const double*>(ws + pl.off_swin)[sb * P + p];
  float dbacc = 0.f;

  const int64_t t0 = (int64_t)s * pl.L;
  const int64_t t1 = min(pl.T, t0 + pl.L);
  const int nchunk = (int)((t1 - t0 + CK - 1) / CK);

  for (int c = nchunk - 1; c >= 0; --c) {
    const int64_t tc = t0 + (int64_t)c * CK;
    const int nt = (int)min((int64_t)CK, t1 - tc);
    float xv[CK], dv[CK], gv[CK];
#pragma unroll
    for (int j = 0; j < CK; ++j) {
      const int64_t row = (int64_t)b * pl.T + tc + j;
      const bool ok = j < nt;
      dv[j] = ok ? __ldg(delta + row * P + p) : 0.f;
      xv[j] = ok ? ld_io<IO>(x + row * P + p) : 0.f;
      gv[j] = (ok && active) ? ld_io<IO>(dy + row * P + p) : 0.f;
    }
    // state at the chunk start: local checkpoint + decayed true segment-start state
    float hs[CK][NS];
    float h[NS];
    {
      const int64_t cc = (int64_t)b * pl.NC + tc / CK;
      float hst[NS];
      load16(reinterpret_cast<const float*>(ws + pl.off_hstart), sb * P * NS, P, p, hst);
      load16(ckpt, cc * P * NS, P, p, h);
      const float csum = __ldg(cs + cc * P + p);
#pragma unroll
      for (int n = 0; n < NS; ++n) h[n] = fmaf(ex2_approx(A2[n] * csum), hst[n], h[n]);
    }
    // forward rebuild
#pragma unroll
    for (int j = 0; j < CK; ++j) {
      if (j < nt) {
        const int64_t row = (int64_t)b * pl.T + tc + j;
        const float4* r4 = reinterpret_cast<const float4*>(bc + row * NBC);
        const float dxj = dv[j] * xv[j];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float4 bt = __ldg(r4 + q);
          const float bb[4] = {bt.x, bt.y, bt.z, bt.w};
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const int n = 4 * q + k;
            h[n] = fmaf(ex2_approx(dv[j] * A2[n]), h[n], dxj * bb[k]);
          }
        }
      }
#pragma unroll
      for (int n = 0; n < NS; ++n) hs[j][n] = h[n];
    }
    // reverse walk
#pragma unroll
    for (int j = CK - 1; j >= 0; --j) {
      if (j < nt) {
        const int64_t t = tc + j;
        const int64_t row = (int64_t)b * pl.T + t;
        float Bt[NS], Ct[NS];
        load_bc(bc + row * NBC, Bt, Ct);
        const float g = gv[j], d = dv[j], xx = xv[j];
        const float dxj = d * xx;
        // mu_i += g_i C_i   (mu already carries abar_{i+1} mu_{i+1})
#pragma unroll
        for (int n = 0; n < NS; ++n) mu[n] = fmaf(g, Ct[n], mu[n]);
        if (!FULL) {
          const int64_t t2 = t + pl.tbar;
          if (t2 < pl.T) {
            // exact exit of token t2 from the window: subtract W_i gC_{t2}, W_i = exp(A * sum_{j=i+1..t2} Delta_j)
            const int64_t row2 = (int64_t)b * pl.T + t2;
            const float d2 = __ldg(delta + row2 * P + p);
            const float swf = (float)sw;
            if (__any_sync(0xffffffffu, swf * A2max > -126.f)) {
              const float g2 = active ? ld_io<IO>(dy + row2 * P + p) : 0.f;
              const float4* c4 = reinterpret_cast<const float4*>(bc + row2 * NBC) + 4;
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                const float4 ct = __ldg(c4 + q);
                const float cc2[4] = {ct.x, ct.y, ct.z, ct.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                  const int n = 4 * q + k;
                  mu[n] = fmaf(-ex2_approx(swf * A2[n]), g2 * cc2[k], mu[n]);
                }
              }
            }
            sw += (double)d - (double)d2;   // window of token t-1: (t-1, t-1+Tbar]
          } else {
            // token t+Tbar does not exist: the (clipped) window sum only grows
            sw += (double)d;
          }
        }
        float v[NBC];
        float ssum = 0.f, dsum = 0.f;
#pragma unroll
        for (int n = 0; n < NS; ++n) {
          const float hn = hs[j][n];
          v[n] = mu[n] * dxj;                    // dB partial
          v[NS + n] = g * hn;                    // dC partial
          ssum = fmaf(mu[n], Bt[n], ssum);
          const float hb = fmaf(-dxj, Bt[n], hn);  // abar_i h_{i-1}
          const float q = mu[n] * hb;
          dsum = fmaf(q, A2[n], dsum);
          dAacc[n] = fmaf(q, d, dAacc[n]);
          mu[n] *= ex2_approx(d * A2[n]);        // ready for token i-1
        }
        const float ddelta = fmaf(dsum, LN2, xx * ssum);
        const float sig = -expm1f(-d);           // sigmoid(u) = 1 - exp(-softplus(u))
        const float duv = ddelta * sig;
        dbacc += duv;
        if (active) {
          st_io<IO>(du + row * pl.du_ld + p, duv);
          st_io<IO>(dxdir + row * P + p, d * ssum);
        }
        // transposing warp reduction: afterwards lane l holds the warp total of v[l]
#pragma unroll
        for (int off = 16, cnt = 16; off >= 1; off >>= 1, cnt >>= 1) {
          const bool up = (lane & off) != 0;
#pragma unroll
          for (int k = 0; k < cnt; ++k) {
            const float send = up ? v[k] : v[k + cnt];
            const float keep = up ? v[k + cnt] : v[k];
            v[k] = keep + __shfl_xor_sync(0xffffffffu, send, off);
          }
        }
        red[warp][j][lane] = v[0];
      }
    }
    __syncthreads();
    for (int e = tid; e < nt * NBC; e += CH) {
      const int j = e / NBC, i = e % NBC;
      float sum = 0.f;
#pragma unroll
      for (int w = 0; w < CH / 32; ++w) sum += red[w][j][i];
      atomicAdd(dbc + ((int64_t)b * pl.T + tc + j) * NBC + i, sum);
    }
    __syncthreads();
  }
  if (active) {
#pragma unroll
    for (int n = 0; n < NS; ++n)
      atomicAdd(dA_log + (int64_t)p * NS + n, dAacc[n] * (A2[n] * LN2));
    atomicAdd(db_delta + p, dbacc);
  }
}

template <typename IO>
__global__ void finish_dx_kernel(int64_t n, const float* __restrict__ acc, const IO* __restrict__ dxdir,
                                 IO* __restrict__ dx) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) st_io<IO>(dx + i, acc[i] + ld_io<IO>(dxdir + i));
}

}  // namespace

// ------------------------------------------------------------------------------------------------
// launchers
// ------------------------------------------------------------------------------------------------
static dim3 seg_grid(const Plan& pl) { return dim3((pl.P + CH - 1) / CH, pl.S, pl.B); }

int launch_prepass(const Plan& pl, const ScanPtrs& sp, bool with_mu, bool with_ckpt, cudaStream_t st) {
  const dim3 g = seg_grid(pl);
#define AS_PRE(IO, MU, CKP) \
  prepass_kernel<IO, MU, CKP><<<g, CH, 0, st>>>(pl, (const IO*)sp.x, (const IO*)sp.dy, sp.A_log, sp.ws)
  if (pl.io == AS_BF16) {
    if (with_mu) AS_PRE(__nv_bfloat16, true, true);
    else if (with_ckpt) AS_PRE(__nv_bfloat16, false, true);
    else AS_PRE(__nv_bfloat16, false, false);
  } else {
    if (with_mu) AS_PRE(float, true, true);
    else if (with_ckpt) AS_PRE(float, false, true);
    else AS_PRE(float, false, false);
  }
#undef AS_PRE
  count_launch();
  return (int)cudaGetLastError();
}

int launch_fixup(const Plan& pl, const ScanPtrs& sp, bool with_mu, cudaStream_t st) {
  const int64_t n = (int64_t)pl.B * pl.P * NS;
  fixup_kernel<<<(unsigned)((n + 127) / 128), 128, 0, st>>>(pl, sp.A_log, sp.ws, with_mu ? 1 : 0);
  count_launch();
  return (int)cudaGetLastError();
}

int launch_forward_y(const Plan& pl, const ScanPtrs& sp, void* y, cudaStream_t st) {
  const dim3 g = seg_grid(pl);
  if (pl.io == AS_BF16)
    forward_y_kernel<__nv_bfloat16><<<g, CH, 0, st>>>(pl, (const __nv_bfloat16*)sp.x, sp.A_log, sp.ws, (__nv_bfloat16*)y);
  else
    forward_y_kernel<float><<<g, CH, 0, st>>>(pl, (const float*)sp.x, sp.A_log, sp.ws, (float*)y);
  count_launch();
  return (int)cudaGetLastError();
}

int launch_adjoint_main(const Plan& pl, const ScanPtrs& sp, float* dA_log, float* db_delta, cudaStream_t st) {
  const dim3 g = seg_grid(pl);
#define AS_MAIN(IO, F) \
  adjoint_main_kernel<IO, F><<<g, CH, 0, st>>>(pl, (const IO*)sp.x, (const IO*)sp.dy, sp.A_log, sp.ws, dA_log, db_delta)
  if (pl.io == AS_BF16) { if (pl.full) AS_MAIN(__nv_bfloat16, true); else AS_MAIN(__nv_bfloat16, false); }
  else { if (pl.full) AS_MAIN(float, true); else AS_MAIN(float, false); }
#undef AS_MAIN
  count_launch();
  return (int)cudaGetLastError();
}

int launch_finish_dx(const Plan& pl, const float* dxacc, const void* dxdir, void* dx, cudaStream_t st) {
  const int64_t n = (int64_t)pl.B * pl.T * pl.P;
  const unsigned blocks = (unsigned)((n + 255) / 256);
  if (pl.io == AS_BF16)
    finish_dx_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(n, dxacc, (const __nv_bfloat16*)dxdir, (__nv_bfloat16*)dx);
  else
    finish_dx_kernel<float><<<blocks, 256, 0, st>>>(n, dxacc, (const float*)dxdir, (float*)dx);
  count_launch();
  return (int)cudaGetLastError();
}

}  // namespace as
