// Matmul form of the forward scan for the scalar structure (one decay rate per channel, Table 1 "Scalar SSM"), bf16 I/O.
//
// With a_p the rate of channel p, cs_t[p] the running sum of Delta inside a chunk of 64 tokens and v_j = Delta_j x_j,
//   y_t[p] = sum_{j<=t} (C_t . B_j) exp(a_p (cs_t - cs_j)) v_j[p]  +  exp(a_p cs_t) (C_t . h_start[p, :])
// The decay factorises around a reference point inside the chunk (its middle token m):
//   exp(a_p (cs_t - cs_j)) = E[t,p] F[j,p],   E = exp(a_p (cs_t - cs_m)),  F = exp(-a_p (cs_j - cs_m)),
// so that one 64 x 64 matrix G = tril(C B^T), shared by all channels, multiplies V[j,p] = F[j,p] v_j[p]:
//   y = E o ( G V + C S'^T ),   S'[p,:] = exp(a_p cs_m) h_start[p,:]            (two tcgen05 GEMMs into one accumulator)
//   h_end[p,:] = exp(a_p (cs_end - cs_m)) ( S'[p,:] + sum_j V[j,p] B_j )        (a third, into a TMEM-resident state)
// One CTA = 128 channels x one segment, one thread (and one TMEM lane) per channel; chunks are walked in order and the
// state stays in tensor memory in fp32 (only the GEMM operands are rounded to bf16).  The exponents are bounded by
// |a_p| times half a chunk's Delta sum; a channel whose bound exceeds 2^+-96 in a chunk takes the plain recurrence for
// that chunk (computed by its own thread) and contributes zeros to the GEMMs.
// Every mbarrier wait is bounded; on a timeout the kernel records AS_ERR_TIMEOUT, frees its TMEM and returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include "as_internal.cuh"

namespace as {
namespace {

constexpr int TCK = 64;    // tokens per chunk
constexpr int MCH = 128;   // channels per CTA
constexpr int MT = 128;    // threads per CTA
// shared-memory map (bytes); every GEMM operand is a K-major tile with 128-byte rows under the 128-byte swizzle
constexpr int SM_E = 0;                  // 4 boxes x [64 tokens][32 channels] fp32: Delta as loaded by TMA, then E in place
constexpr int SM_X = SM_E + 32768;       // x tile [64][128] bf16; reused for the masked G [64 (+64 unused)][64] bf16
constexpr int SM_V = SM_X + 16384;       // V   [128 channels][64 tokens] bf16
constexpr int SM_SP = SM_V + 16384;      // S'  [128 channels][16 states] bf16 (first 32 bytes of each 128-byte row)
constexpr int SM_CT = SM_SP + 16384;     // C   [64 tokens][16 states] bf16 (first 32 bytes of each row)
constexpr int SM_BT = SM_CT + 8192;      // B   [64 tokens][16 states] bf16
constexpr int SM_BTT = SM_BT + 8192;     // B^T [16 states][64 tokens] bf16
constexpr int SM_BC = SM_BTT + 2048;     // staged [B | C] rows, fp32 [64][32]
constexpr int SM_TOTAL = SM_BC + 8192;
constexpr int SMEM_DYN = SM_TOTAL + 1024;   // + alignment slack
// tensor-memory columns
constexpr int TM_Y = 0, TM_G = 128, TM_S = 192, TM_ALLOC = 256;
constexpr float EXP_LIMIT = 96.f;        // largest |log2| of a factor that goes into a bf16 operand
constexpr uint32_t WAIT_LIMIT = 1u << 22;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  const uint32_t addr = smem_u32(bar);
  for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
    if (ok) return true;
  }
  return false;
}
__device__ __forceinline__ void tma_2d(void* dst, const CUtensorMap* tm, int c0, int64_t c1, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(dst)), "l"(tm), "r"(c0), "r"((int)c1), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void bulk_1d(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// K-major operand, 128-byte rows, 128-byte swizzle, groups of 8 rows 1024 bytes apart (descriptor version 1)
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)((16u >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((1024u >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// instruction descriptor: fp32 accumulator, bf16 A and B, both K-major, M = 128, N = n
__device__ __forceinline__ uint32_t idesc_n(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// byte offset of 16-byte piece q of row r in a tile of 128-byte rows under the 128-byte swizzle
__device__ __forceinline__ uint32_t sw128(int r, int q) { return (uint32_t)(r * 128 + ((q ^ (r & 7)) << 4)); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&t);
}

// float offset of (channel pc of the tile, state n) inside a tile block of the scan kernels (thread-major layout:
// 16-byte piece q of scan thread tid at q*128 + tid; scan thread 2k + half owns states 8 half .. 8 half + 7 of channels
// 2k, 2k+1 as units u = 4 ch + m -> states 8 half + 2m, + 1)
__device__ __forceinline__ int tile_block_offset(int pc, int n) {
  const int tid_scan = 2 * (pc >> 1) + (n >> 3);
  const int u = (pc & 1) * 4 + ((n & 7) >> 1);
  return ((u >> 1) * 128 + tid_scan) * 4 + (u & 1) * 2 + (n & 1);
}

__global__ void __launch_bounds__(MT, 2)
scalar_y_mm_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmD, Plan pl,
                   const float* __restrict__ A_log, char* __restrict__ ws, __nv_bfloat16* __restrict__ y) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_ld, bar_g, bar_y;
  __shared__ uint32_t tmem_base_s;
  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);

  const int tile = blockIdx.x, s = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5;
  const int P = pl.P;
  const int64_t T = pl.T;
  const int64_t t0 = (int64_t)s * pl.L, t1 = min(T, t0 + pl.L);
  const int nchunk = (int)((t1 - t0 + TCK - 1) / TCK);
  const int64_t BT = (int64_t)pl.B * T;
  const float* bc = reinterpret_cast<const float*>(ws + pl.off_bc);
  int* status = reinterpret_cast<int*>(ws + pl.off_status);
  const int pch = tile * MCH + tid;                                  // this thread's channel
  const float a2 = -__expf(__ldg(A_log + (int64_t)(b / pl.Bg) * P + pch)) * LOG2E;   // a_p log2(e)

  if (tid == 0) {
    mbar_init(&bar_ld, 1);
    mbar_init(&bar_g, 1);
    mbar_init(&bar_y, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "n"(TM_ALLOC)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tm = tmem_base_s;
  const uint32_t tm_lane = tm + ((uint32_t)(32 * warp) << 16);   // this warp's lanes, column 0

  // true state at the segment start (from the carry pass), this channel's 16 states
  float S[NS];
  {
    const float* hst = reinterpret_cast<const float*>(ws + pl.off_hstart) +
                       (((int64_t)b * pl.S + s) * pl.tiles + tile) * TILE_FLOATS;
#pragma unroll
    for (int n = 0; n < NS; ++n) S[n] = __ldg(hst + tile_block_offset(tid, n));
  }
  float fprev = 1.f;   // exp(a (cs_end - cs_m)) of the previous chunk: brings the TMEM state to that chunk's end
  const uint32_t sm_b = smem_u32(sm);
  bool failed = false;

  for (int c = 0; c < nchunk; ++c) {
    const int64_t tc = t0 + (int64_t)c * TCK;
    const int nt = (int)min((int64_t)TCK, t1 - tc);
    const int64_t row0 = (int64_t)b * T + tc;
    if (tid == 0) {
      const uint32_t bc_bytes = (uint32_t)min((int64_t)TCK, BT - row0) * NBC * 4;
      mbar_expect_tx(&bar_ld, TCK * MCH * 2 + TCK * MCH * 4 + bc_bytes);
      tma_2d(sm + SM_X, &tmX, tile * MCH, row0, &bar_ld);
#pragma unroll
      for (int q = 0; q < 4; ++q) tma_2d(sm + SM_E + q * 8192, &tmD, tile * MCH + 32 * q, row0, &bar_ld);
      bulk_1d(sm + SM_BC, bc + row0 * NBC, bc_bytes, &bar_ld);
    }
    bool ok = mbar_wait(&bar_ld, c & 1);

    // ---- [B | C] rows -> bf16 operand tiles (rows past the segment end as zeros) ----
    if (ok) {
      const int t = tid & 63, which = tid >> 6;   // threads 0..63: B rows, 64..127: C rows
      const float4* src = reinterpret_cast<const float4*>(sm + SM_BC + t * (NBC * 4) + which * (NS * 4));
      float v[NS];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        float4 f = src[q];
        if (t >= nt) f = make_float4(0.f, 0.f, 0.f, 0.f);
        v[4 * q] = f.x; v[4 * q + 1] = f.y; v[4 * q + 2] = f.z; v[4 * q + 3] = f.w;
      }
      uint8_t* dst = sm + (which ? SM_CT : SM_BT);
      *reinterpret_cast<uint4*>(dst + sw128(t, 0)) =
          make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
      *reinterpret_cast<uint4*>(dst + sw128(t, 1)) =
          make_uint4(pack_bf16(v[8], v[9]), pack_bf16(v[10], v[11]), pack_bf16(v[12], v[13]), pack_bf16(v[14], v[15]));
      if (which == 0) {
#pragma unroll
        for (int n = 0; n < NS; ++n)
          *reinterpret_cast<__nv_bfloat16*>(sm + SM_BTT + sw128(n, t >> 3) + (t & 7) * 2) = __float2bfloat16_rn(v[n]);
      }
      fence_async_smem();
    }
    if (__syncthreads_or(ok ? 0 : 1)) { failed = true; break; }
    if (tid == 0) {   // G = C B^T  (64 x 64 useful, issued as 128 x 64: rows 64.. of the A tile are never looked at)
      tc_fence_after();
      umma_bf16(tm + TM_G, make_desc(sm_b + SM_CT), make_desc(sm_b + SM_BT), idesc_n(64), 0u);
      umma_commit(&bar_g);
    }

    // ---- this channel: running Delta sum, E in place of Delta, V = F Delta x ----
    const int bx = tid >> 5, pc = tid & 31, ch4 = pc >> 2, e4 = pc & 3;
    uint8_t* ecol = sm + SM_E + bx * 8192 + e4 * 4;   // element (t, this channel) at + t*128 + ((ch4 ^ (t & 7)) << 4)
    float cs_m = 0.f, cs_end = 0.f;
#pragma unroll 8
    for (int t = 0; t < TCK; ++t) {
      const float d = t < nt ? *reinterpret_cast<const float*>(ecol + t * 128 + ((ch4 ^ (t & 7)) << 4)) : 0.f;
      cs_end += d;
      if (t == TCK / 2 - 1) cs_m = cs_end;
    }
    // exponents stay inside +-EXP_LIMIT on both sides of the reference point?
    const bool slow = fmaxf(cs_m, cs_end - cs_m) * -a2 > EXP_LIMIT;
    {
      const __nv_bfloat16* xcol = reinterpret_cast<const __nv_bfloat16*>(sm + SM_X) + tid;
      float cs = 0.f;
      uint32_t vp[4];
      float vprev = 0.f;
#pragma unroll 8
      for (int t = 0; t < TCK; ++t) {
        float* ep = reinterpret_cast<float*>(ecol + t * 128 + ((ch4 ^ (t & 7)) << 4));
        const float d = t < nt ? *ep : 0.f;
        const float xv = __bfloat162float(xcol[t * MCH]);
        cs += d;
        const float ex = a2 * (cs - cs_m);
        const float E = slow ? 0.f : ex2_approx(ex);
        const float F = ex2_approx(-ex);
        *ep = E;
        const float v = (slow || t >= nt) ? 0.f : F * d * xv;
        if (t & 1) vp[(t & 7) >> 1] = pack_bf16(vprev, v);
        else vprev = v;
        if ((t & 7) == 7) *reinterpret_cast<uint4*>(sm + SM_V + sw128(tid, t >> 3)) = make_uint4(vp[0], vp[1], vp[2], vp[3]);
      }
    }
    // ---- state: bring it to this chunk's reference point, hand it to the GEMMs ----
    if (c > 0) {
      uint32_t r[16];
      tc_fence_after();
      tmem_ld16(tm_lane + TM_S, r);
#pragma unroll
      for (int n = 0; n < NS; ++n) S[n] = __uint_as_float(r[n]) * fprev;   // state at the end of the previous chunk
    }
    if (slow) {
      // plain recurrence for this channel and chunk; y is parked in the E tile and stored by this thread after the
      // epilogue (whose product for this channel is an exact zero)
      const __nv_bfloat16* xcol = reinterpret_cast<const __nv_bfloat16*>(sm + SM_X) + tid;
      for (int t = 0; t < nt; ++t) {
        float* ep = reinterpret_cast<float*>(ecol + t * 128 + ((ch4 ^ (t & 7)) << 4));
        // Delta was overwritten by E = 0 above: recover it from the staged rows is impossible, so keep it simple:
        // this branch re-reads Delta from global memory
        const float d = __ldg(reinterpret_cast<const float*>(ws + pl.off_delta) + (row0 + t) * P + pch);
        const float xv = __bfloat162float(xcol[t * MCH]);
        const float ab = ex2_approx(a2 * d), dx = d * xv;
        const float* brow = reinterpret_cast<const float*>(sm + SM_BC) + t * NBC;
        float acc = 0.f;
#pragma unroll
        for (int n = 0; n < NS; ++n) {
          S[n] = fmaf(ab, S[n], dx * brow[n]);
          acc = fmaf(brow[NS + n], S[n], acc);
        }
        *ep = acc;
      }
    }
    {
      const float f = slow ? 1.f : ex2_approx(a2 * cs_m);
      uint32_t r[16];
      float sp[NS];
#pragma unroll
      for (int n = 0; n < NS; ++n) { sp[n] = S[n] * f; r[n] = __float_as_uint(sp[n]); }
      tmem_st16(tm_lane + TM_S, r);
      // a slow channel keeps its (already advanced) state in TMEM untouched by the GEMMs: zero operand rows
      if (slow) {
#pragma unroll
        for (int n = 0; n < NS; ++n) sp[n] = 0.f;
      }
      *reinterpret_cast<uint4*>(sm + SM_SP + sw128(tid, 0)) =
          make_uint4(pack_bf16(sp[0], sp[1]), pack_bf16(sp[2], sp[3]), pack_bf16(sp[4], sp[5]), pack_bf16(sp[6], sp[7]));
      *reinterpret_cast<uint4*>(sm + SM_SP + sw128(tid, 1)) =
          make_uint4(pack_bf16(sp[8], sp[9]), pack_bf16(sp[10], sp[11]), pack_bf16(sp[12], sp[13]), pack_bf16(sp[14], sp[15]));
      fprev = slow ? 1.f : ex2_approx(a2 * (cs_end - cs_m));
    }
    fence_async_smem();
    tc_fence_before();
    const int any_slow = __syncthreads_or(slow ? 1 : 0);   // x tile fully consumed: its space now takes the masked G

    // ---- G (TMEM) -> lower triangle -> bf16 A operand; rows = tokens = lanes 0..63 ----
    if (warp < 2) {
      ok = mbar_wait(&bar_g, c & 1);
      if (ok) {
        tc_fence_after();
        const int t = tid;
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          uint32_t r[32];
          tmem_ld32(tm_lane + TM_G + 32 * hf, r);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            uint32_t w4[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int j = 32 * hf + 8 * q + 2 * i;
              const float lo = j <= t ? __uint_as_float(r[8 * q + 2 * i]) : 0.f;
              const float hi = j + 1 <= t ? __uint_as_float(r[8 * q + 2 * i + 1]) : 0.f;
              w4[i] = pack_bf16(lo, hi);
            }
            *reinterpret_cast<uint4*>(sm + SM_X + sw128(t, 4 * hf + q)) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
          }
        }
        fence_async_smem();
      }
    }
    tc_fence_before();
    if (__syncthreads_or(ok ? 0 : 1)) { failed = true; break; }
    if (tid == 0) {
      tc_fence_after();
#pragma unroll
      for (int k = 0; k < 4; ++k)   // Y = tril(G) V
        umma_bf16(tm + TM_Y, make_desc(sm_b + SM_X + 32 * k), make_desc(sm_b + SM_V + 32 * k), idesc_n(128), k > 0 ? 1u : 0u);
      umma_bf16(tm + TM_Y, make_desc(sm_b + SM_CT), make_desc(sm_b + SM_SP), idesc_n(128), 1u);   // + C S'^T
#pragma unroll
      for (int k = 0; k < 4; ++k)   // S += V^T B   (rows = channels)
        umma_bf16(tm + TM_S, make_desc(sm_b + SM_V + 32 * k), make_desc(sm_b + SM_BTT + 32 * k), idesc_n(16), 1u);
      umma_commit(&bar_y);
    }
    ok = mbar_wait(&bar_y, c & 1);
    // ---- epilogue: y[t, :] = E[t, :] o Y[t, :] ----
    if (warp < 2 && ok) {
      tc_fence_after();
      const int t = tid;
      __nv_bfloat16* yrow = y + (row0 + t) * P + tile * MCH;
#pragma unroll 1
      for (int cb = 0; cb < 4; ++cb) {
        uint32_t r[32];
        tmem_ld32(tm_lane + TM_Y + 32 * cb, r);
        uint32_t o[16];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const float4 e = *reinterpret_cast<const float4*>(sm + SM_E + cb * 8192 + sw128(t, q));
          o[2 * q] = pack_bf16(__uint_as_float(r[4 * q]) * e.x, __uint_as_float(r[4 * q + 1]) * e.y);
          o[2 * q + 1] = pack_bf16(__uint_as_float(r[4 * q + 2]) * e.z, __uint_as_float(r[4 * q + 3]) * e.w);
        }
        if (t < nt) {
#pragma unroll
          for (int q = 0; q < 4; ++q)
            *reinterpret_cast<uint4*>(yrow + 32 * cb + 8 * q) = make_uint4(o[4 * q], o[4 * q + 1], o[4 * q + 2], o[4 * q + 3]);
        }
      }
    }
    tc_fence_before();
    if (__syncthreads_or(ok ? 0 : 1)) { failed = true; break; }
    if (any_slow) {
      if (slow) {
        for (int t = 0; t < nt; ++t)
          y[(row0 + t) * P + pch] =
              __float2bfloat16_rn(*reinterpret_cast<const float*>(ecol + t * 128 + ((ch4 ^ (t & 7)) << 4)));
      }
      __syncthreads();
    }
  }
  if (failed && tid == 0) {
    mbar_wait(&bar_ld, 0);   // copies already issued still target this CTA's shared memory: one more bounded wait
    atomicExch(status, AS_ERR_TIMEOUT);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base_s), "n"(TM_ALLOC) : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}
// [rows = batches * T, cols = P] row-major, boxes of `bw` channels x TCK tokens
int chunk_map(CUtensorMap* tm, const void* base, const Plan& pl, int elem_bytes, bool is_bf16, int bw, bool swz) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return 1;
  cuuint64_t dims[2] = {(cuuint64_t)pl.P, (cuuint64_t)pl.B * (cuuint64_t)pl.T};
  cuuint64_t strides[1] = {(cuuint64_t)pl.P * elem_bytes};
  cuuint32_t box[2] = {(cuuint32_t)bw, (cuuint32_t)TCK};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(tm, is_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                   const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   swz ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : 1;
}

}  // namespace

bool forward_y_mm_applies(const Plan& pl) { return pl.mm && pl.scalar && pl.io == AS_BF16 && pl.P % MCH == 0; }

int launch_forward_y_mm(const Plan& pl, const ScanPtrs& sp, void* y, cudaStream_t st) {
  CUtensorMap mx, md;
  if (chunk_map(&mx, sp.x, pl, 2, true, MCH, false)) return 1;
  if (chunk_map(&md, sp.ws + pl.off_delta, pl, 4, false, 32, true)) return 1;
  auto kern = scalar_y_mm_kernel;
  static bool done[AS_MAX_DEVICES] = {};
  if (ensure_dynamic_smem(kern, SMEM_DYN, done)) return 1;
  kern<<<dim3(pl.P / MCH, pl.S, pl.B), MT, SMEM_DYN, st>>>(mx, md, pl, sp.A_log, sp.ws, (__nv_bfloat16*)y);
  count_launch();
  return (int)cudaGetLastError();
}

}  // namespace as
