// Matmul form of the forward scan for the scalar structure (one decay rate per channel, Table 1 "Scalar SSM"), bf16 I/O.
//
// With a_p the rate of channel p, cs_t[p] the running sum of Delta and v_j = Delta_j x_j,
//   y_t[p] = sum_{j<=t} (C_t . B_j) exp(a_p (cs_t - cs_j)) v_j[p]  +  exp(a_p cs_t) (C_t . h_start[p, :])
// A chunk of 64 tokens is two halves of 32, each with a reference token r_h in its middle, around which the decay
// factorises:  exp(a_p (cs_t - cs_j)) = E[t,p] F[j,p],  E = exp(a_p (cs_t - cs_r)),  F = exp(-a_p (cs_j - cs_r)).
// With G = tril(C B^T) (64 x 64, shared by all channels), V[j,p] = F[j,p] v_j[p] and S' = exp(a_p cs_r0) h_start:
//   t in half 0:  y = E0 o ( G00 V0 + C S'^T )
//   t in half 1:  y = E1 o ( G11 V1 + X o ( G10 V0 + C S'^T ) ),   X[p] = exp(a_p (cs_r1 - cs_r0))
//   h_end = exp(a_p (cs_end - cs_r0)) ( S' + V0^T B0 ) + exp(a_p (cs_end - cs_r1)) V1^T B1
// All products are tcgen05 MMAs with the channels as the M dimension (one TMEM lane and, per half, one thread per channel):
// the per-channel factors E, F, X then never leave their thread, and the state stays in tensor memory in fp32 (only
// the operands are rounded to bf16).  One CTA = 128 channels x one segment, 256 threads: thread (p, h) owns channel p in
// half h of every chunk.  The exponents are bounded by |a_p| times a quarter chunk's Delta sum; a channel whose bound
// exceeds 2^+-96 in a chunk takes the plain recurrence for that chunk in thread (p, 0) (its TMEM lane is then ignored).
// Every mbarrier wait is bounded; on a timeout the kernel records AS_ERR_TIMEOUT, frees its TMEM and returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include "as_internal.cuh"

namespace as {
namespace {

constexpr int TCK = 64;    // tokens per chunk
constexpr int HCK = 32;    // tokens per half (one reference point each)
constexpr int MCH = 128;   // channels per CTA
constexpr int MT = 256;    // threads per CTA: (channel, half)
// shared-memory map (bytes); every GEMM operand is a K-major tile with 128-byte rows under the 128-byte swizzle
constexpr int SM_D = 0;                  // Delta tile [64 tokens][128 channels] fp32 (TMA, no swizzle)
constexpr int SM_X = SM_D + 32768;       // x tile [64][128] bf16; reused as the y tile [64][128] bf16 of the TMA store
constexpr int SM_V = SM_X + 16384;       // V   [128 channels][64 tokens] bf16
constexpr int SM_SP = SM_V + 16384;      // S'  [128 channels][16 states] bf16 (first 32 bytes of each 128-byte row)
constexpr int SM_CT = SM_SP + 16384;     // C   [64 tokens][16 states] bf16 (first 32 bytes of each row)
constexpr int SM_BT = SM_CT + 8192;      // B   [64 tokens][16 states] bf16
constexpr int SM_GM = SM_BT + 8192;      // tril(G) [64 tokens t][64 tokens j] bf16
constexpr int SM_BTT = SM_GM + 8192;     // B^T [16 states][64 tokens] bf16
constexpr int SM_TOTAL = SM_BTT + 2048;
constexpr int SMEM_DYN = SM_TOTAL + 1024;   // + alignment slack
// tensor-memory columns (lane = channel): G [t][j] lives in lanes 0..63 of columns 0..63 until it has been masked
constexpr int TM_D = 0;       // [0,32): half 0, [32,64): half 1 (own half), [64,96): half 1 (what reaches it from half 0 and before)
constexpr int TM_S0 = 96;     // S' + V0^T B0
constexpr int TM_S1 = 112;    // V1^T B1
constexpr int TM_ALLOC = 128;
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

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tm, const void* src, int c0, int64_t c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(tm), "r"(c0), "r"((int)c1), "r"(smem_u32(src)) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// operand descriptor for the rows from `row` on (a multiple of 8) and the K columns from 16*kstep on
__device__ __forceinline__ uint64_t desc_at(uint32_t tile, int row, int kstep) { return make_desc(tile + row * 128 + kstep * 32); }

// YPASS: the y pass from the true segment-start state.  !YPASS: the segment pass of the forward (local scan from a zero
// state: only V and the state products), which writes the segment's end state and Delta sum for the carry kernel.
template <bool YPASS>
__global__ void __launch_bounds__(MT, 2)
scalar_mm_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmD,
                   const __grid_constant__ CUtensorMap tmY, Plan pl, const float* __restrict__ A_log,
                   char* __restrict__ ws, __nv_bfloat16* __restrict__ y) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_ld, bar_g, bar_y;
  __shared__ uint32_t tmem_base_s;
  __shared__ float xch[4][MCH];   // per channel: Delta sums (to the reference, of the whole half) of half 0 and of half 1
  __shared__ int slow_s[2][MCH];  // per channel and half: 1 if the half left the factorised form in this chunk
  uint8_t* sm = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);   // stays a shared-space pointer

  const int tile = blockIdx.x, s = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5;
  const int pc = tid & (MCH - 1), hf = tid >> 7;   // channel of the tile, half of the chunk
  const int P = pl.P;
  const int64_t T = pl.T;
  const int64_t t0 = (int64_t)s * pl.L, t1 = min(T, t0 + pl.L);
  const int nchunk = (int)((t1 - t0 + TCK - 1) / TCK);
  const float* bc = reinterpret_cast<const float*>(ws + pl.off_bc);
  int* status = reinterpret_cast<int*>(ws + pl.off_status);
  const int pch = tile * MCH + pc;                                   // this thread's channel
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
  const uint32_t tm_lane = tm + ((uint32_t)(32 * (warp & 3)) << 16);   // this warp's lane quarter: lane = channel pc

  // thread (p, 0): true state at the segment start (from the carry pass), this channel's 16 states
  float S[NS];
#pragma unroll
  for (int n = 0; n < NS; ++n) S[n] = 0.f;
  if (YPASS && hf == 0) {
    const float* hst = reinterpret_cast<const float*>(ws + pl.off_hstart) +
                       (((int64_t)b * pl.S + s) * pl.tiles + tile) * TILE_FLOATS;
#pragma unroll
    for (int n = 0; n < NS; ++n) S[n] = __ldg(hst + tile_block_offset(pc, n));
  }
  bool s_in_regs = true;        // thread (p, 0): S[] holds the state at the chunk start (else it is rebuilt from TMEM)
  float xprev = 1.f, fprev = 1.f;   // thread (p, 0): the factors that take S0 and S1 of the previous chunk to its end
  const uint32_t sm_b = smem_u32(sm);
  bool failed = false;
  bool prefetched = false;      // the coming chunk's tiles are already on their way (CTA-uniform)
  float seg_sum = 0.f;          // !YPASS, thread (p, 0): Delta sum of the segment so far

  // [B | C] rows of the coming chunk, 8 values per thread: token tid & 63, part tid >> 6 = (B 0..7, B 8..15, C 0..7, C 8..15)
  const int bt = tid & 63, bpart = tid >> 6;
  float4 bcr[2];
  auto fetch_bc = [&](int64_t row0, int nt) {
    if (bt < nt) {
      const float4* src = reinterpret_cast<const float4*>(bc + (row0 + bt) * NBC + 8 * bpart);
      bcr[0] = __ldg(src); bcr[1] = __ldg(src + 1);
    } else {
      bcr[0] = make_float4(0.f, 0.f, 0.f, 0.f); bcr[1] = bcr[0];
    }
  };
  if (nchunk > 0) fetch_bc((int64_t)b * T + t0, (int)min((int64_t)TCK, t1 - t0));

  for (int c = 0; c < nchunk; ++c) {
    const int64_t tc = t0 + (int64_t)c * TCK;
    const int nt = (int)min((int64_t)TCK, t1 - tc);
    const int64_t row0 = (int64_t)b * T + tc;
    if (tid == 0 && !prefetched) {
      if (YPASS) bulk_wait_read_all();   // the previous chunk's y tile has left the x buffer
      mbar_expect_tx(&bar_ld, TCK * MCH * 2 + TCK * MCH * 4);
      tma_2d(sm + SM_X, &tmX, tile * MCH, row0, &bar_ld);
      tma_2d(sm + SM_D, &tmD, tile * MCH, row0, &bar_ld);
    }
    prefetched = false;
    // ---- [B | C] rows -> bf16 operand tiles (rows past the segment end are zeros) ----
    {
      const float v[8] = {bcr[0].x, bcr[0].y, bcr[0].z, bcr[0].w, bcr[1].x, bcr[1].y, bcr[1].z, bcr[1].w};
      uint8_t* dst = sm + (bpart >= 2 ? SM_CT : SM_BT);
      if (YPASS)
        *reinterpret_cast<uint4*>(dst + sw128(bt, bpart & 1)) =
            make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
      if (bpart < 2) {
#pragma unroll
        for (int n = 0; n < 8; ++n)
          *reinterpret_cast<__nv_bfloat16*>(sm + SM_BTT + sw128(8 * bpart + n, bt >> 3) + (bt & 7) * 2) = __float2bfloat16_rn(v[n]);
      }
      fence_async_smem();
    }
    bool ok = mbar_wait(&bar_ld, c & 1);
    if (__syncthreads_or(ok ? 0 : 1)) { failed = true; break; }
    if (YPASS && tid == 0) {   // G = C B^T into lanes 0..63 of columns 0..63 (issued as 128 x 64: rows 64.. of the A tile are never looked at)
      tc_fence_after();
      umma_bf16(tm + TM_D, make_desc(sm_b + SM_CT), make_desc(sm_b + SM_BT), idesc_n(64), 0u);
      umma_commit(&bar_g);
    }

    // ---- this channel, this half: Delta sums, V = F Delta x ----
    const float* dcol = reinterpret_cast<const float*>(sm + SM_D) + (HCK * hf) * MCH + pc;
    const __nv_bfloat16* xcol = reinterpret_cast<const __nv_bfloat16*>(sm + SM_X) + (HCK * hf) * MCH + pc;
    const int nth = max(0, min(HCK, nt - HCK * hf));   // tokens of this half that exist
    if (nt < TCK) {   // ragged chunk: Delta of the tokens that do not exist is zero, so they add nothing anywhere
      float4* z = reinterpret_cast<float4*>(sm + SM_D + nt * MCH * 4);
      for (int i = tid; i < (TCK - nt) * MCH / 4; i += MT) z[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      __syncthreads();
    }
    // Delta sums outward from the reference token r = 15 of the half: F_j = exp(a (cs_r - cs_j)) is exp(-a sum_{r<i<=j})
    // after it and exp(a sum_{j<i<=r}) before it; V = F Delta x goes out in pieces of eight tokens
    float cs_r, cs_t;
    {
      constexpr int R = HCK / 2 - 1;
      float fv[HCK];
      float up = 0.f, dn = 0.f;
#pragma unroll
      for (int t = R + 1; t < HCK; ++t) {
        const float d = dcol[t * MCH];
        up += d;
        fv[t] = ex2_approx(-a2 * up) * d * __bfloat162float(xcol[t * MCH]);
      }
#pragma unroll
      for (int t = R; t >= 0; --t) {
        const float d = dcol[t * MCH];
        fv[t] = ex2_approx(a2 * dn) * d * __bfloat162float(xcol[t * MCH]);
        dn += d;
      }
      cs_r = dn;            // sum over tokens 0..r
      cs_t = dn + up;       // sum over the half
#pragma unroll
      for (int q = 0; q < HCK / 8; ++q)
        *reinterpret_cast<uint4*>(sm + SM_V + sw128(pc, (HCK * hf) / 8 + q)) =
            make_uint4(pack_bf16(fv[8 * q], fv[8 * q + 1]), pack_bf16(fv[8 * q + 2], fv[8 * q + 3]),
                       pack_bf16(fv[8 * q + 4], fv[8 * q + 5]), pack_bf16(fv[8 * q + 6], fv[8 * q + 7]));
    }
    // a channel whose exponents pass the bound writes whatever it has (possibly infinities): its operand row only
    // reaches its own TMEM lane, which is ignored for this chunk
    const bool slow_half = fmaxf(cs_r, cs_t - cs_r) * -a2 > EXP_LIMIT;
    xch[2 * hf][pc] = cs_r;
    xch[2 * hf + 1][pc] = cs_t;
    slow_s[hf][pc] = slow_half ? 1 : 0;
    // ---- thread (p, 0): state at the chunk start, brought to the reference point of half 0, handed to the GEMMs ----
    if (hf == 0) {   // warps 0..3, warp-uniform
      if (c > 0) {   // the TMEM loads are warp-collective: every lane takes them, a lane whose state is in registers keeps it
        uint32_t r0[16], r1[16];
        tc_fence_after();
        tmem_ld16(tm_lane + TM_S0, r0);
        tmem_ld16(tm_lane + TM_S1, r1);
        if (!s_in_regs) {
#pragma unroll
          for (int n = 0; n < NS; ++n) S[n] = fmaf(xprev, __uint_as_float(r0[n]), fprev * __uint_as_float(r1[n]));
        }
      }
      const float f = ex2_approx(a2 * cs_r);
      uint32_t r[16];
      float sp[NS];
#pragma unroll
      for (int n = 0; n < NS; ++n) { sp[n] = S[n] * f; r[n] = __float_as_uint(sp[n]); }
      tmem_st16(tm_lane + TM_S0, r);
      if (YPASS) {
        *reinterpret_cast<uint4*>(sm + SM_SP + sw128(pc, 0)) =
            make_uint4(pack_bf16(sp[0], sp[1]), pack_bf16(sp[2], sp[3]), pack_bf16(sp[4], sp[5]), pack_bf16(sp[6], sp[7]));
        *reinterpret_cast<uint4*>(sm + SM_SP + sw128(pc, 1)) =
            make_uint4(pack_bf16(sp[8], sp[9]), pack_bf16(sp[10], sp[11]), pack_bf16(sp[12], sp[13]), pack_bf16(sp[14], sp[15]));
      }
    }
    fence_async_smem();
    tc_fence_before();
    const int any_slow = __syncthreads_or(slow_half ? 1 : 0);
    const bool slow = (slow_s[0][pc] | slow_s[1][pc]) != 0;
    if (!YPASS && !any_slow && c + 1 < nchunk) {
      // the segment pass is done with the x and Delta tiles once V is written (no channel needs them for a recurrence):
      // the next chunk's tiles travel while this chunk's products run
      if (tid == 0) {
        mbar_expect_tx(&bar_ld, TCK * MCH * 2 + TCK * MCH * 4);
        tma_2d(sm + SM_X, &tmX, tile * MCH, row0 + TCK, &bar_ld);
        tma_2d(sm + SM_D, &tmD, tile * MCH, row0 + TCK, &bar_ld);
      }
      prefetched = true;
    }

    // ---- G (TMEM lanes 0..63 = tokens t) -> lower triangle -> bf16 operand rows ----
    if (YPASS && warp < 2) {
      ok = mbar_wait(&bar_g, c & 1);
      if (ok) {
        tc_fence_after();
        const int t = tid;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          uint32_t r[32];
          tmem_ld32(tm_lane + TM_D + 32 * hh, r);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            uint32_t w4[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int j = 32 * hh + 8 * q + 2 * i;
              const float lo = j <= t ? __uint_as_float(r[8 * q + 2 * i]) : 0.f;
              const float hi = j + 1 <= t ? __uint_as_float(r[8 * q + 2 * i + 1]) : 0.f;
              w4[i] = pack_bf16(lo, hi);
            }
            *reinterpret_cast<uint4*>(sm + SM_GM + sw128(t, 4 * hh + q)) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
          }
        }
        fence_async_smem();
      }
    }
    if (YPASS) {
      tc_fence_before();
      if (__syncthreads_or(ok ? 0 : 1)) { failed = true; break; }
    }
    if (tid == 0) {
      tc_fence_after();
      const uint32_t V = sm_b + SM_V, GM = sm_b + SM_GM, CT = sm_b + SM_CT, SP = sm_b + SM_SP, BTT = sm_b + SM_BTT;
      if (YPASS) {
      // half 0:  V0 G00^T + S' C0^T
      umma_bf16(tm + TM_D, desc_at(V, 0, 0), desc_at(GM, 0, 0), idesc_n(32), 0u);
      umma_bf16(tm + TM_D, desc_at(V, 0, 1), desc_at(GM, 0, 1), idesc_n(32), 1u);
      umma_bf16(tm + TM_D, desc_at(SP, 0, 0), desc_at(CT, 0, 0), idesc_n(32), 1u);
      // half 1, own half:  V1 G11^T
      umma_bf16(tm + TM_D + 32, desc_at(V, 0, 2), desc_at(GM, 32, 2), idesc_n(32), 0u);
      umma_bf16(tm + TM_D + 32, desc_at(V, 0, 3), desc_at(GM, 32, 3), idesc_n(32), 1u);
      // half 1, what reaches it from half 0 and from before the chunk:  V0 G10^T + S' C1^T
      umma_bf16(tm + TM_D + 64, desc_at(V, 0, 0), desc_at(GM, 32, 0), idesc_n(32), 0u);
      umma_bf16(tm + TM_D + 64, desc_at(V, 0, 1), desc_at(GM, 32, 1), idesc_n(32), 1u);
      umma_bf16(tm + TM_D + 64, desc_at(SP, 0, 0), desc_at(CT, 32, 0), idesc_n(32), 1u);
      }
      // state:  S0 = S' + V0^T B0,  S1 = V1^T B1
      umma_bf16(tm + TM_S0, desc_at(V, 0, 0), desc_at(BTT, 0, 0), idesc_n(16), 1u);
      umma_bf16(tm + TM_S0, desc_at(V, 0, 1), desc_at(BTT, 0, 1), idesc_n(16), 1u);
      umma_bf16(tm + TM_S1, desc_at(V, 0, 2), desc_at(BTT, 0, 2), idesc_n(16), 0u);
      umma_bf16(tm + TM_S1, desc_at(V, 0, 3), desc_at(BTT, 0, 3), idesc_n(16), 1u);
      umma_commit(&bar_y);
    }
    // while the products run: the next chunk's [B | C] rows, and the factors this thread needs below
    if (c + 1 < nchunk) fetch_bc(row0 + TCK, (int)min((int64_t)TCK, t1 - tc - TCK));
    if (!YPASS && hf == 0 && slow) {
      // this channel left the factorised form in this chunk: its state by the plain recurrence (B as the bf16 operand holds it)
      for (int t = 0; t < nt; ++t) {
        const float d = dcol[t * MCH];
        const float ab = ex2_approx(a2 * d), dx = d * __bfloat162float(xcol[t * MCH]);
#pragma unroll
        for (int n = 0; n < NS; ++n)
          S[n] = fmaf(ab, S[n], dx * __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(sm + SM_BTT + sw128(n, t >> 3) + (t & 7) * 2)));
      }
    }
    const float c0r = xch[0][pc], c0t = xch[1][pc], c1r = xch[2][pc], c1t = xch[3][pc];
    const float xoff = (c0t - c0r) + c1r;   // Delta sum between the two reference points
    ok = mbar_wait(&bar_y, c & 1);
    // ---- epilogue: thread (p, h) finishes its 32 tokens of channel p; y goes to the staging tile [t][p] ----
    __nv_bfloat16* ycol = reinterpret_cast<__nv_bfloat16*>(sm + SM_X) + (HCK * hf) * MCH + pc;   // the x tile is consumed
    if (YPASS && ok) {
      tc_fence_after();
      uint32_t r[32], r2[32];
      tmem_ld32(tm_lane + TM_D + 32 * hf, r);
      if (hf == 1) tmem_ld32(tm_lane + TM_D + 64, r2);   // warps 4..7, warp-uniform
      if (!slow) {
        constexpr int R = HCK / 2 - 1;
        float up = 0.f, dn = 0.f;
#pragma unroll
        for (int t = R + 1; t < HCK; ++t) {
          up += dcol[t * MCH];
          float yv = ex2_approx(a2 * up) * __uint_as_float(r[t]);
          // E1 X as one exponential: X alone can underflow where E1 X r2 still matters (E1 is large before the reference)
          if (hf == 1) yv = fmaf(ex2_approx(a2 * (up + xoff)), __uint_as_float(r2[t]), yv);
          ycol[t * MCH] = __float2bfloat16_rn(yv);
        }
#pragma unroll
        for (int t = R; t >= 0; --t) {
          float yv = ex2_approx(-a2 * dn) * __uint_as_float(r[t]);
          if (hf == 1) yv = fmaf(ex2_approx(a2 * (xoff - dn)), __uint_as_float(r2[t]), yv);
          ycol[t * MCH] = __float2bfloat16_rn(yv);
          dn += dcol[t * MCH];
        }
      } else if (hf == 0) {
        // this channel left the factorised form in this chunk: plain recurrence over all its tokens, from the true
        // state at the chunk start (B and C as the bf16 operands hold them); its TMEM lane is not used
        for (int t = 0; t < nt; ++t) {
          const float d = dcol[t * MCH];
          const float xv = __bfloat162float(xcol[t * MCH]);
          const float ab = ex2_approx(a2 * d), dx = d * xv;
          float acc = 0.f;
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            const uint4 bq = *reinterpret_cast<const uint4*>(sm + SM_BT + sw128(t, q));
            const uint4 cq = *reinterpret_cast<const uint4*>(sm + SM_CT + sw128(t, q));
            const uint32_t bw[4] = {bq.x, bq.y, bq.z, bq.w}, cw[4] = {cq.x, cq.y, cq.z, cq.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float2 bf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&bw[i]));
              const float2 cf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&cw[i]));
              const int n = 8 * q + 2 * i;
              S[n] = fmaf(ab, S[n], dx * bf.x);
              S[n + 1] = fmaf(ab, S[n + 1], dx * bf.y);
              acc = fmaf(cf.x, S[n], acc);
              acc = fmaf(cf.y, S[n + 1], acc);
            }
          }
          ycol[t * MCH] = __float2bfloat16_rn(acc);
        }
      }
    }
    if (hf == 0) {   // bookkeeping of thread (p, 0) for the next chunk's state
      s_in_regs = slow;
      xprev = ex2_approx(a2 * (xoff + (c1t - c1r)));   // exp(a (cs_end - cs_r0)): takes S0 to the chunk end
      fprev = ex2_approx(a2 * (c1t - c1r));            // exp(a (cs_end - cs_r1)): takes S1 there
      seg_sum += c0t + c1t;
    }
    fence_async_smem();
    tc_fence_before();
    if (__syncthreads_or(ok ? 0 : 1)) { failed = true; break; }
    if (!YPASS) continue;
    if (nt == TCK) {
      if (tid == 0) { tma_store_2d(&tmY, sm + SM_X, tile * MCH, row0); bulk_commit(); }
    } else {
      // ragged chunk (segment or sequence end): only the rows that exist, by plain stores
      for (int t = 0; t < nth; ++t) y[(row0 + HCK * hf + t) * P + pch] = ycol[t * MCH];
      __syncthreads();   // before the next chunk's x lands in this buffer
    }
  }
  if (!YPASS && !failed && hf == 0) {
    // end state of the local scan and the segment's Delta sum, in the layout the carry kernel reads
    if (nchunk > 0) {   // warp-collective loads: every lane takes them
      uint32_t r0[16], r1[16];
      tc_fence_after();
      tmem_ld16(tm_lane + TM_S0, r0);
      tmem_ld16(tm_lane + TM_S1, r1);
      if (!s_in_regs) {
#pragma unroll
        for (int n = 0; n < NS; ++n) S[n] = fmaf(xprev, __uint_as_float(r0[n]), fprev * __uint_as_float(r1[n]));
      }
    }
    float* hend = reinterpret_cast<float*>(ws + pl.off_hend) + (((int64_t)b * pl.S + s) * pl.tiles + tile) * TILE_FLOATS;
#pragma unroll
    for (int n = 0; n < NS; ++n) hend[tile_block_offset(pc, n)] = S[n];
    reinterpret_cast<float*>(ws + pl.off_segd)[((int64_t)b * pl.S + s) * P + pch] = seg_sum;
  }
  if (tid == 0) {
    bulk_wait_all();
    if (failed) {
      mbar_wait(&bar_ld, 0);   // copies already issued still target this CTA's shared memory: one more bounded wait
      atomicExch(status, AS_ERR_TIMEOUT);
    }
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

bool forward_y_mm_applies(const Plan& pl) { return pl.scalar && pl.io == AS_BF16 && pl.P % MCH == 0; }

int launch_forward_y_mm(const Plan& pl, const ScanPtrs& sp, void* y, cudaStream_t st) {
  CUtensorMap mx, md, my;
  if (chunk_map(&mx, sp.x, pl, 2, true, MCH, false)) return 1;
  if (chunk_map(&md, sp.ws + pl.off_delta, pl, 4, false, MCH, false)) return 1;
  if (chunk_map(&my, y, pl, 2, true, MCH, false)) return 1;
  auto kern = scalar_mm_kernel<true>;
  static bool done[AS_MAX_DEVICES] = {};
  if (ensure_dynamic_smem(kern, SMEM_DYN, done)) return 1;
  kern<<<dim3(pl.P / MCH, pl.S, pl.B), MT, SMEM_DYN, st>>>(mx, md, my, pl, sp.A_log, sp.ws, (__nv_bfloat16*)y);
  count_launch();
  return (int)cudaGetLastError();
}

int launch_forward_state_mm(const Plan& pl, const ScanPtrs& sp, cudaStream_t st) {
  CUtensorMap mx, md;
  if (chunk_map(&mx, sp.x, pl, 2, true, MCH, false)) return 1;
  if (chunk_map(&md, sp.ws + pl.off_delta, pl, 4, false, MCH, false)) return 1;
  auto kern = scalar_mm_kernel<false>;
  static bool done[AS_MAX_DEVICES] = {};
  if (ensure_dynamic_smem(kern, SMEM_DYN, done)) return 1;
  kern<<<dim3(pl.P / MCH, pl.S, pl.B), MT, SMEM_DYN, st>>>(mx, md, mx, pl, sp.A_log, sp.ws, nullptr);
  count_launch();
  return (int)cudaGetLastError();
}

}  // namespace as
