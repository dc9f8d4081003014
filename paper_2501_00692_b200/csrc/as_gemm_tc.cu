// bf16 tensor-core contractions for sm_100a: TMA (cp.async.bulk.tensor, 128-byte swizzle) feeds a
// shared-memory ring, one elected thread issues tcgen05.mma into a TMEM accumulator, eight warps drain it
// with tcgen05.ld, apply the fused epilogue into a swizzled shared-memory staging tile and hand that tile to
// TMA (bulk tensor store, or bulk tensor reduce-add for the split-K weight gradients), so that global memory
// only sees whole rows of 64 bytes.  One kernel template covers the three token-dimension
// contractions of the layer:
//   PROJ : [Delta | B | C] = X Wcat^T            (A K-major, B K-major;  softplus+bias epilogue)
//   DW   : dWcat = Gcat^T X  over all tokens     (A MN-major, B MN-major; split-K, fp32 reduction)
//   DX   : dx = dx_dir + Gcat Wcat               (A K-major, B MN-major; add + bf16 store)
// with Wcat = [W_delta; W_B; W_C] ([P+32, P]) and Gcat = [du | dB | dC] ([tokens, P+32]), both bf16.
// No cluster multicast is used anywhere.  Every mbarrier wait is bounded; on timeout the kernel records
// AS_ERR_TIMEOUT in the status word, stops issuing work, frees its TMEM and returns.
#include <cuda.h>

#include "as_internal.cuh"

namespace as {
namespace {

constexpr int BM = 128, BK = 64, UK = 16, EPI_WARPS = 8, NTHREADS = 64 + 32 * EPI_WARPS;
constexpr int A_BYTES = BM * BK * 2;
constexpr int EPI_TILE_BYTES = 32 * 64;   // staging tile of one epilogue warp: 32 rows of 64 bytes, 64-byte swizzle
// tile width BN is a template parameter: 256 keeps the shared-memory operand traffic per MMA cycle under the
// 128 B/clk an SM can read (a 128x128 tile needs 128 B/clk for the MMA alone), 128 wastes less on narrow outputs
template <int BN> struct Cfg {
  static constexpr int B_BYTES = BN * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = BN >= 208 ? 4 : 6;
  static constexpr int TMEM_COLS = 2 * BN <= 256 ? 256 : 512;   // two accumulators, power-of-two allocation
  static constexpr int SMEM_DYN = STAGES * STAGE_BYTES + 1024 + EPI_WARPS * 2 * EPI_TILE_BYTES;   // + alignment slack + staging
};
constexpr uint32_t WAIT_LIMIT = 1u << 22;

enum { MAJ_K = 0, MAJ_MN = 1 };
enum { TC_PROJ = 0, TC_DW = 1, TC_DX = 2 };

struct TcArgs {
  int64_t M;            // rows of the output tile space (A's MN extent); PROJ / DX: the tokens of all layers
  int N;                // cols of the output (B's MN extent)
  int kblocks;          // number of BK-blocks along K (DW: per layer)
  int splitk;
  int P;                // d_model
  int layers;           // independent problems stacked along the leading dimension of every tensor
  int64_t rows_layer;   // token rows per layer (a multiple of BM when layers > 1)
  const float* bias;    // PROJ: b_delta [layers, P]
  int* status;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// bounded wait: returns false if the phase did not complete within WAIT_LIMIT polls
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  const uint32_t addr = smem_u32(bar);
  for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(addr), "r"(parity)
        : "memory");
    if (ok) return true;
    if (*abort_flag) return false;
  }
  return false;
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* tm, int c0, int c1, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(dst)), "l"(tm), "r"(c0), "r"(c1), "r"(smem_u32(bar))
      : "memory");
}

// shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
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

// softplus(u) = max(u,0) + log(1 + z), z = exp(-|u|) in (0,1]: two MUFU ops (ex2, lg2) and a short series
// for small z, where forming 1 + z would lose z's low bits (relative error of the result < 3e-7)
__device__ __forceinline__ float softplus_f(float u) {
  const float z = ex2_approx(-fabsf(u) * LOG2E);
  float l;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(l) : "f"(1.f + z));
  const float big = l * LN2;
  const float small = z * fmaf(z, fmaf(z, 1.f / 3.f, -0.5f), 1.f);   // z - z^2/2 + z^3/3
  return fmaxf(u, 0.f) + (z < 0.0078125f ? small : big);
}

// ---- TMA stores out of the staging tile (bulk async-groups are tracked per issuing thread) ----
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tm, const void* src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(tm), "r"(c0), "r"(c1), "r"(smem_u32(src)) : "memory");
}
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* tm, const void* src, int c0, int c1) {
  asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(tm), "r"(c0), "r"(c1), "r"(smem_u32(src)) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// byte offset of 16-byte piece q of row r in a [rows][64 B] tile under the 64-byte swizzle
__device__ __forceinline__ uint32_t swz64(int r, int q) { return (uint32_t)(r * 64 + ((q ^ ((r >> 1) & 3)) << 4)); }

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// Persistent, warp-specialised kernel: one CTA per SM walks tiles t = blockIdx.x, + gridDim.x, ...
//   warp 0 (one lane): TMA producer over a STAGES-deep shared-memory ring that runs on across tiles
//   warp 1 (one lane): tcgen05.mma issuer; the accumulator alternates between two 128-column TMEM buffers
//   warps 2..9       : epilogue (two warps per TMEM lane quarter, each taking half of the columns); they drain
//                      buffer a while the issuer already fills buffer a^1 for the next tile
// Tile order: n fastest, then m, then the K split, so concurrently running CTAs share A rows through L2.
// ML: several layers stacked along the leading dimension of every tensor (false compiles the single-layer code).
template <int AMAJ, int BMAJ, int EPI, int BN, bool ML>
__global__ void __launch_bounds__(NTHREADS) gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA,
                                                           const __grid_constant__ CUtensorMap tmB,
                                                           const __grid_constant__ CUtensorMap tmO0,
                                                           const __grid_constant__ CUtensorMap tmO1,
                                                           const __grid_constant__ CUtensorMap tmO2, TcArgs a) {
  constexpr int STAGES = Cfg<BN>::STAGES, B_BYTES = Cfg<BN>::B_BYTES, STAGE_BYTES = Cfg<BN>::STAGE_BYTES;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[STAGES];
  __shared__ __align__(8) uint64_t empty_bar[STAGES];
  __shared__ __align__(8) uint64_t tmem_full_bar[2];
  __shared__ __align__(8) uint64_t tmem_empty_bar[2];
  __shared__ __align__(8) uint64_t ld_bar[EPI_WARPS][2];   // DX: arrival of the dx_dir tile in a staging buffer
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int mt = (int)((a.M + BM - 1) / BM), nt = (a.N + BN - 1) / BN;
  const int ntiles = mt * nt * a.splitk * ((ML && EPI == TC_DW) ? a.layers : 1);
  const int kper = (a.kblocks + a.splitk - 1) / a.splitk;
  const int NWc = a.P + NBC;                       // rows of one layer's Wcat
  volatile int* abortp = &abort_s;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&tmem_full_bar[b], 1); mbar_init(&tmem_empty_bar[b], EPI_WARPS); }
    for (int w2 = 0; w2 < EPI_WARPS; ++w2) { mbar_init(&ld_bar[w2][0], 1); mbar_init(&ld_bar[w2][1], 1); }
    abort_s = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {   // TMEM allocation: two BN-column fp32 accumulators
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(Cfg<BN>::TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_base_s;

  // lay: the layer a tile belongs to.  PROJ / DX tile the token rows of all layers (a tile never straddles two layers);
  // DW has its own set of (m, n, split) tiles per layer and contracts over that layer's tokens only.
  auto decode = [&](int t, int64_t& m0, int& n0, int& kb0, int& nkb, int& lay) {
    const int in = t % nt, im = (t / nt) % mt;
    int ik = t / (nt * mt);
    m0 = (int64_t)im * BM; n0 = in * BN;
    lay = 0;
    if (ML) {
      if (EPI == TC_DW) { lay = ik / a.splitk; ik -= lay * a.splitk; }
      else lay = im / (int)(a.rows_layer / BM);
    }
    kb0 = ik * kper;
    nkb = max(0, min(a.kblocks, kb0 + kper) - kb0);
  };

  if (warp == 0) {
    if (lane == 0) {
      // ---------------- TMA producer ----------------
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB) : "memory");
      int it = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < ntiles && ok; t += gridDim.x) {
        int64_t m0; int n0, kb0, nkb, lay;
        decode(t, m0, n0, kb0, nkb, lay);
        // row offsets of this layer: DW contracts over its token rows (both operands), PROJ / DX read its Wcat rows
        const int ktok = (ML && EPI == TC_DW) ? (int)(lay * a.rows_layer) : 0;
        const int wrow = (ML && EPI != TC_DW) ? lay * NWc : 0;
        for (int i = 0; i < nkb; ++i, ++it) {
          const int s = it % STAGES, round = it / STAGES;
          if (round > 0 && !mbar_wait(&empty_bar[s], (round - 1) & 1, abortp)) { ok = false; break; }
          uint8_t* sa = smem + s * STAGE_BYTES;
          uint8_t* sb = sa + A_BYTES;
          mbar_expect_tx(&full_bar[s], STAGE_BYTES);
          const int k = (kb0 + i) * BK;
          if (AMAJ == MAJ_K) {
            tma_load_2d(sa, &tmA, k, (int)m0, &full_bar[s]);
          } else {
            tma_load_2d(sa, &tmA, (int)m0, ktok + k, &full_bar[s]);
            tma_load_2d(sa + A_BYTES / 2, &tmA, (int)m0 + 64, ktok + k, &full_bar[s]);
          }
          if (BMAJ == MAJ_K) {
            tma_load_2d(sb, &tmB, k, wrow + n0, &full_bar[s]);
          } else {
#pragma unroll
            for (int q = 0; q < BN / 64; ++q)
              tma_load_2d(sb + q * (64 * BK * 2), &tmB, n0 + 64 * q, ktok + wrow + k, &full_bar[s]);
          }
        }
      }
      if (!ok) { *abortp = 1; atomicExch(a.status, AS_ERR_TIMEOUT); }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---------------- MMA issuer ----------------
      const uint32_t idesc0 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)AMAJ << 15) | ((uint32_t)BMAJ << 16) |
                              ((uint32_t)(BM >> 4) << 24);
      int it = 0, ti = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < ntiles && ok; t += gridDim.x, ++ti) {
        int64_t m0; int n0, kb0, nkb, lay;
        decode(t, m0, n0, kb0, nkb, lay);
        const int ab = ti & 1, around = ti >> 1;
        if (around > 0 && !mbar_wait(&tmem_empty_bar[ab], (around - 1) & 1, abortp)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t acc = tmem_base + (uint32_t)(ab * BN);
        // a K-major B tile that sticks out past N only needs the MMA to cover its valid columns (multiple of 16)
        int neff = BN;
        if (BMAJ == MAJ_K && n0 + BN > a.N) neff = ((a.N - n0 + 15) / 16) * 16;
        const uint32_t idesc = idesc0 | ((uint32_t)(neff >> 3) << 17);
        for (int i = 0; i < nkb; ++i, ++it) {
          const int s = it % STAGES, round = it / STAGES;
          if (!mbar_wait(&full_bar[s], round & 1, abortp)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t sa = smem_u32(smem + s * STAGE_BYTES);
          const uint32_t sb = sa + A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / UK; ++k) {
            const uint64_t ad = (AMAJ == MAJ_K) ? make_desc(sa + k * UK * 2, 16, 1024)
                                                : make_desc(sa + k * UK * 128, A_BYTES / 2, 1024);
            const uint64_t bd = (BMAJ == MAJ_K) ? make_desc(sb + k * UK * 2, 16, 1024)
                                                : make_desc(sb + k * UK * 128, 64 * BK * 2, 1024);
            umma_bf16(acc, ad, bd, idesc, (i > 0 || k > 0) ? 1u : 0u);
          }
          umma_commit(&empty_bar[s]);   // frees the stage once these MMAs have read it
        }
        if (ok) umma_commit(&tmem_full_bar[ab]);   // accumulator of this tile complete
      }
      if (!ok) { *abortp = 1; atomicExch(a.status, AS_ERR_TIMEOUT); }
    }
  } else {
    // ---------------- epilogue warps ----------------
    // A warp owns TMEM lanes [32 quarter, 32 quarter + 32) = 32 output rows, one row per lane, and walks its share of
    // the tile's columns in chunks that are 64 bytes wide in the output (16 fp32 or 32 bf16 columns).  A chunk goes
    // registers -> staging tile (two per warp, alternating) -> TMA; lane 0 issues and tracks the bulk operations.
    // Rows and columns past the output's extent are clipped by TMA.
    const int quarter = warp & 3;              // the TMEM lane quarter this warp may read
    const int chalf = (warp - 2) / 4;          // which half of the tile's columns it drains
    constexpr int CW = EPI == TC_DX ? 32 : 16;                 // columns per chunk
    constexpr int NCHUNK = BN / CW;
    constexpr int CSPLIT = (NCHUNK + 1) / 2;                   // first warp of a quarter takes [0, CSPLIT)
    uint8_t* stg = smem + STAGES * STAGE_BYTES + (warp - 2) * 2 * EPI_TILE_BYTES;
    uint64_t* lbar = ld_bar[warp - 2];
    const int c_lo = chalf ? CSPLIT : 0, c_hi = chalf ? NCHUNK : CSPLIT;
    int ti = 0;
    uint32_t nchunks_done = 0;                 // chunks this warp has staged so far (selects buffer and mbarrier phase)
    bool ok = true;
    for (int t = blockIdx.x; t < ntiles && ok; t += gridDim.x, ++ti) {
      int64_t m0; int n0, kb0, nkb, lay;
      decode(t, m0, n0, kb0, nkb, lay);
      const int ab = ti & 1, around = ti >> 1;
      if (nkb > 0) {
        const int mrow = (int)m0 + quarter * 32;      // first output row of this warp
        const float* bias_l = a.bias + (ML ? (int64_t)lay * a.P : 0);
        if (EPI == TC_DX && lane == 0 && n0 + c_lo * CW < a.N) {
          // dx_dir tile of the first chunk; later ones are requested one chunk ahead
          bulk_wait_read<0>();
          const uint32_t bi = nchunks_done & 1;
          mbar_expect_tx(&lbar[bi], EPI_TILE_BYTES);
          tma_load_2d(stg + bi * EPI_TILE_BYTES, &tmO1, n0 + c_lo * CW, mrow, &lbar[bi]);
        }
        if (!mbar_wait(&tmem_full_bar[ab], around & 1, abortp)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll 1
        for (int c = c_lo; c < c_hi; ++c) {
          const int nb = n0 + c * CW;
          if (nb >= a.N) break;                        // warp-uniform
          const uint32_t bi = nchunks_done & 1;
          uint8_t* buf = stg + bi * EPI_TILE_BYTES;
          const uint32_t tcol = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(ab * BN + c * CW);
          if (EPI == TC_DX) {
            if (lane == 0) {
              bulk_wait_read<0>();                      // the other buffer's store has been read out
              if (c + 1 < c_hi && nb + CW < a.N) {
                mbar_expect_tx(&lbar[bi ^ 1], EPI_TILE_BYTES);
                tma_load_2d(stg + (bi ^ 1) * EPI_TILE_BYTES, &tmO1, nb + CW, mrow, &lbar[bi ^ 1]);
              }
            }
            uint32_t r[32];
            tmem_ld32(tcol, r);
            if (!mbar_wait(&lbar[bi], (nchunks_done >> 1) & 1, abortp)) { ok = false; break; }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              uint4* pq = reinterpret_cast<uint4*>(buf + swz64(lane, q));
              const uint4 sv = *pq;
              const __nv_bfloat162* s2 = reinterpret_cast<const __nv_bfloat162*>(&sv);
              uint4 ov;
              __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&ov);
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float2 f = __bfloat1622float2(s2[e]);
                o2[e] = __floats2bfloat162_rn(f.x + __uint_as_float(r[8 * q + 2 * e]), f.y + __uint_as_float(r[8 * q + 2 * e + 1]));
              }
              *pq = ov;
            }
            fence_async_smem();
            __syncwarp();
            if (lane == 0) { tma_store_2d(&tmO0, buf, nb, mrow); bulk_commit(); }
          } else {
            uint32_t r[16];
            tmem_ld16(tcol, r);
            if (lane == 0) bulk_wait_read<1>();         // the operation that last used this buffer has read it
            __syncwarp();
            if (EPI == TC_PROJ && nb < a.P) {
              const float4* b4 = reinterpret_cast<const float4*>(bias_l + nb);
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                const float4 bv = __ldg(b4 + q);
                *reinterpret_cast<float4*>(buf + swz64(lane, q)) =
                    make_float4(softplus_f(__uint_as_float(r[4 * q]) + bv.x), softplus_f(__uint_as_float(r[4 * q + 1]) + bv.y),
                                softplus_f(__uint_as_float(r[4 * q + 2]) + bv.z), softplus_f(__uint_as_float(r[4 * q + 3]) + bv.w));
              }
            } else {
#pragma unroll
              for (int q = 0; q < 4; ++q)
                *reinterpret_cast<uint4*>(buf + swz64(lane, q)) = make_uint4(r[4 * q], r[4 * q + 1], r[4 * q + 2], r[4 * q + 3]);
            }
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
              if (EPI == TC_PROJ) {
                if (nb < a.P) tma_store_2d(&tmO0, buf, nb, mrow);       // Delta
                else tma_store_2d(&tmO1, buf, nb - a.P, mrow);          // [B | C]
              } else {
                // rows of Wcat space: [0, P) dW_delta, [P, P+16) dW_B, [P+16, P+32) dW_C; 16-row groups never straddle
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                  const int mr = mrow + 16 * hh;
                  const void* src = buf + hh * 1024;
                  const int l1 = ML ? lay * a.P : 0, l2 = ML ? lay * NS : 0;   // this layer's rows of the stacked outputs
                  if (mr < a.P) tma_reduce_add_2d(&tmO0, src, nb, l1 + mr);
                  else if (mr < a.P + NS) tma_reduce_add_2d(&tmO1, src, nb, l2 + mr - a.P);
                  else if (mr < a.P + 2 * NS) tma_reduce_add_2d(&tmO2, src, nb, l2 + mr - a.P - NS);
                }
              }
              bulk_commit();
            }
          }
          ++nchunks_done;
        }
        if (!ok) break;
        // hand the accumulator buffer back to the issuer
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(&tmem_empty_bar[ab]);
      }
    }
    if (lane == 0) bulk_wait_all();            // staging tiles must outlive the bulk operations that read them
    if (!ok) { *abortp = 1; if (lane == 0) atomicExch(a.status, AS_ERR_TIMEOUT); }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(Cfg<BN>::TMEM_COLS) : "memory");
  }
}

// ---- small helpers -------------------------------------------------------------------------------
// Wcat[l] = [W_delta[l]; W_B[l]; W_C[l]] for every layer l (blockIdx.y)
__global__ void pack_wcat_kernel(int P, const __nv_bfloat16* __restrict__ Wd, const __nv_bfloat16* __restrict__ WB,
                                 const __nv_bfloat16* __restrict__ WC, __nv_bfloat16* __restrict__ out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t n = (int64_t)(P + NBC) * P;
  if (i >= n) return;
  const int64_t l = blockIdx.y;
  Wd += l * P * P; WB += l * NS * P; WC += l * NS * P; out += l * n;
  const int64_t row = i / P, col = i % P;
  out[i] = row < P ? Wd[i] : (row < P + NS ? WB[(row - P) * P + col] : WC[(row - P - NS) * P + col]);
}

// [dB | dC] fp32 sums -> the last 32 bf16 columns of Gcat; eight values per thread (P and the row pitch are multiples
// of 32 elements on this path, so every access is 16-byte aligned)
__global__ void cvt_dbc_kernel(int64_t rows, int ldg, int P, const float* __restrict__ dbc, __nv_bfloat16* __restrict__ gcat) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;   // one group of 8 columns
  if (i >= rows * (NBC / 8)) return;
  const int64_t row = i / (NBC / 8);
  const int c = (int)(i % (NBC / 8)) * 8;
  const float4 a = __ldg(reinterpret_cast<const float4*>(dbc + row * NBC + c));
  const float4 b = __ldg(reinterpret_cast<const float4*>(dbc + row * NBC + c + 4));
  uint4 o;
  __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&o);
  o2[0] = __floats2bfloat162_rn(a.x, a.y); o2[1] = __floats2bfloat162_rn(a.z, a.w);
  o2[2] = __floats2bfloat162_rn(b.x, b.y); o2[3] = __floats2bfloat162_rn(b.z, b.w);
  *reinterpret_cast<uint4*>(gcat + row * ldg + P + c) = o;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// row-major [rows, cols] tensor with row pitch `ld` elements; box = {box_cols, box_rows}; OOB reads give 0, OOB writes are dropped
int make_map_t(CUtensorMap* tm, CUtensorMapDataType dt, int esz, CUtensorMapSwizzle swz, const void* base, uint64_t rows,
               uint64_t cols, uint64_t ld, uint32_t box_cols, uint32_t box_rows) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return 1;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {ld * (uint64_t)esz};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(tm, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : 1;
}
// bf16 operand: box = {64 cols, box_rows}, 128-byte swizzle
int make_map(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows) {
  return make_map_t(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, CU_TENSOR_MAP_SWIZZLE_128B, base, rows, cols, ld, 64, box_rows);
}
// epilogue tiles: rows of 64 bytes, 64-byte swizzle
int make_map_out_f32(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  return make_map_t(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, CU_TENSOR_MAP_SWIZZLE_64B, base, rows, cols, cols, 16, box_rows);
}
int make_map_out_bf16(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols) {
  return make_map_t(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, CU_TENSOR_MAP_SWIZZLE_64B, base, rows, cols, cols, 32, 32);
}

template <int AMAJ, int BMAJ, int EPI, int BN, bool ML>
int launch_tc_ml(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap (&tmO)[3], const TcArgs& a, cudaStream_t st) {
  auto kern = gemm_tc_kernel<AMAJ, BMAJ, EPI, BN, ML>;
  static bool done[AS_MAX_DEVICES] = {};
  if (ensure_dynamic_smem(kern, Cfg<BN>::SMEM_DYN, done)) return 1;
  const int64_t ntiles = ((a.M + BM - 1) / BM) * ((a.N + BN - 1) / BN) * a.splitk * (EPI == TC_DW ? a.layers : 1);
  const int sms = sm_count();
  const unsigned grid = (unsigned)(ntiles < sms ? ntiles : sms);   // one persistent CTA per SM
  kern<<<grid, NTHREADS, Cfg<BN>::SMEM_DYN, st>>>(tmA, tmB, tmO[0], tmO[1], tmO[2], a);
  count_launch();
  return (int)cudaGetLastError();
}

template <int AMAJ, int BMAJ, int EPI, int BN>
int launch_tc(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap (&tmO)[3], const TcArgs& a, cudaStream_t st) {
  return a.layers > 1 ? launch_tc_ml<AMAJ, BMAJ, EPI, BN, true>(tmA, tmB, tmO, a, st)
                      : launch_tc_ml<AMAJ, BMAJ, EPI, BN, false>(tmA, tmB, tmO, a, st);
}

}  // namespace

constexpr int TBN = 256;   // tile width of the weight-gradient and input-gradient contractions
constexpr int PBN = 208;   // projections: N = P + 32; for P = 768 four 208-wide tiles waste 4 % where 256 wastes 22 %

int tc_pack_wcat(int P, int layers, const as_params_t* pr, void* wcat, cudaStream_t st) {
  const int64_t n = (int64_t)(P + NBC) * P;
  pack_wcat_kernel<<<dim3((unsigned)((n + 255) / 256), (unsigned)layers), 256, 0, st>>>(
      P, (const __nv_bfloat16*)pr->W_delta, (const __nv_bfloat16*)pr->W_B, (const __nv_bfloat16*)pr->W_C,
      (__nv_bfloat16*)wcat);
  count_launch();
  return (int)cudaGetLastError();
}

// The layers of a call go out as one launch when no 128-row tile straddles two layers (token rows per layer a
// multiple of BM); otherwise one launch per layer, on that layer's slab of every tensor.
struct LayerLoop { int first, count; };
static inline int layer_groups(const Plan& pl, LayerLoop* g) {
  const int64_t rows = (int64_t)pl.Bg * pl.T;
  if (pl.KL == 1 || rows % BM == 0) { g[0] = {0, pl.KL}; return 1; }
  return 0;   // the caller loops over single layers
}

int tc_projections(const Plan& pl, const as_params_t* pr, const void* wcat, const void* x, char* ws, cudaStream_t st) {
  const int64_t rows = (int64_t)pl.Bg * pl.T;
  const int P = pl.P, NW = P + NBC;
  LayerLoop one;
  const bool batched = layer_groups(pl, &one) == 1;
  for (int l0 = 0; l0 < pl.KL; l0 += batched ? pl.KL : 1) {
    const int nl = batched ? pl.KL : 1;
    const int64_t M = rows * nl;
    CUtensorMap tmA, tmB;
    if (make_map(&tmA, (const char*)x + (size_t)l0 * rows * P * 2, M, P, P, BM)) return 1;
    if (make_map(&tmB, (const char*)wcat + (size_t)l0 * NW * P * 2, (uint64_t)NW * nl, P, P, PBN)) return 1;
    TcArgs a{};
    a.M = M; a.N = NW; a.kblocks = (P + BK - 1) / BK; a.splitk = 1; a.P = P; a.layers = nl; a.rows_layer = rows;
    a.bias = pr->b_delta + (size_t)l0 * P;
    a.status = (int*)(ws + pl.off_status);
    CUtensorMap tmO[3];
    if (make_map_out_f32(&tmO[0], ws + pl.off_delta + (size_t)l0 * rows * P * 4, M, P, 32)) return 1;
    if (make_map_out_f32(&tmO[1], ws + pl.off_bc + (size_t)l0 * rows * NBC * 4, M, NBC, 32)) return 1;
    tmO[2] = tmO[1];
    const int e = launch_tc<MAJ_K, MAJ_K, TC_PROJ, PBN>(tmA, tmB, tmO, a, st);
    if (e) return e;
  }
  return 0;
}

int tc_weight_grads(const Plan& pl, const void* x, const as_grads_t* out, char* ws, cudaStream_t st) {
  const int64_t rows = (int64_t)pl.Bg * pl.T;
  const int64_t Mall = rows * pl.KL;
  const int P = pl.P, NW = P + NBC;
  cvt_dbc_kernel<<<(unsigned)((Mall * (NBC / 8) + 255) / 256), 256, 0, st>>>(Mall, NW, P, (const float*)(ws + pl.off_dbc),
                                                                       (__nv_bfloat16*)(ws + pl.off_du));
  count_launch();
  if (cudaGetLastError() != cudaSuccess) return 1;
  LayerLoop one;
  const bool batched = layer_groups(pl, &one) == 1;
  for (int l0 = 0; l0 < pl.KL; l0 += batched ? pl.KL : 1) {
    const int nl = batched ? pl.KL : 1;
    CUtensorMap tmA, tmB;
    if (make_map(&tmA, ws + pl.off_du + (size_t)l0 * rows * NW * 2, rows * nl, NW, NW, 64)) return 1;   // Gcat as [K=tokens, M=P+32]
    if (make_map(&tmB, (const char*)x + (size_t)l0 * rows * P * 2, rows * nl, P, P, 64)) return 1;       // X as [K=tokens, N=P]
    TcArgs a{};
    a.M = NW; a.N = P; a.kblocks = (int)((rows + BK - 1) / BK); a.P = P; a.layers = nl; a.rows_layer = rows;
    const int tiles = ((NW + BM - 1) / BM) * ((P + TBN - 1) / TBN) * nl;
    int sk = sm_count() / tiles;   // about one tile per persistent CTA (two measured 3 % slower at C3: more reduce-adds)
    if (sk > a.kblocks) sk = a.kblocks;
    if (sk < 1) sk = 1;
    const int kper = (a.kblocks + sk - 1) / sk;
    a.splitk = (a.kblocks + kper - 1) / kper;   // no empty split: every tile has at least one K block
    a.status = (int*)(ws + pl.off_status);
    CUtensorMap tmO[3];
    if (make_map_out_f32(&tmO[0], out->dW_delta + (size_t)l0 * P * P, (uint64_t)P * nl, P, 16)) return 1;
    if (make_map_out_f32(&tmO[1], out->dW_B + (size_t)l0 * NS * P, (uint64_t)NS * nl, P, 16)) return 1;
    if (make_map_out_f32(&tmO[2], out->dW_C + (size_t)l0 * NS * P, (uint64_t)NS * nl, P, 16)) return 1;
    const int e = launch_tc<MAJ_MN, MAJ_MN, TC_DW, TBN>(tmA, tmB, tmO, a, st);
    if (e) return e;
  }
  return 0;
}

int tc_input_grad(const Plan& pl, const void* wcat, void* dx, char* ws, cudaStream_t st) {
  const int64_t rows = (int64_t)pl.Bg * pl.T;
  const int P = pl.P, NW = P + NBC;
  LayerLoop one;
  const bool batched = layer_groups(pl, &one) == 1;
  for (int l0 = 0; l0 < pl.KL; l0 += batched ? pl.KL : 1) {
    const int nl = batched ? pl.KL : 1;
    const int64_t M = rows * nl;
    CUtensorMap tmA, tmB;
    if (make_map(&tmA, ws + pl.off_du + (size_t)l0 * rows * NW * 2, M, NW, NW, BM)) return 1;            // Gcat as [M=tokens, K=P+32]
    if (make_map(&tmB, (const char*)wcat + (size_t)l0 * NW * P * 2, (uint64_t)NW * nl, P, P, 64)) return 1;   // Wcat as [K=P+32, N=P]
    TcArgs a{};
    a.M = M; a.N = P; a.kblocks = (NW + BK - 1) / BK; a.splitk = 1; a.P = P; a.layers = nl; a.rows_layer = rows;
    a.status = (int*)(ws + pl.off_status);
    CUtensorMap tmO[3];
    if (make_map_out_bf16(&tmO[0], (char*)dx + (size_t)l0 * rows * P * 2, M, P)) return 1;
    if (make_map_out_bf16(&tmO[1], ws + pl.off_dxdir + (size_t)l0 * rows * P * 2, M, P)) return 1;
    tmO[2] = tmO[1];
    const int e = launch_tc<MAJ_K, MAJ_MN, TC_DX, TBN>(tmA, tmB, tmO, a, st);
    if (e) return e;
  }
  return 0;
}

}  // namespace as
