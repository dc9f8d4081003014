// Internal declarations shared by the translation units of libadjoint_ssm (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <atomic>

#include "../../include/adjoint_ssm.h"

namespace as {

extern std::atomic<int64_t> g_launches;   // kernels launched by this library (diagnostic)
inline void count_launch(int n = 1) { g_launches.fetch_add(n); }

// Function attributes (the dynamic shared-memory limit) belong to a device: remember per device, per kernel
// instantiation, whether the limit has been raised.  `done` is a static array of the launcher, one flag per device.
constexpr int AS_MAX_DEVICES = 64;
template <typename K>
inline int ensure_dynamic_smem(K kern, int bytes, bool (&done)[AS_MAX_DEVICES]) {   // idempotent: a race between host threads only repeats the call
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= AS_MAX_DEVICES) return 1;
  if (!done[dev]) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return 1;
    done[dev] = true;
  }
  return 0;
}

// Number of SMs of the current device (grids are sized in multiples of it); queried once per device.  The cache is
// a plain array of atomics: concurrent first calls from several host threads at worst query twice.
inline int sm_count() {
  static std::atomic<int> cached[AS_MAX_DEVICES] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= AS_MAX_DEVICES) return 148;
  int n = cached[dev].load(std::memory_order_relaxed);
  if (n <= 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev].store(n, std::memory_order_relaxed);
  }
  return n;
}

constexpr int NS = 16;        // d_state handled by the scan kernels
constexpr int CK = 8;         // tokens per checkpoint chunk (h of one chunk lives in registers)
constexpr int NCH = 2;        // channels per thread of the scan kernels (1 or 2)
constexpr int NTHR = 128;     // threads per CTA of the scan kernels; two threads share a channel set, 8 states each
constexpr int CH = NTHR / 2 * NCH;   // channels per CTA
constexpr int NU = 4 * NCH;   // packed state pairs (f32x2) a thread owns
constexpr int TILE_FLOATS = CH * NS;   // one (channel tile, all states) block of a per-segment / per-chunk array
constexpr int NBC = 2 * NS;   // per-token row of [B_t | C_t] (and of [dB_t | dC_t])
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;

// ---- I/O element access ---------------------------------------------------------------------
template <typename T> __device__ __forceinline__ float ld_io(const T* p);
template <> __device__ __forceinline__ float ld_io<float>(const float* p) { return __ldg(p); }
template <> __device__ __forceinline__ float ld_io<__nv_bfloat16>(const __nv_bfloat16* p) {
  return __bfloat162float(__ldg(p));
}
template <typename T> __device__ __forceinline__ void st_io(T* p, float v);
template <> __device__ __forceinline__ void st_io<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void st_io<__nv_bfloat16>(__nv_bfloat16* p, float v) {
  *p = __float2bfloat16_rn(v);
}

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---- time segmentation and scratch layout ---------------------------------------------------
// Time is cut into S segments of L tokens (L a multiple of CK); a CTA owns (segment, batch element,
// CH channels).  Per-(segment, channel, state) and per-(chunk, channel, state) arrays are stored as
// blocks of TILE_FLOATS floats per channel tile, in the order the owning thread keeps them in registers
// (float4 q of thread tid at float offset (q*NTHR + tid)*4), so one bulk copy moves a CTA's block and
// every thread's access is a contiguous 16 bytes.
struct Plan {
  int KL;           // layers handled by one call (independent problems that share dy); 1 for the single-layer entry points
  int Bg;           // batch elements per layer
  int B, P;         // B = KL * Bg: the kernels see (layer, batch element) as one batch index; layer = b / Bg
  int64_t T;
  int64_t tbar;     // clamped to T
  int full;         // tbar >= T
  int L;            // segment length (tokens)
  int S;            // number of segments
  int64_t NC;       // number of CK-token chunks = ceil(T/CK)
  int m;            // tbar / L   (whole segments inside a window that starts on a segment boundary)
  int r;            // tbar % L   (tokens of the following partial segment)
  int io;           // as_dtype_t
  int scalar;       // 1: one decay rate per channel (A_log is [P]), 0: one per (channel, state)
  int tiles;        // ceil(P / CH) channel tiles
  int bw;           // channels per staged row: min(CH, P)
  int tc;           // 1: bf16 tensor-core contractions (bf16 I/O and d_model % 32 == 0), 0: FP32-pipe GEMMs
  int du_ld;        // row pitch (elements) of the du buffer: P, or P+32 when it is the left part of Gcat = [du|dB|dC]
  // byte offsets into the workspace
  size_t off_status, off_delta, off_bc, off_ckpt, off_cs, off_hend, off_muloc, off_mupart, off_segd,
      off_partd, off_hstart, off_carry, off_swin, off_du, off_dxdir, off_dbc, off_dxacc,
      off_bptt_ckpt, off_wcat, total_fwd, total_grad;
};

int make_plan(const as_shape_t* sh, int64_t tbar, int layers, Plan* pl);
// elements of A_log (and dA_log) per layer
inline int64_t a_stride(const Plan& pl) { return pl.scalar ? (int64_t)pl.P : (int64_t)pl.P * NS; }

// ---- launchers (each returns a cudaError_t as int) ------------------------------------------
// C[m, coff + n] (ldc) = epi( sum_k A(m,k) B(n,k) ), fp32 accumulation on the FP32 pipe.
enum { EPI_STORE = 0, EPI_SOFTPLUS_BIAS = 1, EPI_ATOMIC = 2, EPI_ACCUM = 3 };
struct GemmArgs {
  const void* A; int a_bf16; int64_t a_sm, a_sk;   // element strides of A(m,k)
  const void* Bm; int b_bf16; int64_t b_sn, b_sk;  // element strides of B(n,k)
  float* C; int64_t ldc; int64_t coff;
  const float* bias;
  int64_t M; int N; int64_t K;
  int epi;
  int splitk;                                      // >1 only with EPI_ATOMIC
};
int launch_gemm_simt(const GemmArgs& g, cudaStream_t st);

struct ScanPtrs {
  const void *x, *dy;
  const float* A_log;
  char* ws;
};
int launch_prepass(const Plan& pl, const ScanPtrs& sp, bool with_mu, cudaStream_t st);
int launch_fixup(const Plan& pl, const ScanPtrs& sp, bool with_mu, cudaStream_t st);
int launch_forward_y(const Plan& pl, const ScanPtrs& sp, void* y, cudaStream_t st);
// matmul form of the y pass (as_scan_mm.cu): scalar structure with bf16 I/O and d_model % 128 == 0
bool forward_y_mm_applies(const Plan& pl);
int launch_forward_y_mm(const Plan& pl, const ScanPtrs& sp, void* y, cudaStream_t st);
int launch_forward_state_mm(const Plan& pl, const ScanPtrs& sp, cudaStream_t st);   // the segment pass in the same form
int launch_adjoint_main(const Plan& pl, const ScanPtrs& sp, float* dA_log, float* db_delta, cudaStream_t st);
int launch_wait_selftest(int* status, unsigned limit, cudaStream_t st);
int launch_finish_dx(const Plan& pl, const float* dxacc, const void* dxdir, void* dx, cudaStream_t st);

// bf16 tensor-core path (as_gemm_tc.cu)
int tc_pack_wcat(int P, int layers, const as_params_t* pr, void* wcat, cudaStream_t st);
int tc_projections(const Plan& pl, const as_params_t* pr, const void* wcat, const void* x, char* ws, cudaStream_t st);
int tc_weight_grads(const Plan& pl, const void* x, const as_grads_t* out, char* ws, cudaStream_t st);
int tc_input_grad(const Plan& pl, const void* wcat, void* dx, char* ws, cudaStream_t st);

int launch_bptt(const Plan& pl, const ScanPtrs& sp, float* dA_log, float* db_delta, cudaStream_t st);

// device address of the library's built-in scratch array on the current device (as_noalloc.cu); AS_OK or an error code
int static_scratch_address(void** out);

// regions to clear in one launch (each 16-byte aligned, length a multiple of 16 bytes)
struct ZeroList { void* ptr[8]; size_t bytes[8]; int n; };
int launch_zero_regions(const ZeroList& z, cudaStream_t st);

int launch_rmsnorm_fwd(const as_shape_t* sh, const void* y, void* yhat, float eps, cudaStream_t st);
int launch_residual_add(const as_shape_t* sh, const void* a, const void* b, void* out, cudaStream_t st);
int launch_rmsnorm_bwd_add(const as_shape_t* sh, const void* y, const void* dyhat, void* G, float eps,
                           cudaStream_t st);

}  // namespace as
