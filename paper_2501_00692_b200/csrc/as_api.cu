// extern "C" entry points: argument checks, scratch layout, and the launch sequence of each call.
#include <atomic>

#include "as_internal.cuh"

using namespace as;

namespace as {
std::atomic<int64_t> g_launches{0};
}

namespace {

// Phase timing is a diagnostic with process-wide state: one set of events, no locking.  It is meant for one host
// thread driving one stream (as the header says); everything else in the library is free of shared mutable state.
bool g_timing = false;
bool g_timing_valid = false;
cudaEvent_t g_ev[AS_NUM_PHASES + 1];

void mark(int i, cudaStream_t st) {
  if (g_timing) cudaEventRecord(g_ev[i], st);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_shape(const as_shape_t* sh) {
  if (!sh) return AS_ERR_NULL;
  if (sh->batch < 1 || sh->seqlen < 1 || sh->d_model < 1) return AS_ERR_SHAPE;
  if (sh->d_state != NS) return AS_ERR_SHAPE;
  if (sh->a_structure != AS_A_DIAGONAL && sh->a_structure != AS_A_SCALAR) return AS_ERR_SHAPE;
  if (sh->io != AS_F32 && sh->io != AS_BF16) return AS_ERR_DTYPE;
  if (sh->d_model % 8 != 0) return AS_ERR_ALIGN;
  if (sh->batch > 65535) return AS_ERR_SHAPE;
  // token rows are addressed with 32-bit TMA coordinates (row + window lookahead + one chunk), and the time
  // segments (at most 2048 tokens each) fill gridDim.y
  if ((int64_t)sh->batch * sh->seqlen + sh->seqlen + 2 * CK >= ((int64_t)1 << 31)) return AS_ERR_LIMIT;
  return AS_OK;
}

int check_params(const as_params_t* pr) {
  if (!pr || !pr->W_delta || !pr->b_delta || !pr->W_B || !pr->W_C || !pr->A_log) return AS_ERR_NULL;
  if (!aligned16(pr->W_delta) || !aligned16(pr->b_delta) || !aligned16(pr->W_B) || !aligned16(pr->W_C) ||
      !aligned16(pr->A_log) || !aligned16(pr->Wcat))
    return AS_ERR_ALIGN;
  return AS_OK;
}

#define AS_TRY(expr)                      \
  do {                                    \
    int e__ = (expr);                     \
    if (e__ != 0) return AS_ERR_CUDA;     \
  } while (0)

// Wcat of the call: the caller's packed copy if it gave one, else packed here into the scratch
int wcat_of(const Plan& pl, const as_params_t* pr, char* ws, cudaStream_t st, const void** wcat) {
  if (pr->Wcat) { *wcat = pr->Wcat; return AS_OK; }
  AS_TRY(tc_pack_wcat(pl.P, pl.KL, pr, ws + pl.off_wcat, st));
  *wcat = ws + pl.off_wcat;
  return AS_OK;
}

// steps 1-3 of SSM(.): Delta = softplus(x W_delta^T + b), B = x W_B^T, C = x W_C^T  (every layer of the call)
int projections(const Plan& pl, const as_params_t* pr, const void* wcat, const void* x, char* ws, cudaStream_t st) {
  if (pl.tc) {
    AS_TRY(tc_projections(pl, pr, wcat, x, ws, st));
    return AS_OK;
  }
  const int bf = pl.io == AS_BF16;
  const size_t e = bf ? 2 : 4;
  const int64_t M = (int64_t)pl.Bg * pl.T;
  const size_t P = pl.P;
  for (int l = 0; l < pl.KL; ++l) {
    GemmArgs g{};
    g.A = (const char*)x + l * M * P * e; g.a_bf16 = bf; g.a_sm = pl.P; g.a_sk = 1;
    g.b_bf16 = bf; g.b_sn = pl.P; g.b_sk = 1;
    g.M = M; g.K = pl.P; g.splitk = 1;
    g.Bm = (const char*)pr->W_delta + l * P * P * e; g.N = pl.P;
    g.C = reinterpret_cast<float*>(ws + pl.off_delta) + l * M * P; g.ldc = pl.P; g.coff = 0;
    g.bias = pr->b_delta + l * P; g.epi = EPI_SOFTPLUS_BIAS;
    AS_TRY(launch_gemm_simt(g, st));
    g.epi = EPI_STORE; g.bias = nullptr; g.N = NS; g.C = reinterpret_cast<float*>(ws + pl.off_bc) + l * M * NBC; g.ldc = NBC;
    g.Bm = (const char*)pr->W_B + l * NS * P * e; g.coff = 0;
    AS_TRY(launch_gemm_simt(g, st));
    g.Bm = (const char*)pr->W_C + l * NS * P * e; g.coff = NS;
    AS_TRY(launch_gemm_simt(g, st));
  }
  return AS_OK;
}

int pick_splitk(int64_t tiles, int64_t K) {
  int64_t s = ((int64_t)sm_count() * 4 + tiles - 1) / tiles;
  const int64_t maxs = (K + 255) / 256;
  if (s > maxs) s = maxs;
  if (s < 1) s = 1;
  if (s > 1024) s = 1024;
  return (int)s;
}

// the net-VJPs: weight gradients (contractions over all tokens) and the input gradient, for every layer of the call
int contractions(const Plan& pl, const as_params_t* pr, const void* wcat, const void* x, const as_grads_t* out, char* ws,
                 cudaStream_t st) {
  const int bf = pl.io == AS_BF16;
  const size_t e = bf ? 2 : 4;
  const int64_t M = (int64_t)pl.Bg * pl.T;
  const int P = pl.P;
  if (pl.tc) {
    AS_TRY(tc_weight_grads(pl, x, out, ws, st));
    mark(5, st);
    if (out->dx) AS_TRY(tc_input_grad(pl, wcat, out->dx, ws, st));
    mark(6, st);
    return AS_OK;
  }
  for (int l = 0; l < pl.KL; ++l) {
    const void* du = ws + pl.off_du + (size_t)l * M * pl.du_ld * e;
    const float* dbc = reinterpret_cast<const float*>(ws + pl.off_dbc) + (size_t)l * M * NBC;
    const void* xl = (const char*)x + (size_t)l * M * P * e;
    // dW_delta[i,j] = sum_m du[m,i] x[m,j]
    GemmArgs g{};
    g.A = du; g.a_bf16 = bf; g.a_sm = 1; g.a_sk = P;
    g.Bm = xl; g.b_bf16 = bf; g.b_sn = 1; g.b_sk = P;
    g.C = out->dW_delta + (size_t)l * P * P; g.ldc = P; g.coff = 0; g.M = P; g.N = P; g.K = M; g.epi = EPI_ATOMIC;
    g.splitk = pick_splitk((int64_t)((P + 63) / 64) * ((P + 63) / 64), M);
    AS_TRY(launch_gemm_simt(g, st));
    // dW_B, dW_C
    g.A = dbc; g.a_bf16 = 0; g.a_sm = 1; g.a_sk = NBC; g.M = NS;
    g.splitk = pick_splitk((P + 63) / 64, M);
    g.C = out->dW_B + (size_t)l * NS * P;
    AS_TRY(launch_gemm_simt(g, st));
    g.A = dbc + NS; g.C = out->dW_C + (size_t)l * NS * P;
    AS_TRY(launch_gemm_simt(g, st));
  }
  mark(5, st);
  if (out->dx) {  // dx = dx_dir + du W_delta + dB W_B + dC W_C
    for (int l = 0; l < pl.KL; ++l) {
      const void* du = ws + pl.off_du + (size_t)l * M * pl.du_ld * e;
      const float* dbc = reinterpret_cast<const float*>(ws + pl.off_dbc) + (size_t)l * M * NBC;
      float* acc = reinterpret_cast<float*>(ws + pl.off_dxacc) + (size_t)l * M * P;
      GemmArgs g{};
      g.A = du; g.a_bf16 = bf; g.a_sm = P; g.a_sk = 1;
      g.Bm = (const char*)pr->W_delta + (size_t)l * P * P * e; g.b_bf16 = bf; g.b_sn = 1; g.b_sk = P;
      g.C = acc; g.ldc = P; g.coff = 0; g.M = M; g.N = P; g.K = P; g.epi = EPI_STORE; g.splitk = 1;
      AS_TRY(launch_gemm_simt(g, st));
      g.A = dbc; g.a_bf16 = 0; g.a_sm = NBC; g.a_sk = 1; g.K = NS; g.epi = EPI_ACCUM;
      g.Bm = (const char*)pr->W_B + (size_t)l * NS * P * e;
      AS_TRY(launch_gemm_simt(g, st));
      g.A = dbc + NS; g.Bm = (const char*)pr->W_C + (size_t)l * NS * P * e;
      AS_TRY(launch_gemm_simt(g, st));
    }
    AS_TRY(launch_finish_dx(pl, reinterpret_cast<const float*>(ws + pl.off_dxacc), ws + pl.off_dxdir, out->dx, st));
  }
  mark(6, st);
  return AS_OK;
}

int check_grad_args(const as_shape_t* sh, const as_params_t* pr, const void* x, const void* dy,
                    const as_grads_t* out, void* ws) {
  int e = check_shape(sh);
  if (e) return e;
  e = check_params(pr);
  if (e) return e;
  if (!x || !dy || !out || !ws) return AS_ERR_NULL;
  if (!out->dW_delta || !out->db_delta || !out->dW_B || !out->dW_C || !out->dA_log) return AS_ERR_NULL;
  if (!aligned16(x) || !aligned16(dy) || !aligned16(ws) || !aligned16(out->dW_delta) || !aligned16(out->db_delta) ||
      !aligned16(out->dW_B) || !aligned16(out->dW_C) || !aligned16(out->dA_log) || !aligned16(out->dx))
    return AS_ERR_ALIGN;
  return AS_OK;
}

int zero_outputs(const Plan& pl, uint32_t flags, const as_grads_t* out, char* ws, cudaStream_t st) {
  const size_t P = pl.P, K = pl.KL;
  ZeroList z{};
  auto add = [&](void* p, size_t bytes) { z.ptr[z.n] = p; z.bytes[z.n] = (bytes + 15) / 16 * 16; ++z.n; };
  add(ws + pl.off_status, 256);
  add(ws + pl.off_dbc, (size_t)pl.B * pl.T * NBC * 4);
  if (!(flags & AS_ACCUMULATE)) {
    add(out->dW_delta, K * P * P * 4);
    add(out->db_delta, K * P * 4);
    add(out->dW_B, K * NS * P * 4);
    add(out->dW_C, K * NS * P * 4);
    add(out->dA_log, K * (pl.scalar ? P : P * NS) * 4);
  }
  AS_TRY(launch_zero_regions(z, st));
  return AS_OK;
}

}  // namespace

extern "C" {

int as_version(void) { return AS_VERSION; }

const char* as_strerror(int code) {
  switch (code) {
    case AS_OK: return "ok";
    case AS_ERR_NULL: return "a required pointer is NULL";
    case AS_ERR_SHAPE: return "bad shape (non-positive dimension or d_state != 16)";
    case AS_ERR_DTYPE: return "unsupported io dtype";
    case AS_ERR_TBAR: return "tbar must be >= 1";
    case AS_ERR_WORKSPACE: return "workspace too small";
    case AS_ERR_ALIGN: return "pointer not 16-byte aligned or d_model not a multiple of 8";
    case AS_ERR_CUDA: return "CUDA runtime call or launch failed";
    case AS_ERR_TIMEOUT: return "bounded device-side wait gave up";
    case AS_ERR_LIMIT: return "size exceeds a fixed capacity of this entry point";
    default: return "unknown status code";
  }
}

int as_workspace_bytes(const as_shape_t* shape, int64_t tbar, size_t* fwd_bytes, size_t* grad_bytes) {
  int e = check_shape(shape);
  if (e) return e;
  if (tbar < 1) return AS_ERR_TBAR;
  Plan pl;
  e = make_plan(shape, tbar, 1, &pl);
  if (e) return e;
  if (fwd_bytes) *fwd_bytes = pl.total_fwd;
  if (grad_bytes) *grad_bytes = pl.total_grad;
  return AS_OK;
}

int as_check_status(const void* ws, void* stream) {
  if (!ws) {   // the built-in scratch array of as_ssm_forward_static on the current device
    void* p = nullptr;
    const int e = static_scratch_address(&p);
    if (e) return e;
    ws = p;
  }
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  int word = 0;
  if (cudaMemcpyAsync(&word, ws, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return AS_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return AS_ERR_CUDA;
  return word;
}

int as_ssm_forward(const as_shape_t* shape, const as_params_t* params, const void* x, void* y, void* ws,
                   size_t ws_bytes, void* stream) {
  int e = check_shape(shape);
  if (e) return e;
  e = check_params(params);
  if (e) return e;
  if (!x || !y || !ws) return AS_ERR_NULL;
  if (!aligned16(x) || !aligned16(y) || !aligned16(ws)) return AS_ERR_ALIGN;
  Plan pl;
  e = make_plan(shape, shape->seqlen, 1, &pl);
  if (e) return e;
  if (ws_bytes < pl.total_fwd) return AS_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  char* w = reinterpret_cast<char*>(ws);
  AS_TRY((int)cudaMemsetAsync(w + pl.off_status, 0, 256, st));
  const void* wcat = nullptr;
  if (pl.tc) { e = wcat_of(pl, params, w, st, &wcat); if (e) return e; }
  e = projections(pl, params, wcat, x, w, st);
  if (e) return e;
  ScanPtrs sp{x, nullptr, params->A_log, w};
  const bool mm = forward_y_mm_applies(pl);
  if (mm) AS_TRY(launch_forward_state_mm(pl, sp, st));
  else AS_TRY(launch_prepass(pl, sp, false, st));
  AS_TRY(launch_fixup(pl, sp, false, st));
  if (mm) AS_TRY(launch_forward_y_mm(pl, sp, y, st));
  else AS_TRY(launch_forward_y(pl, sp, y, st));
  return AS_OK;
}

int as_adjoint_grad(const as_shape_t* shape, const as_params_t* params, const void* x, const void* dy, int64_t tbar,
                    uint32_t flags, const as_grads_t* out, void* ws, size_t ws_bytes, void* stream) {
  return as_adjoint_grad_layers(shape, 1, params, x, dy, tbar, flags, out, ws, ws_bytes, stream);
}

int as_workspace_bytes_layers(const as_shape_t* shape, int32_t layers, int64_t tbar, size_t* grad_bytes) {
  int e = check_shape(shape);
  if (e) return e;
  if (tbar < 1) return AS_ERR_TBAR;
  if (layers < 1) return AS_ERR_SHAPE;
  if ((int64_t)layers * shape->batch * shape->seqlen + shape->seqlen + 2 * CK >= ((int64_t)1 << 31)) return AS_ERR_LIMIT;
  Plan pl;
  e = make_plan(shape, tbar, layers, &pl);
  if (e) return e;
  if (grad_bytes) *grad_bytes = pl.total_grad;
  return AS_OK;
}

size_t as_wcat_bytes(const as_shape_t* shape, int32_t layers) {
  if (check_shape(shape) != AS_OK || layers < 1) return 0;
  return (size_t)layers * (shape->d_model + NBC) * shape->d_model * (shape->io == AS_BF16 ? 2 : 4);
}

int as_pack_weights(const as_shape_t* shape, int32_t layers, const as_params_t* params, void* wcat, void* stream) {
  int e = check_shape(shape);
  if (e) return e;
  e = check_params(params);
  if (e) return e;
  if (!wcat) return AS_ERR_NULL;
  if (!aligned16(wcat)) return AS_ERR_ALIGN;
  if (layers < 1) return AS_ERR_SHAPE;
  if (shape->io != AS_BF16) return AS_ERR_DTYPE;   // only the bf16 tensor-core contractions read a packed copy
  AS_TRY(tc_pack_wcat(shape->d_model, layers, params, wcat, reinterpret_cast<cudaStream_t>(stream)));
  return AS_OK;
}

int as_adjoint_grad_layers(const as_shape_t* shape, int32_t layers, const as_params_t* params, const void* x,
                           const void* dy, int64_t tbar, uint32_t flags, const as_grads_t* out, void* ws,
                           size_t ws_bytes, void* stream) {
  int e = check_grad_args(shape, params, x, dy, out, ws);
  if (e) return e;
  if (tbar < 1) return AS_ERR_TBAR;
  if (layers < 1) return AS_ERR_SHAPE;
  if ((int64_t)layers * shape->batch * shape->seqlen + shape->seqlen + 2 * CK >= ((int64_t)1 << 31)) return AS_ERR_LIMIT;
  Plan pl;
  e = make_plan(shape, tbar, layers, &pl);
  if (e) return e;
  if (ws_bytes < pl.total_grad) return AS_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  char* w = reinterpret_cast<char*>(ws);
  mark(0, st);
  e = zero_outputs(pl, flags, out, w, st);
  if (e) return e;
  const void* wcat = nullptr;
  if (pl.tc) { e = wcat_of(pl, params, w, st, &wcat); if (e) return e; }
  e = projections(pl, params, wcat, x, w, st);
  if (e) return e;
  mark(1, st);
  ScanPtrs sp{x, dy, params->A_log, w};
  AS_TRY(launch_prepass(pl, sp, true, st));
  mark(2, st);
  AS_TRY(launch_fixup(pl, sp, true, st));
  mark(3, st);
  AS_TRY(launch_adjoint_main(pl, sp, out->dA_log, out->db_delta, st));
  mark(4, st);
  e = contractions(pl, params, wcat, x, out, w, st);
  if (g_timing && e == AS_OK) g_timing_valid = true;
  return e;
}

int as_full_bptt_grad(const as_shape_t* shape, const as_params_t* params, const void* x, const void* dy,
                      uint32_t flags, const as_grads_t* out, void* ws, size_t ws_bytes, void* stream) {
  int e = check_grad_args(shape, params, x, dy, out, ws);
  if (e) return e;
  Plan pl;
  e = make_plan(shape, shape->seqlen, 1, &pl);
  if (e) return e;
  if (ws_bytes < pl.total_grad) return AS_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  char* w = reinterpret_cast<char*>(ws);
  e = zero_outputs(pl, flags, out, w, st);
  if (e) return e;
  const void* wcat = nullptr;
  if (pl.tc) { e = wcat_of(pl, params, w, st, &wcat); if (e) return e; }
  e = projections(pl, params, wcat, x, w, st);
  if (e) return e;
  ScanPtrs sp{x, dy, params->A_log, w};
  AS_TRY(launch_bptt(pl, sp, out->dA_log, out->db_delta, st));
  return contractions(pl, params, wcat, x, out, w, st);
}

int as_rmsnorm_fwd(const as_shape_t* shape, const void* y, void* yhat, float eps, void* stream) {
  int e = check_shape(shape);
  if (e) return e;
  if (!y || !yhat) return AS_ERR_NULL;
  AS_TRY(launch_rmsnorm_fwd(shape, y, yhat, eps, reinterpret_cast<cudaStream_t>(stream)));
  return AS_OK;
}

int as_residual_add(const as_shape_t* shape, const void* y_in, const void* ytilde, void* y_out, void* stream) {
  int e = check_shape(shape);
  if (e) return e;
  if (!y_in || !ytilde || !y_out) return AS_ERR_NULL;
  AS_TRY(launch_residual_add(shape, y_in, ytilde, y_out, reinterpret_cast<cudaStream_t>(stream)));
  return AS_OK;
}

int as_rmsnorm_bwd_add(const as_shape_t* shape, const void* y, const void* dyhat, void* G_inout, float eps,
                       void* stream) {
  int e = check_shape(shape);
  if (e) return e;
  if (!y || !dyhat || !G_inout) return AS_ERR_NULL;
  AS_TRY(launch_rmsnorm_bwd_add(shape, y, dyhat, G_inout, eps, reinterpret_cast<cudaStream_t>(stream)));
  return AS_OK;
}

int as_wait_selftest(void* ws, size_t ws_bytes, uint32_t poll_limit, void* stream) {
  if (!ws) return AS_ERR_NULL;
  if (ws_bytes < 256) return AS_ERR_WORKSPACE;
  if (!aligned16(ws)) return AS_ERR_ALIGN;
  if (poll_limit == 0 || poll_limit > (1u << 20)) return AS_ERR_LIMIT;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  AS_TRY((int)cudaMemsetAsync(ws, 0, 256, st));
  AS_TRY(launch_wait_selftest(reinterpret_cast<int*>(ws), poll_limit, st));
  return AS_OK;
}

int64_t as_launch_count(int reset) {
  const int64_t v = as::g_launches.load();
  if (reset) as::g_launches.store(0);
  return v;
}

int as_sm_count(void) { return sm_count(); }

int as_set_timing(int enable) {
  static bool created = false;
  if (enable && !created) {
    for (int i = 0; i <= AS_NUM_PHASES; ++i)
      if (cudaEventCreate(&g_ev[i]) != cudaSuccess) return AS_ERR_CUDA;
    created = true;
  }
  g_timing = enable != 0;
  g_timing_valid = false;
  return AS_OK;
}

int as_get_timing(float* ms, int n) {
  if (!ms) return AS_ERR_NULL;
  if (!g_timing || !g_timing_valid) return AS_ERR_NULL;
  if (cudaEventSynchronize(g_ev[AS_NUM_PHASES]) != cudaSuccess) return AS_ERR_CUDA;
  for (int i = 0; i < n && i < AS_NUM_PHASES; ++i)
    if (cudaEventElapsedTime(&ms[i], g_ev[i], g_ev[i + 1]) != cudaSuccess) return AS_ERR_CUDA;
  return AS_OK;
}

}  // extern "C"
