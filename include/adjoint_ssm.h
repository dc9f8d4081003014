/*
 * adjoint_ssm.h - C ABI of the B200 (sm_100a) library that computes the gradients of a diagonal
 * selective state-space layer with the adjoint method, in full and truncated-window form.
 *
 * Layer (Section 3.1 "State-space models", the five steps of SSM(.), with the diagonal selective
 * structure of Section 4.5), per sequence, t = 1..T, h_0 = 0:
 *     Delta_t = softplus(W_delta x_t + b_delta)  [P]     B_t = W_B x_t, C_t = W_C x_t  [N]
 *     A = -exp(A_log) [P,N]     h_t[p,n] = exp(Delta_t[p] A[p,n]) h_{t-1}[p,n] + Delta_t[p] B_t[n] x_t[p]
 *     y_t[p] = sum_n C_t[n] h_t[p,n]
 *
 * Conventions for every entry point
 *   - Every tensor pointer is a DEVICE pointer owned by the caller, contiguous, row-major (last index
 *     fastest) and 16-byte aligned.  Activations are [batch, seqlen, d_model]; "io dtype" is fp32 or
 *     bf16 as selected by as_shape_t.io.  The library never allocates or frees device memory, and keeps none
 *     between calls, with one exception: the fixed scratch array of as_ssm_forward_static (see there).
 *   - All work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = the legacy default
 *     stream).  No entry point synchronises except as_check_status.
 *   - `ws` is caller-provided scratch of at least the size reported by as_workspace_bytes; its
 *     contents on entry are ignored and on return are unspecified.
 *   - Return value: AS_OK (0) or a negative AS_ERR_* code.  Nothing is launched when an argument
 *     check fails.  No exceptions, no aborts, no printing.
 *   - Threads: the entry points keep no shared mutable state, so several host threads may call them at once
 *     (each call with its own `ws`), except for the phase-timing diagnostic (one thread, one stream) and the
 *     shared array of as_ssm_forward_static.  The library uses the CUDA runtime API, i.e. each device's primary context.
 *   - Size limits (AS_ERR_LIMIT): batch * seqlen + seqlen + 16 < 2^31 (token rows are 32-bit TMA coordinates) and
 *     seqlen <= 65527 * 2048 (time segments fill one grid dimension).
 *   - Device-side waits: every wait on staged data (mbarrier waits on TMA / bulk copies and on tensor-core commits)
 *     is bounded and ends in AS_ERR_TIMEOUT.  The one wait that has no software bound is the hardware allocation of
 *     tensor memory (tcgen05.alloc) at the start of the contraction, adjoint and matmul-form forward kernels: it blocks until enough of
 *     the SM's 512 columns are free, which happens when CTAs that hold them finish; a kernel of this library frees
 *     its columns on every exit path and never waits for another CTA while holding them, so the allocation of a
 *     later CTA always completes.
 *   - Results are deterministic up to floating-point summation order (fp32 atomics are used for the
 *     sums over channels, segments and the batch).
 */
#ifndef ADJOINT_SSM_H_
#define ADJOINT_SSM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define AS_VERSION 104

typedef enum { AS_F32 = 0, AS_BF16 = 1 } as_dtype_t;

/* Structure of A (Table 1 of Section 4.5): AS_A_DIAGONAL, one decay rate per (channel, state), A_log [P,N];
 * AS_A_SCALAR, one decay rate per channel shared by its N states ("Scalar SSM": A^t is a multiple of the identity on
 * each channel), A_log [P] and dA_log [P] (the sum over n of the diagonal layer's dA_log[p,n]).  With AS_A_SCALAR,
 * io == AS_BF16 and d_model % 128 == 0, as_ssm_forward runs its scans in the matmul form this structure admits (chunks of
 * 64 tokens as tensor-core products of tril(C B^T) with the decay-scaled inputs, state carried in tensor memory);
 * every other shape and every other entry point uses the scan kernels. */
typedef enum { AS_A_DIAGONAL = 0, AS_A_SCALAR = 1 } as_structure_t;

enum {
  AS_OK = 0,
  AS_ERR_NULL = -1,       /* a required pointer is NULL */
  AS_ERR_SHAPE = -2,      /* non-positive dimension, d_state != 16, or an unknown a_structure */
  AS_ERR_DTYPE = -3,      /* io is neither AS_F32 nor AS_BF16 */
  AS_ERR_TBAR = -4,       /* tbar < 1 */
  AS_ERR_WORKSPACE = -5,  /* ws_bytes smaller than as_workspace_bytes reports */
  AS_ERR_ALIGN = -6,      /* a pointer is not 16-byte aligned, or d_model is not a multiple of 8 */
  AS_ERR_CUDA = -7,       /* a CUDA runtime call or kernel launch failed */
  AS_ERR_TIMEOUT = -8,    /* a bounded device-side wait gave up (reported by as_check_status) */
  AS_ERR_LIMIT = -9       /* a size exceeds a fixed capacity of the entry point */
};

/* flags */
#define AS_ACCUMULATE 1u  /* add into the parameter-gradient buffers instead of overwriting them */

typedef struct {
  int32_t batch;      /* Bsz >= 1 */
  int64_t seqlen;     /* T >= 1 */
  int32_t d_model;    /* P >= 8, multiple of 8 */
  int32_t d_state;    /* N, must be 16 */
  int32_t io;         /* as_dtype_t of x, y, dy, dx and the W_* matrices */
  int32_t a_structure; /* as_structure_t */
} as_shape_t;

typedef struct {          /* parameters of one layer (device pointers) */
  const void  *W_delta;   /* [P,P] (out,in), io dtype */
  const float *b_delta;   /* [P]   fp32 */
  const void  *W_B;       /* [N,P] io dtype */
  const void  *W_C;       /* [N,P] io dtype */
  const float *A_log;     /* [P,N] fp32 (AS_A_SCALAR: [P]), A = -exp(A_log) */
  const void  *Wcat;      /* optional, may be NULL: [P+32, P] io dtype, the rows of W_delta, W_B, W_C stacked, as written
                             by as_pack_weights.  Only the bf16 tensor-core contractions read it (bf16 io, P % 32 == 0);
                             when NULL they pack a copy into the scratch on every call (one more small kernel). */
} as_params_t;

typedef struct {          /* gradient outputs (device pointers); parameter gradients are fp32, summed over the batch */
  float *dW_delta;        /* [P,P] */
  float *db_delta;        /* [P]   */
  float *dW_B;            /* [N,P] */
  float *dW_C;            /* [N,P] */
  float *dA_log;          /* [P,N] (AS_A_SCALAR: [P]) */
  void  *dx;              /* [Bsz,T,P] io dtype, always overwritten; may be NULL (input gradient skipped) */
} as_grads_t;

/* Library version (AS_VERSION of the build). */
int as_version(void);

/* Static description of a status code. */
const char *as_strerror(int code);

/* Scratch sizes in bytes for a shape: *fwd_bytes for as_ssm_forward, *grad_bytes for as_adjoint_grad and
 * as_full_bptt_grad (the larger of the two).  Either output pointer may be NULL.  `tbar` as for as_adjoint_grad. */
int as_workspace_bytes(const as_shape_t *shape, int64_t tbar, size_t *fwd_bytes, size_t *grad_bytes);

/* Synchronises `stream` and returns the status word the kernels keep at the start of `ws`
 * (AS_OK, or AS_ERR_TIMEOUT if a bounded device-side wait ran out).  ws == NULL selects the built-in scratch
 * array of as_ssm_forward_static on the current device. */
int as_check_status(const void *ws, void *stream);

/* SSM(X) = Y (Section 3.1, steps 1-5; Alg. 1 line 5 for one layer).
 * x [Bsz,T,P] io -> y [Bsz,T,P] io.  The three projections run as one dense contraction, the recurrence as
 * a time-segmented scan (local scan per segment, sequential carry over segments, final pass). */
int as_ssm_forward(const as_shape_t *shape, const as_params_t *params, const void *x, void *y,
                   void *ws, size_t ws_bytes, void *stream);

/* Adjoint-method gradient of L = sum_t l^t(y^t) w.r.t. the layer parameters and x, given dy = dl^t/dy^t
 * (Proposition 2; with tbar < T the truncated form, Eq. 7 of Section 4.3; Algorithms 2-4 for one layer).
 * Token t contributes A-net and B-net vector-Jacobian products only for source tokens i in
 * [max(1, t+1-tbar), t]; the C-net term is never truncated.  tbar >= seqlen selects the full form.
 * The adjoint states lambda^{t,i} are never materialised: the cotangents of all tokens t whose window
 * contains i are summed on chip (a reverse-time recurrence with the exact removal of the term that
 * leaves the window) and each source token's three VJPs are evaluated once.
 * Self-contained: recomputes the forward quantities it needs from x; no prior as_ssm_forward call needed.
 * dx also uses the windowed sum for the A/B paths and the exact C path. */
int as_adjoint_grad(const as_shape_t *shape, const as_params_t *params, const void *x, const void *dy,
                    int64_t tbar, uint32_t flags, const as_grads_t *out,
                    void *ws, size_t ws_bytes, void *stream);

/* The K layers of a residual stack in one call (Proposition 3 and Section 4.2: given the stored layer inputs and the
 * one upstream gradient dL/dy_K, the adjoint states of a layer depend only on that layer's own A and C, so all
 * layers' vector-Jacobian products are independent; Alg. 4's loop over k).  Every phase - projections, segment
 * pre-pass, carries, main adjoint kernel, the two contractions - runs as ONE launch over (layer, batch element)
 * instead of one launch per layer.
 *   layers  K >= 1;
 *   params  every pointer addresses K contiguous copies of the single-layer tensor: W_delta [K,P,P], b_delta [K,P],
 *           W_B, W_C [K,N,P], A_log [K,P,N] ([K,P] for AS_A_SCALAR), Wcat [K,P+32,P] or NULL;
 *   x       [K,Bsz,T,P] io: the input of each layer (for the stack: Norm(y_{k-1}));
 *   dy      [Bsz,T,P] io: shared by all layers;
 *   out     every pointer addresses K contiguous copies: dW_delta [K,P,P], ..., dA_log [K,P,N]; dx [K,Bsz,T,P] or NULL;
 *   ws      at least as_workspace_bytes_layers bytes.
 * Layer k's results equal as_adjoint_grad on (params[k], x[k], dy).  The bf16 contractions go out as one launch when
 * Bsz*T is a multiple of 128 (no 128-row tile then straddles two layers), otherwise as one launch per layer; fp32 io
 * runs its FP32-pipe contractions layer by layer.  K = 1 is exactly as_adjoint_grad.
 * Limits: K * Bsz <= 65535 and K * Bsz * T + T + 16 < 2^31 (AS_ERR_LIMIT). */
int as_adjoint_grad_layers(const as_shape_t *shape, int32_t layers, const as_params_t *params, const void *x,
                           const void *dy, int64_t tbar, uint32_t flags, const as_grads_t *out,
                           void *ws, size_t ws_bytes, void *stream);

/* Scratch size of as_adjoint_grad_layers. */
int as_workspace_bytes_layers(const as_shape_t *shape, int32_t layers, int64_t tbar, size_t *grad_bytes);

/* Packed weights for the bf16 tensor-core contractions: Wcat[k] = [W_delta[k]; W_B[k]; W_C[k]], [layers, P+32, P].
 * as_wcat_bytes gives the buffer size (0 for a bad shape); as_pack_weights writes it (bf16 io only, AS_ERR_DTYPE
 * otherwise).  Pack once per parameter update and pass the pointer as as_params_t.Wcat: the forward and gradient
 * calls then skip their own packing kernel.  The packed copy must be re-made whenever W_delta, W_B or W_C change. */
size_t as_wcat_bytes(const as_shape_t *shape, int32_t layers);
int as_pack_weights(const as_shape_t *shape, int32_t layers, const as_params_t *params, void *wcat, void *stream);

/* The same outputs by plain backpropagation through time (the sequential nested accumulation that the
 * adjoint method replaces, Section 3.3): one reverse sweep per channel carrying dL/dh_t.  Separately coded
 * and deliberately simple; it exists for comparison with as_adjoint_grad at tbar >= seqlen. */
int as_full_bptt_grad(const as_shape_t *shape, const as_params_t *params, const void *x, const void *dy,
                      uint32_t flags, const as_grads_t *out, void *ws, size_t ws_bytes, void *stream);

/* Forward for callers that cannot allocate device memory (the paper has no counterpart: this is a deployment
 * convenience, not part of the method).  Meant for code running as a guest of a host program that owns all
 * device memory and forbids cudaMalloc from guest code (a plug-in in an inference server with a frozen memory
 * budget, a latency-critical loop that cannot afford cudaMalloc's device-wide synchronisation).  Same result as
 * as_ssm_forward, but the scratch is a fixed AS_STATIC_SCRATCH_BYTES array inside the library's device image:
 *   - every GPU context that loads the library holds that much memory until exit;
 *   - a shape whose forward scratch (as_workspace_bytes, fwd_bytes) is larger returns AS_ERR_LIMIT, nothing runs;
 *   - the first call on a device resolves the array's device address (a synchronous runtime query made with that
 *     device current): make it during set-up, before any stream capture;
 *   - all calls on a device share the array and it keeps the previous call's contents (what must start at zero is
 *     cleared by the call); calls whose kernels may overlap on the GPU race on it - order them on one stream;
 *   - the status word of the call's kernels sits at the head of the array: read it with as_check_status(NULL, stream);
 *   - the array belongs to the device's primary context (the one the CUDA runtime API uses);
 *   - neither this call nor anything it launches calls cudaMalloc, cudaFree or another allocating routine.
 * x, y: [Bsz,T,P] io dtype device buffers supplied by the caller, as for as_ssm_forward. */
#define AS_STATIC_SCRATCH_BYTES (32u << 20)
int as_ssm_forward_static(const as_shape_t *shape, const as_params_t *params, const void *x, void *y, void *stream);

/* Residual-stack glue (Section 3.2; Alg. 1 lines 6-7): gain-free RMSNorm over d_model.
 * yhat = y / sqrt(mean_p(y^2) + eps), io dtype in and out, fp32 arithmetic. */
int as_rmsnorm_fwd(const as_shape_t *shape, const void *y, void *yhat, float eps, void *stream);

/* y_out = y_in + ytilde (the residual connection y_k = y_{k-1} + SSM_k(Norm(y_{k-1}))); y_out may alias y_in. */
int as_residual_add(const as_shape_t *shape, const void *y_in, const void *ytilde, void *y_out, void *stream);

/* Backward of the glue: G_inout += RMSNormVJP(y, dyhat) = (dyhat - yhat * mean_p(dyhat*yhat)) / rms(y).
 * G_inout [Bsz,T,P] io dtype is the upstream gradient of y (read and overwritten). */
int as_rmsnorm_bwd_add(const as_shape_t *shape, const void *y, const void *dyhat, void *G_inout,
                       float eps, void *stream);

/* ---- diagnostics ------------------------------------------------------------------------------------ */

/* Self test of the failure-reporting path.  Every device-side wait of this library (mbarrier waits on staged
 * tiles) is bounded: after a fixed number of polls the kernel stops, writes AS_ERR_TIMEOUT into the status word at
 * the head of `ws` and returns, leaving the context usable.  This call enqueues a one-warp kernel that waits, with
 * `poll_limit` polls (1 .. 2^20), for an mbarrier phase that nothing completes; as_check_status(ws, stream) must
 * then return AS_ERR_TIMEOUT.  `ws` needs 256 bytes.  Nothing faults, traps or spins without bound. */
int as_wait_selftest(void *ws, size_t ws_bytes, uint32_t poll_limit, void *stream);

/* host-side bookkeeping only; no effect on results */

/* Number of SMs of the current device as the library sees it (grids are sized in multiples of it). */
int as_sm_count(void);

/* Number of kernels this library has launched in this process since the last reset; reset != 0 zeroes it. */
int64_t as_launch_count(int reset);

/* Phase timing of as_adjoint_grad (process-wide state, not thread-safe: use it from one host thread driving one
 * stream).  as_set_timing(1) makes every later as_adjoint_grad call record CUDA
 * events on its stream between its phases (this creates the events once; timing mode is opt-in and is the one
 * place where the library creates CUDA objects).  as_get_timing synchronises on the last event of the most
 * recent call and writes elapsed milliseconds into ms[0..AS_NUM_PHASES): projections (S1, incl. zeroing),
 * segment pre-pass, carry fix-up, main adjoint kernel, weight-gradient contractions, input-gradient
 * contractions.  Returns AS_OK, or AS_ERR_NULL if timing is off or no call was recorded. */
#define AS_NUM_PHASES 6
int as_set_timing(int enable);
int as_get_timing(float *ms, int n);

#ifdef __cplusplus
}
#endif
#endif /* ADJOINT_SSM_H_ */
