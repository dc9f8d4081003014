/* Plain-C caller of the adjoint_ssm C ABI: no Python, no torch - device memory from the CUDA runtime, raw fp32
 * tensors from a file, results to a file.
 *
 *   demo_c_abi <batch> <seqlen> <d_model> <tbar> <in.bin> <out.bin>
 *
 * in.bin  (fp32, in this order): W_delta[P*P] b_delta[P] W_B[16*P] W_C[16*P] A_log[P*16] x[B*T*P] dy[B*T*P]
 * out.bin (fp32, in this order): y[B*T*P] dW_delta[P*P] db_delta[P] dW_B[16*P] dW_C[16*P] dA_log[P*16] dx[B*T*P]
 * Exit code 0 on success, 1 on a usage/IO error, 2 on a CUDA error, 3 on a library error. */
#include <cuda_runtime.h>
#include <stdio.h>
#include <stdlib.h>

#include "../../include/adjoint_ssm.h"

#define CK(x) do { if ((x) != cudaSuccess) { fprintf(stderr, "CUDA error at %s:%d\n", __FILE__, __LINE__); return 2; } } while (0)
#define AS(x) do { int e_ = (x); if (e_ != AS_OK) { fprintf(stderr, "%s -> %s\n", #x, as_strerror(e_)); return 3; } } while (0)

static float *upload(FILE *f, size_t n) {
  float *h = (float *)malloc(n * sizeof(float)), *d = NULL;
  if (!h || fread(h, sizeof(float), n, f) != n) { free(h); return NULL; }
  if (cudaMalloc((void **)&d, n * sizeof(float)) != cudaSuccess ||
      cudaMemcpy(d, h, n * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess) { free(h); return NULL; }
  free(h);
  return d;
}

static int download(FILE *f, const float *d, size_t n) {
  float *h = (float *)malloc(n * sizeof(float));
  if (!h || cudaMemcpy(h, d, n * sizeof(float), cudaMemcpyDeviceToHost) != cudaSuccess) { free(h); return 1; }
  int bad = fwrite(h, sizeof(float), n, f) != n;
  free(h);
  return bad;
}

int main(int argc, char **argv) {
  if (argc != 7) { fprintf(stderr, "usage: %s batch seqlen d_model tbar in.bin out.bin\n", argv[0]); return 1; }
  as_shape_t sh;
  sh.batch = atoi(argv[1]); sh.seqlen = atoll(argv[2]); sh.d_model = atoi(argv[3]); sh.d_state = 16;
  sh.io = AS_F32; sh.a_structure = AS_A_DIAGONAL;
  const long long tbar = atoll(argv[4]);
  const size_t P = (size_t)sh.d_model, N = 16, BTP = (size_t)sh.batch * (size_t)sh.seqlen * P;
  FILE *in = fopen(argv[5], "rb");
  if (!in) return 1;
  float *W_delta = upload(in, P * P), *b_delta = upload(in, P), *W_B = upload(in, N * P), *W_C = upload(in, N * P),
        *A_log = upload(in, P * N), *x = upload(in, BTP), *dy = upload(in, BTP);
  fclose(in);
  if (!W_delta || !b_delta || !W_B || !W_C || !A_log || !x || !dy) { fprintf(stderr, "short input\n"); return 1; }

  size_t fwd_bytes = 0, grad_bytes = 0;
  AS(as_workspace_bytes(&sh, tbar, &fwd_bytes, &grad_bytes));
  void *ws = NULL;
  float *y, *dW_delta, *db_delta, *dW_B, *dW_C, *dA_log, *dx;
  CK(cudaMalloc(&ws, grad_bytes));
  CK(cudaMalloc((void **)&y, BTP * 4)); CK(cudaMalloc((void **)&dx, BTP * 4));
  CK(cudaMalloc((void **)&dW_delta, P * P * 4)); CK(cudaMalloc((void **)&db_delta, P * 4));
  CK(cudaMalloc((void **)&dW_B, N * P * 4)); CK(cudaMalloc((void **)&dW_C, N * P * 4)); CK(cudaMalloc((void **)&dA_log, P * N * 4));

  as_params_t pr = {W_delta, b_delta, W_B, W_C, A_log};
  as_grads_t gr = {dW_delta, db_delta, dW_B, dW_C, dA_log, dx};
  cudaStream_t st;
  CK(cudaStreamCreate(&st));
  AS(as_ssm_forward(&sh, &pr, x, y, ws, grad_bytes, st));
  AS(as_adjoint_grad(&sh, &pr, x, dy, tbar, 0u, &gr, ws, grad_bytes, st));
  AS(as_check_status(ws, st));

  FILE *out = fopen(argv[6], "wb");
  if (!out) return 1;
  int bad = download(out, y, BTP) | download(out, dW_delta, P * P) | download(out, db_delta, P) | download(out, dW_B, N * P) |
            download(out, dW_C, N * P) | download(out, dA_log, P * N) | download(out, dx, BTP);
  fclose(out);
  printf("adjoint_ssm %d: forward + adjoint gradient of a [%d, %lld, %d] layer, window %lld: %s\n", as_version(), sh.batch,
         (long long)sh.seqlen, sh.d_model, tbar, bad ? "write failed" : "ok");
  return bad ? 1 : 0;
}
