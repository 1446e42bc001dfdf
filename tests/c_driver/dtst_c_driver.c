/* Plain-C driver for the DTST library: no Python, no C++.  It links against libdtst.so and the CUDA runtime,
 * reads a real field x[B][C_in][N...] (fp32) and weights W[C_in][C_out][M] (complex64) from binary files, runs
 * forward -> spectral_mul -> inverse through the C ABI with a caller-owned workspace, and writes Xhat and y back
 * to binary files.  The test that calls it compares those files with the float64 oracle.
 *
 * usage: dtst_c_driver d N_0..N_{d-1} k_0..k_{d-1} B C_in C_out x.bin W.bin Xhat.bin y.bin
 */
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#include <cuda_runtime_api.h>

#include "dtst.h"

static int fail(const char* what, int code) {
  fprintf(stderr, "dtst_c_driver: %s failed (%d: %s)\n", what, code, dtst_status_string(code));
  return 1;
}

static void* read_file(const char* path, size_t bytes) {
  FILE* f = fopen(path, "rb");
  void* buf = malloc(bytes);
  if (!f || !buf || fread(buf, 1, bytes, f) != bytes) {
    fprintf(stderr, "dtst_c_driver: cannot read %zu bytes from %s\n", bytes, path);
    exit(2);
  }
  fclose(f);
  return buf;
}

static void write_file(const char* path, const void* buf, size_t bytes) {
  FILE* f = fopen(path, "wb");
  if (!f || fwrite(buf, 1, bytes, f) != bytes) {
    fprintf(stderr, "dtst_c_driver: cannot write %s\n", path);
    exit(2);
  }
  fclose(f);
}

#define CUDA_OK(call)                                                                   \
  do {                                                                                  \
    cudaError_t e_ = (call);                                                            \
    if (e_ != cudaSuccess) {                                                            \
      fprintf(stderr, "dtst_c_driver: %s: %s\n", #call, cudaGetErrorString(e_));        \
      return 3;                                                                         \
    }                                                                                   \
  } while (0)

int main(int argc, char** argv) {
  if (argc < 2) return 64;
  const int d = atoi(argv[1]);
  if (d < 1 || d > DTST_MAX_DIMS || argc != 2 + 2 * d + 3 + 4) {
    fprintf(stderr, "usage: %s d N.. k.. B C_in C_out x.bin W.bin Xhat.bin y.bin\n", argv[0]);
    return 64;
  }
  int64_t N[DTST_MAX_DIMS], K[DTST_MAX_DIMS], M = 0;
  int32_t kmax[DTST_MAX_DIMS];
  size_t points = 1;
  for (int j = 0; j < d; ++j) {
    N[j] = atoll(argv[2 + j]);
    kmax[j] = atoi(argv[2 + d + j]);
    points *= (size_t)N[j];
  }
  const int B = atoi(argv[2 + 2 * d]), C_in = atoi(argv[3 + 2 * d]), C_out = atoi(argv[4 + 2 * d]);
  const char* fx = argv[5 + 2 * d];
  const char* fW = argv[6 + 2 * d];
  const char* fX = argv[7 + 2 * d];
  const char* fy = argv[8 + 2 * d];

  dtst_plan* plan = NULL;
  dtst_status st = dtst_plan_create(&plan, d, N, kmax, B, C_in, C_out);
  if (st != DTST_OK) return fail("dtst_plan_create", st);
  st = dtst_plan_num_modes(plan, &M, K);
  if (st != DTST_OK) return fail("dtst_plan_num_modes", st);
  printf("dtst %d: d=%d modes=%lld\n", dtst_version(), d, (long long)M);

  const size_t x_bytes = (size_t)B * C_in * points * sizeof(float);
  const size_t y_bytes = (size_t)B * C_out * points * sizeof(float);
  const size_t W_bytes = (size_t)C_in * C_out * (size_t)M * 8;
  const size_t X_bytes = (size_t)B * C_in * (size_t)M * 8;
  const size_t Y_bytes = (size_t)B * C_out * (size_t)M * 8;
  void* hx = read_file(fx, x_bytes);
  void* hW = read_file(fW, W_bytes);

  size_t ws_bytes = 0;
  st = dtst_plan_workspace_bytes(plan, &ws_bytes);
  if (st != DTST_OK) return fail("dtst_plan_workspace_bytes", st);
  void *ws = NULL, *dx = NULL, *dW = NULL, *dX = NULL, *dY = NULL, *dy = NULL;
  CUDA_OK(cudaMalloc(&ws, ws_bytes ? ws_bytes : 16));
  CUDA_OK(cudaMalloc(&dx, x_bytes));
  CUDA_OK(cudaMalloc(&dW, W_bytes));
  CUDA_OK(cudaMalloc(&dX, X_bytes));
  CUDA_OK(cudaMalloc(&dY, Y_bytes));
  CUDA_OK(cudaMalloc(&dy, y_bytes));
  st = dtst_plan_set_workspace(plan, ws, ws_bytes);
  if (st != DTST_OK) return fail("dtst_plan_set_workspace", st);
  CUDA_OK(cudaMemcpy(dx, hx, x_bytes, cudaMemcpyHostToDevice));
  CUDA_OK(cudaMemcpy(dW, hW, W_bytes, cudaMemcpyHostToDevice));

  cudaStream_t stream;
  CUDA_OK(cudaStreamCreate(&stream));
  st = dtst_forward(plan, (const float*)dx, dX, stream);
  if (st != DTST_OK) return fail("dtst_forward", st);
  st = dtst_spectral_mul(plan, dX, dW, dY, stream);
  if (st != DTST_OK) return fail("dtst_spectral_mul", st);
  st = dtst_inverse(plan, dY, (float*)dy, stream);
  if (st != DTST_OK) return fail("dtst_inverse", st);
  st = dtst_plan_status(plan, stream);   /* synchronises the stream and reads the device status word */
  if (st != DTST_OK) return fail("dtst_plan_status", st);

  void* hX = malloc(X_bytes);
  void* hy = malloc(y_bytes);
  if (!hX || !hy) return 2;
  CUDA_OK(cudaMemcpy(hX, dX, X_bytes, cudaMemcpyDeviceToHost));
  CUDA_OK(cudaMemcpy(hy, dy, y_bytes, cudaMemcpyDeviceToHost));
  write_file(fX, hX, X_bytes);
  write_file(fy, hy, y_bytes);

  int64_t launches = 0;
  dtst_plan_launch_count(plan, &launches);
  printf("kernel launches: %lld\n", (long long)launches);
  dtst_plan_destroy(plan);
  cudaFree(ws); cudaFree(dx); cudaFree(dW); cudaFree(dX); cudaFree(dY); cudaFree(dy);
  cudaStreamDestroy(stream);
  free(hx); free(hW); free(hX); free(hy);
  return 0;
}
