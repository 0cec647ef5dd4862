/*
 * A plain C99 client of the AdaCons C ABI (include/adacons.h): no Python, no torch.
 *
 *   adacons_client N d beta steps [pitch]   < gradients
 *
 * reads steps * N * d float32 values (text, row-major, worker by worker) from standard input,
 * aggregates them step by step on the current CUDA device and prints, per step, one line each
 * of "gamma", "m" (momentum state), "out" and "flags".  With `pitch` > d the rows are placed
 * `pitch` elements apart on the device (ADACONS_OPT_ROW_PITCH) and the padding is filled with NaN.
 * Exit code: 0 on success, 1 on a usage or input error, 2 when a library or CUDA call fails.
 */
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#include <cuda_runtime_api.h>

#include "adacons.h"

#define CHECK_AC(call)                                                                   \
  do {                                                                                   \
    int rc_ = (call);                                                                    \
    if (rc_ != ADACONS_OK) {                                                             \
      fprintf(stderr, "%s: %s (code %d)\n", #call, adacons_strerror(rc_), rc_);          \
      return 2;                                                                          \
    }                                                                                    \
  } while (0)
#define CHECK_CUDA(call)                                                                 \
  do {                                                                                   \
    cudaError_t e_ = (call);                                                             \
    if (e_ != cudaSuccess) {                                                             \
      fprintf(stderr, "%s: %s\n", #call, cudaGetErrorString(e_));                        \
      return 2;                                                                          \
    }                                                                                    \
  } while (0)

int main(int argc, char **argv) {
  if (argc < 5) {
    fprintf(stderr, "usage: %s N d beta steps [pitch] < gradients\n", argv[0]);
    return 1;
  }
  const int N = atoi(argv[1]);
  const long long d = atoll(argv[2]);
  const double beta = atof(argv[3]);
  const int steps = atoi(argv[4]);
  const long long pitch = argc > 5 ? atoll(argv[5]) : d;
  if (N < 1 || d < 1 || steps < 1 || pitch < d) return 1;

  float *host = (float *)malloc(sizeof(float) * (size_t)N * (size_t)pitch);
  float *host_out = (float *)malloc(sizeof(float) * (size_t)d);
  double *gamma = (double *)malloc(sizeof(double) * (size_t)N);
  double *m = (double *)malloc(sizeof(double) * (size_t)N);
  if (!host || !host_out || !gamma || !m) return 2;

  float *dev_g = NULL, *dev_out = NULL;
  cudaStream_t stream;
  CHECK_CUDA(cudaMalloc((void **)&dev_g, sizeof(float) * (size_t)N * (size_t)pitch));
  CHECK_CUDA(cudaMalloc((void **)&dev_out, sizeof(float) * (size_t)d));
  CHECK_CUDA(cudaStreamCreate(&stream));

  adacons_ctx *ctx = NULL;
  CHECK_AC(adacons_create(&ctx, N, (int64_t)d, ADACONS_F32, NULL, 0));
  CHECK_AC(adacons_set_option(ctx, ADACONS_OPT_BETA, beta));
  if (pitch != d) CHECK_AC(adacons_set_option(ctx, ADACONS_OPT_ROW_PITCH, (double)pitch));

  for (int t = 0; t < steps; ++t) {
    for (int i = 0; i < N; ++i) {
      for (long long k = 0; k < pitch; ++k) {
        float x = NAN;
        if (k < d && scanf("%f", &x) != 1) {
          fprintf(stderr, "input ended early (step %d, worker %d, element %lld)\n", t, i, k);
          return 1;
        }
        host[(size_t)i * (size_t)pitch + (size_t)k] = x;
      }
    }
    CHECK_CUDA(cudaMemcpyAsync(dev_g, host, sizeof(float) * (size_t)N * (size_t)pitch, cudaMemcpyHostToDevice, stream));
    CHECK_AC(adacons_aggregate(ctx, dev_g, dev_out, stream));
    CHECK_CUDA(cudaMemcpyAsync(host_out, dev_out, sizeof(float) * (size_t)d, cudaMemcpyDeviceToHost, stream));
    CHECK_AC(adacons_get_coeffs(ctx, ADACONS_COEFF_GAMMA, gamma, stream));   /* synchronises the stream */
    int64_t step = 0;
    uint32_t flags = 0;
    CHECK_AC(adacons_get_state(ctx, m, &step, stream));
    CHECK_AC(adacons_get_status(ctx, &flags, stream));
    if (step != t + 1) {
      fprintf(stderr, "step counter is %lld after %d aggregations\n", (long long)step, t + 1);
      return 2;
    }
    printf("gamma");
    for (int i = 0; i < N; ++i) printf(" %.17g", gamma[i]);
    printf("\nm");
    for (int i = 0; i < N; ++i) printf(" %.17g", m[i]);
    printf("\nout");
    for (long long k = 0; k < d; ++k) printf(" %.9g", (double)host_out[k]);
    printf("\nflags %u\n", (unsigned)flags);
  }

  CHECK_AC(adacons_destroy(ctx));
  CHECK_CUDA(cudaStreamDestroy(stream));
  CHECK_CUDA(cudaFree(dev_g));
  CHECK_CUDA(cudaFree(dev_out));
  free(host); free(host_out); free(gamma); free(m);
  return 0;
}
