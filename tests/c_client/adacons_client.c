/*
 * A plain C99 client of the AdaCons C ABI (include/adacons.h): no Python, no torch.
 *
 *   adacons_client N d beta steps [pitch [shards]]   < gradients
 *
 * reads steps * N * d float32 values (text, row-major, worker by worker) from standard input,
 * aggregates them step by step on the current CUDA device and prints, per step, one line each
 * of "gamma", "m" (momentum state), "out" and "flags".  With `pitch` > d the rows are placed
 * `pitch` elements apart on the device (ADACONS_OPT_ROW_PITCH) and the padding is filled with NaN.
 * With `shards` > 1 the columns are split into that many consecutive ranges, each with a context of
 * its own on the same device buffer, and every step runs in two halves (adacons_pass1 on every
 * range, then adacons_finish on every range with all the statistics records); the printed
 * coefficients are those of the first range, after a check that all ranges hold the same.
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
    fprintf(stderr, "usage: %s N d beta steps [pitch [shards]] < gradients\n", argv[0]);
    return 1;
  }
  const int N = atoi(argv[1]);
  const long long d = atoll(argv[2]);
  const double beta = atof(argv[3]);
  const int steps = atoi(argv[4]);
  const long long pitch = argc > 5 ? atoll(argv[5]) : d;
  const int shards = argc > 6 ? atoi(argv[6]) : 1;
  if (N < 1 || d < 1 || steps < 1 || pitch < d || shards < 1 || shards > 16 || shards > d) return 1;

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

  adacons_ctx *ctxs[16];
  long long col0[17];
  for (int r = 0; r <= shards; ++r) col0[r] = d * r / shards;
  for (int r = 0; r < shards; ++r) {
    ctxs[r] = NULL;
    CHECK_AC(adacons_create(&ctxs[r], N, (int64_t)(col0[r + 1] - col0[r]), ADACONS_F32, NULL, 0));
    CHECK_AC(adacons_set_option(ctxs[r], ADACONS_OPT_BETA, beta));
    if (pitch != col0[r + 1] - col0[r]) CHECK_AC(adacons_set_option(ctxs[r], ADACONS_OPT_ROW_PITCH, (double)pitch));
  }
  adacons_ctx *ctx = ctxs[0];
  int64_t rec = 0;
  CHECK_AC(adacons_get_info(ctx, ADACONS_INFO_STATS_DOUBLES, &rec));
  if (rec != 2 * N + 1) {
    fprintf(stderr, "a statistics record has %lld doubles, expected %d\n", (long long)rec, 2 * N + 1);
    return 2;
  }
  double *dev_stats = NULL;
  double *gamma_r = (double *)malloc(sizeof(double) * (size_t)N);
  if (!gamma_r) return 2;
  CHECK_CUDA(cudaMalloc((void **)&dev_stats, sizeof(double) * (size_t)rec * (size_t)shards));

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
    if (shards == 1) {
      CHECK_AC(adacons_aggregate(ctx, dev_g, dev_out, stream));
    } else {
      for (int r = 0; r < shards; ++r)
        CHECK_AC(adacons_pass1(ctxs[r], dev_g + col0[r], dev_stats + (size_t)r * (size_t)rec, stream));
      for (int r = 0; r < shards; ++r)
        CHECK_AC(adacons_finish(ctxs[r], dev_g + col0[r], dev_out + col0[r], dev_stats, shards, stream));
    }
    CHECK_CUDA(cudaMemcpyAsync(host_out, dev_out, sizeof(float) * (size_t)d, cudaMemcpyDeviceToHost, stream));
    CHECK_AC(adacons_get_coeffs(ctx, ADACONS_COEFF_GAMMA, gamma, stream));   /* synchronises the stream */
    int64_t step = 0;
    uint32_t flags = 0;
    CHECK_AC(adacons_get_state(ctx, m, &step, stream));
    CHECK_AC(adacons_get_status(ctx, &flags, stream));
    for (int r = 1; r < shards; ++r) {
      CHECK_AC(adacons_get_coeffs(ctxs[r], ADACONS_COEFF_GAMMA, gamma_r, stream));
      for (int i = 0; i < N; ++i)
        if (gamma_r[i] != gamma[i]) {
          fprintf(stderr, "range %d disagrees with range 0 on gamma[%d]\n", r, i);
          return 2;
        }
      uint32_t flags_r = 0;
      CHECK_AC(adacons_get_status(ctxs[r], &flags_r, stream));
      flags |= flags_r;
    }
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

  for (int r = 0; r < shards; ++r) CHECK_AC(adacons_destroy(ctxs[r]));
  CHECK_CUDA(cudaFree(dev_stats));
  free(gamma_r);
  CHECK_CUDA(cudaStreamDestroy(stream));
  CHECK_CUDA(cudaFree(dev_g));
  CHECK_CUDA(cudaFree(dev_out));
  free(host); free(host_out); free(gamma); free(m);
  return 0;
}
