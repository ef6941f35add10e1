/*
 * fb4_hostcost -- what one call of the C ABI costs on the host, without any Python in the way.
 *
 * Small tensors are launch-bound (App. D.2 of the paper names kernel launches as the main overhead of the
 * method), so the time the host spends inside fb4_quantize / fb4_dequantize matters there.  The program
 * enqueues batches of quantize + decode pairs on a 256 x 3072 bf16 tensor and reports
 *   host_us_per_call : wall-clock time of the enqueueing loop / number of calls (minimum over the batches),
 *   gpu_us_per_pair  : CUDA-event time of a batch / number of pairs (the GPU side of the same stream).
 * Usage: fb4_hostcost [pairs per batch] [batches]; prints one JSON line.  Plain C99 against include/fb4.h.
 */
#define _POSIX_C_SOURCE 200809L
#include <cuda_runtime_api.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <time.h>

#include "fb4.h"

static double now_us(void) {
  struct timespec ts;
  clock_gettime(CLOCK_MONOTONIC, &ts);
  return ts.tv_sec * 1e6 + ts.tv_nsec * 1e-3;
}

#define CK(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) { fprintf(stderr, "%s: %s\n", #call, cudaGetErrorString(e_)); return 2; } } while (0)
#define FB(call) do { int r_ = (call); if (r_ != FB4_OK) { fprintf(stderr, "%s: %s\n", #call, fb4_strerror(r_)); return 3; } } while (0)

int main(int argc, char** argv) {
  const int pairs = argc > 1 ? atoi(argv[1]) : 200;
  const int batches = argc > 2 ? atoi(argv[2]) : 20;
  const int64_t T = 256, C = 3072;
  fb4_ctx* ctx = NULL;
  FB(fb4_init(&ctx, 0, NULL, NULL, NULL));
  uint16_t* hx = (uint16_t*)malloc((size_t)(T * C) * 2);
  uint32_t s = 12345u;
  for (int64_t i = 0; i < T * C; ++i) {           /* finite bf16 patterns with moderate exponents */
    s = s * 1664525u + 1013904223u;
    hx[i] = (uint16_t)(((s >> 16) & 0x807f) | (uint16_t)((120 + ((s >> 8) & 15)) << 7));
  }
  void *x, *codes, *meta, *out;
  CK(cudaMalloc(&x, (size_t)(T * C) * 2));
  CK(cudaMalloc(&codes, (size_t)(T * C / 2)));
  CK(cudaMalloc(&meta, (size_t)(T * C / 32) * 2));
  CK(cudaMalloc(&out, (size_t)(T * C) * 4));
  CK(cudaMemcpy(x, hx, (size_t)(T * C) * 2, cudaMemcpyHostToDevice));
  cudaStream_t st;
  CK(cudaStreamCreate(&st));
  cudaEvent_t e0, e1;
  CK(cudaEventCreate(&e0));
  CK(cudaEventCreate(&e1));
  for (int i = 0; i < 20; ++i) {
    FB(fb4_quantize(ctx, x, T, C, C, (uint8_t*)codes, (uint16_t*)meta, st));
    FB(fb4_dequantize(ctx, (const uint8_t*)codes, (const uint16_t*)meta, T, C, NULL, 0, NULL, NULL, out, 0, st));
  }
  CK(cudaStreamSynchronize(st));
  double best_host = 1e30, best_gpu = 1e30, best_q = 1e30;
  for (int b = 0; b < batches; ++b) {
    CK(cudaEventRecord(e0, st));
    const double t0 = now_us();
    for (int i = 0; i < pairs; ++i) {
      FB(fb4_quantize(ctx, x, T, C, C, (uint8_t*)codes, (uint16_t*)meta, st));
      FB(fb4_dequantize(ctx, (const uint8_t*)codes, (const uint16_t*)meta, T, C, NULL, 0, NULL, NULL, out, 0, st));
    }
    const double t1 = now_us();
    CK(cudaEventRecord(e1, st));
    CK(cudaStreamSynchronize(st));
    float ms = 0.f;
    CK(cudaEventElapsedTime(&ms, e0, e1));
    const double host = (t1 - t0) / (2.0 * pairs), gpu = ms * 1e3 / pairs;
    if (host < best_host) best_host = host;
    if (gpu < best_gpu) best_gpu = gpu;
    /* quantize alone */
    const double q0 = now_us();
    for (int i = 0; i < pairs; ++i) FB(fb4_quantize(ctx, x, T, C, C, (uint8_t*)codes, (uint16_t*)meta, st));
    const double q1 = now_us();
    CK(cudaStreamSynchronize(st));
    if ((q1 - q0) / pairs < best_q) best_q = (q1 - q0) / pairs;
  }
  uint32_t status = 0;
  FB(fb4_device_status(ctx, &status));
  printf("{\"tensor\": \"256x3072 bf16\", \"pairs_per_batch\": %d, \"batches\": %d, \"host_us_per_call\": %.3f, "
         "\"host_us_per_quantize_call\": %.3f, \"gpu_us_per_pair\": %.3f, \"device_status\": %u}\n",
         pairs, batches, best_host, best_q, best_gpu, status);
  fb4_destroy(ctx);
  return status ? 4 : 0;
}
