/*
 * The library used from plain C through include/razor.h alone: sizes, create, compress, append, decode.
 * One sequence, two fp32 heads of 64 dimensions, 40 prompt tokens + 1 appended token; head 0 keeps everything,
 * head 1 keeps 2 sinks + a window of 8 and the compensation token.  The outputs are checked against the two
 * formulas written out in double precision below (softmax attention; Eq. 5 with the mean of Eq. 4).
 * Exit code 0 and "c abi example ok" on success.  Built and run by tests/test_zy_c_example.py on a GPU.
 */
#include <cuda_runtime_api.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#include "razor.h"

#define H 2
#define D 64
#define N 40
#define NSINK 2
#define WINDOW 8
#define TOTAL (N + 1)

#define CHECK_RZ(call)                                                              \
  do {                                                                              \
    int rc_ = (call);                                                               \
    if (rc_ != 0) {                                                                 \
      fprintf(stderr, "%s -> %d (%s)\n", #call, rc_, razor_status_string(rc_));     \
      return 1;                                                                     \
    }                                                                               \
  } while (0)
#define CHECK_CUDA(call)                                                            \
  do {                                                                              \
    cudaError_t e_ = (call);                                                        \
    if (e_ != cudaSuccess) {                                                        \
      fprintf(stderr, "%s -> %s\n", #call, cudaGetErrorString(e_));                 \
      return 1;                                                                     \
    }                                                                               \
  } while (0)

static float K[H][TOTAL][D], V[H][TOTAL][D], q[H][D], out[H][D];

static float next_value(uint32_t* state) { /* small exact values: multiples of 1/8 in [-2, 2) */
  *state = *state * 1664525u + 1013904223u;
  return (float)((int)((*state >> 20) & 31) - 16) / 8.0f;
}

/* Eq. 5 (or plain softmax attention when nothing is dropped) for one head, in double precision. */
static void expected(int h, int keeps_all, double scale, double* o) {
  double logit[TOTAL + 1], weight[TOTAL + 1], vals[TOTAL + 1][D];
  int n = 0, first_recent = TOTAL - WINDOW, n_drop = keeps_all ? 0 : first_recent - NSINK;
  for (int p = 0; p < TOTAL; ++p) {
    if (!keeps_all && p >= NSINK && p < first_recent) continue; /* dropped */
    double s = 0;
    for (int d = 0; d < D; ++d) s += (double)q[h][d] * K[h][p][d];
    logit[n] = s * scale;
    weight[n] = 1.0;
    for (int d = 0; d < D; ++d) vals[n][d] = V[h][p][d];
    ++n;
  }
  if (n_drop > 0) { /* the compensation token: mean of the dropped keys and values, weight N_d */
    double s = 0;
    for (int d = 0; d < D; ++d) {
      double mk = 0, mv = 0;
      for (int p = NSINK; p < first_recent; ++p) {
        mk += K[h][p][d];
        mv += V[h][p][d];
      }
      s += (double)q[h][d] * (mk / n_drop);
      vals[n][d] = mv / n_drop;
    }
    logit[n] = s * scale;
    weight[n] = (double)n_drop;
    ++n;
  }
  double mx = logit[0], den = 0;
  for (int i = 1; i < n; ++i) mx = logit[i] > mx ? logit[i] : mx;
  for (int d = 0; d < D; ++d) o[d] = 0;
  for (int i = 0; i < n; ++i) {
    const double w = weight[i] * exp(logit[i] - mx);
    den += w;
    for (int d = 0; d < D; ++d) o[d] += w * vals[i][d];
  }
  for (int d = 0; d < D; ++d) o[d] /= den;
}

int main(void) {
  uint32_t state = 12345u;
  for (int h = 0; h < H; ++h)
    for (int p = 0; p < TOTAL; ++p)
      for (int d = 0; d < D; ++d) {
        K[h][p][d] = next_value(&state);
        V[h][p][d] = next_value(&state);
      }
  for (int h = 0; h < H; ++h)
    for (int d = 0; d < D; ++d) q[h][d] = next_value(&state);

  razor_config_t cfg;
  cfg.batch = 1; cfg.n_layers = 1; cfg.n_q_heads = H; cfg.n_kv_heads = H; cfg.head_dim = D;
  cfg.dtype = RAZOR_F32; cfg.page_tokens = 16; cfg.n_sink = NSINK; cfg.max_ctx_len = N; cfg.max_new_tokens = 1;
  cfg.use_compensation = 1; cfg.page_shuffle_seed = 0; cfg.sm_scale = 0.0f;
  const int32_t ctx_len[1] = {N}, window[1] = {WINDOW};
  const uint8_t retrieval[H] = {1, 0};

  size_t pool_bytes = 0, ws_bytes = 0;
  CHECK_RZ(razor_query_bytes(&cfg, ctx_len, window, retrieval, &pool_bytes, &ws_bytes));
  void *pool = NULL, *ws = NULL, *dK = NULL, *dV = NULL, *dq = NULL, *dk1 = NULL, *dv1 = NULL, *dout = NULL;
  CHECK_CUDA(cudaMalloc(&pool, pool_bytes));
  CHECK_CUDA(cudaMalloc(&ws, ws_bytes));
  CHECK_CUDA(cudaMalloc(&dK, sizeof(float) * H * N * D));
  CHECK_CUDA(cudaMalloc(&dV, sizeof(float) * H * N * D));
  CHECK_CUDA(cudaMalloc(&dq, sizeof(q)));
  CHECK_CUDA(cudaMalloc(&dk1, sizeof(float) * H * D));
  CHECK_CUDA(cudaMalloc(&dv1, sizeof(float) * H * D));
  CHECK_CUDA(cudaMalloc(&dout, sizeof(out)));
  float k1[H][D], v1[H][D];
  for (int h = 0; h < H; ++h) { /* dense prompt [1, H, N, D]; the appended token [1, H, D] */
    CHECK_CUDA(cudaMemcpy((float*)dK + (size_t)h * N * D, K[h], sizeof(float) * N * D, cudaMemcpyHostToDevice));
    CHECK_CUDA(cudaMemcpy((float*)dV + (size_t)h * N * D, V[h], sizeof(float) * N * D, cudaMemcpyHostToDevice));
    for (int d = 0; d < D; ++d) {
      k1[h][d] = K[h][N][d];
      v1[h][d] = V[h][N][d];
    }
  }
  CHECK_CUDA(cudaMemcpy(dk1, k1, sizeof(k1), cudaMemcpyHostToDevice));
  CHECK_CUDA(cudaMemcpy(dv1, v1, sizeof(v1), cudaMemcpyHostToDevice));
  CHECK_CUDA(cudaMemcpy(dq, q, sizeof(q), cudaMemcpyHostToDevice));

  razor_cache_t* cache = NULL;
  CHECK_RZ(razor_cache_create(&cache, &cfg, pool, pool_bytes, ws, ws_bytes, NULL));
  CHECK_RZ(razor_compress(cache, 0, dK, dV, (int64_t)H * N * D, (int64_t)N * D, D, ctx_len, retrieval, NSINK, window,
                          NULL));
  CHECK_RZ(razor_append(cache, 0, dk1, dv1, NULL));
  CHECK_RZ(razor_decode_attention(cache, 0, dq, (float*)dout, NULL));
  CHECK_CUDA(cudaMemcpy(out, dout, sizeof(out), cudaMemcpyDeviceToHost));
  int32_t status = -1;
  CHECK_RZ(razor_cache_device_status(cache, &status, NULL));
  if (status != 0) {
    fprintf(stderr, "device status %d\n", status);
    return 1;
  }

  double worst = 0;
  for (int h = 0; h < H; ++h) {
    double want[D];
    expected(h, retrieval[h], 1.0 / sqrt((double)D), want);
    for (int d = 0; d < D; ++d) {
      const double err = fabs((double)out[h][d] - want[d]);
      worst = err > worst ? err : worst;
    }
  }
  /* the same decode step as ONE call: compress again (same pages), then razor_decode_step */
  CHECK_RZ(razor_compress(cache, 0, dK, dV, (int64_t)H * N * D, (int64_t)N * D, D, ctx_len, retrieval, NSINK, window,
                          NULL));
  CHECK_RZ(razor_decode_step(cache, 0, dk1, dv1, dq, (float*)dout, NULL));
  CHECK_CUDA(cudaMemcpy(out, dout, sizeof(out), cudaMemcpyDeviceToHost));
  CHECK_RZ(razor_cache_device_status(cache, &status, NULL));
  if (status != 0) {
    fprintf(stderr, "device status %d after razor_decode_step\n", status);
    return 1;
  }
  for (int h = 0; h < H; ++h) {
    double want[D];
    expected(h, retrieval[h], 1.0 / sqrt((double)D), want);
    for (int d = 0; d < D; ++d) {
      const double err = fabs((double)out[h][d] - want[d]);
      worst = err > worst ? err : worst;
    }
  }
  CHECK_RZ(razor_cache_destroy(cache));
  cudaFree(pool); cudaFree(ws); cudaFree(dK); cudaFree(dV); cudaFree(dq); cudaFree(dk1); cudaFree(dv1); cudaFree(dout);
  if (!(worst <= 1e-5)) {
    fprintf(stderr, "max abs error %g\n", worst);
    return 1;
  }
  printf("c abi example ok: max abs error %.3g\n", worst);
  return 0;
}
