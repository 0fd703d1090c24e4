/* A host written in plain C against include/step.h: no Python, no torch.  It owns the device memory (cudaMalloc),
 * drives one problem through the library - InitTraces, cache writes, decode attention, step scoring, the memory
 * trigger with eviction - and checks every result against arithmetic done right here in double precision.
 * Values are small multiples of 1/8, exact in bf16, so the only rounding is the kernel's own.
 * Prints "C-HOST OK" and exits 0 when everything agrees. */
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <cuda_runtime_api.h>

#include "step.h"

#define CHECK(x) do { int rc_ = (x); if (rc_ != 0) { fprintf(stderr, "%s failed: %d (line %d)\n", #x, rc_, __LINE__); return 1; } } while (0)

enum { L = 2, HQ = 8, HKV = 2, D = 128, P = 16, NB = 24, T = 4, MAXP = 6, PREFIX = 20, EXTRA = 15, SD = 64, SM = 64 };

static uint16_t bf16_of(float x) { uint32_t u; memcpy(&u, &x, 4); return (uint16_t)(u >> 16); }   /* exact for these values */
static float pattern(int a, int b, int c, int d) { return (float)(((a * 7 + b * 13 + c * 5 + d * 3) % 17) - 8) / 8.0f; }

/* K/V value of (trace, position, layer, head, dim); the first PREFIX positions are the shared prompt */
static float kval(int t, int pos, int l, int h, int d) { return pos < PREFIX ? pattern(pos, l, h, d) : pattern(pos + 31 * t, l + 2, h, d); }
static float vval(int t, int pos, int l, int h, int d) { return pos < PREFIX ? pattern(pos + 3, l, h, d + 1) : pattern(pos + 17 * t, l + 1, h, d + 2); }
static float qval(int t, int h, int d) { return pattern(t, h, d, 1) / 4.0f; }

int main(void) {
  kv_pool_config cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.num_layers = L; cfg.num_q_heads = HQ; cfg.num_kv_heads = HKV; cfg.head_dim = D; cfg.page_size = P;
  cfg.num_blocks = NB; cfg.max_traces = T; cfg.max_pages_per_trace = MAXP; cfg.dtype = STEP_BF16;
  cfg.max_score_rows = T; cfg.unscored_score = 1.0f;
  size_t kvb = 0, mb = 0;
  CHECK(kv_pool_required_bytes(&cfg, &kvb, &mb));
  CHECK(cudaMalloc(&cfg.kv_storage, kvb)); CHECK(cudaMalloc(&cfg.meta_storage, mb));
  cfg.kv_bytes = kvb; cfg.meta_bytes = mb;
  step_pool* pool = NULL;
  CHECK(kv_pool_create(&cfg, &pool));
  cudaStream_t s;
  CHECK(cudaStreamCreate(&s));

  /* InitTraces: T traces share a PREFIX-token prompt */
  size_t npre = (size_t)L * HKV * PREFIX * D;
  uint16_t *hk = malloc(npre * 2), *hv = malloc(npre * 2);
  for (int l = 0; l < L; ++l) for (int h = 0; h < HKV; ++h) for (int p = 0; p < PREFIX; ++p) for (int d = 0; d < D; ++d) {
    size_t i = (((size_t)l * HKV + h) * PREFIX + p) * D + d;
    hk[i] = bf16_of(kval(0, p, l, h, d)); hv[i] = bf16_of(vval(0, p, l, h, d));
  }
  void *dk, *dv;
  CHECK(cudaMalloc(&dk, npre * 2)); CHECK(cudaMalloc(&dv, npre * 2));
  CHECK(cudaMemcpy(dk, hk, npre * 2, cudaMemcpyHostToDevice)); CHECK(cudaMemcpy(dv, hv, npre * 2, cudaMemcpyHostToDevice));
  int32_t ids[T];
  CHECK(kv_pool_fork_prefix(pool, T, PREFIX, dk, dv, ids, s));
  for (int t = 0; t < T; ++t) if (ids[t] != t) { fprintf(stderr, "trace ids\n"); return 1; }

  /* NextToken's cache writes: EXTRA tokens per trace in one call */
  size_t nnew = (size_t)T * EXTRA * L * HKV * D;
  uint16_t *nk = malloc(nnew * 2), *nv = malloc(nnew * 2);
  for (int t = 0; t < T; ++t) for (int j = 0; j < EXTRA; ++j) for (int l = 0; l < L; ++l) for (int h = 0; h < HKV; ++h) for (int d = 0; d < D; ++d) {
    size_t i = ((((size_t)t * EXTRA + j) * L + l) * HKV + h) * D + d;
    nk[i] = bf16_of(kval(t, PREFIX + j, l, h, d)); nv[i] = bf16_of(vval(t, PREFIX + j, l, h, d));
  }
  void *dnk, *dnv; int32_t* dids;
  CHECK(cudaMalloc(&dnk, nnew * 2)); CHECK(cudaMalloc(&dnv, nnew * 2)); CHECK(cudaMalloc((void**)&dids, sizeof ids));
  CHECK(cudaMemcpy(dnk, nk, nnew * 2, cudaMemcpyHostToDevice)); CHECK(cudaMemcpy(dnv, nv, nnew * 2, cudaMemcpyHostToDevice));
  CHECK(cudaMemcpy(dids, ids, sizeof ids, cudaMemcpyHostToDevice));
  CHECK(append_kv(pool, dids, T, EXTRA, dnk, dnv, s));
  int used, free_, total, live;
  CHECK(kv_pool_stats(pool, &used, &free_, &total, &live, s));
  /* 1 shared full page + per trace: the private partial prompt page and one more page (20 + 15 = 35 tokens = 3 pages) */
  if (used != 1 + T * 2 || live != T || used + free_ != total) { fprintf(stderr, "stats %d %d %d %d\n", used, free_, total, live); return 1; }

  /* decode attention of layer 1 through the pool's own tables, against the definition in double */
  int32_t *bt, *sl; float* ts;
  CHECK(kv_pool_device_views(pool, &bt, &sl, &ts, NULL, NULL, NULL, NULL));
  size_t nq = (size_t)T * HQ * D;
  uint16_t* hq = malloc(nq * 2);
  for (int t = 0; t < T; ++t) for (int h = 0; h < HQ; ++h) for (int d = 0; d < D; ++d) hq[((size_t)t * HQ + h) * D + d] = bf16_of(qval(t, h, d));
  void* dq; float* dout;
  CHECK(cudaMalloc(&dq, nq * 2)); CHECK(cudaMalloc((void**)&dout, nq * 4));
  CHECK(cudaMemcpy(dq, hq, nq * 2, cudaMemcpyHostToDevice));
  CHECK(decode_attention(pool, 1, dq, bt, sl, T, dout, s));
  float* hout = malloc(nq * 4);
  CHECK(cudaMemcpyAsync(hout, dout, nq * 4, cudaMemcpyDeviceToHost, s));
  CHECK(cudaStreamSynchronize(s));
  const int S = PREFIX + EXTRA, G = HQ / HKV;
  double worst = 0.0;
  for (int t = 0; t < T; ++t) for (int h = 0; h < HQ; ++h) {
    double logit[PREFIX + EXTRA], mx = -1e300, den = 0.0;
    for (int j = 0; j < S; ++j) {
      double acc = 0.0;
      for (int d = 0; d < D; ++d) acc += (double)qval(t, h, d) * kval(t, j, 1, h / G, d);
      logit[j] = acc / sqrt((double)D);
      if (logit[j] > mx) mx = logit[j];
    }
    for (int j = 0; j < S; ++j) den += exp(logit[j] - mx);
    for (int d = 0; d < D; ++d) {
      double o = 0.0;
      for (int j = 0; j < S; ++j) o += exp(logit[j] - mx) / den * vval(t, j, 1, h / G, d);
      double e = fabs(o - hout[((size_t)t * HQ + h) * D + d]);
      if (e > worst) worst = e;
    }
  }
  if (!(worst <= 1e-2)) { fprintf(stderr, "attention error %g\n", worst); return 1; }

  /* step scorer: every trace ends a step; W1 = 1/8 on the diagonal block, so y = sigmoid(sum_j w2_j ReLU(h_j / 8 + b1_j) + b2) */
  uint16_t *hW1 = calloc((size_t)SM * SD, 2), hb1[SM], hw2[SM], *hh = malloc((size_t)T * SD * 2);
  for (int j = 0; j < SM; ++j) { hW1[(size_t)j * SD + j] = bf16_of(0.125f); hb1[j] = bf16_of((float)(j % 3 - 1) / 8.0f); hw2[j] = bf16_of((float)(j % 5 - 2) / 8.0f); }
  for (int t = 0; t < T; ++t) for (int k = 0; k < SD; ++k) hh[(size_t)t * SD + k] = bf16_of(pattern(t, k, 2, 0) * (float)(t + 1));
  void *dW1, *db1, *dw2, *dh; uint8_t* dmask; float* dys;
  CHECK(cudaMalloc(&dW1, (size_t)SM * SD * 2)); CHECK(cudaMalloc(&db1, SM * 2)); CHECK(cudaMalloc(&dw2, SM * 2));
  CHECK(cudaMalloc(&dh, (size_t)T * SD * 2)); CHECK(cudaMalloc((void**)&dmask, T)); CHECK(cudaMalloc((void**)&dys, T * 4));
  CHECK(cudaMemcpy(dW1, hW1, (size_t)SM * SD * 2, cudaMemcpyHostToDevice)); CHECK(cudaMemcpy(db1, hb1, SM * 2, cudaMemcpyHostToDevice));
  CHECK(cudaMemcpy(dw2, hw2, SM * 2, cudaMemcpyHostToDevice)); CHECK(cudaMemcpy(dh, hh, (size_t)T * SD * 2, cudaMemcpyHostToDevice));
  CHECK(cudaMemset(dmask, 1, T));
  scorer_weights w;
  w.W1 = dW1; w.b1 = db1; w.w2 = dw2; w.b2 = 0.25f; w.D = SD; w.m = SM; w.dtype = STEP_BF16;
  CHECK(score_steps(pool, dh, dmask, NULL, T, &w, dys, s));
  float ys[T], tsc[T];
  CHECK(cudaMemcpyAsync(ys, dys, sizeof ys, cudaMemcpyDeviceToHost, s));
  CHECK(cudaMemcpyAsync(tsc, ts, sizeof tsc, cudaMemcpyDeviceToHost, s));
  CHECK(cudaStreamSynchronize(s));
  double want[T];
  int argmin = 0;
  for (int t = 0; t < T; ++t) {
    double z = 0.25;
    for (int j = 0; j < SM; ++j) {
      double pre = pattern(t, j, 2, 0) * (t + 1) * 0.125 + (j % 3 - 1) / 8.0;
      z += (j % 5 - 2) / 8.0 * (pre > 0 ? pre : 0);
    }
    want[t] = 1.0 / (1.0 + exp(-z));
    if (fabs(want[t] - ys[t]) > 1e-3 || fabs(want[t] - tsc[t]) > 1e-3) { fprintf(stderr, "score %d: %g vs %g / %g\n", t, want[t], ys[t], tsc[t]); return 1; }
    if (want[t] < want[argmin]) argmin = t;
  }

  /* the memory trigger with the paper's rule (evict the argmin) at a threshold the pool is over */
  int32_t *dpr, *dnp, pr[T], np_;
  CHECK(cudaMalloc((void**)&dpr, sizeof pr)); CHECK(cudaMalloc((void**)&dnp, 4));
  CHECK(prune_if_saturated(pool, NULL, 0.3f, -1.0f, dpr, dnp, s));
  CHECK(cudaMemcpyAsync(pr, dpr, sizeof pr, cudaMemcpyDeviceToHost, s)); CHECK(cudaMemcpyAsync(&np_, dnp, 4, cudaMemcpyDeviceToHost, s));
  CHECK(cudaStreamSynchronize(s));
  if (np_ != 1 || pr[0] != argmin) { fprintf(stderr, "prune: %d evicted, first %d, expected trace %d\n", np_, pr[0], argmin); return 1; }
  CHECK(kv_pool_stats(pool, &used, &free_, &total, &live, s));
  if (live != T - 1 || used != 1 + (T - 1) * 2) { fprintf(stderr, "after prune: used %d live %d\n", used, live); return 1; }
  unsigned mask = 0;
  CHECK(kv_pool_last_error(pool, &mask, s));
  if (mask) { fprintf(stderr, "device status %u\n", mask); return 1; }
  CHECK(kv_pool_destroy(pool));
  printf("C-HOST OK (attention max err %.2e, %s)\n", worst, step_version());
  return 0;
}
