// scorer_train_step: one optimisation step of the step scorer (Sec. 3.1 "Training Objective"; appendix
// "Training Parameters": batch 128, Adam, learning rate 1e-4, weight decay 1e-5, BCE-with-logits).
//
//   pre = H W1^T + b1,  a = ReLU(pre),  z = a . w2 + b2
//   L   = -(1/B) sum_b ( alpha y_b log sigmoid(z_b) + (1 - y_b) log(1 - sigmoid(z_b)) ),  alpha = K- / K+
//   dz_b = ((1 - y_b) sigmoid(z_b) - alpha y_b (1 - sigmoid(z_b))) / B
//   dw2 = a^T dz,  db2 = sum dz,  dpre = (dz w2^T) * [pre > 0],  db1 = sum_b dpre,  dW1 = dpre^T H
//   Adam with L2 weight decay folded into the gradient (g += wd * p), bias-corrected moments.
//
// Parameters, moments and gradients are fp32.  The batch is small (the paper trains with 128 rows), so the two
// products (B x m x D each) are plain fp32 tiled GEMMs on CUDA cores: forward split over K across CTAs with the
// partial sums added in a fixed order, backward as a rank-B update with one CTA per 64 x 64 tile of dW1.  Between
// them a CTA per batch row makes the logit, loss term and dz, and a thread per hidden unit the small gradients.
// Everything is deterministic (no floating-point atomics).
#include "step_internal.cuh"

#include <math.h>

using namespace stepk;

namespace {

constexpr int kTile = 64, kKStep = 16, kSplitK = 32;   // 32 K-slices: several CTAs per SM hide the load latency
constexpr int kUnitRows = 16;                          // row slices of train_unit_kernel

template <typename T> __device__ inline float ldf(const T* p);
template <> __device__ inline float ldf<float>(const float* p) { return *p; }
template <> __device__ inline float ldf<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }

// part[s][b][j] = sum over the s-th slice of k of H[b][k] * W1[j][k].   grid (m tiles, B tiles, kSplitK), 256 threads,
// a thread owns a 4 x 4 block of the 64 x 64 tile.
template <typename T>
__global__ void __launch_bounds__(256)
train_fwd_kernel(const T* __restrict__ H, const float* __restrict__ W1, float* __restrict__ part, int B, int D, int m) {
  __shared__ float sA[kKStep][kTile + 1], sB[kKStep][kTile + 1];
  const int j0 = blockIdx.x * kTile, b0 = blockIdx.y * kTile;
  const int k_per = (D + kSplitK - 1) / kSplitK;
  const int k_lo = blockIdx.z * k_per, k_hi = min(D, k_lo + k_per);
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[4][4] = {};
  // the next tile's elements travel in registers while the current tile is multiplied
  float ra[4], rb[4];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int i = threadIdx.x + q * 256, r = i / kKStep, k = k0 + i % kKStep;
      ra[q] = (b0 + r < B && k < k_hi) ? ldf(H + (size_t)(b0 + r) * D + k) : 0.f;
      rb[q] = (j0 + r < m && k < k_hi) ? W1[(size_t)(j0 + r) * D + k] : 0.f;
    }
  };
  if (k_lo < k_hi) fetch(k_lo);
  for (int k0 = k_lo; k0 < k_hi; k0 += kKStep) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int i = threadIdx.x + q * 256;
      sA[i % kKStep][i / kKStep] = ra[q];
      sB[i % kKStep][i / kKStep] = rb[q];
    }
    __syncthreads();
    if (k0 + kKStep < k_hi) fetch(k0 + kKStep);
#pragma unroll
    for (int kk = 0; kk < kKStep; ++kk) {
      float av[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { av[i] = sA[kk][ty * 4 + i]; bv[i] = sB[kk][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
  float* out = part + (size_t)blockIdx.z * B * m;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int b = b0 + ty * 4 + i, u = j0 + tx * 4 + j;
      if (b < B && u < m) out[(size_t)b * m + u] = acc[i][j];
    }
}

// One CTA per batch row: pre (slices added in order, + b1, kept in part[0]) -> z, the row's loss term and dz.
__global__ void __launch_bounds__(256)
train_row_kernel(float* __restrict__ part, const float* __restrict__ labels, const float* __restrict__ b1,
                 const float* __restrict__ w2, const float* __restrict__ b2, int B, int m, float pos_weight,
                 float* __restrict__ dz, float* __restrict__ loss_terms) {
  __shared__ float s_red[8];
  const int b = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float z = 0.f;
  for (int j = threadIdx.x; j < m; j += blockDim.x) {
    const size_t i = (size_t)b * m + j;
    float p = 0.f;
    for (int s = 0; s < kSplitK; ++s) p += part[(size_t)s * B * m + i];
    p += b1[j];
    part[i] = p;
    z = fmaf(fmaxf(p, 0.f), w2[j], z);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
  if (lane == 0) s_red[warp] = z;
  __syncthreads();
  if (threadIdx.x == 0) {
    z = b2[0];
    for (int w = 0; w < 8; ++w) z += s_red[w];
    const float y = labels[b];
    // log sigmoid(z) = -softplus(-z), log(1 - sigmoid(z)) = -softplus(z), softplus(x) = max(x, 0) + log1p(exp(-|x|))
    const float sp_pos = fmaxf(z, 0.f) + log1pf(expf(-fabsf(z)));        // softplus(z)
    const float sp_neg = sp_pos - z;                                     // softplus(-z)
    const float sig = 1.f / (1.f + expf(-z));
    loss_terms[b] = pos_weight * y * sp_neg + (1.f - y) * sp_pos;
    dz[b] = ((1.f - y) * sig - pos_weight * y * (1.f - sig)) / (float)B;
  }
}

// dw2, db1 and dpre (in place) for 32 hidden units per CTA: thread (unit, slice) walks every kUnitRows-th row, the
// slices are added in order through shared memory; thread 0 of CTA 0 adds up the loss and db2.
__global__ void __launch_bounds__(32 * kUnitRows)
train_unit_kernel(float* __restrict__ part, const float* __restrict__ w2, const float* __restrict__ dz,
                  const float* __restrict__ loss_terms, int B, int m, float* __restrict__ g_b1, float* __restrict__ g_w2,
                  float* __restrict__ g_b2, float* __restrict__ loss_out) {
  __shared__ float s_gw[kUnitRows][32], s_gb[kUnitRows][32];
  const int u = threadIdx.x & 31, r = threadIdx.x >> 5;
  const int j = blockIdx.x * 32 + u;
  float gw = 0.f, gb = 0.f;
  if (j < m) {
    const float wj = w2[j];
    for (int b = r; b < B; b += kUnitRows) {
      const float p = part[(size_t)b * m + j], d = dz[b];
      gw = fmaf(fmaxf(p, 0.f), d, gw);
      const float dp = p > 0.f ? d * wj : 0.f;
      gb += dp;
      part[(size_t)b * m + j] = dp;
    }
  }
  s_gw[r][u] = gw; s_gb[r][u] = gb;
  __syncthreads();
  if (r == 0 && j < m) {
    gw = 0.f; gb = 0.f;
    for (int q = 0; q < kUnitRows; ++q) { gw += s_gw[q][u]; gb += s_gb[q][u]; }
    g_w2[j] = gw; g_b1[j] = gb;
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    float l = 0.f, sum = 0.f;
    for (int b = 0; b < B; ++b) { l += loss_terms[b]; sum += dz[b]; }
    *loss_out = l / (float)B;
    *g_b2 = sum;
  }
}

// g_W1[j][k] = sum_b dpre[b][j] * H[b][k].   grid (D tiles, m tiles), 256 threads, 4 x 4 outputs per thread.
template <typename T>
__global__ void __launch_bounds__(256)
train_bwd_kernel(const float* __restrict__ dpre, const T* __restrict__ H, float* __restrict__ g_W1, int B, int D, int m) {
  __shared__ float sA[kKStep][kTile + 1], sB[kKStep][kTile + 1];
  const int k0 = blockIdx.x * kTile, j0 = blockIdx.y * kTile;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[4][4] = {};
  float ra[4], rb[4];
  auto fetch = [&](int r0) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int i = threadIdx.x + q * 256, b = r0 + i / kTile, c = i % kTile;
      ra[q] = (b < B && j0 + c < m) ? dpre[(size_t)b * m + j0 + c] : 0.f;
      rb[q] = (b < B && k0 + c < D) ? ldf(H + (size_t)b * D + k0 + c) : 0.f;
    }
  };
  fetch(0);
  for (int r0 = 0; r0 < B; r0 += kKStep) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int i = threadIdx.x + q * 256;
      sA[i / kTile][i % kTile] = ra[q];
      sB[i / kTile][i % kTile] = rb[q];
    }
    __syncthreads();
    if (r0 + kKStep < B) fetch(r0 + kKStep);
#pragma unroll
    for (int rr = 0; rr < kKStep; ++rr) {
      float av[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { av[i] = sA[rr][ty * 4 + i]; bv[i] = sB[rr][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int u = j0 + ty * 4 + i, k = k0 + tx * 4 + j;
      if (u < m && k < D) g_W1[(size_t)u * D + k] = acc[i][j];
    }
}

// Adam over the four parameter tensors laid out one after another: W1 [m*D], b1 [m], w2 [m], b2 [1].
__global__ void __launch_bounds__(256)
train_adam_kernel(float* __restrict__ W1, float* __restrict__ b1, float* __restrict__ w2, float* __restrict__ b2,
                  const float* __restrict__ g_W1, const float* __restrict__ g_b1, const float* __restrict__ g_w2,
                  const float* __restrict__ g_b2, float* __restrict__ mom, float* __restrict__ var, size_t n_w1, int m,
                  scorer_train_hyper h, float c1, float c2) {      // c1, c2: 1 - beta^step, worked out on the host
  const size_t total = n_w1 + 2 * (size_t)m + 1;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    float* p;
    float g;
    if (i < n_w1) { p = W1 + i; g = g_W1[i]; }
    else if (i < n_w1 + m) { p = b1 + (i - n_w1); g = g_b1[i - n_w1]; }
    else if (i < n_w1 + 2 * (size_t)m) { p = w2 + (i - n_w1 - m); g = g_w2[i - n_w1 - m]; }
    else { p = b2; g = g_b2[0]; }
    const float w = *p;
    g = fmaf(h.weight_decay, w, g);
    const float mi = h.beta1 * mom[i] + (1.f - h.beta1) * g;
    const float vi = h.beta2 * var[i] + (1.f - h.beta2) * g * g;
    mom[i] = mi; var[i] = vi;
    *p = w - h.lr * (mi / c1) / (sqrtf(vi / c2) + h.eps);
  }
}

struct TrainLayout { size_t part, dz, loss_terms, g_W1, g_b1, g_w2, g_b2, total; };
TrainLayout train_layout(int B, int D, int m) {
  TrainLayout l;
  size_t off = 0;
  auto take = [&](size_t floats) { size_t o = off; off += (floats * 4 + 255) / 256 * 256; return o; };
  l.part = take((size_t)kSplitK * B * m);
  l.dz = take(B);
  l.loss_terms = take(B);
  l.g_W1 = take((size_t)m * D);
  l.g_b1 = take(m);
  l.g_w2 = take(m);
  l.g_b2 = take(1);
  l.total = off;
  return l;
}

}  // namespace

extern "C" {

size_t scorer_train_workspace_bytes(int B, int D, int m) {
  if (B < 1 || D < 1 || m < 1) return 0;
  return train_layout(B, D, m).total;
}

int scorer_train_step(const void* hidden, int hidden_dtype, const float* labels, int B, float* W1, float* b1,
                      float* w2, float* b2, int D, int m, float* adam_m, float* adam_v,
                      const scorer_train_hyper* h, void* workspace, size_t workspace_bytes, float* loss_out,
                      void* stream) {
  if (!hidden || !labels || !W1 || !b1 || !w2 || !b2 || !adam_m || !adam_v || !h || !workspace || !loss_out)
    return STEP_ERR_INVALID_ARG;
  if (B < 1 || D < 1 || m < 1 || h->step < 1) return STEP_ERR_INVALID_ARG;
  if (hidden_dtype != STEP_BF16 && hidden_dtype != STEP_FP32) return STEP_ERR_INVALID_ARG;
  if (!(h->beta1 >= 0.f && h->beta1 < 1.f) || !(h->beta2 >= 0.f && h->beta2 < 1.f) || !(h->eps > 0.f)) return STEP_ERR_INVALID_ARG;
  const TrainLayout l = train_layout(B, D, m);
  if (workspace_bytes < l.total || ((uintptr_t)workspace & 255)) return STEP_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  char* ws = (char*)workspace;
  float* part = (float*)(ws + l.part);
  float* dz = (float*)(ws + l.dz);
  float* loss_terms = (float*)(ws + l.loss_terms);
  float* g_W1 = (float*)(ws + l.g_W1);
  float* g_b1 = (float*)(ws + l.g_b1);
  float* g_w2 = (float*)(ws + l.g_w2);
  float* g_b2 = (float*)(ws + l.g_b2);
  const dim3 gf((m + kTile - 1) / kTile, (B + kTile - 1) / kTile, kSplitK);
  const dim3 gb((D + kTile - 1) / kTile, (m + kTile - 1) / kTile);
  if (hidden_dtype == STEP_BF16)
    train_fwd_kernel<__nv_bfloat16><<<gf, 256, 0, s>>>((const __nv_bfloat16*)hidden, W1, part, B, D, m);
  else
    train_fwd_kernel<float><<<gf, 256, 0, s>>>((const float*)hidden, W1, part, B, D, m);
  train_row_kernel<<<B, 256, 0, s>>>(part, labels, b1, w2, b2, B, m, h->pos_weight, dz, loss_terms);
  train_unit_kernel<<<(m + 31) / 32, 32 * kUnitRows, 0, s>>>(part, w2, dz, loss_terms, B, m, g_b1, g_w2, g_b2, loss_out);
  if (hidden_dtype == STEP_BF16)
    train_bwd_kernel<__nv_bfloat16><<<gb, 256, 0, s>>>(part, (const __nv_bfloat16*)hidden, g_W1, B, D, m);
  else
    train_bwd_kernel<float><<<gb, 256, 0, s>>>(part, (const float*)hidden, g_W1, B, D, m);
  const size_t n_w1 = (size_t)m * D;
  size_t blocks = (n_w1 + 2 * (size_t)m + 1 + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  const float c1 = (float)(1.0 - pow((double)h->beta1, (double)h->step));
  const float c2 = (float)(1.0 - pow((double)h->beta2, (double)h->step));
  train_adam_kernel<<<(unsigned)blocks, 256, 0, s>>>(W1, b1, w2, b2, g_W1, g_b1, g_w2, g_b2, adam_m, adam_v, n_w1, m, *h,
                                                     c1, c2);
  return launch_ok();
}

}  // extern "C"
