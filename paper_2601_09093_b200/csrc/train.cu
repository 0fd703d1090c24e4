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
// partial sums added in a fixed order, backward as a rank-B update with one CTA per 64 x 128 tile of dW1, which
// applies Adam to its tile straight from the accumulators (dW1 is never written out).  Between
// them a CTA per batch row makes the logit, loss term and dz, and a thread per hidden unit the small gradients.
// Every output element's sum runs over k (forward: within its K-slice) or over the batch rows (backward) in
// ascending order with one fused multiply-add per term, whatever the tiling: in Adam's first steps a gradient entry
// near zero decides its parameter's direction by its sign, so the order of summation is part of the result that the
// parameter tolerance (5e-6 against a double-precision run) was established with.  Everything is deterministic (no
// floating-point atomics).
#include "step_internal.cuh"

#include <math.h>

using namespace stepk;

namespace {

constexpr int kKStep = 16, kSplitK = 32;               // 32 K-slices: several CTAs per SM hide the load latency
constexpr int kFwdRows = 128, kFwdUnits = 64;          // forward tile: batch rows x hidden units, 8 x 4 outputs per thread
constexpr int kBwdUnits = 64, kBwdCols = 128;          // dW1 tile: hidden units x input dims, 4 x 8 outputs per thread
constexpr int kUnitRows = 16;                          // row slices of train_unit_kernel

template <typename T> __device__ inline float ldf(const T* p);
template <> __device__ inline float ldf<float>(const float* p) { return *p; }
template <> __device__ inline float ldf<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }

// One Adam step of one parameter (L2 decay folded into the gradient; c1, c2 = 1 - beta^step).
__device__ __forceinline__ void adam_update(float& w, float& mo, float& va, float g, const scorer_train_hyper& h, float c1, float c2) {
  g = fmaf(h.weight_decay, w, g);
  mo = h.beta1 * mo + (1.f - h.beta1) * g;
  va = h.beta2 * va + (1.f - h.beta2) * g * g;
  w = w - h.lr * (mo / c1) / (sqrtf(va / c2) + h.eps);
}

// part[s][b][j] = sum over the s-th slice of k of H[b][k] * W1[j][k].   grid (m tiles, B tiles, kSplitK), 256 threads,
// a thread owns an 8 x 4 block of the 128 x 64 tile: per k, two 16-byte reads of H values and one of W1 values from
// shared memory feed 32 multiply-adds.
template <typename T>
__global__ void __launch_bounds__(256)
train_fwd_kernel(const T* __restrict__ H, const float* __restrict__ W1, float* __restrict__ part, int B, int D, int m) {
  __shared__ __align__(16) float sA[kKStep][kFwdRows + 4], sB[kKStep][kFwdUnits + 4];
  const int j0 = blockIdx.x * kFwdUnits, b0 = blockIdx.y * kFwdRows;
  const int k_per = (D + kSplitK - 1) / kSplitK;
  const int k_lo = blockIdx.z * k_per, k_hi = min(D, k_lo + k_per);
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  dependents_may_launch();                               // the row kernel may take its places meanwhile
  float acc[8][4] = {};
  // the next tile's elements travel in registers while the current tile is multiplied
  float ra[8], rb[4];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int i = threadIdx.x + q * 256, r = i / kKStep, k = k0 + i % kKStep;
      ra[q] = (b0 + r < B && k < k_hi) ? ldf(H + (size_t)(b0 + r) * D + k) : 0.f;
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int i = threadIdx.x + q * 256, r = i / kKStep, k = k0 + i % kKStep;
      rb[q] = (j0 + r < m && k < k_hi) ? W1[(size_t)(j0 + r) * D + k] : 0.f;
    }
  };
  if (k_lo < k_hi) fetch(k_lo);
  for (int k0 = k_lo; k0 < k_hi; k0 += kKStep) {
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int i = threadIdx.x + q * 256;
      sA[i % kKStep][i / kKStep] = ra[q];
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int i = threadIdx.x + q * 256;
      sB[i % kKStep][i / kKStep] = rb[q];
    }
    __syncthreads();
    if (k0 + kKStep < k_hi) fetch(k0 + kKStep);
#pragma unroll
    for (int kk = 0; kk < kKStep; ++kk) {
      const float4 a0 = *reinterpret_cast<const float4*>(&sA[kk][ty * 8]);
      const float4 a1 = *reinterpret_cast<const float4*>(&sA[kk][ty * 8 + 4]);
      const float4 bq = *reinterpret_cast<const float4*>(&sB[kk][tx * 4]);
      const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float bv[4] = {bq.x, bq.y, bq.z, bq.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
  float* out = part + (size_t)blockIdx.z * B * m;
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int b = b0 + ty * 8 + i, u = j0 + tx * 4 + j;
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
  dependents_may_launch();
  wait_for_primary();                                    // the forward product
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
  dependents_may_launch();
  wait_for_primary();                                    // the rows' dz
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

// dW1[j][k] = sum_b dpre[b][j] * H[b][k], and Adam on W1 with it.   grid (D tiles, m tiles), 256 threads, 4 x (4 + 4)
// outputs of the 64 x 128 tile per thread; the gradient goes from the accumulators straight into the update of W1 and its
// moments (W1 is not read by this kernel's products, and the forward pass that read it is over).
template <typename T>
__global__ void __launch_bounds__(256)
train_bwd_adam_kernel(const float* __restrict__ dpre, const T* __restrict__ H, float* __restrict__ W1,
                      float* __restrict__ mom, float* __restrict__ var, int B, int D, int m, scorer_train_hyper h,
                      float c1, float c2) {
  __shared__ __align__(16) float sA[kKStep][kBwdUnits + 4], sB[kKStep][kBwdCols + 4];
  const int k0 = blockIdx.x * kBwdCols, j0 = blockIdx.y * kBwdUnits;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[4][8] = {};
  float ra[4], rb[8];
  // (a dependent of the small Adam kernel, which has itself waited for the kernel that leaves dpre)
  wait_for_primary();
  auto fetch = [&](int r0) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int i = threadIdx.x + q * 256, b = r0 + i / kBwdUnits, c = i % kBwdUnits;
      ra[q] = (b < B && j0 + c < m) ? dpre[(size_t)b * m + j0 + c] : 0.f;
    }
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int i = threadIdx.x + q * 256, b = r0 + i / kBwdCols, c = i % kBwdCols;
      rb[q] = (b < B && k0 + c < D) ? ldf(H + (size_t)b * D + k0 + c) : 0.f;
    }
  };
  fetch(0);
  for (int r0 = 0; r0 < B; r0 += kKStep) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int i = threadIdx.x + q * 256;
      sA[i / kBwdUnits][i % kBwdUnits] = ra[q];
    }
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int i = threadIdx.x + q * 256;
      sB[i / kBwdCols][i % kBwdCols] = rb[q];
    }
    __syncthreads();
    if (r0 + kKStep < B) fetch(r0 + kKStep);
#pragma unroll
    for (int rr = 0; rr < kKStep; ++rr) {
      const float4 aq = *reinterpret_cast<const float4*>(&sA[rr][ty * 4]);
      const float4 b0 = *reinterpret_cast<const float4*>(&sB[rr][tx * 4]);
      const float4 b1 = *reinterpret_cast<const float4*>(&sB[rr][kBwdCols / 2 + tx * 4]);
      const float av[4] = {aq.x, aq.y, aq.z, aq.w};
      const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
  // this thread's outputs: rows j0 + 4 ty + i, columns k0 + 4 tx + (0..3) and k0 + 64 + 4 tx + (0..3) - so that the
  // sixteen threads of a row group touch 256 contiguous bytes of W1 and of each moment at a time
  const bool vec = D % 4 == 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int u = j0 + ty * 4 + i;
    if (u >= m) continue;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const int k = k0 + half * (kBwdCols / 2) + tx * 4;
      const size_t idx = (size_t)u * D + k;
      if (vec && k + 3 < D) {
        float4 w = *reinterpret_cast<const float4*>(W1 + idx);
        float4 mo = *reinterpret_cast<const float4*>(mom + idx);
        float4 va = *reinterpret_cast<const float4*>(var + idx);
        adam_update(w.x, mo.x, va.x, acc[i][half * 4 + 0], h, c1, c2);
        adam_update(w.y, mo.y, va.y, acc[i][half * 4 + 1], h, c1, c2);
        adam_update(w.z, mo.z, va.z, acc[i][half * 4 + 2], h, c1, c2);
        adam_update(w.w, mo.w, va.w, acc[i][half * 4 + 3], h, c1, c2);
        *reinterpret_cast<float4*>(W1 + idx) = w;
        *reinterpret_cast<float4*>(mom + idx) = mo;
        *reinterpret_cast<float4*>(var + idx) = va;
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (k + j >= D) continue;
          float w = W1[idx + j], mo = mom[idx + j], va = var[idx + j];
          adam_update(w, mo, va, acc[i][half * 4 + j], h, c1, c2);
          W1[idx + j] = w; mom[idx + j] = mo; var[idx + j] = va;
        }
      }
    }
  }
}

// Adam for b1 [m], w2 [m], b2 [1]; their moments follow those of W1 [m * D] in mom / var.
__global__ void __launch_bounds__(256)
train_adam_small_kernel(float* __restrict__ b1, float* __restrict__ w2, float* __restrict__ b2,
                        const float* __restrict__ g_b1, const float* __restrict__ g_w2, const float* __restrict__ g_b2,
                        float* __restrict__ mom, float* __restrict__ var, size_t n_w1, int m,
                        scorer_train_hyper h, float c1, float c2) {      // c1, c2: 1 - beta^step, worked out on the host
  const int total = 2 * m + 1;
  dependents_may_launch();
  wait_for_primary();                                    // the small gradients
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
    float* p;
    float g;
    if (i < m) { p = b1 + i; g = g_b1[i]; }
    else if (i < 2 * m) { p = w2 + (i - m); g = g_w2[i - m]; }
    else { p = b2; g = g_b2[0]; }
    float w = *p, mo = mom[n_w1 + i], va = var[n_w1 + i];
    adam_update(w, mo, va, g, h, c1, c2);
    *p = w; mom[n_w1 + i] = mo; var[n_w1 + i] = va;
  }
}

struct TrainLayout { size_t part, dz, loss_terms, g_b1, g_w2, g_b2, total; };
TrainLayout train_layout(int B, int D, int m) {
  TrainLayout l;
  size_t off = 0;
  auto take = [&](size_t floats) { size_t o = off; off += (floats * 4 + 255) / 256 * 256; return o; };
  l.part = take((size_t)kSplitK * B * m);
  l.dz = take(B);
  l.loss_terms = take(B);
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
  float* g_b1 = (float*)(ws + l.g_b1);
  float* g_w2 = (float*)(ws + l.g_w2);
  float* g_b2 = (float*)(ws + l.g_b2);
  const dim3 gf((m + kFwdUnits - 1) / kFwdUnits, (B + kFwdRows - 1) / kFwdRows, kSplitK);
  const dim3 gb((D + kBwdCols - 1) / kBwdCols, (m + kBwdUnits - 1) / kBwdUnits);
  const float c1 = (float)(1.0 - pow((double)h->beta1, (double)h->step));
  const float c2 = (float)(1.0 - pow((double)h->beta2, (double)h->step));
  const size_t n_w1 = (size_t)m * D;
  if (hidden_dtype == STEP_BF16)
    train_fwd_kernel<__nv_bfloat16><<<gf, 256, 0, s>>>((const __nv_bfloat16*)hidden, W1, part, B, D, m);
  else
    train_fwd_kernel<float><<<gf, 256, 0, s>>>((const float*)hidden, W1, part, B, D, m);
  // the four launches behind the forward product are programmatic dependents of one another: each is scheduled while
  // the one before it drains and waits for it at its top
  bool ok = launch_dependent(train_row_kernel, dim3(B), dim3(256), 0, s, part, labels, (const float*)b1, (const float*)w2,
                             (const float*)b2, B, m, h->pos_weight, dz, loss_terms) == cudaSuccess;
  ok = ok && launch_dependent(train_unit_kernel, dim3((m + 31) / 32), dim3(32 * kUnitRows), 0, s, part, (const float*)w2,
                              (const float*)dz, (const float*)loss_terms, B, m, g_b1, g_w2, g_b2, loss_out) == cudaSuccess;
  // (the small tensors first: the unit kernel's w2 and the row kernel's b1 / b2 have been read by now)
  ok = ok && launch_dependent(train_adam_small_kernel, dim3((2 * m + 1 + 255) / 256), dim3(256), 0, s, b1, w2, b2,
                              (const float*)g_b1, (const float*)g_w2, (const float*)g_b2, adam_m, adam_v, n_w1, m, *h, c1, c2) == cudaSuccess;
  if (hidden_dtype == STEP_BF16)
    ok = ok && launch_dependent(train_bwd_adam_kernel<__nv_bfloat16>, gb, dim3(256), 0, s, (const float*)part,
                                (const __nv_bfloat16*)hidden, W1, adam_m, adam_v, B, D, m, *h, c1, c2) == cudaSuccess;
  else
    ok = ok && launch_dependent(train_bwd_adam_kernel<float>, gb, dim3(256), 0, s, (const float*)part, (const float*)hidden,
                                W1, adam_m, adam_v, B, D, m, *h, c1, c2) == cudaSuccess;
  if (!ok) return STEP_ERR_CUDA;
  return launch_ok();
}

}  // extern "C"
