// score_steps: the step scorer at step boundaries and the running-mean trace score.
//
//   y = sigmoid(w2 . ReLU(W1 h + b1) + b2)        (Sec. 3.1, "Model Architecture")
//   score_t = (1/n) sum_{i<=n} y_i^t               (Sec. 3.3)
//
// Only rows whose boundary flag is set are scored (Algorithm 1 runs the scorer when the new
// token ends a step), so one launch is
//   compact : ascending list of boundary rows (prefix sums within and across the CTAs of a cluster), NaN into the other rows;
//             it also decides, from the number of rows found, which first-layer kernel does the work
//   mlp     : few rows (a decode step: about one boundary per 64 traces) - score_mlp_kernel, CUDA
//             cores: for a tile of listed rows and a slice of the m hidden units the partial
//             w2 . ReLU(W1 h + b1), hidden rows staged in shared memory as fp32, W1 rows streamed with
//             16-byte loads;  many rows (batched scoring) - the tcgen05 kernel of scorer_tc.cu.
//             Both accumulate in fp32 and never round the activations.
//   finish  : fixed-order sum of the slices, + b2, sigmoid, scatter to the row; then every trace's new
//             scores are folded into its (sum, count) in ascending row order (per 512-row CTA, the
//             CTA partials in CTA order) and the mean is refreshed.
// A call with at most kSmallRows candidate rows - the shape of a decode step, one row per trace - does all of
// that in ONE launch (score_small_kernel): the three-launch form costs more in launch gaps than such a call
// has work.
#include "step_internal.cuh"
#include "block_scan.cuh"

#include <cooperative_groups.h>
#include <math.h>

using namespace stepk;

namespace {

constexpr int kCompactThreads = 1024;
constexpr int kRowTile = 8;       // listed rows per CTA
constexpr int kSplits = kScoreSplits;   // slices of the m hidden units
constexpr int kMlpWarps = 4;
constexpr int kFinishThreads = 1024;

template <typename T> __device__ inline float cvt(T x);
template <> __device__ inline float cvt<float>(float x) { return x; }
template <> __device__ inline float cvt<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

// tc_min_rows: 0 = the tensor-core kernel is not available for this launch; otherwise the smallest
// number of boundary rows that goes to it.  m: hidden units; num_sms: for the tiling choice.
// A thread looks at kRowsPerThread consecutive rows per pass.
// The step-end flag of row i is either mask[i] (tokens == nullptr) or, when the caller hands over the
// sampled token ids instead, table[tokens[i]]: a token ends a step if its text contains "\n\n" (Sec. 3.1,
// footnote), which the table records per vocabulary entry.  In that case the flags are also written to
// mask_out if it is given.  An id outside the vocabulary ends no step and is flagged.
constexpr int kRowsPerThread = 8;

__device__ inline bool row_flag(const FlagSource& f, int i, int32_t* counters) {
  if (f.live && !f.live[i]) {
    if (f.mask_out) f.mask_out[i] = 0;
    return false;
  }
  if (!f.tokens) return f.mask[i] != 0;
  const int id = f.tokens[i];
  bool e = false;
  if (id < 0 || id >= f.vocab) flag_error(counters, STEP_ERR_INVALID_ARG);
  else e = f.table[id] != 0;
  if (f.mask_out) f.mask_out[i] = e ? 1 : 0;
  return e;
}

// A cluster of kCompactCtas CTAs; CTA r owns the r-th contiguous share of the rows.  Pass 1 counts the step-end
// rows of the share, the counts are exchanged through distributed shared memory, pass 2 writes the row list
// (ascending over the whole launch) and NaN into the other rows.
constexpr int kCompactCtas = 8;

__global__ void __cluster_dims__(kCompactCtas, 1, 1) __launch_bounds__(kCompactThreads, 1)
score_compact_kernel(DevViews v, FlagSource src, int M, float* __restrict__ step_scores,
                     int tc_min_rows, int m, int num_sms) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank(), C = (int)cluster.num_blocks();
  __shared__ int s_warp[33];
  __shared__ int s_count, s_base, s_all;
  dependents_may_launch();       // the first-layer kernel may set itself up on the other SMs meanwhile
  const float nan = __int_as_float(0x7fc00000);
  const int span = blockDim.x * kRowsPerThread;
  const int share = ((M + C - 1) / C + span - 1) / span * span;       // rows per CTA, whole passes
  const int lo = min(M, rank * share), hi = min(M, lo + share);
  // pass 1: count (the flags of the share's first pass stay in a register for pass 2)
  int mine = 0;
  unsigned first_flags = 0;
  for (int base = lo; base < hi; base += span) {
    const int i0 = base + threadIdx.x * kRowsPerThread;
    unsigned flags = 0;
#pragma unroll
    for (int j = 0; j < kRowsPerThread; ++j)
      if (i0 + j < hi && row_flag(src, i0 + j, v.counters)) flags |= 1u << j;
    if (base == lo) first_flags = flags;
    mine += __popc(flags);
  }
  {
    int total;
    block_excl_scan(mine, s_warp, &total);
    if (threadIdx.x == 0) s_count = total;
  }
  cluster.sync();
  if (threadIdx.x == 0) {
    int before = 0, all = 0;
    for (int r = 0; r < C; ++r) {
      const int c = *cluster.map_shared_rank(&s_count, r);
      if (r < rank) before += c;
      all += c;
    }
    s_base = before; s_all = all;
  }
  __syncthreads();
  // pass 2: place
  int running = s_base;
  for (int base = lo; base < hi; base += span) {
    const int i0 = base + threadIdx.x * kRowsPerThread;
    unsigned flags = first_flags;
    if (base != lo) {
      flags = 0;
#pragma unroll
      for (int j = 0; j < kRowsPerThread; ++j)
        if (i0 + j < hi && row_flag(src, i0 + j, v.counters)) flags |= 1u << j;
    }
    int total;
    int at = running + block_excl_scan(__popc(flags), s_warp, &total);
#pragma unroll
    for (int j = 0; j < kRowsPerThread; ++j) {
      if (flags & (1u << j)) v.score_idx[at++] = i0 + j;
      else if (i0 + j < hi) step_scores[i0 + j] = nan;
    }
    running += total;
  }
  if (rank == 0 && threadIdx.x == 0) {
    const int nb = s_all;
    v.counters[C_SCORE_NB] = nb;
    v.counters[C_SCORE_TICKET] = 0;
    int N = 0;
    if (tc_min_rows > 0 && nb >= tc_min_rows) {
      // widest slice of hidden units per CTA (best reuse of the gathered rows) that still gives every SM
      // an item; else the narrowest, which spreads a small launch over the most SMs
      const int tiles = (nb + 127) / 128;
      for (int cand = 256; cand >= 64; cand >>= 1) {
        if (m % cand != 0 || m / cand > kSplits) continue;
        N = cand;
        if (tiles * (m / cand) >= num_sms) break;
      }
      // items of 256 rows (two accumulators sharing each W1 tile) if there are still enough of them
      v.counters[C_SCORE_TILE] = ((nb + 255) / 256) * (m / N) >= num_sms ? 256 : 128;
    }
    v.counters[C_SCORE_TC] = N;
    v.counters[C_SCORE_SLICES] = N ? m / N : kSplits;
  }
  cluster.sync();                        // no CTA leaves while its count may still be read
}

// grid (kSplits, row tiles).  Dynamic shared memory: kRowTile * D floats.
template <typename T>
__global__ void __launch_bounds__(kMlpWarps * 32)
score_mlp_kernel(DevViews v, const T* __restrict__ hidden, const T* __restrict__ W1, const T* __restrict__ b1,
                 const T* __restrict__ w2, int D, int m) {
  extern __shared__ float s_h[];                      // [kRowTile][D]
  __shared__ float s_part[kMlpWarps][kRowTile];
  if (v.counters[C_SCORE_TC] != 0) return;            // this launch's rows belong to the tensor-core kernel
  const int nb = v.counters[C_SCORE_NB];
  const int r0 = blockIdx.y * kRowTile;
  if (r0 >= nb) return;
  const int rows = min(kRowTile, nb - r0);
  const int split = blockIdx.x;
  const int per = (m + kSplits - 1) / kSplits;
  const int j0 = split * per, j1 = min(m, j0 + per);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int r = 0; r < kRowTile; ++r) {
    if (r < rows) {
      const T* src = hidden + (size_t)v.score_idx[r0 + r] * D;
      for (int k = threadIdx.x; k < D; k += blockDim.x) s_h[r * D + k] = cvt(src[k]);
    } else {
      for (int k = threadIdx.x; k < D; k += blockDim.x) s_h[r * D + k] = 0.f;
    }
  }
  __syncthreads();
  float zpart[kRowTile];
#pragma unroll
  for (int r = 0; r < kRowTile; ++r) zpart[r] = 0.f;
  for (int j = j0 + warp; j < j1; j += kMlpWarps) {
    const T* wrow = W1 + (size_t)j * D;
    float acc[kRowTile];
#pragma unroll
    for (int r = 0; r < kRowTile; ++r) acc[r] = 0.f;
    for (int k = lane; k < D; k += 32) {
      const float w = cvt(wrow[k]);
#pragma unroll
      for (int r = 0; r < kRowTile; ++r) acc[r] += w * s_h[r * D + k];
    }
    const float bj = cvt(b1[j]), wj = cvt(w2[j]);
#pragma unroll
    for (int r = 0; r < kRowTile; ++r) {
      float a = acc[r];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
      a += bj;
      zpart[r] += wj * fmaxf(a, 0.f);
    }
  }
  if (lane == 0)
    for (int r = 0; r < kRowTile; ++r) s_part[warp][r] = zpart[r];
  __syncthreads();
  if (threadIdx.x < rows) {
    float z = 0.f;
    for (int w = 0; w < kMlpWarps; ++w) z += s_part[w][threadIdx.x];
    v.score_z[(size_t)(r0 + threadIdx.x) * kSplits + split] = z;
  }
}

// Finishing kernel.  CTA c owns listed rows [c * kScoreFoldRows, ...):
//   1. per row: slices in fixed order, + b2, sigmoid, scatter to step_scores;
//   2. per trace: the sum and count of this CTA's rows that belong to it, rows in ascending order
//      (a thread per trace walks the CTA's rows in shared memory), written as one partial;
//   3. the CTA that finishes last adds the partials of every trace in CTA order to the trace's running
//      (sum, count) and refreshes the mean - a fixed order, whichever CTA happens to be last.
__global__ void __launch_bounds__(kFinishThreads)
score_finish_kernel(DevViews v, Geo g, const int32_t* __restrict__ row_trace, int row_base, float b2,
                    float unscored, float* __restrict__ step_scores) {
  __shared__ float s_y[kScoreFoldRows];
  __shared__ int s_tr[kScoreFoldRows];
  __shared__ float2 s_run[kFinishThreads];
  __shared__ int s_last;
  wait_for_primary();            // launched as a dependent of the first-layer kernel
  const int nb = v.counters[C_SCORE_NB], ns = v.counters[C_SCORE_SLICES];
  const int chunks = (nb + kScoreFoldRows - 1) / kScoreFoldRows;
  const int c = blockIdx.x;
  if (c >= chunks) return;
  const int r0 = c * kScoreFoldRows, n = min(kScoreFoldRows, nb - r0);
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    const int r = r0 + i;
    float z = 0.f;
    for (int s = 0; s < ns; ++s) z += v.score_z[(size_t)r * kSplits + s];
    z += b2;
    const float y = 1.f / (1.f + expf(-z));
    const int row = v.score_idx[r];
    step_scores[row] = y;
    const int tr = row_trace ? row_trace[row] : row + row_base;
    if (tr < 0 || tr >= g.max_traces) flag_error(v.counters, STEP_ERR_BAD_TRACE);   // names no trace of this pool
    s_y[i] = y; s_tr[i] = tr;
  }
  __syncthreads();
  for (int t = threadIdx.x; t < g.max_traces; t += blockDim.x) {
    float sum = 0.f;
    int cnt = 0;
    for (int i = 0; i < n; ++i)
      if (s_tr[i] == t) { sum += s_y[i]; ++cnt; }
    v.score_part[(size_t)c * g.max_traces + t] = make_float2(sum, __int_as_float(cnt));
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = atomicAdd(&v.counters[C_SCORE_TICKET], 1) == chunks - 1;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  // every trace's partials are summed by `groups` threads, each over a contiguous run of CTAs, and the runs are
  // then added in order: the same fixed order whoever is last, with the loads spread over the whole CTA
  const int T = g.max_traces;
  const int Tc = min(T, (int)blockDim.x), groups = max(1, (int)blockDim.x / Tc);
  const int cpg = (chunks + groups - 1) / groups;
  const int tl = threadIdx.x % Tc, grp = threadIdx.x / Tc;
  for (int base = 0; base < T; base += Tc) {
    const int t = base + tl;
    float sum = 0.f;
    int cnt = 0;
    if (grp < groups && t < T) {
      const int k_end = min(chunks, (grp + 1) * cpg);
      for (int k0 = grp * cpg; k0 < k_end; k0 += 8) {
        float2 p[8];                       // eight loads in flight, then added in CTA order
#pragma unroll
        for (int j = 0; j < 8; ++j)
          p[j] = k0 + j < k_end ? __ldcg(&v.score_part[(size_t)(k0 + j) * T + t]) : make_float2(0.f, 0.f);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int pc = __float_as_int(p[j].y);
          if (pc) { sum += p[j].x; cnt += pc; }
        }
      }
    }
    s_run[threadIdx.x] = make_float2(sum, __int_as_float(cnt));
    __syncthreads();
    if (grp == 0 && t < T) {
      float tot = v.score_sum[t];
      int n_tot = v.score_cnt[t];
      for (int q = 0; q < groups; ++q) {
        const float2 r = s_run[q * Tc + tl];
        const int rc = __float_as_int(r.y);
        if (rc) { tot += r.x; n_tot += rc; }
      }
      v.score_sum[t] = tot; v.score_cnt[t] = n_tot;
      v.trace_scores[t] = n_tot > 0 ? tot / (float)n_tot : unscored;
    }
    __syncthreads();
  }
}

// ---------------------------------------------------------------- one launch for a decode step's rows
// grid = S CTAs, CTA c owns hidden units [c * mu, (c + 1) * mu).  Every CTA builds the same ascending list of
// step-end rows from the flags (M <= kSmallRows, one thread per row; only CTA 0 writes mask_out and error flags),
// then, for tiles of kRowTile listed rows staged in shared memory as fp32, its warps take the CTA's units one by
// one (lanes over D, 16-byte loads of the W1 row) and the CTA's partial w2 . ReLU(W1 h + b1) per row goes to
// score_zs[row][c].  The CTA that finishes last adds the partials in CTA order, applies b2 and the sigmoid, writes
// every row's output (NaN where no step ends), folds the new scores into the traces' running means in ascending
// row order and refreshes the means.  Dynamic shared memory: kRowTile * D floats.
template <typename T> __device__ inline void load4(const T* p, float (&w)[4]);
template <> __device__ inline void load4<float>(const float* p, float (&w)[4]) {
  const float4 x = *reinterpret_cast<const float4*>(p);
  w[0] = x.x; w[1] = x.y; w[2] = x.z; w[3] = x.w;
}
template <> __device__ inline void load4<__nv_bfloat16>(const __nv_bfloat16* p, float (&w)[4]) {
  const uint2 x = *reinterpret_cast<const uint2*>(p);
  w[0] = __uint_as_float(x.x << 16); w[1] = __uint_as_float(x.x & 0xffff0000u);
  w[2] = __uint_as_float(x.y << 16); w[3] = __uint_as_float(x.y & 0xffff0000u);
}

constexpr int kSmallThreads = 256;
constexpr int kSmallWarps = kSmallThreads / 32;

template <typename T>
__global__ void __launch_bounds__(kSmallThreads)
score_small_kernel(DevViews v, Geo g, FlagSource src, const T* __restrict__ hidden, const int32_t* __restrict__ row_trace,
                   int M, const T* __restrict__ W1, const T* __restrict__ b1, const T* __restrict__ w2, float b2,
                   int D, int m, float unscored, float* __restrict__ step_scores, float* __restrict__ trace_scores_out, int n_out) {
  extern __shared__ float s_h[];                      // [kRowTile][D]
  __shared__ int s_list[kSmallRows];
  __shared__ int s_wcnt[kSmallWarps + 1];
  __shared__ float s_part[kSmallWarps][kRowTile];
  __shared__ float s_y[kSmallRows];
  __shared__ int s_tr[kSmallRows];
  __shared__ int s_last;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int S = gridDim.x, c = blockIdx.x;
  const int mu = (m + S - 1) / S;
  const int j0 = c * mu, j1 = min(m, j0 + mu);
  const bool vec4 = D % 4 == 0 && ((uintptr_t)W1 & 15) == 0;
  // The W1 row of this warp's first unit does not depend on which rows end a step: its loads (the first kPrefetch
  // steps of four elements per lane) are issued before anything else, so that their latency - W1 is usually not in
  // the L2 - runs alongside the flag scan and the staging of the hidden rows.
  constexpr int kPrefetch = 32;
  float wpre[kPrefetch][4];
  if (vec4 && j0 + warp < j1) {
    const T* wrow = W1 + (size_t)(j0 + warp) * D;
#pragma unroll
    for (int u = 0; u < kPrefetch; ++u)
      if (lane * 4 + u * 128 < D) load4(wrow + lane * 4 + u * 128, wpre[u]);
  }
  // ---- the list of step-end rows (the same in every CTA)
  FlagSource quiet = src;
  if (c != 0) quiet.mask_out = nullptr;
  int32_t* err = c == 0 ? v.counters : nullptr;
  bool f = false;
  if ((int)threadIdx.x < M) {
    if (quiet.live && !quiet.live[threadIdx.x]) { if (quiet.mask_out) quiet.mask_out[threadIdx.x] = 0; }
    else if (!quiet.tokens) f = quiet.mask[threadIdx.x] != 0;
    else {
      const int id = quiet.tokens[threadIdx.x];
      if (id < 0 || id >= quiet.vocab) { if (err) flag_error(err, STEP_ERR_INVALID_ARG); }
      else f = quiet.table[id] != 0;
      if (quiet.mask_out) quiet.mask_out[threadIdx.x] = f ? 1 : 0;
    }
  }
  const unsigned bal = __ballot_sync(0xffffffffu, f);
  if (lane == 0) s_wcnt[warp] = __popc(bal);
  __syncthreads();
  int before = 0, nb = 0;
  for (int w = 0; w < kSmallWarps; ++w) { if (w < warp) before += s_wcnt[w]; nb += s_wcnt[w]; }
  if (f) s_list[before + __popc(bal & ((1u << lane) - 1))] = threadIdx.x;
  __syncthreads();
  // ---- this CTA's units, tile by tile of the listed rows
  for (int r0 = 0; r0 < nb && j0 < j1; r0 += kRowTile) {
    const int rows = min(kRowTile, nb - r0);
    if (vec4 && ((uintptr_t)hidden & 15) == 0) {
      // all rows' loads first (four elements per thread and step), then the stores
      for (int k = threadIdx.x * 4; k < D; k += blockDim.x * 4) {
        float hv[kRowTile][4];
#pragma unroll
        for (int r = 0; r < kRowTile; ++r)
          if (r < rows) load4(hidden + (size_t)s_list[r0 + r] * D + k, hv[r]);
#pragma unroll
        for (int r = 0; r < kRowTile; ++r)
          *reinterpret_cast<float4*>(&s_h[r * D + k]) = r < rows ? make_float4(hv[r][0], hv[r][1], hv[r][2], hv[r][3])
                                                               : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    } else {
      for (int r = 0; r < kRowTile; ++r) {
        if (r < rows) {
          const T* hs = hidden + (size_t)s_list[r0 + r] * D;
          for (int k = threadIdx.x; k < D; k += blockDim.x) s_h[r * D + k] = cvt(hs[k]);
        } else {
          for (int k = threadIdx.x; k < D; k += blockDim.x) s_h[r * D + k] = 0.f;
        }
      }
    }
    __syncthreads();
    float zpart[kRowTile];
#pragma unroll
    for (int r = 0; r < kRowTile; ++r) zpart[r] = 0.f;
    for (int j = j0 + warp; j < j1; j += kSmallWarps) {
      const T* wrow = W1 + (size_t)j * D;
      float acc[kRowTile];
#pragma unroll
      for (int r = 0; r < kRowTile; ++r) acc[r] = 0.f;
      if (vec4) {
        // four consecutive k per lane and step: one 8- or 16-byte load of the W1 row, one 16-byte load per staged
        // hidden row.  W1 is usually not in the L2 (the attention launches before this call stream gigabytes through
        // it), so the loads of eight steps are issued together: what this loop costs is its dependent round trips.
        int k_from = lane * 4;
        if (j == j0 + warp) {
          // this warp's first unit: the prefetched part of its row
#pragma unroll
          for (int u = 0; u < kPrefetch; ++u) {
            if (lane * 4 + u * 128 < D) {
#pragma unroll
              for (int r = 0; r < kRowTile; ++r) {
                const float4 hv = *reinterpret_cast<const float4*>(&s_h[r * D + lane * 4 + u * 128]);
                acc[r] += wpre[u][0] * hv.x + wpre[u][1] * hv.y + wpre[u][2] * hv.z + wpre[u][3] * hv.w;
              }
            }
          }
          k_from += kPrefetch * 128;
        }
        for (int k0 = k_from; k0 < D; k0 += 128 * 8) {
          float wv[8][4];
#pragma unroll
          for (int u = 0; u < 8; ++u)
            if (k0 + u * 128 < D) load4(wrow + k0 + u * 128, wv[u]);
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            if (k0 + u * 128 < D) {
#pragma unroll
              for (int r = 0; r < kRowTile; ++r) {
                const float4 hv = *reinterpret_cast<const float4*>(&s_h[r * D + k0 + u * 128]);
                acc[r] += wv[u][0] * hv.x + wv[u][1] * hv.y + wv[u][2] * hv.z + wv[u][3] * hv.w;
              }
            }
          }
        }
      } else {
        for (int k = lane; k < D; k += 32) {
          const float wv = cvt(wrow[k]);
#pragma unroll
          for (int r = 0; r < kRowTile; ++r) acc[r] += wv * s_h[r * D + k];
        }
      }
      const float bj = cvt(b1[j]), wj = cvt(w2[j]);
#pragma unroll
      for (int r = 0; r < kRowTile; ++r) {
        float x = acc[r];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
        zpart[r] += wj * fmaxf(x + bj, 0.f);
      }
    }
    if (lane == 0)
      for (int r = 0; r < kRowTile; ++r) s_part[warp][r] = zpart[r];
    __syncthreads();
    if ((int)threadIdx.x < rows) {
      float z = 0.f;
      for (int w = 0; w < kSmallWarps; ++w) z += s_part[w][threadIdx.x];       // warps in order: a fixed sum
      v.score_zs[(size_t)(r0 + threadIdx.x) * kSmallCtas + c] = z;
    }
    __syncthreads();
  }
  // ---- whoever finishes last completes the call
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = atomicAdd(&v.counters[C_SCORE_TICKET], 1) == S - 1;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const int used = min(S, (m + mu - 1) / mu);                                   // CTAs that own units
  const float nan = __int_as_float(0x7fc00000);
  if ((int)threadIdx.x < M && !f) step_scores[threadIdx.x] = nan;
  // a warp per listed row: lane l adds the partials of CTAs l, l + 32, ... in that order, then the lanes are added
  // in a fixed tree - the same sum whoever is last
  for (int i = warp; i < nb; i += kSmallWarps) {
    float z = 0.f;
    for (int k = lane; k < used; k += 32) z += __ldcg(&v.score_zs[(size_t)i * kSmallCtas + k]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    if (lane == 0) {
      z += b2;
      const float y = 1.f / (1.f + expf(-z));
      const int row = s_list[i];
      step_scores[row] = y;
      const int tr = row_trace ? row_trace[row] : row;
      if (tr < 0 || tr >= g.max_traces) flag_error(v.counters, STEP_ERR_BAD_TRACE);   // names no trace of this pool
      s_y[i] = y; s_tr[i] = tr;
    }
  }
  __syncthreads();
  for (int t = threadIdx.x; t < g.max_traces; t += blockDim.x) {
    float sum = v.score_sum[t];
    int cnt = v.score_cnt[t];
    for (int i = 0; i < nb; ++i)
      if (s_tr[i] == t) { sum += s_y[i]; ++cnt; }
    v.score_sum[t] = sum; v.score_cnt[t] = cnt;
    const float mean = cnt > 0 ? sum / (float)cnt : unscored;
    v.trace_scores[t] = mean;
    if (trace_scores_out && t < n_out) trace_scores_out[t] = mean;
  }
  if (threadIdx.x == 0) {
    v.counters[C_SCORE_TICKET] = 0;
    v.counters[C_SCORE_NB] = nb; v.counters[C_SCORE_TC] = 0; v.counters[C_SCORE_SLICES] = used;
  }
}

// step-end detection alone: mask[i] = table[tokens[i]]
__global__ void __launch_bounds__(256)
step_end_kernel(FlagSource src, int M, int32_t* counters) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < M; i += gridDim.x * blockDim.x) row_flag(src, i, counters);
}

}  // namespace

extern "C" int score_steps(step_pool* pool, const void* hidden, const uint8_t* boundary_mask,
                           const int32_t* row_trace, int M, const scorer_weights* w,
                           float* step_scores_out, void* stream) {
  if (!pool || M < 0 || !w) return STEP_ERR_INVALID_ARG;
  if (M == 0) return STEP_OK;
  if (!boundary_mask) return STEP_ERR_INVALID_ARG;
  FlagSource src{boundary_mask, nullptr, nullptr, 0, nullptr, nullptr};
  return score_steps_impl(pool, hidden, src, row_trace, M, w, step_scores_out, nullptr, 0, stream);
}

extern "C" int score_steps_tokens(step_pool* pool, const void* hidden, const int32_t* token_ids,
                                  const uint8_t* step_end_table, int vocab, const int32_t* row_trace, int M,
                                  const scorer_weights* w, float* step_scores_out, uint8_t* boundary_mask_out,
                                  void* stream) {
  if (!pool || M < 0 || !w) return STEP_ERR_INVALID_ARG;
  if (M == 0) return STEP_OK;
  if (!token_ids || !step_end_table || vocab < 1) return STEP_ERR_INVALID_ARG;
  FlagSource src{nullptr, token_ids, step_end_table, vocab, boundary_mask_out, nullptr};
  return score_steps_impl(pool, hidden, src, row_trace, M, w, step_scores_out, nullptr, 0, stream);
}

extern "C" int detect_step_ends(step_pool* pool, const int32_t* token_ids, int M, const uint8_t* step_end_table,
                                int vocab, uint8_t* boundary_mask_out, void* stream) {
  if (!pool || M < 0) return STEP_ERR_INVALID_ARG;
  if (M == 0) return STEP_OK;
  if (!token_ids || !step_end_table || vocab < 1 || !boundary_mask_out) return STEP_ERR_INVALID_ARG;
  FlagSource src{nullptr, token_ids, step_end_table, vocab, boundary_mask_out, nullptr};
  int ctas = (M + 255) / 256;
  if (ctas > pool->num_sms * 8) ctas = pool->num_sms * 8;
  step_end_kernel<<<ctas, 256, 0, (cudaStream_t)stream>>>(src, M, pool->v.counters);
  return launch_ok();
}

extern "C" int step_end_table_from_vocab(const char* const* token_text, const int32_t* text_len, int vocab,
                                         uint8_t* table_out) {
  if (!token_text || vocab < 0 || !table_out) return STEP_ERR_INVALID_ARG;
  for (int v = 0; v < vocab; ++v) {
    const char* t = token_text[v];
    uint8_t hit = 0;
    if (t) {
      if (text_len) {
        for (int i = 0; i + 1 < text_len[v]; ++i)
          if (t[i] == '\n' && t[i + 1] == '\n') { hit = 1; break; }
      } else {
        for (int i = 0; t[i] && t[i + 1]; ++i)
          if (t[i] == '\n' && t[i + 1] == '\n') { hit = 1; break; }
      }
    }
    table_out[v] = hit;
  }
  return STEP_OK;
}

int stepk::score_steps_impl(step_pool* pool, const void* hidden, FlagSource src, const int32_t* row_trace, int M,
                            const scorer_weights* w, float* step_scores_out, float* trace_scores_out, int n_out, void* stream) {
  if (!hidden || !step_scores_out) return STEP_ERR_INVALID_ARG;
  if (!w->W1 || !w->b1 || !w->w2 || w->D < 1 || w->m < 1) return STEP_ERR_INVALID_ARG;
  if (w->dtype != STEP_BF16 && w->dtype != STEP_FP32) return STEP_ERR_INVALID_ARG;
  const size_t smem = (size_t)kRowTile * w->D * sizeof(float);
  cudaStream_t s = (cudaStream_t)stream;
  Geo g = geo_of(pool);
  // a decode step's shape: everything in one launch (unless the tensor-core kernel was asked for by name)
  if (M <= kSmallRows && pool->scorer_mode <= 0 && smem <= 200 * 1024) {
    int S = (w->m + 3) / 4;                                        // about four hidden units per CTA
    const int cap = pool->num_sms < kSmallCtas ? pool->num_sms : kSmallCtas;
    if (S > cap) S = cap;
    if (w->dtype == STEP_BF16) {
      auto kern = score_small_kernel<__nv_bfloat16>;
      if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return STEP_ERR_CUDA;
      kern<<<S, kSmallThreads, smem, s>>>(pool->v, g, src, (const __nv_bfloat16*)hidden, row_trace, M, (const __nv_bfloat16*)w->W1,
                                          (const __nv_bfloat16*)w->b1, (const __nv_bfloat16*)w->w2, w->b2, w->D, w->m,
                                          pool->cfg.unscored_score, step_scores_out, trace_scores_out, n_out);
    } else {
      auto kern = score_small_kernel<float>;
      if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return STEP_ERR_CUDA;
      kern<<<S, kSmallThreads, smem, s>>>(pool->v, g, src, (const float*)hidden, row_trace, M, (const float*)w->W1, (const float*)w->b1,
                                          (const float*)w->w2, w->b2, w->D, w->m, pool->cfg.unscored_score, step_scores_out,
                                          trace_scores_out, n_out);
    }
    return launch_ok();
  }
  const size_t eb = w->dtype == STEP_BF16 ? 2 : 4;
  const bool tc = pool->scorer_mode >= 0 && score_tc_supported(w, hidden);
  const int tc_min_rows = !tc ? 0 : (pool->scorer_mode > 0 ? 1 : pool->scorer_tc_min_rows);
  for (int off = 0; off < M; off += pool->max_score_rows) {
    const int Mc = M - off < pool->max_score_rows ? M - off : pool->max_score_rows;
    const char* hid = (const char*)hidden + (size_t)off * w->D * eb;
    const int32_t* rt = row_trace ? row_trace + off : nullptr;
    FlagSource part = src;
    if (part.mask) part.mask += off;
    if (part.tokens) part.tokens += off;
    if (part.mask_out) part.mask_out += off;
    if (part.live) part.live += off;
    score_compact_kernel<<<kCompactCtas, kCompactThreads, 0, s>>>(pool->v, part, Mc, step_scores_out + off,
                                                       tc_min_rows, w->m, pool->num_sms);
    // the CUDA-core kernel only ever sees launches with fewer than tc_min_rows boundary rows
    const int scalar_rows = tc_min_rows > 0 && tc_min_rows - 1 < Mc ? tc_min_rows - 1 : Mc;
    if (scalar_rows > 0) {
      if (smem > 200 * 1024) return STEP_ERR_INVALID_ARG;           // the CUDA-core kernel stages 8 hidden rows as fp32
      dim3 grid(kSplits, (scalar_rows + kRowTile - 1) / kRowTile);
      if (w->dtype == STEP_BF16) {
        auto kern = score_mlp_kernel<__nv_bfloat16>;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return STEP_ERR_CUDA;
        kern<<<grid, kMlpWarps * 32, smem, s>>>(pool->v, (const __nv_bfloat16*)hid, (const __nv_bfloat16*)w->W1,
                                               (const __nv_bfloat16*)w->b1, (const __nv_bfloat16*)w->w2, w->D, w->m);
      } else {
        auto kern = score_mlp_kernel<float>;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return STEP_ERR_CUDA;
        kern<<<grid, kMlpWarps * 32, smem, s>>>(pool->v, (const float*)hid, (const float*)w->W1, (const float*)w->b1,
                                               (const float*)w->w2, w->D, w->m);
      }
    }
    if (tc_min_rows > 0 && Mc >= tc_min_rows) {
      const int st = score_tc_launch(pool, hid, Mc, w, s);
      if (st != STEP_OK) return st;
    }
    // row_trace == NULL means row i is trace i, counted from the start of the whole call
    if (launch_dependent(score_finish_kernel, dim3((Mc + kScoreFoldRows - 1) / kScoreFoldRows), dim3(kFinishThreads), 0, s,
                         pool->v, g, rt, off, w->b2, pool->cfg.unscored_score, step_scores_out + off) != cudaSuccess)
      return STEP_ERR_CUDA;
  }
  if (trace_scores_out && n_out > 0)
    STEP_CUDA_OK(cudaMemcpyAsync(trace_scores_out, pool->v.trace_scores, (size_t)(n_out < g.max_traces ? n_out : g.max_traces) * sizeof(float),
                                 cudaMemcpyDeviceToDevice, s));
  return launch_ok();
}

extern "C" int kv_pool_set_scorer_config(step_pool* pool, int mode, int tc_min_rows) {
  if (!pool || mode < -1 || mode > 1 || tc_min_rows < 0) return STEP_ERR_INVALID_ARG;
  pool->scorer_mode = mode;
  if (tc_min_rows > 0) pool->scorer_tc_min_rows = tc_min_rows;
  return STEP_OK;
}

extern "C" int kv_pool_score_launch_info(step_pool* pool, int* n_rows, int* tc_units, void* stream) {
  if (!pool) return STEP_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  int32_t c[C_SCORE_SLICES + 1];
  STEP_CUDA_OK(cudaMemcpyAsync(c, pool->v.counters, sizeof(c), cudaMemcpyDeviceToHost, s));
  STEP_CUDA_OK(cudaStreamSynchronize(s));
  if (n_rows) *n_rows = c[C_SCORE_NB];
  if (tc_units) *tc_units = c[C_SCORE_TC];
  return STEP_OK;
}
