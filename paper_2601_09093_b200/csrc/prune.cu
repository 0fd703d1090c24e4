// prune_if_saturated: memory trigger, ranking and KV release (Sec. 3.2; Algorithm 1, the
// GPUMemoryFull branch: t* = argmin score_t, ReleaseKVCache(t*), T <- T \ {t*}).
//
// One CTA does the whole call (the trace set is tiny; the block-id traffic is a few hundred KB):
//   1. predicate   used + need > floor(threshold * total)
//   2. rank        every live trace counts the live traces that order before it
//                  (score descending, id ascending, NaN last) - a warp per trace, lanes over rivals
//   3. list        evicted ids in ascending order by a block-wide prefix sum
//   4. release     all (trace, page) entries drop one reference in parallel; the entry that is the
//                  LAST in (trace, page) order to name a block whose count reached zero owns the
//                  push, and a block-wide prefix sum over the entries in order gives each push its
//                  place - so the free list comes out exactly as a serial walk would leave it.
#include "step_internal.cuh"

#include <math.h>

using namespace stepk;

namespace {

constexpr int kPruneThreads = 1024;

// Exclusive prefix sum of one int per thread over the CTA; *total gets the sum.
__device__ inline int block_excl_scan(int x, int* s_warp, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = x;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  __syncthreads();                       // s_warp may still be read from the previous call
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = s_warp[lane];
    int wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += v;
    }
    s_warp[lane] = wi - w;               // exclusive offset of each warp
    if (lane == 31) s_warp[32] = wi;
  }
  __syncthreads();
  *total = s_warp[32];
  return s_warp[warp] + incl - x;
}

// true if trace a orders strictly before trace b (a is the better one)
__device__ inline bool orders_before(float sa, int a, float sb, int b) {
  const bool na = isnan(sa), nb = isnan(sb);
  if (na != nb) return nb;               // a number beats NaN
  if (!na && sa != sb) return sa > sb;
  return a < b;
}

// Releases the traces listed in v.prune_list[0 .. n_list) (processed in list order).
__device__ void release_listed(DevViews& v, const Geo& g, int n_list, float unscored, int* s_warp) {
  // offsets of each trace's entries in the global (trace, page) order
  if (threadIdx.x == 0) {
    int off = 0;
    for (int k = 0; k < n_list; ++k) {
      v.prune_off[k] = off;
      const int S = v.seq_lens[v.prune_list[k]];
      off += (S + g.P - 1) / g.P;
    }
    v.prune_off[n_list] = off;
  }
  __syncthreads();
  // pass A: drop references, find the last entry naming each block
  for (int k = 0; k < n_list; ++k) {
    const int t = v.prune_list[k], off = v.prune_off[k], np = v.prune_off[k + 1] - off;
    const int32_t* row = v.block_table + (size_t)t * g.max_pages;
    for (int p = threadIdx.x; p < np; p += blockDim.x) {
      const int b = row[p];
      if (b < 0 || b >= g.num_blocks) { flag_error(v.counters, STEP_ERR_BAD_BLOCK); continue; }
      atomicSub(&v.refcount[b], 1);
      atomicMax(&v.claim[b], off + p);
    }
  }
  __syncthreads();
  // pass B: pushes in (trace, page) order
  const int fc = v.counters[C_FREE_COUNT];
  int pushed = 0;
  for (int k = 0; k < n_list; ++k) {
    const int t = v.prune_list[k], off = v.prune_off[k], np = v.prune_off[k + 1] - off;
    int32_t* row = v.block_table + (size_t)t * g.max_pages;
    for (int base = 0; base < np; base += blockDim.x) {
      const int p = base + threadIdx.x;
      int b = -1, f = 0;
      if (p < np) {
        b = row[p];
        row[p] = -1;
        if (b >= 0 && b < g.num_blocks && v.claim[b] == off + p) {
          v.claim[b] = -1;
          f = v.refcount[b] == 0;
        }
      }
      int chunk_total;
      const int at = block_excl_scan(f, s_warp, &chunk_total);
      if (f) v.free_list[fc + pushed + at] = b;
      pushed += chunk_total;
    }
  }
  for (int k = threadIdx.x; k < n_list; k += blockDim.x) {
    const int t = v.prune_list[k];
    v.seq_lens[t] = 0; v.live[t] = 0;
    v.score_sum[t] = 0.f; v.score_cnt[t] = 0; v.trace_scores[t] = unscored;
  }
  __syncthreads();
  if (threadIdx.x == 0) v.counters[C_FREE_COUNT] = fc + pushed;
}

__global__ void __launch_bounds__(kPruneThreads)
prune_kernel(DevViews v, Geo g, const float* __restrict__ scores_in, float threshold, float keep_frac,
             float unscored, int32_t* __restrict__ pruned_ids_out, int32_t* __restrict__ n_pruned_out) {
  __shared__ int s_warp[33];
  __shared__ int s_nlive, s_need, s_go, s_nkeep;
  const float* scores = scores_in ? scores_in : v.trace_scores;
  const int T = g.max_traces;
  if (threadIdx.x == 0) { s_nlive = 0; s_need = 0; }
  __syncthreads();
  // ---- 1. the trigger
  int nl = 0, nd = 0;
  for (int t = threadIdx.x; t < T; t += blockDim.x)
    if (v.live[t]) { ++nl; nd += (v.seq_lens[t] % g.P) == 0; }
  if (nl) atomicAdd(&s_nlive, nl);
  if (nd) atomicAdd(&s_need, nd);
  __syncthreads();
  if (threadIdx.x == 0) {
    const int used = g.num_blocks - v.counters[C_FREE_COUNT];
    const long long limit = (long long)floor((double)threshold * (double)g.num_blocks);
    int go = (long long)used + s_need > limit;
    int n_keep = 0;
    if (go) {
      n_keep = keep_frac < 0.f ? s_nlive - 1 : (int)ceil((double)keep_frac * (double)s_nlive - 1e-6);
      if (keep_frac >= 0.f && n_keep < 1) n_keep = 1;
      if (s_nlive == 0 || n_keep >= s_nlive) go = 0;
    }
    s_go = go; s_nkeep = n_keep;
    if (!go) *n_pruned_out = 0;
  }
  __syncthreads();
  if (!s_go) return;
  const int n_keep = s_nkeep;
  // ---- 2. rank by counting: a warp per trace, lanes over rivals
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  for (int t = warp; t < T; t += nwarps) {
    int evict = 0;
    if (v.live[t]) {
      const float st = scores[t];
      int ahead = 0;
      for (int u = lane; u < T; u += 32)
        if (u != t && v.live[u] && orders_before(scores[u], u, st, t)) ++ahead;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ahead += __shfl_xor_sync(0xffffffffu, ahead, o);
      evict = ahead >= n_keep;
    }
    if (lane == 0) v.prune_rank[t] = evict;
  }
  __syncthreads();
  // ---- 3. evicted ids, ascending
  int n_list = 0;
  for (int base = 0; base < T; base += blockDim.x) {
    const int t = base + threadIdx.x;
    const int f = t < T ? v.prune_rank[t] : 0;
    int chunk_total;
    const int at = block_excl_scan(f, s_warp, &chunk_total);
    if (f) { v.prune_list[n_list + at] = t; pruned_ids_out[n_list + at] = t; }
    n_list += chunk_total;
  }
  __syncthreads();
  if (threadIdx.x == 0) *n_pruned_out = n_list;
  // ---- 4. release
  release_listed(v, g, n_list, unscored, s_warp);
}

__global__ void __launch_bounds__(kPruneThreads)
release_kernel(DevViews v, Geo g, const int32_t* __restrict__ ids, int n, float unscored) {
  __shared__ int s_warp[33];
  __shared__ int s_n;
  // keep the valid, live ids in the order given
  if (threadIdx.x == 0) {
    int k = 0;
    for (int i = 0; i < n; ++i) {
      const int t = ids[i];
      if (t < 0 || t >= g.max_traces || !v.live[t]) { flag_error(v.counters, STEP_ERR_BAD_TRACE); continue; }
      v.prune_list[k++] = t;
    }
    s_n = k;
  }
  __syncthreads();
  release_listed(v, g, s_n, unscored, s_warp);
}

}  // namespace

extern "C" {

int prune_if_saturated(step_pool* pool, const float* scores, float threshold, float keep_frac,
                       int32_t* pruned_ids_out, int32_t* n_pruned_out, void* stream) {
  if (!pool || !pruned_ids_out || !n_pruned_out) return STEP_ERR_INVALID_ARG;
  if (!(threshold > 0.f) || threshold > 1.f) return STEP_ERR_INVALID_ARG;
  if (isnan(keep_frac) || keep_frac == 0.f || keep_frac > 1.f) return STEP_ERR_INVALID_ARG;
  prune_kernel<<<1, kPruneThreads, 0, (cudaStream_t)stream>>>(pool->v, geo_of(pool), scores, threshold, keep_frac,
                                                              pool->cfg.unscored_score, pruned_ids_out, n_pruned_out);
  return launch_ok();
}

int kv_pool_release_traces(step_pool* pool, const int32_t* trace_ids, int n, void* stream) {
  if (!pool || n < 0) return STEP_ERR_INVALID_ARG;
  if (n == 0) return STEP_OK;
  if (!trace_ids || n > pool->cfg.max_traces) return STEP_ERR_INVALID_ARG;
  release_kernel<<<1, kPruneThreads, 0, (cudaStream_t)stream>>>(pool->v, geo_of(pool), trace_ids, n,
                                                                pool->cfg.unscored_score);
  return launch_ok();
}

}  // extern "C"
