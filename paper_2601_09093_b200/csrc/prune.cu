// prune_if_saturated: memory trigger, ranking and KV release (Sec. 3.2; Algorithm 1, the
// GPUMemoryFull branch: t* = argmin score_t, ReleaseKVCache(t*), T <- T \ {t*}).
//
// One thread-block cluster of eight CTAs does the whole call:
//   1. predicate   used + need > floor(threshold * total)              (every CTA; all leave if it is false)
//   2. rank        every live trace counts the live traces that order before it
//                  (score descending, id ascending, NaN last) - a warp per trace, lanes over rivals
//   3. list        evicted ids in ascending order by a block-wide prefix sum          (2, 3: the leading CTA)
//   4. release     all (trace, page) entries drop one reference in parallel; the entry that is the
//                  LAST in (trace, page) order to name a block whose count reached zero owns the
//                  push; prefix sums within each CTA and push counts exchanged through distributed shared
//                  memory give each push its place - so the free list comes out exactly as a serial walk
//                  would leave it.  The entries are spread over the cluster's eight SMs because a release is
//                  bound by how many scattered 4-byte requests one SM can issue.
#include "release.cuh"

using namespace stepk;

namespace {

// A cluster of kClusterCtas CTAs.  Every CTA evaluates the trigger (same inputs, same answer); rank 0 ranks the
// traces and lists the evicted ones; the cluster releases them together.
__global__ void __cluster_dims__(kClusterCtas, 1, 1) __launch_bounds__(kPruneThreads, 1)
prune_kernel(DevViews v, Geo g, const float* __restrict__ scores_in, float threshold, float keep_frac,
             float unscored, int32_t* __restrict__ pruned_ids_out, int32_t* __restrict__ n_pruned_out) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  const bool leader = cluster.block_rank() == 0;
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
    if (!go && leader) *n_pruned_out = 0;
  }
  __syncthreads();
  if (!s_go) return;                      // the whole cluster leaves: nothing has been written yet
  const int n_keep = s_nkeep;
  if (leader) {
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
    if (threadIdx.x == 0) { *n_pruned_out = n_list; v.counters[C_PRUNE_N] = n_list; v.counters[C_N_EVICTED] += n_list; }
    __threadfence();
  }
  cluster.sync();
  // ---- 4. release
  release_listed_cluster(v, g, __ldcg(&v.counters[C_PRUNE_N]), unscored, s_warp);
}

__global__ void __cluster_dims__(kClusterCtas, 1, 1) __launch_bounds__(kPruneThreads, 1)
release_kernel(DevViews v, Geo g, const int32_t* __restrict__ ids, int n, float unscored) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  __shared__ int s_warp[33];
  // keep the valid, live ids in the order given; an id listed twice is released once (at its first place) and the
  // repeat flagged - counting it twice would take two references off every one of its blocks
  if (cluster.block_rank() == 0) {
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
      const int t = ids[i];
      if (t >= 0 && t < g.max_traces) v.prune_rank[t] = 0;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      int k = 0;
      for (int i = 0; i < n; ++i) {
        const int t = ids[i];
        if (t < 0 || t >= g.max_traces || !v.live[t] || v.prune_rank[t]) { flag_error(v.counters, STEP_ERR_BAD_TRACE); continue; }
        v.prune_rank[t] = 1;
        v.prune_list[k++] = t;
      }
      v.counters[C_PRUNE_N] = k;
      __threadfence();
    }
  }
  cluster.sync();
  release_listed_cluster(v, g, __ldcg(&v.counters[C_PRUNE_N]), unscored, s_warp);
}

}  // namespace

extern "C" {

int prune_if_saturated(step_pool* pool, const float* scores, float threshold, float keep_frac,
                       int32_t* pruned_ids_out, int32_t* n_pruned_out, void* stream) {
  if (!pool || !pruned_ids_out || !n_pruned_out) return STEP_ERR_INVALID_ARG;
  if (!(threshold > 0.f) || threshold > 1.f) return STEP_ERR_INVALID_ARG;
  if (isnan(keep_frac) || keep_frac == 0.f || keep_frac > 1.f) return STEP_ERR_INVALID_ARG;
  prune_kernel<<<kClusterCtas, kPruneThreads, 0, (cudaStream_t)stream>>>(pool->v, geo_of(pool), scores, threshold, keep_frac,
                                                              pool->cfg.unscored_score, pruned_ids_out, n_pruned_out);
  return launch_ok();
}

int kv_pool_release_traces(step_pool* pool, const int32_t* trace_ids, int n, void* stream) {
  if (!pool || n < 0) return STEP_ERR_INVALID_ARG;
  if (n == 0) return STEP_OK;
  if (!trace_ids || n > pool->cfg.max_traces) return STEP_ERR_INVALID_ARG;
  release_kernel<<<kClusterCtas, kPruneThreads, 0, (cudaStream_t)stream>>>(pool->v, geo_of(pool), trace_ids, n,
                                                                pool->cfg.unscored_score);
  return launch_ok();
}

}  // extern "C"
