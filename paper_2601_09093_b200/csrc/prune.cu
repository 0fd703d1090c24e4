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

__global__ void __cluster_dims__(kClusterCtas, 1, 1) __launch_bounds__(kPruneThreads, 1)
prune_kernel(DevViews v, Geo g, const float* __restrict__ scores_in, float threshold, float keep_frac,
             float unscored, int32_t* __restrict__ pruned_ids_out, int32_t* __restrict__ n_pruned_out) {
  __shared__ int s_warp[33];
  trigger_and_evict_cluster(v, g, scores_in, threshold, keep_frac, unscored, pruned_ids_out, n_pruned_out, s_warp);
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
