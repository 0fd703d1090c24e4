// Device helpers shared by the kernels that give KV blocks back (prune.cu, algorithm1.cu):
// a block-wide exclusive prefix sum, the ranking order of traces, and the ordered release of a list of traces.
#pragma once

#include "step_internal.cuh"
#include "block_scan.cuh"

#include <cooperative_groups.h>
#include <math.h>

namespace stepk {

constexpr int kPruneThreads = 1024;

// true if trace a orders strictly before trace b (a is the better one)
__device__ inline bool orders_before(float sa, int a, float sb, int b) {
  const bool na = isnan(sa), nb = isnan(sb);
  if (na != nb) return nb;               // a number beats NaN
  if (!na && sa != sb) return sa > sb;
  return a < b;
}

// Position of entry e of the flattened (trace, page) order: k = index into the list with off[k] <= e < off[k+1].
__device__ inline int find_list_index(const int32_t* off, int n_list, int e) {
  int lo = 0, hi = n_list - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (off[mid] <= e) lo = mid; else hi = mid - 1;
  }
  return lo;
}

constexpr int kClusterCtas = 8;         // CTAs (one per SM) that share one release
constexpr int kListInSmem = 1024;      // lists up to this long are staged in shared memory
constexpr int kMaskRows = 64;          // rows of blockDim entries whose decisions a thread keeps in registers

// Releases the traces listed in v.prune_list[0 .. n_list) (processed in list order).
//
// Called by every CTA of a thread-block cluster with the same n_list, after a cluster barrier that follows the
// writing of the list.  The (trace, page) entries of all listed traces form one sequence in list order;
// every block whose reference count reaches zero is pushed on the free list at the place a serial walk of
// that sequence would give it.  One SM can issue only so many scattered 4-byte requests per microsecond,
// and a release is nothing but such requests, so the sequence is cut into one contiguous range per CTA:
//   A   every entry drops one reference (atomicSub) and bids for its block with its position (atomicMax);
//   B1  the entry that won the bid (the last, in order, to name the block) owns it; it pushes the block if
//       the count is now zero; each CTA counts its pushes and shows the count to the cluster through
//       distributed shared memory;
//   B2  a CTA's pushes start after those of all lower-ranked CTAs; block-wide prefix sums place them.
// Cluster barriers separate the phases (hardware barriers; nothing spins).
__device__ inline void release_listed_cluster(DevViews& v, const Geo& g, int n_list, float unscored, int* s_warp) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank(), C = (int)cluster.num_blocks();
  __shared__ int32_t s_off[kListInSmem + 1], s_list[kListInSmem];
  __shared__ int s_count, s_base, s_total;
  const bool staged = n_list <= kListInSmem;
  // ---- entry offsets of each listed trace (every CTA for itself; rank 0 also keeps them in global memory)
  {
    int running = 0;
    for (int base = 0; base < n_list || base == 0; base += blockDim.x) {
      const int k = base + threadIdx.x;
      int pages = 0, t = 0;
      if (k < n_list) { t = v.prune_list[k]; pages = (v.seq_lens[t] + g.P - 1) / g.P; }
      int chunk_total;
      const int at = running + block_excl_scan(pages, s_warp, &chunk_total);
      if (k < n_list) {
        if (staged) { s_off[k] = at; s_list[k] = t; }
        if (rank == 0) v.prune_off[k] = at;
      }
      running += chunk_total;
    }
    if (threadIdx.x == 0) {
      if (staged) s_off[n_list] = running;
      if (rank == 0) v.prune_off[n_list] = running;
      s_total = running;
    }
  }
  __threadfence();
  cluster.sync();                        // (long lists read rank 0's global copy)
  const int32_t* off = staged ? s_off : v.prune_off;
  const int32_t* list = staged ? s_list : v.prune_list;
  const int E = s_total;
  const int R = ((E + C - 1) / C + blockDim.x - 1) / blockDim.x * blockDim.x;   // entries per CTA, whole rows
  const int lo = min(E, rank * R), hi = min(E, lo + R);
  const int fc = v.counters[C_FREE_COUNT];
  // ---- A: drop references, bid for the blocks
  for (int base = lo; base < hi; base += blockDim.x) {
    const int e = base + threadIdx.x;
    if (e >= hi) continue;
    const int k = find_list_index(off, n_list, e);
    const int b = v.block_table[(size_t)list[k] * g.max_pages + (e - off[k])];
    if (b < 0 || b >= g.num_blocks) { flag_error(v.counters, STEP_ERR_BAD_BLOCK); continue; }
    atomicSub(&v.refcount[b], 1);
    atomicMax(&v.claim[b], e);
  }
  __threadfence();
  cluster.sync();
  // ---- B1: who owns, who pushes
  unsigned long long own = 0, push = 0;
  int my_pushes = 0;
  {
    int r = 0;
    for (int base = lo; base < hi; base += blockDim.x, ++r) {
      const int e = base + threadIdx.x;
      if (e >= hi) continue;
      const int k = find_list_index(off, n_list, e);
      const int b = v.block_table[(size_t)list[k] * g.max_pages + (e - off[k])];
      if (b < 0 || b >= g.num_blocks) continue;
      if (__ldcg(&v.claim[b]) == e) {
        const bool p = __ldcg(&v.refcount[b]) == 0;
        if (r < kMaskRows) { own |= 1ull << r; if (p) push |= 1ull << r; }
        my_pushes += p;
      }
    }
  }
  {
    int total;
    block_excl_scan(my_pushes, s_warp, &total);
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
    s_base = fc + before;
    if (rank == 0) v.counters[C_FREE_COUNT] = fc + all;
  }
  __syncthreads();
  // ---- B2: place the pushes, clear the table entries and the bids
  {
    int at_base = s_base, r = 0;
    for (int base = lo; base < hi; base += blockDim.x, ++r) {
      const int e = base + threadIdx.x;
      int b = -1;
      bool o = false, p = false;
      if (e < hi) {
        const int k = find_list_index(off, n_list, e);
        int32_t* slot = v.block_table + (size_t)list[k] * g.max_pages + (e - off[k]);
        b = *slot;
        *slot = -1;
        if (b >= 0 && b < g.num_blocks) {
          if (r < kMaskRows) { o = (own >> r) & 1; p = (push >> r) & 1; }
          else if (__ldcg(&v.claim[b]) == e) { o = true; p = __ldcg(&v.refcount[b]) == 0; }
        }
      }
      int row_total;
      const int at = at_base + block_excl_scan(p ? 1 : 0, s_warp, &row_total);
      if (p) v.free_list[at] = b;
      if (o) v.claim[b] = -1;
      at_base += row_total;
    }
  }
  if (rank == 0)
    for (int k = threadIdx.x; k < n_list; k += blockDim.x) {
      const int t = list[k];
      v.seq_lens[t] = 0; v.live[t] = 0;
      v.score_sum[t] = 0.f; v.score_cnt[t] = 0; v.trace_scores[t] = unscored;
    }
  cluster.sync();                        // no CTA leaves while its count may still be read
}

// The memory trigger and the eviction (Sec. 3.2; Algorithm 1, the GPUMemoryFull branch) for a cluster of kClusterCtas
// CTAs: every CTA evaluates the trigger (same inputs, same answer); rank 0 ranks the traces and lists the evicted
// ones; the cluster releases them together.
// Called by every CTA of the cluster; true if the trigger fired (the same answer in every CTA).
__device__ inline bool trigger_and_evict_cluster(DevViews& v, const Geo& g, const float* __restrict__ scores_in, float threshold,
                                                 float keep_frac, float unscored, int32_t* __restrict__ pruned_ids_out,
                                                 int32_t* __restrict__ n_pruned_out, int* s_warp) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  const bool leader = cluster.block_rank() == 0;
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
  if (!s_go) return false;                // the whole cluster leaves: nothing has been written yet
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
  return true;
}


}  // namespace stepk
