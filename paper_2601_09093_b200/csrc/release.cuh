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

}  // namespace stepk
