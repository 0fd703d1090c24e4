// Paged KV pool: creation, InitTraces prefix fork, append_kv, accessors.
// (Algorithm 1: InitTraces and the cache write of NextToken; block bookkeeping is the
// library's own since the paper delegates it to its inference engine.)
#include "step_internal.cuh"

#include <new>
#include <vector>

using namespace stepk;

namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

bool config_valid(const kv_pool_config* c) {
  if (!c) return false;
  if (c->num_layers < 1 || c->num_q_heads < 1 || c->num_kv_heads < 1 || c->head_dim < 1) return false;
  if (c->page_size < 1 || c->num_blocks < 1 || c->max_traces < 1 || c->max_pages_per_trace < 1) return false;
  if (c->num_q_heads % c->num_kv_heads != 0) return false;
  if (c->num_q_heads / c->num_kv_heads > 16) return false;
  if (c->dtype != STEP_BF16 && c->dtype != STEP_FP32) return false;
  int eb = c->dtype == STEP_BF16 ? 2 : 4;
  if ((c->head_dim * eb) % 16 != 0 || c->head_dim > 512) return false;   // rows move as 16-byte chunks
  if (c->max_score_rows < 0) return false;
  if ((long long)c->max_traces * c->max_pages_per_trace > (1ll << 31) - 1) return false;
  return true;
}

MetaLayout make_layout(const kv_pool_config* c) {
  MetaLayout l;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const size_t T = c->max_traces, NB = c->num_blocks;
  const size_t rows = c->max_score_rows > 0 ? c->max_score_rows : c->max_traces;
  const int G = c->num_q_heads / c->num_kv_heads;
  l.block_table = take(T * c->max_pages_per_trace * 4);
  l.seq_lens = take(T * 4);
  l.live = take(T);
  l.score_sum = take(T * 4);
  l.score_cnt = take(T * 4);
  l.trace_scores = take(T * 4);
  l.refcount = take(NB * 4);
  l.free_list = take(NB * 4);
  l.claim = take(NB * 4);
  l.counters = take(C_NUM * 4);
  l.append_base = take(T * 4);
  l.prune_rank = take(T * 4);
  l.prune_list = take(T * 4);
  l.prune_off = take((T + 1) * 4);
  l.score_idx = take(rows * 4);
  l.score_z = take(rows * kScoreSplits * 4);
  l.score_part = take((rows + kScoreFoldRows - 1) / kScoreFoldRows * T * 8);
  l.score_zs = take((size_t)kSmallRows * kSmallCtas * 4);
  // attention partials: two slots per equal share, then (tensor-core shape only) one per chunk handed out at run time
  const bool mma = c->dtype == STEP_BF16 && c->head_dim == 128 && c->page_size == 16;
  const size_t slots = (size_t)kMaxPartitions * 2 + (mma ? kMaxDynChunks : 0);
  l.attn_ml = take(slots * G * 2 * 4);
  l.attn_o = take(slots * G * c->head_dim * 4);
  l.attn_sched = take(4);
  // shared-prefix attention: partials of its first pass (16 query rows per slot) and that pass's result per (trace, head)
  l.pre_ws_ml = take(mma ? (size_t)kPrefixPartitions * 2 * 16 * 2 * 4 : 0);
  l.pre_ws_o = take(mma ? (size_t)kPrefixPartitions * 2 * 16 * c->head_dim * 4 : 0);
  l.pre_ml = take(mma ? T * c->num_q_heads * 2 * 4 : 0);
  l.pre_o = take(mma ? T * c->num_q_heads * c->head_dim * 4 : 0);
  l.final_score = take(T * 4);
  l.answer = take(T * 4);
  l.finished = take(T);
  l.it_ids = take(T * 4);
  l.it_fin = take(T * 4);
  l.it_pruned = take(T * 4);
  l.it_tokens = take(T * 4);
  l.it_scores = take(T * 4);
  l.total = off;
  return l;
}

size_t kv_bytes_of(const kv_pool_config* c) {
  size_t eb = c->dtype == STEP_BF16 ? 2 : 4;
  return (size_t)c->num_layers * c->num_blocks * c->num_kv_heads * 2 * c->page_size * c->head_dim * eb;
}

__global__ void init_meta_kernel(DevViews v, Geo g, float unscored) {
  const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  const size_t nbt = (size_t)g.max_traces * g.max_pages;
  for (size_t i = tid; i < nbt; i += stride) v.block_table[i] = -1;
  for (size_t i = tid; i < (size_t)g.max_traces; i += stride) {
    v.seq_lens[i] = 0; v.live[i] = 0; v.score_sum[i] = 0.f; v.score_cnt[i] = 0;
    v.trace_scores[i] = unscored; v.append_base[i] = -1;
    v.final_score[i] = 0.f; v.answer[i] = -1; v.finished[i] = 0;
  }
  for (size_t i = tid; i < (size_t)g.num_blocks; i += stride) {
    v.refcount[i] = 0; v.claim[i] = -1;
    v.free_list[i] = g.num_blocks - 1 - (int)i;       // a stack: the first pop is block 0
  }
  for (size_t i = tid; i < (size_t)C_NUM; i += stride) v.counters[i] = (i == C_FREE_COUNT) ? g.num_blocks : 0;
  if (tid == 0) v.attn_sched[0] = 0;
}

// ---------------------------------------------------------------- InitTraces (fork)
__global__ void fork_alloc_kernel(DevViews v, Geo g, int n_traces, int prefix_len) {
  __shared__ int s_ok, s_fc, s_first;
  const int full = prefix_len / g.P, rem = prefix_len % g.P;
  const int needed = full + (rem ? n_traces : 0);
  if (threadIdx.x == 0) {
    // trace ids are handed out here, on the device, and only by a fork that goes through: a fork that fails
    // consumes none, so a retry after blocks were freed gets the ids the failed one would have got
    const int first = v.counters[C_NEXT_TRACE];
    s_first = first;
    s_fc = v.counters[C_FREE_COUNT];
    const bool fits = first + n_traces <= g.max_traces;
    s_ok = fits && needed <= s_fc;
    v.counters[C_FORK_OK] = s_ok;
    v.counters[C_FORK_FIRST] = first;
    if (!fits) flag_error(v.counters, STEP_ERR_CAPACITY);
    else if (!s_ok) flag_error(v.counters, STEP_ERR_NO_BLOCKS);
    if (s_ok) v.counters[C_NEXT_TRACE] = first + n_traces;
  }
  __syncthreads();
  if (!s_ok) return;
  const int fc = s_fc, first_trace = s_first;
  // shared full pages: pop in page order
  for (int p = threadIdx.x; p < full; p += blockDim.x) v.refcount[v.free_list[fc - 1 - p]] = n_traces;
  for (int j = 0; j < n_traces; ++j) {
    int32_t* row = v.block_table + (size_t)(first_trace + j) * g.max_pages;
    for (int p = threadIdx.x; p < full; p += blockDim.x) row[p] = v.free_list[fc - 1 - p];
  }
  // private copy of the partial last page, one block per trace in trace order
  for (int j = threadIdx.x; j < n_traces; j += blockDim.x) {
    const int t = first_trace + j;
    if (rem) {
      int b = v.free_list[fc - 1 - full - j];
      v.refcount[b] = 1;
      v.block_table[(size_t)t * g.max_pages + full] = b;
    }
    v.seq_lens[t] = prefix_len;
    v.live[t] = 1;
    v.score_sum[t] = 0.f; v.score_cnt[t] = 0;
  }
  __syncthreads();
  if (threadIdx.x == 0) v.counters[C_FREE_COUNT] = fc - needed;
}

// The prompt's K and V rows go into their pages.  A CTA owns one prompt position and a range of layers; the
// position's block (one shared block, or one private block per trace for a partial last page) is looked up once.
// k_prefix, v_prefix: [layer, head, position, chunk].  grid (prefix_len, layer splits).
__global__ void __launch_bounds__(256)
fork_write_kernel(DevViews v, Geo g, uint4* __restrict__ kv, const uint4* __restrict__ kpre,
                  const uint4* __restrict__ vpre, int n_traces, int prefix_len, int cpr,
                  int layers_per_cta) {
  if (!v.counters[C_FORK_OK]) return;
  const int first_trace = v.counters[C_FORK_FIRST];
  const int pos = blockIdx.x, page = pos / g.P, slot = pos % g.P;
  const int copies = page < prefix_len / g.P ? 1 : n_traces;     // the partial page is private per trace
  const int l0 = blockIdx.y * layers_per_cta, l1 = min(g.L, l0 + layers_per_cta);
  const int per_kv = g.Hkv * cpr;
  const size_t page_chunks = (size_t)g.P * cpr;
  const size_t layer_stride = (size_t)g.num_blocks * g.Hkv * 2 * page_chunks;
  for (int i = threadIdx.x; i < 2 * per_kv; i += blockDim.x) {
    const int which = i >= per_kv;
    const int r = which ? i - per_kv : i;
    const int head = r / cpr, c = r - head * cpr;
    const int cdst = g.swizzle ? ((c & ~7) | ((c ^ slot) & 7)) : c;
    const uint4* src = (which ? vpre : kpre) + ((size_t)head * prefix_len + pos) * cpr + c;
    const size_t src_layer = (size_t)g.Hkv * prefix_len * cpr;
    for (int j = 0; j < copies; ++j) {
      const int b = v.block_table[(size_t)(first_trace + j) * g.max_pages + page];
      const size_t dst0 = (((size_t)b * g.Hkv + head) * 2 + which) * page_chunks + (size_t)slot * cpr + cdst;
      for (int l = l0; l < l1; ++l) kv[(size_t)l * layer_stride + dst0] = src[(size_t)l * src_layer];
    }
  }
}

// ---------------------------------------------------------------- append_kv
// Two forms.  Pools of up to kFusedMaxTraces traces, and the live-trace form of the Algorithm 1 loop: one launch,
// append_fused_kernel (further down).  Larger pools: two launches -
// phase 1 (one CTA): decide, in list order, which traces get their pages; pop blocks.
// n_dev (may be null): only the first min(n, *n_dev) listed traces take part; the rest are passed over in silence.
__global__ void append_alloc_kernel(DevViews v, Geo g, const int32_t* __restrict__ ids, int n, int n_tokens,
                                    const int32_t* __restrict__ n_dev) {
  extern __shared__ int sm[];
  dependents_may_launch();                               // the kernel that writes the rows may set itself up meanwhile
  const int n_eff = n_dev ? min(n, max(*n_dev, 0)) : n;
  int* s_need = sm;            // pages wanted, or -1 if the trace is skipped
  int* s_off = sm + n;         // pops that precede this trace's
  int* s_have = sm + 2 * n;
  __shared__ int s_fc;
  // a trace listed twice is served once, at its first place in the list; the repeats are flagged and skipped
  // (v.prune_rank, scratch of max_traces ints, records the first place that names each trace)
  for (int i = threadIdx.x; i < n_eff; i += blockDim.x) {
    const int t = ids[i];
    if (t >= 0 && t < g.max_traces) v.prune_rank[t] = 0x7fffffff;
  }
  __syncthreads();
  for (int i = threadIdx.x; i < n_eff; i += blockDim.x) {
    const int t = ids[i];
    if (t >= 0 && t < g.max_traces) atomicMin(&v.prune_rank[t], i);
  }
  __syncthreads();
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    int need = -1, have = 0;
    if (i >= n_eff) { s_need[i] = need; s_have[i] = have; continue; }
    const int t = ids[i];
    if (t < 0 || t >= g.max_traces || !v.live[t] || v.prune_rank[t] != i) {
      flag_error(v.counters, STEP_ERR_BAD_TRACE);
    } else {
      const int S = v.seq_lens[t];
      have = (S + g.P - 1) / g.P;
      const long long want = ((long long)S + n_tokens + g.P - 1) / g.P;
      if (want > g.max_pages) flag_error(v.counters, STEP_ERR_CAPACITY);
      else need = (int)want - have;
    }
    s_need[i] = need; s_have[i] = have;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const int fc = v.counters[C_FREE_COUNT];
    int remaining = fc;
    for (int i = 0; i < n; ++i) {
      const int need = s_need[i];
      if (need < 0) continue;
      if (need > remaining) { s_need[i] = -1; flag_error(v.counters, STEP_ERR_NO_BLOCKS); continue; }
      s_off[i] = fc - remaining;
      remaining -= need;
    }
    s_fc = fc;
    v.counters[C_FREE_COUNT] = remaining;
  }
  __syncthreads();
  const int fc = s_fc;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  for (int i = warp; i < n; i += nwarps) {
    const int need = s_need[i];
    if (need < 0) { if (lane == 0) v.append_base[i] = -1; continue; }
    const int t = ids[i];
    int32_t* row = v.block_table + (size_t)t * g.max_pages;
    for (int p = lane; p < need; p += 32) {
      const int b = v.free_list[fc - 1 - s_off[i] - p];
      row[s_have[i] + p] = b;
      v.refcount[b] = 1;
    }
    if (lane == 0) {
      const int S = v.seq_lens[t];
      v.append_base[i] = S;
      v.seq_lens[t] = S + n_tokens;
    }
  }
}

// Phase 2: the new rows go into their pages.  A CTA owns one (listed trace, new token) pair and a range of
// layers: where the token lands (page, slot, block) is worked out once per CTA, and per layer the threads move the
// 16-byte chunks of the K and V rows of all KV heads with nothing but adds in the loop.
// grid (n * n_tokens, layer splits).
__global__ void __launch_bounds__(256)
append_write_kernel(DevViews v, Geo g, uint4* __restrict__ kv, const uint4* __restrict__ knew,
                    const uint4* __restrict__ vnew, const int32_t* __restrict__ ids,
                    int n_tokens, int cpr, int layers_per_cta, int src_by_id) {
  const int idx = blockIdx.x / n_tokens, j = blockIdx.x - idx * n_tokens;
  wait_for_primary();                                            // launched as a dependent of the allocation kernel
  const int base = v.append_base[idx];
  if (base < 0) return;                                          // this trace's request was not met
  const int t = ids[idx];
  const int pos = base + j, page = pos / g.P, slot = pos % g.P;
  const int b = v.block_table[(size_t)t * g.max_pages + page];
  const int l0 = blockIdx.y * layers_per_cta, l1 = min(g.L, l0 + layers_per_cta);
  const int per_kv = g.Hkv * cpr;                                // chunks of the K (or V) rows of one layer
  // the new rows are laid out [row, token, layer, head, chunk]; row = position in the list, or the trace id
  const size_t row = src_by_id ? (size_t)t : (size_t)idx;
  const size_t src_token = (row * n_tokens + j) * (size_t)g.L * per_kv;
  const size_t page_chunks = (size_t)g.P * cpr;                  // 16-byte chunks of one K (or V) page
  for (int i = threadIdx.x; i < 2 * per_kv; i += blockDim.x) {
    const int which = i >= per_kv;
    const int r = which ? i - per_kv : i;
    const int head = r / cpr, c = r - head * cpr;
    const int cdst = g.swizzle ? ((c & ~7) | ((c ^ slot) & 7)) : c;
    const uint4* src = (which ? vnew : knew) + src_token + r;
    // chunk index of (layer, b, head, which, slot, cdst): pages are [layer][block][head][K|V]
    const size_t dst0 = (((size_t)b * g.Hkv + head) * 2 + which) * page_chunks + (size_t)slot * cpr + cdst;
    const size_t layer_stride = (size_t)g.num_blocks * g.Hkv * 2 * page_chunks;
    for (int l = l0; l < l1; ++l) kv[(size_t)l * layer_stride + dst0] = src[(size_t)l * per_kv];
  }
}

// append_kv in ONE launch, for pools of up to kFusedMaxTraces traces (a list's first-place table must fit shared
// memory; the live-trace form needs none).  grid (listed entries x new tokens, splits of the layer range), as for
// append_write_kernel; every CTA works out the allocation of the whole call for itself - it is a pure function of the
// list, the lengths, the live flags and the free count, none of which changes before every CTA has read them:
//   1. first place of every trace in the list (a repeat is flagged and not served);
//   2. every entry's length S and page need; sum of the needs in front of this CTA's entry, and of all;
//      if the free list covers the sum nobody is skipped and entry i pops the blocks
//      free_list[fc - 1 - before_i - p]; otherwise one thread replays the serial rule (in list order, an entry whose
//      need exceeds what is left is skipped whole) for exactly the same outcome;
//   3. a ticket: the CTA that draws the last one knows that every CTA has finished reading, and writes what the
//      others read - the new lengths, the free count (and, for the live-trace form, the lists of the iteration);
//   4. the CTA of an entry's first token and first layer range records the entry's new pages (block table, reference
//      counts); every CTA moves its rows, taking the block of a new page straight from the free list.
// Nothing waits for anything.
// ids == nullptr (the loop of Algorithm 1, whose row i is trace i): entry i is trace i and is served if the trace is
// live; the last CTA also leaves the live traces in ascending order in v.it_ids and, if tokens is given, those of them
// whose sampled token is eos in v.it_fin (the traces that complete in this iteration), the counts in C_IT_NLIVE /
// C_IT_NFIN.  n_dev (may be null, lists only): only the first min(n, *n_dev) entries take part.
constexpr int kFusedMaxTraces = 4096;

__global__ void __launch_bounds__(256)
append_fused_kernel(DevViews v, Geo g, uint4* __restrict__ kv, const uint4* __restrict__ knew,
                    const uint4* __restrict__ vnew, const int32_t* __restrict__ ids, int n, int n_tokens,
                    const int32_t* __restrict__ n_dev, const int32_t* __restrict__ tokens, int eos,
                    int cpr, int layers_per_cta, int src_by_id) {
  extern __shared__ int sm[];
  int* s_S = sm;                 // [n] length before the call; -1: the entry is not served
  int* s_need = sm + n;          // [n] new pages; -1: not served
  int* s_first = sm + 2 * n;     // [max_traces] first place in the list that names the trace (lists only)
  __shared__ int s_red[2][8];
  __shared__ int s_fc, s_last, s_off, s_granted;
  const int idx = blockIdx.x / n_tokens, j = blockIdx.x - idx * n_tokens;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool reporter = blockIdx.x == 0 && blockIdx.y == 0;        // raises the status bits (once is enough)
  const int n_eff = (ids && n_dev) ? min(n, max(*n_dev, 0)) : n;
  // ---- 1. first places
  if (ids) {
    for (int i = threadIdx.x; i < g.max_traces; i += blockDim.x) s_first[i] = 0x7fffffff;
    __syncthreads();
    for (int i = threadIdx.x; i < n_eff; i += blockDim.x) {
      const int t = ids[i];
      if (t >= 0 && t < g.max_traces) atomicMin(&s_first[t], i);
    }
    __syncthreads();
  }
  // ---- 2. lengths and needs
  int before = 0, all = 0;
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    int S = -1, need = -1;
    if (i < n_eff) {
      const int t = ids ? ids[i] : i;
      if (ids) {
        if (t < 0 || t >= g.max_traces || !v.live[t] || s_first[t] != i) { if (reporter) flag_error(v.counters, STEP_ERR_BAD_TRACE); }
        else S = v.seq_lens[t];
      } else if (v.live[t]) {
        S = v.seq_lens[t];
      }
      if (S >= 0) {
        const int have = (S + g.P - 1) / g.P;
        const long long want = ((long long)S + n_tokens + g.P - 1) / g.P;
        if (want > g.max_pages) { if (reporter) flag_error(v.counters, STEP_ERR_CAPACITY); S = -1; }
        else need = (int)want - have;
      }
    }
    s_S[i] = S; s_need[i] = need;
    if (need > 0) { all += need; if (i < idx) before += need; }
  }
  if (threadIdx.x == 0) s_fc = v.counters[C_FREE_COUNT];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { before += __shfl_xor_sync(0xffffffffu, before, o); all += __shfl_xor_sync(0xffffffffu, all, o); }
  if (lane == 0) { s_red[0][warp] = before; s_red[1][warp] = all; }
  __syncthreads();                 // every value this CTA reads from the pool's state has arrived (it sits in shared memory)
  // ---- 3. the ticket
  const int total_ctas = gridDim.x * gridDim.y;
  if (threadIdx.x == 0) {
    __threadfence();
    s_last = atomicAdd(&v.counters[C_APPEND_TICKET], 1) == total_ctas - 1;
  }
  before = 0; all = 0;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { before += s_red[0][w]; all += s_red[1][w]; }
  const int fc = s_fc;
  if (all > fc) {
    // the free list cannot serve everybody: the serial rule decides who is skipped
    if (threadIdx.x == 0) {
      int remaining = fc, off = 0;
      for (int i = 0; i < n; ++i) {
        const int need = s_need[i];
        if (need < 0) continue;
        if (need > remaining) { s_need[i] = -1; s_S[i] = -1; if (reporter) flag_error(v.counters, STEP_ERR_NO_BLOCKS); continue; }
        if (i == idx) off = fc - remaining;
        remaining -= need;
      }
      s_off = off; s_granted = fc - remaining;
    }
  } else if (threadIdx.x == 0) {
    s_off = before; s_granted = all;
  }
  __syncthreads();
  const int S = s_S[idx], need = s_need[idx], off = s_off;
  const bool served = S >= 0;
  const int t = ids ? (served ? ids[idx] : 0) : idx;
  const int have = served ? (S + g.P - 1) / g.P : 0;
  // ---- 4a. this entry's new pages
  if (served && j == 0 && blockIdx.y == 0) {
    int32_t* row = v.block_table + (size_t)t * g.max_pages;
    for (int p = threadIdx.x; p < need; p += blockDim.x) {
      const int b = v.free_list[fc - 1 - off - p];
      row[have + p] = b;
      v.refcount[b] = 1;
    }
  }
  // ---- 3b. the last CTA to have read writes what was read
  if (s_last) {
    for (int i = threadIdx.x; i < n; i += blockDim.x)
      if (s_S[i] >= 0) v.seq_lens[ids ? ids[i] : i] = s_S[i] + n_tokens;
    if (threadIdx.x == 0) { v.counters[C_FREE_COUNT] = fc - s_granted; v.counters[C_APPEND_TICKET] = 0; }
    if (!ids) {
      // the lists of the Algorithm 1 iteration: traces that were live before this call, and those of them that have
      // just sampled the end-of-sequence token (ascending ids)
      __shared__ int s_cnt[2][8];
      int n_live = 0, n_fin = 0;
      for (int base = 0; base < n; base += blockDim.x) {
        const int u = base + threadIdx.x;
        const bool lv = u < n && v.live[u];
        const bool fin = lv && tokens && tokens[u] == eos;
        const unsigned bl = __ballot_sync(0xffffffffu, lv), bf = __ballot_sync(0xffffffffu, fin);
        __syncthreads();                                 // the counts of the pass before have been read
        if (lane == 0) { s_cnt[0][warp] = __popc(bl); s_cnt[1][warp] = __popc(bf); }
        __syncthreads();
        int bl_before = 0, bf_before = 0, bl_all = 0, bf_all = 0;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) {
          if (w < warp) { bl_before += s_cnt[0][w]; bf_before += s_cnt[1][w]; }
          bl_all += s_cnt[0][w]; bf_all += s_cnt[1][w];
        }
        const unsigned below = (1u << lane) - 1;
        if (lv) v.it_ids[n_live + bl_before + __popc(bl & below)] = u;
        if (fin) v.it_fin[n_fin + bf_before + __popc(bf & below)] = u;
        n_live += bl_all; n_fin += bf_all;
      }
      if (threadIdx.x == 0) { v.counters[C_IT_NLIVE] = n_live; v.counters[C_IT_NFIN] = n_fin; }
    }
  }
  // ---- 4b. the rows
  if (!served) return;
  const int pos = S + j, page = pos / g.P, slot = pos % g.P;
  const int b = page < have ? v.block_table[(size_t)t * g.max_pages + page] : v.free_list[fc - 1 - off - (page - have)];
  const int l0 = blockIdx.y * layers_per_cta, l1 = min(g.L, l0 + layers_per_cta);
  const int per_kv = g.Hkv * cpr;                                // chunks of the K (or V) rows of one layer
  const size_t row = src_by_id ? (size_t)t : (size_t)idx;
  const size_t src_token = (row * n_tokens + j) * (size_t)g.L * per_kv;
  const size_t page_chunks = (size_t)g.P * cpr;                  // 16-byte chunks of one K (or V) page
  for (int i = threadIdx.x; i < 2 * per_kv; i += blockDim.x) {
    const int which = i >= per_kv;
    const int r = which ? i - per_kv : i;
    const int head = r / cpr, c = r - head * cpr;
    const int cdst = g.swizzle ? ((c & ~7) | ((c ^ slot) & 7)) : c;
    const uint4* src = (which ? vnew : knew) + src_token + r;
    const size_t dst0 = (((size_t)b * g.Hkv + head) * 2 + which) * page_chunks + (size_t)slot * cpr + cdst;
    const size_t layer_stride = (size_t)g.num_blocks * g.Hkv * 2 * page_chunks;
    for (int l = l0; l < l1; ++l) kv[(size_t)l * layer_stride + dst0] = src[(size_t)l * per_kv];
  }
}

// ---------------------------------------------------------------- read-back of logical rows
__global__ void read_kv_kernel(Geo g, const uint4* __restrict__ kv, int layer, int head,
                               const int32_t* __restrict__ block_row, int seq_len, uint4* __restrict__ k_out,
                               uint4* __restrict__ v_out, int cpr, int cpe, int32_t* counters) {
  const size_t total = (size_t)seq_len * cpr * 2;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int which = i >= (size_t)seq_len * cpr;
    size_t r = which ? i - (size_t)seq_len * cpr : i;
    const int c = r % cpr; const int pos = r / cpr;
    const int page = pos / g.P, slot = pos % g.P;
    const int b = block_row[page];
    uint4 val = make_uint4(0, 0, 0, 0);
    if (b < 0 || b >= g.num_blocks) {
      flag_error(counters, STEP_ERR_BAD_BLOCK);
    } else {
      const int csrc = g.swizzle ? ((c & ~7) | ((c ^ slot) & 7)) : c;
      const size_t e = kv_page_base(g, layer, b, head, which) + (size_t)slot * g.d;
      val = kv[e / cpe + csrc];
    }
    (which ? v_out : k_out)[(size_t)pos * cpr + c] = val;
  }
}

int grid_for(size_t items, int threads, int num_sms) {
  size_t blocks = (items + threads - 1) / threads;
  size_t cap = (size_t)num_sms * 16;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  return (int)blocks;
}

}  // namespace

extern "C" {

const char* step_version(void) { return "libstep 0.1 (sm_100a)"; }

int kv_pool_required_bytes(const kv_pool_config* cfg, size_t* kv_bytes, size_t* meta_bytes) {
  if (!config_valid(cfg)) return STEP_ERR_INVALID_ARG;
  if (kv_bytes) *kv_bytes = kv_bytes_of(cfg);
  if (meta_bytes) *meta_bytes = make_layout(cfg).total;
  return STEP_OK;
}

int kv_pool_create(const kv_pool_config* cfg, step_pool** out) {
  if (!out) return STEP_ERR_INVALID_ARG;
  *out = nullptr;
  if (!config_valid(cfg)) return STEP_ERR_INVALID_ARG;
  if (!cfg->kv_storage || !cfg->meta_storage) return STEP_ERR_INVALID_ARG;
  if (((uintptr_t)cfg->kv_storage | (uintptr_t)cfg->meta_storage) & 255) return STEP_ERR_INVALID_ARG;
  MetaLayout lay = make_layout(cfg);
  if (cfg->kv_bytes < kv_bytes_of(cfg) || cfg->meta_bytes < lay.total) return STEP_ERR_INVALID_ARG;
  int dev = 0, sms = 0;
  STEP_CUDA_OK(cudaGetDevice(&dev));
  STEP_CUDA_OK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  step_pool* p = new (std::nothrow) step_pool();
  if (!p) return STEP_ERR_INVALID_ARG;
  p->cfg = *cfg;
  p->G = cfg->num_q_heads / cfg->num_kv_heads;
  p->elem_bytes = cfg->dtype == STEP_BF16 ? 2 : 4;
  p->swizzle = (cfg->dtype == STEP_BF16 && cfg->head_dim % 64 == 0) ? 1 : 0;
  p->max_score_rows = cfg->max_score_rows > 0 ? cfg->max_score_rows : cfg->max_traces;
  p->num_sms = sms;
  p->attn_grid = sms;
  p->attn_dyn16 = 4;
  p->attn_dyn_chunk = 16;
  p->fast_path = 1;
  p->wait_limit_ns = 2000000000ull;
  p->scorer_mode = 0;
  p->scorer_tc_min_rows = 1;
  p->tmap_w1 = nullptr; p->tmap_D = 0; p->tmap_m = 0; p->tc_smem_set = false;
  p->tmap_h_ptr = nullptr; p->tmap_h_D = 0; p->tmap_h_M = 0;
  p->device = dev;
  p->lay = lay;
  char* m = static_cast<char*>(cfg->meta_storage);
  DevViews& v = p->v;
  v.block_table = (int32_t*)(m + lay.block_table); v.seq_lens = (int32_t*)(m + lay.seq_lens);
  v.live = (uint8_t*)(m + lay.live); v.score_sum = (float*)(m + lay.score_sum);
  v.score_cnt = (int32_t*)(m + lay.score_cnt); v.trace_scores = (float*)(m + lay.trace_scores);
  v.refcount = (int32_t*)(m + lay.refcount); v.free_list = (int32_t*)(m + lay.free_list);
  v.claim = (int32_t*)(m + lay.claim); v.counters = (int32_t*)(m + lay.counters);
  v.append_base = (int32_t*)(m + lay.append_base); v.prune_rank = (int32_t*)(m + lay.prune_rank);
  v.prune_list = (int32_t*)(m + lay.prune_list); v.prune_off = (int32_t*)(m + lay.prune_off);
  v.score_idx = (int32_t*)(m + lay.score_idx); v.score_z = (float*)(m + lay.score_z);
  v.score_part = (float2*)(m + lay.score_part);
  v.score_zs = (float*)(m + lay.score_zs);
  v.attn_ml = (float*)(m + lay.attn_ml); v.attn_o = (float*)(m + lay.attn_o); v.attn_sched = (int32_t*)(m + lay.attn_sched);
  const bool mma = lay.pre_ws_o != lay.pre_ml;      // the regions are zero-sized for other shapes
  v.pre_ws_ml = mma ? (float*)(m + lay.pre_ws_ml) : nullptr; v.pre_ws_o = mma ? (float*)(m + lay.pre_ws_o) : nullptr;
  v.pre_ml = mma ? (float*)(m + lay.pre_ml) : nullptr; v.pre_o = mma ? (float*)(m + lay.pre_o) : nullptr;
  v.final_score = (float*)(m + lay.final_score); v.answer = (int32_t*)(m + lay.answer);
  v.finished = (uint8_t*)(m + lay.finished); v.it_ids = (int32_t*)(m + lay.it_ids);
  v.it_fin = (int32_t*)(m + lay.it_fin); v.it_pruned = (int32_t*)(m + lay.it_pruned);
  v.it_tokens = (int32_t*)(m + lay.it_tokens); v.it_scores = (float*)(m + lay.it_scores);
  int st = kv_pool_reset(p, nullptr);
  if (st == STEP_OK && cudaStreamSynchronize(nullptr) != cudaSuccess) st = STEP_ERR_CUDA;
  if (st != STEP_OK) { delete p; return st; }
  *out = p;
  return STEP_OK;
}

int kv_pool_destroy(step_pool* pool) {
  if (!pool) return STEP_ERR_INVALID_ARG;
  delete pool;
  return STEP_OK;
}

int kv_pool_reset(step_pool* pool, void* stream) {
  if (!pool) return STEP_ERR_INVALID_ARG;
  Geo g = geo_of(pool);
  size_t items = (size_t)g.max_traces * g.max_pages;
  if ((size_t)g.num_blocks > items) items = g.num_blocks;
  init_meta_kernel<<<grid_for(items, 256, pool->num_sms), 256, 0, (cudaStream_t)stream>>>(pool->v, g, pool->cfg.unscored_score);
  return launch_ok();
}

int kv_pool_fork_prefix(step_pool* pool, int n_traces, int prefix_len, const void* k_prefix,
                        const void* v_prefix, int32_t* trace_ids_out, void* stream) {
  if (!pool || n_traces < 1 || prefix_len < 0) return STEP_ERR_INVALID_ARG;
  if (prefix_len > 0 && (!k_prefix || !v_prefix)) return STEP_ERR_INVALID_ARG;
  Geo g = geo_of(pool);
  if (n_traces > g.max_traces) return STEP_ERR_CAPACITY;
  if ((prefix_len + g.P - 1) / g.P > g.max_pages) return STEP_ERR_CAPACITY;
  cudaStream_t s = (cudaStream_t)stream;
  fork_alloc_kernel<<<1, 256, 0, s>>>(pool->v, g, n_traces, prefix_len);
  if (prefix_len > 0) {
    const int cpe = 16 / pool->elem_bytes, cpr = g.d / cpe;
    int splits = (2 * pool->num_sms + prefix_len - 1) / prefix_len;
    if (splits > g.L) splits = g.L;
    if (splits < 1) splits = 1;
    const int layers_per_cta = (g.L + splits - 1) / splits;
    splits = (g.L + layers_per_cta - 1) / layers_per_cta;
    fork_write_kernel<<<dim3((unsigned)prefix_len, (unsigned)splits), 256, 0, s>>>(
        pool->v, g, (uint4*)pool->cfg.kv_storage, (const uint4*)k_prefix, (const uint4*)v_prefix,
        n_traces, prefix_len, cpr, layers_per_cta);
  }
  const int st = launch_ok();
  if (st != STEP_OK || !trace_ids_out) return st;
  // the ids were decided on the device: fetch the outcome (the one synchronising path of this call)
  int32_t h[C_FORK_FIRST + 1];
  STEP_CUDA_OK(cudaMemcpyAsync(h, pool->v.counters, sizeof(h), cudaMemcpyDeviceToHost, s));
  STEP_CUDA_OK(cudaStreamSynchronize(s));
  for (int j = 0; j < n_traces; ++j) trace_ids_out[j] = h[C_FORK_OK] ? h[C_FORK_FIRST] + j : -1;
  return STEP_OK;
}

int append_kv(step_pool* pool, const int32_t* trace_ids, int n, int n_tokens, const void* k_new,
              const void* v_new, void* stream) {
  if (!trace_ids && n > 0 && n_tokens > 0) return STEP_ERR_INVALID_ARG;
  return stepk::append_kv_impl(pool, trace_ids, n, n_tokens, k_new, v_new, nullptr, 0, (cudaStream_t)stream, nullptr, 0);
}

}  // extern "C"

int stepk::append_kv_impl(step_pool* pool, const int32_t* trace_ids, int n, int n_tokens, const void* k_new,
                          const void* v_new, const int32_t* n_dev, int src_by_id, cudaStream_t s,
                          const int32_t* live_tokens, int eos) {
  if (!pool || n < 0 || n_tokens < 0) return STEP_ERR_INVALID_ARG;
  if (n == 0 || n_tokens == 0) return STEP_OK;
  if (!k_new || !v_new) return STEP_ERR_INVALID_ARG;
  if (n > pool->cfg.max_traces) return STEP_ERR_INVALID_ARG;   // ids must be distinct
  Geo g = geo_of(pool);
  const int cpe = 16 / pool->elem_bytes, cpr = g.d / cpe;
  const size_t row_chunks = (size_t)n_tokens * g.L * g.Hkv * cpr;   // 16-byte chunks of K (or V) per trace
  constexpr int kListChunk = 2048;                                  // traces per launch (24 KiB of shared memory for the scan)
  if (!trace_ids && (n > kListChunk || !src_by_id)) return STEP_ERR_INVALID_ARG;   // the live-trace form is one launch, rows by trace id
  for (int off = 0; off < n; off += kListChunk) {
    const int m = n - off < kListChunk ? n - off : kListChunk;
    if (n_dev && off > 0) return STEP_ERR_INVALID_ARG;              // a device-side count covers one launch only
    const size_t src_off = src_by_id ? 0 : row_chunks * off;
    // enough CTAs to occupy the device: (trace, token) pairs x splits of the layer range
    const long long pairs = (long long)m * n_tokens;
    if (pairs > 0x7fffffffll) return STEP_ERR_INVALID_ARG;
    int splits = (int)((2ll * pool->num_sms + pairs - 1) / pairs);
    if (splits > g.L) splits = g.L;
    if (splits < 1) splits = 1;
    const int layers_per_cta = (g.L + splits - 1) / splits;
    splits = (g.L + layers_per_cta - 1) / layers_per_cta;
    if (!trace_ids || g.max_traces <= kFusedMaxTraces) {
      // one launch does it all
      const size_t smem = ((size_t)2 * m + (trace_ids ? g.max_traces : 0)) * sizeof(int);
      append_fused_kernel<<<dim3((unsigned)pairs, (unsigned)splits), 256, smem, s>>>(
          pool->v, g, (uint4*)pool->cfg.kv_storage, (const uint4*)k_new + src_off, (const uint4*)v_new + src_off,
          trace_ids ? trace_ids + off : nullptr, m, n_tokens, n_dev, live_tokens, eos, cpr, layers_per_cta, src_by_id);
      if (launch_ok() != STEP_OK) return STEP_ERR_CUDA;
      continue;
    }
    // larger pools: the allocation in a kernel of its own (its table of first places lives in global memory), the rows
    // by its programmatic dependent: scheduled while that one runs, waits for it before its first read
    append_alloc_kernel<<<1, 256, (size_t)m * 3 * sizeof(int), s>>>(pool->v, g, trace_ids + off, m, n_tokens, n_dev);
    if (launch_dependent(append_write_kernel, dim3((unsigned)pairs, (unsigned)splits), dim3(256), 0, s, pool->v, g,
                         (uint4*)pool->cfg.kv_storage, (const uint4*)k_new + src_off, (const uint4*)v_new + src_off,
                         trace_ids + off, n_tokens, cpr, layers_per_cta, src_by_id) != cudaSuccess)
      return STEP_ERR_CUDA;
  }
  return launch_ok();
}

extern "C" {

int kv_pool_stats(step_pool* pool, int* used, int* free_, int* total, int* live_traces, void* stream) {
  if (!pool) return STEP_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  int fc = 0;
  std::vector<uint8_t> live(pool->cfg.max_traces);
  STEP_CUDA_OK(cudaMemcpyAsync(&fc, pool->v.counters + C_FREE_COUNT, sizeof(int), cudaMemcpyDeviceToHost, s));
  STEP_CUDA_OK(cudaMemcpyAsync(live.data(), pool->v.live, live.size(), cudaMemcpyDeviceToHost, s));
  STEP_CUDA_OK(cudaStreamSynchronize(s));
  int nl = 0;
  for (uint8_t b : live) nl += b != 0;
  if (used) *used = pool->cfg.num_blocks - fc;
  if (free_) *free_ = fc;
  if (total) *total = pool->cfg.num_blocks;
  if (live_traces) *live_traces = nl;
  return STEP_OK;
}

int kv_pool_device_views(step_pool* pool, int32_t** block_table, int32_t** seq_lens, float** trace_scores,
                         int32_t** free_list, int32_t** free_count, int32_t** refcount, uint8_t** live) {
  if (!pool) return STEP_ERR_INVALID_ARG;
  if (block_table) *block_table = pool->v.block_table;
  if (seq_lens) *seq_lens = pool->v.seq_lens;
  if (trace_scores) *trace_scores = pool->v.trace_scores;
  if (free_list) *free_list = pool->v.free_list;
  if (free_count) *free_count = pool->v.counters + C_FREE_COUNT;
  if (refcount) *refcount = pool->v.refcount;
  if (live) *live = pool->v.live;
  return STEP_OK;
}

int kv_pool_score_views(step_pool* pool, float** score_sum, int32_t** score_cnt) {
  if (!pool) return STEP_ERR_INVALID_ARG;
  if (score_sum) *score_sum = pool->v.score_sum;
  if (score_cnt) *score_cnt = pool->v.score_cnt;
  return STEP_OK;
}

int kv_pool_last_error(step_pool* pool, unsigned* mask_out, void* stream) {
  if (!pool) return STEP_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  unsigned mask = 0;
  STEP_CUDA_OK(cudaMemcpyAsync(&mask, pool->v.counters + C_STATUS, sizeof(mask), cudaMemcpyDeviceToHost, s));
  STEP_CUDA_OK(cudaMemsetAsync(pool->v.counters + C_STATUS, 0, sizeof(int), s));
  STEP_CUDA_OK(cudaStreamSynchronize(s));
  if (mask_out) *mask_out = mask;
  for (int code = 1; code < 32; ++code)
    if (mask & (1u << code)) return code;
  return STEP_OK;
}

int kv_pool_read_kv(step_pool* pool, int layer, int kv_head, const int32_t* block_row, int seq_len,
                    void* k_out, void* v_out, void* stream) {
  if (!pool || !block_row || seq_len < 0) return STEP_ERR_INVALID_ARG;
  Geo g = geo_of(pool);
  if (layer < 0 || layer >= g.L || kv_head < 0 || kv_head >= g.Hkv) return STEP_ERR_INVALID_ARG;
  if ((seq_len + g.P - 1) / g.P > g.max_pages) return STEP_ERR_INVALID_ARG;
  if (seq_len == 0) return STEP_OK;
  if (!k_out || !v_out) return STEP_ERR_INVALID_ARG;
  const int cpe = 16 / pool->elem_bytes, cpr = g.d / cpe;
  size_t chunks = (size_t)seq_len * cpr * 2;
  read_kv_kernel<<<grid_for(chunks, 256, pool->num_sms), 256, 0, (cudaStream_t)stream>>>(
      g, (const uint4*)pool->cfg.kv_storage, layer, kv_head, block_row, seq_len, (uint4*)k_out, (uint4*)v_out,
      cpr, cpe, pool->v.counters);
  return launch_ok();
}

int kv_pool_set_wait_limit_ns(step_pool* pool, unsigned long long ns) {
  if (!pool) return STEP_ERR_INVALID_ARG;
  pool->wait_limit_ns = ns;
  return STEP_OK;
}

int kv_pool_set_attention_config(step_pool* pool, int grid_ctas, int fast_path) {
  if (!pool || grid_ctas < 0) return STEP_ERR_INVALID_ARG;
  if (grid_ctas > 0) pool->attn_grid = grid_ctas;
  if (fast_path != 0) pool->fast_path = fast_path > 0 ? 1 : -1;
  return STEP_OK;
}

int kv_pool_set_attention_balance(step_pool* pool, int dynamic_sixteenths, int min_chunk_pages) {
  if (!pool || dynamic_sixteenths < 0 || dynamic_sixteenths > 12 || min_chunk_pages < 0) return STEP_ERR_INVALID_ARG;
  pool->attn_dyn16 = dynamic_sixteenths;
  if (min_chunk_pages > 0) pool->attn_dyn_chunk = min_chunk_pages;
  return STEP_OK;
}

}  // extern "C"
