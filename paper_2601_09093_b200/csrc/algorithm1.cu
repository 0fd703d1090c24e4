// Algorithm 1 as a loop over device-resident state.
//
//   T <- InitTraces(P, N)
//   while T is not empty:
//     for each trace t in T:  (x, h) <- NextToken(t);  if x ends a step: y <- f(h), update score_t
//                             if GPUMemoryFull: evict argmin score_t, release its KV, drop it from T
//   answer <- WeightedVote(T, {score_t})                                 (Sec. 3.3, last paragraph)
//
// The model's forward pass is not part of this library, so NextToken is represented by its inputs and
// outputs: the caller supplies, per iteration, the sampled token of every trace, the new K/V rows, the
// queries of every layer and the last-layer hidden states; this file chains the library's own steps on
// them - cache write, attention over the paged cache, step-end detection, scorer, completion of traces
// that sampled the end-of-sequence token, memory trigger and eviction (four launches besides the attention's) -
// without a host round trip: row i
// of every input is trace i, and traces that are no longer live are passed over on the device.
// One trigger check is made per iteration (a batch of NextToken calls), after the batch's cache writes.
//
// A trace that completes keeps what the vote needs (its final score_t and its answer) and gives its KV
// back at once; the vote runs over the completed traces - the evicted ones never vote.
#include "release.cuh"

#include <string.h>

#include <vector>

using namespace stepk;

namespace {

// Completion: every valid, live listed trace records (score_t, answer) for the vote, then the cluster
// releases their KV exactly as an eviction would.  n_dev (may be null) caps the list on the device;
// answers are indexed by trace id (by_trace) or by position in the list.
__device__ inline void finish_listed_cluster(DevViews& v, const Geo& g, const int32_t* __restrict__ ids, int n,
                                             const int32_t* __restrict__ n_dev, const int32_t* __restrict__ answers,
                                             int by_trace, float unscored, int* s_warp) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  if (n_dev && *n_dev <= 0) return;      // nobody completes (every CTA reads the same count: the whole cluster passes)
  if (cluster.block_rank() == 0) {
    const int n_eff = n_dev ? min(n, max(*n_dev, 0)) : n;
    // an id listed twice completes once, at its first place in the list (v.prune_rank records that place)
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
    int k = 0;
    for (int base = 0; base < n_eff; base += blockDim.x) {
      const int i = base + threadIdx.x;
      int t = -1, ok = 0;
      if (i < n_eff) {
        t = ids[i];
        ok = t >= 0 && t < g.max_traces && v.live[t] && v.prune_rank[t] == i;
        if (!ok) flag_error(v.counters, STEP_ERR_BAD_TRACE);
      }
      int total;
      const int at = block_excl_scan(ok, s_warp, &total);
      if (ok) {
        v.prune_list[k + at] = t;
        v.final_score[t] = v.trace_scores[t];
        v.answer[t] = answers ? answers[by_trace ? t : i] : -1;
        v.finished[t] = 1;
      }
      k += total;
    }
    if (threadIdx.x == 0) { v.counters[C_PRUNE_N] = k; v.counters[C_N_FINISHED] += k; }
    __threadfence();
  }
  cluster.sync();
  release_listed_cluster(v, g, __ldcg(&v.counters[C_PRUNE_N]), unscored, s_warp);
}

__global__ void __cluster_dims__(kClusterCtas, 1, 1) __launch_bounds__(kPruneThreads, 1)
finish_kernel(DevViews v, Geo g, const int32_t* __restrict__ ids, int n, const int32_t* __restrict__ n_dev,
              const int32_t* __restrict__ answers, int by_trace, float unscored) {
  __shared__ int s_warp[33];
  finish_listed_cluster(v, g, ids, n, n_dev, answers, by_trace, unscored, s_warp);
}

// The end of one iteration of the loop in a single launch: the live traces that sampled the end-of-sequence token
// complete (v.it_fin, listed by the iteration's cache-write kernel), then the memory trigger is tested and the
// eviction rule applied up to `tests` times, each test seeing the pool the one before it left.
__global__ void __cluster_dims__(kClusterCtas, 1, 1) __launch_bounds__(kPruneThreads, 1)
iter_tail_kernel(DevViews v, Geo g, int n, const int32_t* __restrict__ answers, float threshold, float keep_frac, int tests,
                 float unscored, int32_t* __restrict__ pruned_ids_out, int32_t* __restrict__ n_pruned_out) {
  __shared__ int s_warp[33];
  finish_listed_cluster(v, g, v.it_fin, n, v.counters + C_IT_NFIN, answers, 1, unscored, s_warp);
  for (int k = 0; k < tests; ++k)
    if (!trigger_and_evict_cluster(v, g, nullptr, threshold, keep_frac, unscored, pruned_ids_out, n_pruned_out, s_warp)) break;
}

// WeightedVote: total[a] = sum of final scores of the completed traces that answered a; the largest total
// wins, equal totals go to the smaller answer id.  A warp per completed trace sums the scores of all traces
// with the same answer (lanes over traces in a fixed pattern, so equal answers get bit-equal totals).
__global__ void __launch_bounds__(1024)
vote_kernel(DevViews v, Geo g, int32_t* __restrict__ answer_out, float* __restrict__ weight_out,
            int32_t* __restrict__ n_finished_out) {
  __shared__ float s_best_w[32];
  __shared__ int s_best_a[32], s_cnt[32];
  const int T = g.max_traces;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  float best_w = -1.f;
  int best_a = -1, cnt = 0;
  for (int t = warp; t < T; t += nwarps) {
    if (!v.finished[t]) continue;                    // warp-uniform
    ++cnt;
    const int a = v.answer[t];
    if (a < 0) continue;                             // completed without an answer: takes no part in the vote
    float acc = 0.f;
    for (int u = lane; u < T; u += 32)
      if (v.finished[u] && v.answer[u] == a) acc += v.final_score[u];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (best_a < 0 || acc > best_w || (acc == best_w && a < best_a)) { best_w = acc; best_a = a; }
  }
  if (lane == 0) { s_best_w[warp] = best_w; s_best_a[warp] = best_a; s_cnt[warp] = cnt; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float bw = -1.f;
    int ba = -1, n = 0;
    for (int w = 0; w < nwarps; ++w) {
      n += s_cnt[w];
      if (s_best_a[w] < 0) continue;
      if (ba < 0 || s_best_w[w] > bw || (s_best_w[w] == bw && s_best_a[w] < ba)) { bw = s_best_w[w]; ba = s_best_a[w]; }
    }
    *answer_out = ba;
    if (weight_out) *weight_out = ba < 0 ? 0.f : bw;
    if (n_finished_out) *n_finished_out = n;
  }
}

}  // namespace

extern "C" {

int kv_pool_finish_traces(step_pool* pool, const int32_t* trace_ids, const int32_t* answers, int n, void* stream) {
  if (!pool || n < 0) return STEP_ERR_INVALID_ARG;
  if (n == 0) return STEP_OK;
  if (!trace_ids || n > pool->cfg.max_traces) return STEP_ERR_INVALID_ARG;
  finish_kernel<<<kClusterCtas, kPruneThreads, 0, (cudaStream_t)stream>>>(pool->v, geo_of(pool), trace_ids, n, nullptr,
                                                                          answers, 0, pool->cfg.unscored_score);
  return launch_ok();
}

int weighted_vote(step_pool* pool, int32_t* answer_out, float* weight_out, int32_t* n_finished_out, void* stream) {
  if (!pool || !answer_out) return STEP_ERR_INVALID_ARG;
  vote_kernel<<<1, 1024, 0, (cudaStream_t)stream>>>(pool->v, geo_of(pool), answer_out, weight_out, n_finished_out);
  return launch_ok();
}

int kv_pool_vote_views(step_pool* pool, float** final_score, int32_t** answer, uint8_t** finished) {
  if (!pool) return STEP_ERR_INVALID_ARG;
  if (final_score) *final_score = pool->v.final_score;
  if (answer) *answer = pool->v.answer;
  if (finished) *finished = pool->v.finished;
  return STEP_OK;
}

int algorithm1_iteration(step_pool* pool, const step_iteration* it, void* stream) {
  if (!pool || !it) return STEP_ERR_INVALID_ARG;
  const int n = it->n_traces;
  if (n < 1 || n > pool->cfg.max_traces) return STEP_ERR_INVALID_ARG;
  if (!it->token_ids || !it->step_end_table || it->vocab < 1 || !it->k_new || !it->v_new || !it->hidden ||
      !it->scorer || !it->step_scores_out)
    return STEP_ERR_INVALID_ARG;
  if (it->n_layers_attention < 0 || it->n_layers_attention > pool->cfg.num_layers) return STEP_ERR_INVALID_ARG;
  if (it->n_layers_attention > 0 && (!it->q || !it->attn_out)) return STEP_ERR_INVALID_ARG;
  if (!(it->threshold > 0.f) || it->threshold > 1.f) return STEP_ERR_INVALID_ARG;
  if (isnan(it->keep_frac) || it->keep_frac == 0.f || it->keep_frac > 1.f) return STEP_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  Geo g = geo_of(pool);
  DevViews& v = pool->v;
  int st;
  // NextToken's cache write for the live traces (row t of k_new / v_new belongs to trace t); the same kernel lists
  // who is live and who completes
  st = append_kv_impl(pool, nullptr, n, 1, it->k_new, it->v_new, nullptr, 1, s, it->token_ids, it->eos_token);
  if (st != STEP_OK) return st;
  // NextToken's attention, layer by layer (traces that are not live have length 0 and get zeros)
  st = decode_attention_layers(pool, 0, it->n_layers_attention, it->q, v.block_table, v.seq_lens, n, it->attn_out, stream);
  if (st != STEP_OK) return st;
  // `if x ends a step: y <- f(h); update score_t`
  FlagSource src{nullptr, it->token_ids, it->step_end_table, it->vocab, it->boundary_mask_out, v.live};
  st = score_steps_impl(pool, it->hidden, src, nullptr, n, it->scorer, it->step_scores_out, it->trace_scores_out, n, stream);
  if (st != STEP_OK) return st;
  // traces that sampled the end-of-sequence token complete; `if GPUMemoryFull: evict`
  int32_t* pruned = it->pruned_ids_out ? it->pruned_ids_out : v.it_pruned;
  int32_t* n_pruned = it->n_pruned_out ? it->n_pruned_out : v.counters + C_IT_NPRUNED;
  const int tests = it->max_evictions > 1 ? it->max_evictions : 1;
  iter_tail_kernel<<<kClusterCtas, kPruneThreads, 0, s>>>(v, g, n, it->answers, it->threshold, it->keep_frac, tests,
                                                          pool->cfg.unscored_score, pruned, n_pruned);
  if (launch_ok() != STEP_OK) return STEP_ERR_CUDA;
  return STEP_OK;
}

int algorithm1_run(step_pool* pool, const step_run_args* a, step_run_result* res, void* stream) {
  if (!pool || !a || !res) return STEP_ERR_INVALID_ARG;
  if (a->max_iterations < 1 || a->ring < 1 || a->check_every < 1 || !a->token_ids) return STEP_ERR_INVALID_ARG;
  const int n = a->n_traces;
  if (n < 1 || n > pool->cfg.max_traces) return STEP_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  Geo g = geo_of(pool);
  const int La = a->n_layers_attention;
  const size_t eb = pool->elem_bytes;
  const size_t q_slot = (size_t)La * n * g.Hq * g.d * eb;
  const size_t kv_slot = (size_t)n * g.L * g.Hkv * g.d * eb;
  const size_t h_slot = a->scorer ? (size_t)n * a->scorer->D * (a->scorer->dtype == STEP_BF16 ? 2 : 4) : 0;
  // With use_graphs the launches of one iteration are recorded once per ring slot and replayed: what changes from
  // one use of a slot to the next (the tokens, the row of the score history) goes through fixed staging rows.
  bool graphs = a->use_graphs != 0 && s != nullptr && s != cudaStreamLegacy;
  if (graphs) {
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(s, &cs) != cudaSuccess || cs != cudaStreamCaptureStatusNone) graphs = false;
  }
  std::vector<cudaGraphExec_t> execs(graphs ? a->ring : 0, nullptr);
  auto drop_graphs = [&]() { for (cudaGraphExec_t e : execs) if (e) cudaGraphExecDestroy(e); };
  int done = 0, live = -1;
  for (int i = 0; i < a->max_iterations; ++i) {
    const int slot = i % a->ring;
    step_iteration it;
    it.n_traces = n;
    it.token_ids = graphs ? pool->v.it_tokens : a->token_ids + (size_t)i * n;
    it.eos_token = a->eos_token;
    it.step_end_table = a->step_end_table; it.vocab = a->vocab;
    it.answers = a->answers;
    it.n_layers_attention = La;
    it.q = a->q ? (const char*)a->q + slot * q_slot : nullptr;
    it.k_new = (const char*)a->k_new + slot * kv_slot;
    it.v_new = (const char*)a->v_new + slot * kv_slot;
    it.hidden = (const char*)a->hidden + slot * h_slot;
    it.attn_out = a->attn_out;
    it.step_scores_out = a->step_scores_out;
    it.boundary_mask_out = nullptr;
    it.scorer = a->scorer;
    it.threshold = a->threshold; it.keep_frac = a->keep_frac;
    it.max_evictions = a->max_evictions;
    it.pruned_ids_out = nullptr; it.n_pruned_out = nullptr;
    float* hist_row = a->score_history ? a->score_history + (size_t)i * n : nullptr;
    it.trace_scores_out = graphs ? (hist_row ? pool->v.it_scores : nullptr) : hist_row;
    if (!graphs) {
      const int st = algorithm1_iteration(pool, &it, stream);
      if (st != STEP_OK) return st;
    } else {
      if (!execs[slot]) {
        cudaGraph_t graph = nullptr;
        if (cudaStreamBeginCapture(s, cudaStreamCaptureModeThreadLocal) != cudaSuccess) { drop_graphs(); return STEP_ERR_CUDA; }
        const int st = algorithm1_iteration(pool, &it, stream);
        const cudaError_t e = cudaStreamEndCapture(s, &graph);          // always leaves capture mode
        if (st != STEP_OK || e != cudaSuccess || !graph) {
          if (graph) cudaGraphDestroy(graph);
          drop_graphs();
          cudaGetLastError();
          return st != STEP_OK ? st : STEP_ERR_CUDA;
        }
        const cudaError_t e2 = cudaGraphInstantiate(&execs[slot], graph, 0);
        cudaGraphDestroy(graph);
        if (e2 != cudaSuccess) { execs[slot] = nullptr; drop_graphs(); return STEP_ERR_CUDA; }
      }
      cudaError_t e = cudaMemcpyAsync(pool->v.it_tokens, a->token_ids + (size_t)i * n, (size_t)n * sizeof(int32_t),
                                      cudaMemcpyDeviceToDevice, s);
      if (e == cudaSuccess) e = cudaGraphLaunch(execs[slot], s);
      if (e == cudaSuccess && hist_row)
        e = cudaMemcpyAsync(hist_row, pool->v.it_scores, (size_t)n * sizeof(float), cudaMemcpyDeviceToDevice, s);
      if (e != cudaSuccess) { drop_graphs(); return STEP_ERR_CUDA; }
    }
    done = i + 1;
    if (done % a->check_every == 0 || done == a->max_iterations) {
      // the only host round trip of the loop: is anyone still live?
      const int st2 = kv_pool_stats(pool, nullptr, nullptr, nullptr, &live, stream);
      if (st2 != STEP_OK) { drop_graphs(); return st2; }
      if (live == 0) break;
    }
  }
  if (graphs) {
    if (cudaStreamSynchronize(s) != cudaSuccess) { drop_graphs(); return STEP_ERR_CUDA; }
    drop_graphs();
  }
  int32_t* out = pool->v.it_pruned;                 // free between iterations: answer, count; weight as float bits
  const int st = weighted_vote(pool, out, reinterpret_cast<float*>(out + 1), out + 2, stream);
  if (st != STEP_OK) return st;
  int32_t h[3];
  int32_t c[C_NUM];
  STEP_CUDA_OK(cudaMemcpyAsync(h, out, sizeof(h), cudaMemcpyDeviceToHost, s));
  STEP_CUDA_OK(cudaMemcpyAsync(c, pool->v.counters, sizeof(c), cudaMemcpyDeviceToHost, s));
  STEP_CUDA_OK(cudaStreamSynchronize(s));
  res->iterations = done;
  res->answer = h[0];
  memcpy(&res->answer_weight, &h[1], sizeof(float));
  res->n_finished = h[2];
  res->n_evicted = c[C_N_EVICTED];
  res->live_left = live;
  return STEP_OK;
}

}  // extern "C"
