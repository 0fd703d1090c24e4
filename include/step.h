/*
 * libstep - C ABI of the STEP parallel-trace decode hot path on one B200 (sm_100a).
 *
 * STEP (Step-level Trace Evaluation and Pruning) samples N reasoning traces of one
 * problem in parallel, scores every finished reasoning step with a small MLP on the
 * step-end token's last-layer hidden state, and - when the KV-cache memory is full -
 * evicts the trace with the lowest mean step score and releases its KV cache at once
 * (Algorithm 1; Sec. 3.1 "Step Scorer"; Sec. 3.2 "Memory Constraint as Trigger";
 * Sec. 3.3 running-average equation).  This library is the data-parallel part of one
 * decode iteration of Algorithm 1 on device-resident state:
 *
 *   kv_pool_create / kv_pool_fork_prefix   InitTraces(P, N): N traces share one prompt
 *   append_kv                              store the new token's K/V (NextToken's cache write)
 *   decode_attention                       the attention of NextToken over the paged cache
 *   score_steps                            y = f(h) at step ends; update score_t
 *   prune_if_saturated                     if GPUMemoryFull: evict, ReleaseKVCache
 *
 * Conventions
 *  - Every call returns a step_status.  Argument checks are made on the host and fail
 *    at once with nothing launched.  Conditions only the device can see (free list empty,
 *    block table full, bad trace id, bad block id) never trap: the kernel skips the
 *    affected trace, ORs (1 << code) into a sticky device status word and carries on;
 *    kv_pool_last_error reads and clears that word.
 *  - The library allocates no device memory.  KV storage, metadata (which includes all
 *    kernel scratch) and every input/output buffer belong to the caller and must outlive
 *    the pool / the call.  Pointers are DEVICE pointers unless marked "host".
 *  - `stream` is a cudaStream_t passed as void*.  Calls are asynchronous on it and ordered
 *    by it, except those documented as synchronising.  One pool must not be used from two
 *    streams at once.
 *  - dtype: STEP_BF16 (0) or STEP_FP32 (1) is the storage type of K/V, q, hidden states and
 *    scorer weights.  Accumulation and all outputs are fp32.
 *  - Query head h reads KV head h / G, G = num_q_heads / num_kv_heads.
 *  - Decode order: append_kv for the new token comes BEFORE decode_attention; the query
 *    attends to all S_t stored positions including its own; there is no mask.
 *  - The physical layout of kv_storage is private to the library (kv_pool_read_kv returns
 *    logical rows).  Metadata arrays are visible through kv_pool_device_views.
 */
#ifndef STEP_H_
#define STEP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct step_pool step_pool; /* opaque, host object */

typedef enum {
  STEP_OK = 0,
  STEP_ERR_INVALID_ARG = 1, /* host-side argument check failed                          */
  STEP_ERR_NO_BLOCKS = 2,   /* free list too short for the request                      */
  STEP_ERR_BAD_TRACE = 3,   /* trace id out of range or not live                        */
  STEP_ERR_CAPACITY = 4,    /* trace would exceed max_pages_per_trace / max_traces      */
  STEP_ERR_CUDA = 5,        /* a CUDA runtime call failed (no device, launch error...)  */
  STEP_ERR_TIMEOUT = 6,     /* a bounded device-side wait ran out                       */
  STEP_ERR_BAD_BLOCK = 7    /* a block-table entry read by a kernel was out of range    */
} step_status;

enum { STEP_BF16 = 0, STEP_FP32 = 1 };

typedef struct {
  int num_layers, num_q_heads, num_kv_heads, head_dim, page_size;
  int num_blocks;          /* a block holds page_size tokens of ALL layers and KV heads  */
  int max_traces, max_pages_per_trace;
  int dtype;               /* STEP_BF16 | STEP_FP32                                       */
  int max_score_rows;      /* largest M one score_steps launch handles; 0 = max_traces    */
  float unscored_score;    /* score_t of a trace with no scored step yet (paper: 0/0)     */
  void* kv_storage;   size_t kv_bytes;   /* device memory, 256-byte aligned              */
  void* meta_storage; size_t meta_bytes; /* device memory, 256-byte aligned              */
} kv_pool_config;

/* Step scorer parameters (Sec. 3.1 "Model Architecture"): W1 [m, D] row-major, b1 [m],
 * w2 [m] in `dtype`; b2 scalar.  Device pointers. */
typedef struct {
  const void* W1; const void* b1; const void* w2;
  float b2;
  int D, m;
  int dtype;
} scorer_weights;

/* Bytes the caller must provide for a configuration (storage pointers in cfg are ignored).
 * Host-only, needs no GPU. */
int kv_pool_required_bytes(const kv_pool_config* cfg, size_t* kv_bytes, size_t* meta_bytes);

/* InitTraces, part 1: build a pool over caller memory.  All blocks free (the free list is a
 * stack holding [num_blocks-1 .. 0], so the first allocation is block 0), no live trace.
 * Initialises the metadata on the legacy default stream and synchronises. */
int kv_pool_create(const kv_pool_config* cfg, step_pool** out);
int kv_pool_destroy(step_pool* pool);
/* Back to the freshly created state (asynchronous on stream). */
int kv_pool_reset(step_pool* pool, void* stream);

/* InitTraces, part 2 (Algorithm 1, first line): start n_traces traces that share one prompt.
 * k_prefix, v_prefix: [num_layers, num_kv_heads, prefix_len, head_dim] in pool dtype.
 * Full prompt pages are allocated once and shared (refcount = n_traces); if prefix_len is
 * not a multiple of page_size every trace gets a private copy of the last, partial page.
 * Trace ids are consecutive, continuing from the last fork that went through; they are handed out on the
 * device.  trace_ids_out (HOST, n_traces ints, may be NULL): if given, the call synchronises the stream and
 * writes the ids there, or -1 in every entry if the fork failed on the device; with NULL the call is
 * asynchronous and the ids are the next n_traces in sequence.  n_traces > max_traces or a prompt longer than
 * max_pages_per_trace pages is STEP_ERR_CAPACITY at once.  Checked on the device: more traces than max_traces
 * in all (CAPACITY) or a free list too short (NO_BLOCKS) - the fork is then a no-op that consumes no ids and no
 * blocks, the status word is set, and the call still returns STEP_OK. */
int kv_pool_fork_prefix(step_pool* pool, int n_traces, int prefix_len,
                        const void* k_prefix, const void* v_prefix,
                        int32_t* trace_ids_out, void* stream);

/* Store K/V of n_tokens new positions for each of the n listed traces (the cache write of
 * NextToken).  k_new, v_new: [n, n_tokens, num_layers, num_kv_heads, head_dim].
 * Traces are served in the order listed, pages in ascending order; a trace whose request
 * cannot be met (not live, table full, free list too short) is skipped whole and flagged. */
int append_kv(step_pool* pool, const int32_t* trace_ids, int n, int n_tokens,
              const void* k_new, const void* v_new, void* stream);

/* Decode attention of one layer for n traces:
 *   out[i][h] = sum_j softmax_j(q[i][h] . K_i[j] / sqrt(d)) V_i[j],  j in [0, seq_lens[i])
 * where position j of row i lives in block block_table[i][j / page_size], slot j % page_size.
 * q: [n, num_q_heads, head_dim] pool dtype; block_table: [n, max_pages_per_trace] int32;
 * seq_lens: [n] int32; out: [n, num_q_heads, head_dim] fp32.  seq_lens[i] = 0 gives zeros.
 * The pool's own block_table / seq_lens (kv_pool_device_views) may be passed directly. */
int decode_attention(step_pool* pool, int layer, const void* q,
                     const int32_t* block_table, const int32_t* seq_lens, int n,
                     void* out, void* stream);

/* decode_attention of n_layers consecutive layers, layer0 .. layer0 + n_layers - 1, over the same block table and
 * lengths: q [n_layers, n, num_q_heads, head_dim], out [n_layers, n, num_q_heads, head_dim] fp32.  The results are
 * those of n_layers decode_attention calls, bit for bit.  For callers that hold the queries of several layers at once
 * (NextToken is outside this library, so the loop of Algorithm 1 is given all layers' queries of an iteration: see
 * algorithm1_iteration).  Every launch after the first is made a programmatic dependent of the one before it, so the
 * SMs pass from layer to layer one by one and the KV stream does not drain at layer boundaries.  A later layer's launch
 * may read its queries, the tables and the cache while an earlier layer is still writing its output: q, block_table
 * and seq_lens must not overlap out.  Errors as decode_attention; layer0 + n_layers > num_layers is
 * STEP_ERR_INVALID_ARG with nothing launched. */
int decode_attention_layers(step_pool* pool, int layer0, int n_layers, const void* q,
                            const int32_t* block_table, const int32_t* seq_lens, int n,
                            void* out, void* stream);

/* decode_attention for a caller that runs the model layer by layer (the attention inside NextToken of Algorithm 1: the
 * query of layer l + 1 is computed from the output of layer l, so the queries of all layers are never at hand
 * together and decode_attention_layers does not apply).  Same arguments and the same result, bit for bit, as
 * decode_attention.  The launch is made a programmatic dependent of whatever kernel directly precedes it in the
 * stream - meant to be the caller's kernel that writes q: its CTAs are scheduled while that kernel is finishing, work
 * out their shares from seq_lens, start their first page copies through block_table, and wait for that kernel's
 * completion (and with it for everything earlier in the stream) only in front of their first read of q.
 * Requirement: the kernel directly before this call in the stream must not write seq_lens, block_table or this
 * layer's cache (do not issue it directly after append_kv or a prune), and it must itself be ordered after
 * everything before it, as any kernel launched the ordinary way is.  Shapes the tensor-core kernel does not cover
 * are launched the ordinary way. */
int decode_attention_dependent(step_pool* pool, int layer, const void* q,
                               const int32_t* block_table, const int32_t* seq_lens, int n,
                               void* out, void* stream);

/* decode_attention for traces that share their first pages (the prompt pages kv_pool_fork_prefix allocates once for
 * all traces of a problem: Algorithm 1, InitTraces):
 *   out[i] = attention of q[i] over the prefix_pages * page_size positions stored in blocks prefix_blocks[0 ..
 *            prefix_pages) followed by positions [prefix_pages * page_size, seq_lens[i]) of row i of block_table,
 * which is decode_attention's result whenever block_table[i][p] == prefix_blocks[p] for every listed row and
 * p < prefix_pages (prefix_blocks may point at any such row).  The shared pages are read once per 16 / G traces
 * instead of once per trace.  prefix_blocks: [prefix_pages] int32, device.  prefix_pages = 0 is decode_attention.
 * A row with seq_lens[i] = 0 gives zeros; a row shorter than the prefix gives zeros and sets the
 * STEP_ERR_INVALID_ARG bit of the device status word.  Only for pools the tensor-core kernel covers (bf16, head_dim
 * 128, page_size 16, G <= 16) and n <= min(max_traces, 2048); otherwise STEP_ERR_INVALID_ARG, nothing launched. */
int decode_attention_shared_prefix(step_pool* pool, int layer, const void* q,
                                   const int32_t* block_table, const int32_t* seq_lens, int n,
                                   const int32_t* prefix_blocks, int prefix_pages, void* out, void* stream);

/* decode_attention without any caller-provided or allocated scratch.  (The paper has no
 * counterpart: this entry point exists for hosts, not for the method.)
 *
 * Same result as decode_attention, for callers that cannot obtain device memory when they need
 * attention: a plug-in running inside another framework's pool-managed region, a serving loop that
 * bans allocator calls after start-up, an embedder that can only pass the buffers it was given.
 * The kernel's split partials live in a fixed array inside the library image (about 9.9 MB per GPU
 * that loads the library, held until the process exits); the call itself performs no cudaMalloc /
 * cudaFree and calls no allocating routine.
 *
 * Limits (fixed by that array): bf16 pools with head_dim 128 and page_size 16 only (else
 * STEP_ERR_INVALID_ARG); num_q_heads / num_kv_heads <= 8, n <= 2048 and n * num_kv_heads <= 16384, else
 * STEP_ERR_CAPACITY with nothing launched.  The launch uses at most 148 CTAs whatever kv_pool_set_attention_config says.
 * The pool's device must be the current device.
 *
 * First use on a device: the first call on each device looks up the array's device address
 * (cudaGetSymbolAddress) before it launches.  Make that first call outside any stream capture.
 *
 * Sharing: all calls on a device - from every pool and every stream - use the same array, and it
 * keeps whatever the previous call left.  Nothing in it needs clearing: each call writes every partial
 * before it reads it.  A call whose bounded device wait ran out (STEP_ERR_TIMEOUT in the pool's status word)
 * leaves some partials unwritten and its outputs are
 * undefined; the next call starts clean all the same.  Two calls that overlap in time on the GPU race on
 * the array: keep calls of this entry point ordered, e.g. on one stream. */
int decode_attention_static(step_pool* pool, int layer, const void* q,
                            const int32_t* block_table, const int32_t* seq_lens, int n,
                            void* out, void* stream);

/* Step scorer at step boundaries (Sec. 3.1) and running-mean update (Sec. 3.3):
 * for every row i with boundary_mask[i] != 0:
 *   y = sigmoid(w2 . ReLU(W1 hidden[i] + b1) + b2);  step_scores_out[i] = y;
 *   trace t = row_trace ? row_trace[i] : i:  sum_t += y, cnt_t += 1 (rows in ascending order).
 * Rows with mask 0 get NaN in step_scores_out.  Then score_t = sum_t / cnt_t is refreshed
 * for every trace (unscored_score while cnt_t = 0).
 * hidden: [M, D] in weights dtype; boundary_mask: [M] u8; row_trace: [M] int32 or NULL. */
int score_steps(step_pool* pool, const void* hidden, const uint8_t* boundary_mask,
                const int32_t* row_trace, int M, const scorer_weights* weights,
                float* step_scores_out, void* stream);

/* Step-end detection (Sec. 3.1 "Step Representation" and its footnote; Algorithm 1: `if "\n\n" in x`):
 * a sampled token ends a reasoning step if its text contains two consecutive newline characters.
 * step_end_table_from_vocab fills table_out[v] (HOST, vocab bytes) with 1 for such vocabulary entries and 0
 * for the others; token_text[v] (HOST) is the entry's text, text_len[v] its length in bytes, or text_len =
 * NULL for NUL-terminated strings; a NULL entry counts as empty.  Needs no GPU. */
int step_end_table_from_vocab(const char* const* token_text, const int32_t* text_len, int vocab,
                              uint8_t* table_out);
/* boundary_mask_out[i] = step_end_table[token_ids[i]] for M sampled tokens (device pointers; the table is a
 * device copy of what step_end_table_from_vocab made).  An id outside [0, vocab) ends no step and sets the
 * STEP_ERR_INVALID_ARG bit of the device status word. */
int detect_step_ends(step_pool* pool, const int32_t* token_ids, int M, const uint8_t* step_end_table,
                     int vocab, uint8_t* boundary_mask_out, void* stream);
/* score_steps with the step-end flags taken from the sampled tokens instead of a mask: row i is scored iff
 * step_end_table[token_ids[i]] != 0 (one pass less over the rows than detect_step_ends + score_steps).
 * The flags are also written to boundary_mask_out (device, [M]) unless it is NULL.  Everything else as
 * score_steps. */
int score_steps_tokens(step_pool* pool, const void* hidden, const int32_t* token_ids,
                       const uint8_t* step_end_table, int vocab, const int32_t* row_trace, int M,
                       const scorer_weights* weights, float* step_scores_out, uint8_t* boundary_mask_out,
                       void* stream);

/* Memory trigger and eviction (Sec. 3.2, Algorithm 1):
 *   used = total - free_count; need = #{live t: S_t % page_size == 0};
 *   saturated <=> used + need > floor((double)threshold * total).
 * If saturated, rank live traces by (score descending, id ascending, NaN last), keep the
 * first n_keep and evict the rest: keep_frac < 0 -> n_keep = n_live - 1 (the paper's rule:
 * evict the argmin only); keep_frac in (0,1] -> n_keep = max(1, ceil(keep_frac*n_live - 1e-6)).
 * Evicted traces (ascending id, pages ascending) drop one reference per block; blocks that
 * reach zero are pushed on the free list in that order; the trace's table, length, live flag
 * and score state are cleared.
 * scores: [max_traces] fp32 or NULL for the pool's running means.
 * pruned_ids_out: [max_traces] int32 (ascending ids, rest untouched); n_pruned_out: 1 int32. */
int prune_if_saturated(step_pool* pool, const float* scores, float threshold, float keep_frac,
                       int32_t* pruned_ids_out, int32_t* n_pruned_out, void* stream);

/* A trace that finished on its own gives its KV back (same reclaim as an eviction; the traces are reclaimed in the
 * order listed, each one's pages in ascending order).  trace_ids: [n] device, distinct; invalid or dead ids are flagged
 * (STEP_ERR_BAD_TRACE) and skipped. */
int kv_pool_release_traces(step_pool* pool, const int32_t* trace_ids, int n, void* stream);

/* ---- Algorithm 1 as a loop over device-resident state ----
 * The model's forward pass is outside this library, so NextToken(t) -> (x, h) is represented by what goes in
 * and comes out of it: per iteration the caller supplies, for every trace, the sampled token x, the new K/V
 * rows, the queries of the layers whose attention is to be run and the last-layer hidden state h.  In all of
 * these ROW i IS TRACE i (the traces are ids 0 .. n_traces-1 of the pool, forked before the first iteration),
 * and rows of traces that are no longer live are passed over on the device, so the host never needs to know
 * who is live.  One memory-trigger check is made per iteration, after the iteration's cache writes. */

/* A trace that completed: its current score_t and its answer id (>= 0) are kept for the vote, then its KV is
 * released as for an eviction.  trace_ids, answers: [n] device; a trace whose answer is negative, or all of
 * them if answers is NULL, completes without taking part in the vote.  Ids must be distinct; invalid or dead
 * ids are flagged (STEP_ERR_BAD_TRACE) and skipped. */
int kv_pool_finish_traces(step_pool* pool, const int32_t* trace_ids, const int32_t* answers, int n, void* stream);

/* WeightedVote(T, {score_t}) (Algorithm 1, last line; Sec. 3.3): over the completed traces, the answer with the
 * largest sum of final trace scores; equal sums go to the smaller answer id.  Evicted traces do not vote.
 * answer_out [1] int32 (-1 if no trace completed), weight_out [1] float (may be NULL), n_finished_out [1] int32
 * (may be NULL): device pointers. */
int weighted_vote(step_pool* pool, int32_t* answer_out, float* weight_out, int32_t* n_finished_out, void* stream);

typedef struct {
  int n_traces;                       /* rows of every per-trace input below                                      */
  const int32_t* token_ids;           /* [n] the token each trace sampled                                         */
  int eos_token;                      /* a live trace that sampled it completes in this iteration                 */
  const uint8_t* step_end_table;      /* [vocab] see step_end_table_from_vocab                                    */
  int vocab;
  const int32_t* answers;             /* [n] answer id trace i reports if it completes now (may be NULL)          */
  int n_layers_attention;             /* decode_attention is run for layers 0 .. this-1 (0: none)                 */
  const void* q;                      /* [n_layers_attention, n, num_q_heads, head_dim] pool dtype                */
  const void* k_new; const void* v_new; /* [n, 1, num_layers, num_kv_heads, head_dim] pool dtype                  */
  const void* hidden;                 /* [n, D] scorer dtype                                                      */
  void* attn_out;                     /* [n_layers_attention, n, num_q_heads, head_dim] fp32; must not overlap q   */
  float* step_scores_out;             /* [n] as score_steps                                                       */
  uint8_t* boundary_mask_out;         /* [n] step-end flags of the live rows (may be NULL)                        */
  float* trace_scores_out;            /* [n] score_t of every trace right after this iteration's scoring, i.e. what
                                         completion records and eviction ranks by (may be NULL)                    */
  const scorer_weights* scorer;
  float threshold, keep_frac;         /* as prune_if_saturated; keep_frac < 0 with threshold 1 is the paper's rule */
  int max_evictions;                  /* the trigger is tested, and the rule applied, up to this many times in a row
                                         (0 or 1: once); each further test sees the pool the last eviction left      */
  int32_t* pruned_ids_out;            /* [max_traces], may be NULL; holds the last test's evictions               */
  int32_t* n_pruned_out;              /* [1], may be NULL                                                         */
} step_iteration;

/* One iteration of the while loop of Algorithm 1 for all traces, chained on the stream with no host round trip:
 * append_kv of the live traces' new token -> decode_attention per layer -> step-end detection + score_steps ->
 * completion (kv_pool_finish_traces) of the live traces whose token is eos_token -> prune_if_saturated on the
 * pool's running means (max_evictions times: with the paper's one-eviction rule a single eviction may not free
 * enough blocks for the next step when many traces reach a page boundary together).  All pointers are device pointers except `it` and it->scorer (host structs). */
int algorithm1_iteration(step_pool* pool, const step_iteration* it, void* stream);

typedef struct {
  int n_traces, max_iterations;
  const int32_t* token_ids;           /* [max_iterations, n] sampled tokens, iteration-major                      */
  int eos_token;
  const uint8_t* step_end_table; int vocab;
  const int32_t* answers;             /* [n]                                                                      */
  int ring;                           /* the per-iteration tensors below hold `ring` slots; iteration i uses i % ring */
  int n_layers_attention;
  const void* q;                      /* [ring, n_layers_attention, n, num_q_heads, head_dim]                     */
  const void* k_new; const void* v_new; /* [ring, n, 1, num_layers, num_kv_heads, head_dim]                       */
  const void* hidden;                 /* [ring, n, D]                                                             */
  void* attn_out;                     /* [n_layers_attention, n, num_q_heads, head_dim] fp32, overwritten each iteration */
  float* step_scores_out;             /* [n]                                                                      */
  const scorer_weights* scorer;
  float threshold, keep_frac;
  int max_evictions;                  /* as in step_iteration                                                     */
  int check_every;                    /* the host asks for the number of live traces every this many iterations   */
  float* score_history;               /* [max_iterations, n] score_t after each iteration's scoring, or NULL      */
  int use_graphs;                     /* != 0: the launches of one iteration are recorded once per ring slot as a CUDA
                                         graph and replayed (one graph launch per iteration instead of a dozen kernel
                                         launches; worth it when an iteration is short).  Needs a stream that can be
                                         captured (not the default stream, not already capturing), else ignored.  The
                                         graphs are private to the call and destroyed before it returns (whatever memory
                                         the CUDA runtime takes for them is the one exception to "allocates nothing"). */
} step_run_args;

typedef struct {
  int iterations;                     /* iterations executed                                                      */
  int answer; float answer_weight;    /* the vote's result (-1 if no trace completed)                             */
  int n_finished, n_evicted, live_left;
} step_run_result;

/* The whole loop: iterations until no trace is live (checked every check_every iterations; iterations with no
 * live trace do nothing) or max_iterations, then the weighted vote.  res is a HOST struct; synchronises. */
int algorithm1_run(step_pool* pool, const step_run_args* args, step_run_result* res, void* stream);

/* ---- training the step scorer (Sec. 3.1 "Training Objective"; appendix "Training Parameters") ----
 * One optimisation step on a batch of B (hidden state, label) pairs:
 *   L = -(1/B) sum_b ( pos_weight * y_b * log yhat_b + (1 - y_b) * log(1 - yhat_b) ),  yhat = f(h),
 * pos_weight = alpha = K- / K+ (negative over positive samples of the training set); then Adam with the weight decay
 * added to the gradient (g += weight_decay * p) and bias-corrected moments.  The paper's values: B = 128,
 * lr = 1e-4, weight_decay = 1e-5; beta1 = 0.9, beta2 = 0.999, eps = 1e-8 are the optimiser's usual defaults (the
 * paper does not list them).  `step` is the 1-based number of this update (for the bias correction). */
typedef struct {
  float lr, beta1, beta2, eps, weight_decay, pos_weight;
  int step;
} scorer_train_hyper;

/* Bytes of device workspace scorer_train_step needs (pre-activations and gradients); host-only, 0 on bad arguments. */
size_t scorer_train_workspace_bytes(int B, int D, int m);

/* hidden: [B, D] in hidden_dtype (STEP_BF16 | STEP_FP32); labels: [B] fp32 in {0, 1}; W1 [m, D], b1 [m], w2 [m],
 * b2 [1]: fp32 parameters, updated in place; adam_m, adam_v: [m*D + 2m + 1] fp32 moments in the order W1, b1, w2, b2
 * (zero before the first step), updated in place; workspace: 256-byte aligned, at least
 * scorer_train_workspace_bytes(B, D, m); loss_out: [1] fp32, the loss BEFORE the update.  All device pointers except
 * `h`.  Asynchronous on the stream; deterministic. */
int scorer_train_step(const void* hidden, int hidden_dtype, const float* labels, int B, float* W1, float* b1,
                      float* w2, float* b2, int D, int m, float* adam_m, float* adam_v,
                      const scorer_train_hyper* h, void* workspace, size_t workspace_bytes, float* loss_out,
                      void* stream);

/* ---- accessors for tests and benchmarks ---- */
/* Vote state: final_score [max_traces] f32, answer [max_traces] i32, finished [max_traces] u8 (device). */
int kv_pool_vote_views(step_pool* pool, float** final_score, int32_t** answer, uint8_t** finished);
/* Host ints; synchronises the stream. */
int kv_pool_stats(step_pool* pool, int* used, int* free_, int* total, int* live_traces, void* stream);
/* Device pointers into meta_storage (any may be NULL):
 * block_table [max_traces, max_pages_per_trace] i32 (-1 = unmapped), seq_lens [max_traces] i32,
 * trace_scores [max_traces] f32, free_list [num_blocks] i32, free_count [1] i32,
 * refcount [num_blocks] i32, live [max_traces] u8. */
int kv_pool_device_views(step_pool* pool, int32_t** block_table, int32_t** seq_lens,
                         float** trace_scores, int32_t** free_list, int32_t** free_count,
                         int32_t** refcount, uint8_t** live);
/* Further views: score_sum [max_traces] f32, score_cnt [max_traces] i32. */
int kv_pool_score_views(step_pool* pool, float** score_sum, int32_t** score_cnt);
/* Reads and clears the sticky device status word (synchronises).  Returns the lowest error
 * code that was set (STEP_OK if none); *mask_out (host, may be NULL) gets the full bit mask. */
int kv_pool_last_error(step_pool* pool, unsigned* mask_out, void* stream);
/* Logical K and V rows [0, seq_len) of one trace, layer and KV head, gathered through the
 * given block-table row into k_out, v_out: [seq_len, head_dim] pool dtype. */
int kv_pool_read_kv(step_pool* pool, int layer, int kv_head, const int32_t* block_row,
                    int seq_len, void* k_out, void* v_out, void* stream);
/* Tuning knobs of decode_attention (0 keeps the current value): CTAs per launch, and whether
 * the tensor-core bf16 path may be used (1) or the scalar kernel is forced (-1). */
int kv_pool_set_attention_config(step_pool* pool, int grid_ctas, int fast_path);
/* How decode_attention's tensor-core launch spreads the KV pages over the SMs.  Of every (trace, KV head)
 * sequence the last dynamic_sixteenths / 16 of its pages (0 .. 12; default 4) are cut into chunks of at least
 * min_chunk_pages pages (0 keeps the current value; default 16) that warps fetch from a device counter when they
 * have finished their equal share of the other pages; 0 sixteenths = equal shares only.  The outputs are the same
 * bits whichever warp processes which chunk.  decode_attention_static and the shared pages' pass of
 * decode_attention_shared_prefix always use equal shares.  STEP_ERR_INVALID_ARG outside the ranges. */
int kv_pool_set_attention_balance(step_pool* pool, int dynamic_sixteenths, int min_chunk_pages);
/* How long the tensor-core kernel of decode_attention (all its entry points) waits for a page copy before it gives
 * up: the warp then sets the STEP_ERR_TIMEOUT bit of the status word, waits (with
 * the full limit) for the copies it still has in flight, and leaves; outputs of such a launch are undefined (the
 * launches after it are unaffected: no state of the kernel outlives a launch).  Default 2,000,000,000 ns.
 * 0 = no waiting at all: a page that has not landed by the time it is first looked at counts as timed out - for testing this path, which no healthy device otherwise reaches. */
int kv_pool_set_wait_limit_ns(step_pool* pool, unsigned long long ns);
/* Which first-layer kernel score_steps uses for bf16 scorers whose shape the tensor-core kernel covers
 * (D a multiple of 64, m a multiple of 64 and <= 1024, 16-byte aligned W1 and hidden): mode 0 (default)
 * sends a launch to the tensor cores when it has at least tc_min_rows boundary rows (the count is taken
 * on the device) and to the CUDA-core kernel otherwise; mode 1 always uses the tensor cores, mode -1 never.
 * tc_min_rows = 0 keeps the current value (default 1: measured faster than the CUDA-core kernel from the
 * first row on; fp32 scorers and other shapes always take the CUDA-core kernel). */
int kv_pool_set_scorer_config(step_pool* pool, int mode, int tc_min_rows);
/* What the most recent score_steps launch did (of its last chunk, if M exceeded max_score_rows):
 * *n_rows = boundary rows it found, *tc_units = hidden units per CTA of the tensor-core kernel, or 0 if
 * the CUDA-core kernel scored the rows.  Host ints, either may be NULL; synchronises the stream. */
int kv_pool_score_launch_info(step_pool* pool, int* n_rows, int* tc_units, void* stream);
/* Measurement aid (the paper has no counterpart): the rate at which this device's HBM feeds the copy structure of
 * decode_attention when no arithmetic is attached - one CTA per SM, eight warps, each streaming an equal
 * contiguous share of buf through a ring of three 8 KiB bulk copies into shared memory and dropping the data.
 * n_launches launches over the same buffer; chained != 0 makes every launch after the first a programmatic
 * dependent of the one before it, as decode_attention_layers does with its layers.  buf: device, 16-byte aligned,
 * bytes >= 8192 (a multiple of 8192 is read); err_flag: [1] int32 device, set to 1 if a bounded wait ran out.
 * Asynchronous on the stream; time it with events around the call. */
int step_read_stream_probe(const void* buf, size_t bytes, int n_launches, int chained, int32_t* err_flag,
                           void* stream);
/* Library build tag, for logs. */
const char* step_version(void);

#ifdef __cplusplus
}
#endif
#endif /* STEP_H_ */
