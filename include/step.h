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
 * Trace ids are consecutive, continuing from earlier forks; they are written to
 * trace_ids_out (HOST, n_traces ints, may be NULL).  Errors: CAPACITY, NO_BLOCKS (checked on
 * the device: the fork is then a no-op and the status word is set). */
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
 * STEP_ERR_INVALID_ARG); num_q_heads / num_kv_heads <= 8 and n <= 2048, else STEP_ERR_CAPACITY with
 * nothing launched.  The launch uses at most 148 CTAs whatever kv_pool_set_attention_config says.
 * The pool's device must be the current device.
 *
 * First use on a device: the first call on each device looks up the array's device address
 * (cudaGetSymbolAddress) before it launches.  Make that first call outside any stream capture.
 *
 * Sharing: all calls on a device - from every pool and every stream - use the same array, and it
 * keeps whatever the previous call left.  Nothing in it has to start at zero (each call writes every
 * partial before it reads it), but two calls that overlap in time on the GPU race on it: keep
 * calls of this entry point ordered, e.g. on one stream. */
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

/* A trace that finished on its own gives its KV back (same reclaim as an eviction). */
int kv_pool_release_traces(step_pool* pool, const int32_t* trace_ids, int n, void* stream);

/* ---- accessors for tests and benchmarks ---- */
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
/* Library build tag, for logs. */
const char* step_version(void);

#ifdef __cplusplus
}
#endif
#endif /* STEP_H_ */
