// Internal definitions shared by the translation units of libstep (never installed).
//
// Physical KV layout (private to the library):
//   kv[layer][block][kv_head][K|V][slot][dim]          slot in [0, page_size)
// so that one page of one KV head (K rows then V rows) is a single contiguous run of
// 2 * page_size * head_dim elements - 8 KiB for bf16, page 16, d 128 - which one bulk async
// copy brings into shared memory.  For bf16 pools whose head_dim is a multiple of 64 the 16-byte
// chunks of every row are stored XOR-swizzled with the slot number (chunk' = chunk ^ (slot & 7)
// on the low three bits): the page then lands in shared memory already in the bank-conflict-free
// arrangement that ldmatrix wants, without a tensor map.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/step.h"

namespace stepk {

constexpr int kMaxPartitions = 4096;   // upper bound on independent KV-stream partitions of one launch
constexpr int kPrefixPartitions = 1184; // partitions of the shared-prefix pass of decode_attention_shared_prefix (148 SMs x 8 warps)
constexpr int kMaxDynChunks = 8192;    // upper bound on the chunks of one attention launch handed out at run time (partial slots beyond those of the shares)
constexpr int kMaxTracesFast = 2048;   // traces per decode_attention call on the tensor-core path
constexpr int kScoreSplits = 16;       // slices of the scorer's hidden units; score_z holds this many floats per row
constexpr int kSmallRows = 256;       // candidate rows up to which score_steps is one launch (a decode step's shape)
constexpr int kSmallCtas = 148;       // CTAs of that launch at most; score_zs holds this many partial sums per listed row
constexpr int kScoreFoldRows = 512;    // listed rows one CTA of the scorer's finishing kernel folds into per-trace partials

// C_SCORE_TC: 0 = the launch's boundary rows go through the CUDA-core MLP kernel; otherwise the
// number of hidden units (UMMA N) each CTA of the tensor-core kernel covers.  C_SCORE_SLICES:
// how many partial sums per row the MLP kernels leave in score_z.
enum Counter { C_FREE_COUNT = 0, C_STATUS = 1, C_FORK_OK = 2, C_SCORE_NB = 3, C_PRUNE_N = 4,
               C_SCORE_TC = 5, C_SCORE_SLICES = 6, C_SCORE_TICKET = 7,
               // Algorithm 1 driver: live / finishing traces of the current iteration, running totals
               C_IT_NLIVE = 8, C_IT_NFIN = 9, C_N_FINISHED = 10, C_N_EVICTED = 11, C_IT_NPRUNED = 12,
               C_SCORE_TILE = 13,   // rows per work item of the tensor-core scorer kernel (128 or 256)
               C_NEXT_TRACE = 14,   // id the next successful fork starts at
               C_FORK_FIRST = 15,   // first id of the most recent fork (valid when C_FORK_OK is set)
               C_APPEND_TICKET = 16, // CTAs of the current append launch that have read the pool's state; zero between launches
               C_NUM = 64 };

struct MetaLayout {
  size_t block_table, seq_lens, live, score_sum, score_cnt, trace_scores;
  size_t refcount, free_list, claim, counters;
  size_t append_base, prune_rank, prune_list, prune_off;
  size_t score_idx, score_z, score_part, score_zs;
  size_t attn_ml, attn_o, attn_sched;
  size_t pre_ws_ml, pre_ws_o, pre_ml, pre_o;   // shared-prefix attention (zero-sized for pools the tensor-core kernel does not cover)
  size_t final_score, answer, finished, it_ids, it_fin, it_pruned, it_tokens, it_scores;
  size_t total;
};

struct DevViews {
  int32_t* block_table; int32_t* seq_lens; uint8_t* live;
  float* score_sum; int32_t* score_cnt; float* trace_scores;
  int32_t* refcount; int32_t* free_list; int32_t* claim; int32_t* counters;
  int32_t* append_base; int32_t* prune_rank; int32_t* prune_list; int32_t* prune_off;
  int32_t* score_idx; float* score_z; float2* score_part; float* score_zs;
  float* attn_ml; float* attn_o; int32_t* attn_sched;
  float* pre_ws_ml; float* pre_ws_o; float* pre_ml; float* pre_o;   // null when zero-sized
  float* final_score; int32_t* answer; uint8_t* finished;     // traces that completed: what the vote needs
  int32_t* it_ids; int32_t* it_fin; int32_t* it_pruned;       // per-iteration lists of the Algorithm 1 driver
  int32_t* it_tokens; float* it_scores;                       // staging rows of algorithm1_run's recorded iterations
};

}  // namespace stepk

struct step_pool {
  kv_pool_config cfg;
  int G;
  int elem_bytes;
  int swizzle;        // 1: rows stored with XOR-swizzled 16-byte chunks
  int max_score_rows;
  int num_sms;
  int attn_grid;      // CTAs of the tensor-core attention launch
  int attn_dyn16;     // sixteenths of every sequence's pages handed out at run time (0: equal shares only)
  int attn_dyn_chunk; // smallest chunk handed out, in pages
  int fast_path;      // 1 allowed, -1 forced off
  unsigned long long wait_limit_ns;   // limit of decode_attention's wait for a page copy (kv_pool_set_wait_limit_ns)
  int scorer_mode;    // 0: tensor-core MLP for launches with >= scorer_tc_min_rows boundary rows; 1: always; -1: never
  int scorer_tc_min_rows;
  // the tensor map of the last W1 the tensor-core scorer was given (encoding it costs a few host microseconds)
  alignas(64) unsigned char tmap_bytes[128];
  const void* tmap_w1; int tmap_D, tmap_m;
  // ... and of the last array of candidate rows it was given
  alignas(64) unsigned char tmap_h_bytes[128];
  const void* tmap_h_ptr; int tmap_h_D, tmap_h_M;
  bool tc_smem_set;   // the scorer kernel's dynamic shared memory limit has been raised on this pool's device
  int device;
  stepk::MetaLayout lay;
  stepk::DevViews v;
};

namespace stepk {

// Geometry handed to kernels by value.
struct Geo {
  int L, Hq, Hkv, d, P, num_blocks, max_traces, max_pages, G, swizzle;
};

inline Geo geo_of(const step_pool* p) {
  Geo g;
  g.L = p->cfg.num_layers; g.Hq = p->cfg.num_q_heads; g.Hkv = p->cfg.num_kv_heads;
  g.d = p->cfg.head_dim; g.P = p->cfg.page_size; g.num_blocks = p->cfg.num_blocks;
  g.max_traces = p->cfg.max_traces; g.max_pages = p->cfg.max_pages_per_trace;
  g.G = p->G; g.swizzle = p->swizzle;
  return g;
}

// Element offset of (layer, block, head, kv, slot, dim) in kv_storage.
__host__ __device__ inline size_t kv_page_base(const Geo& g, int layer, int block, int head, int kv) {
  return ((((size_t)layer * g.num_blocks + block) * g.Hkv + head) * 2 + kv) * ((size_t)g.P * g.d);
}
// Offset inside a page of (slot, dim); `cpe` = elements per 16-byte chunk.
__host__ __device__ inline int kv_in_page(const Geo& g, int slot, int dim, int cpe) {
  int chunk = dim / cpe, within = dim % cpe;
  if (g.swizzle) chunk = (chunk & ~7) | ((chunk ^ slot) & 7);
  return slot * g.d + chunk * cpe + within;
}

__device__ inline void flag_error(int32_t* counters, int code) {
  atomicOr(reinterpret_cast<unsigned*>(counters + C_STATUS), 1u << code);
}

#define STEP_CUDA_OK(expr)                                  \
  do {                                                      \
    cudaError_t e__ = (expr);                               \
    if (e__ != cudaSuccess) return STEP_ERR_CUDA;           \
  } while (0)

inline int launch_ok() { return cudaGetLastError() == cudaSuccess ? STEP_OK : STEP_ERR_CUDA; }

// Programmatic dependent launch.  A kernel launched with launch_dependent() may be scheduled while the kernel before
// it in the stream is still running (as soon as every CTA of that kernel has called dependents_may_launch() or has
// exited); it must call wait_for_primary() before it touches anything the earlier kernel writes - the call returns
// once that kernel has completed and its writes are visible.  Both calls do nothing in a kernel launched the plain way.
__device__ inline void dependents_may_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ inline void wait_for_primary() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... Params, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                    Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);
}

// ---- pieces the Algorithm 1 driver (algorithm1.cu) chains together
// append_kv with extras: *n_dev (device, may be null) caps the number of listed traces on the device; src_by_id makes
// trace t read row t of k_new / v_new instead of row (position in the list); trace_ids == nullptr (with src_by_id, one
// token) appends to every live trace among 0 .. n-1 - the list is made on the device (v.it_ids, C_IT_NLIVE) together
// with the list of those whose sampled token live_tokens[t] equals eos (v.it_fin, C_IT_NFIN; live_tokens may be null).
int append_kv_impl(step_pool* pool, const int32_t* trace_ids, int n, int n_tokens, const void* k_new,
                   const void* v_new, const int32_t* n_dev, int src_by_id, cudaStream_t s,
                   const int32_t* live_tokens, int eos);

// Where score_steps takes a row's step-end flag from: mask[i], or table[tokens[i]] (a token ends a step if its
// text contains two newlines in a row; the table records that per vocabulary entry).  live (may be null)
// additionally requires live[i] != 0 - for callers whose row i is trace i.
struct FlagSource {
  const uint8_t* mask;       // [M], or nullptr
  const int32_t* tokens;     // [M], or nullptr
  const uint8_t* table;      // [vocab]
  int vocab;
  uint8_t* mask_out;         // [M], or nullptr
  const uint8_t* live;       // [M], or nullptr
};
// trace_scores_out (may be null): its first n_out entries get the trace scores as they stand after this call.
int score_steps_impl(step_pool* pool, const void* hidden, FlagSource src, const int32_t* row_trace, int M,
                     const scorer_weights* w, float* step_scores_out, float* trace_scores_out, int n_out, void* stream);

// ---- tensor-core scorer (scorer_tc.cu)
// True if the tcgen05 kernel covers this scorer shape and these pointers.
bool score_tc_supported(const scorer_weights* w, const void* hidden);
// Launches the persistent kernel for a chunk of Mc candidate rows (at most one CTA per SM); it reads
// C_SCORE_NB / C_SCORE_TC on the device and returns at once when C_SCORE_TC is 0.
int score_tc_launch(step_pool* pool, const void* hidden, int Mc, const scorer_weights* w, cudaStream_t s);

}  // namespace stepk
