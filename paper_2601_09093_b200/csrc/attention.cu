// decode_attention: grouped-query decode attention over the paged KV pool.
//
//   out[i][h] = sum_j softmax_j(q[i][h] . K_i[j] / sqrt(d)) V_i[j]      (the attention inside
// NextToken of Algorithm 1; decoding is where Table 3 / Fig. 2c put the non-waiting time).
//
// Two implementations:
//  * attn_scalar_kernel - any dtype / head_dim / page size, one CTA per (trace, query head).
//    Used for fp32 pools and for shapes the tensor-core kernel does not cover.
//  * attn_mma_kernel + attn_merge_kernel - bf16, head_dim 128, page 16, G <= 16.  HBM-bound design:
//      - of the launch's KV stream (for every trace, for every KV head, its pages in order) the first pages of
//        every sequence are cut into gridDim * kWarps equal contiguous shares, one per warp, so every SM gets
//        the same number of pages whatever the mix of trace lengths; the last pages of every sequence are cut
//        into chunks that a warp fetches from a device counter when its share is done (SMs do not all stream
//        at the same rate);
//      - a page of one KV head (K 4 KiB + V 4 KiB, contiguous, pre-swizzled in HBM) is brought
//        into shared memory by ONE bulk async copy that signals an mbarrier; every warp keeps
//        its own ring of kStages pages in flight and never synchronises with another warp;
//      - all G query heads of the group are served from that single read of K and V:
//        S = Q K^T and O += P V run on mma.sync m16n8k16 (bf16 in, fp32 accumulate) with the
//        heads on the M axis, ldmatrix (plain for K, transposed for V) feeding the B operand;
//      - running (max, sum) softmax state per head in fp32, exp2 with the scale folded in;
//      - a warp that has read a whole (trace, head) sequence writes the output directly; otherwise it leaves an
//        (m, l, o) partial in the piece's slot, and attn_merge_kernel - a programmatic dependent of the
//        streaming kernel, resident beside it - combines every sequence's partials in a fixed order;
//      - a launch that directly follows another attention launch (the next layer of a decode step:
//        decode_attention_layers) is made a programmatic dependent too: it starts on every SM the earlier
//        launch has left, reads and accumulates at once, and waits for that launch's completion only in
//        front of its own first write, so the stream of KV reads does not stop at layer boundaries.
#include "step_internal.cuh"
#include "async_copy.cuh"

#include <math.h>

using namespace stepk;

namespace {

// =============================================================== scalar kernel
template <typename T> __device__ inline float ld_f32(const T* p);
template <> __device__ inline float ld_f32<float>(const float* p) { return *p; }
template <> __device__ inline float ld_f32<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }

constexpr int kScalarWarps = 4;
constexpr int kMaxDimsPerLane = 16;   // head_dim <= 512

template <typename T>
__global__ void __launch_bounds__(kScalarWarps * 32)
attn_scalar_kernel(Geo g, const T* __restrict__ kv, int layer, const T* __restrict__ q,
                   const int32_t* __restrict__ block_table, const int32_t* __restrict__ seq_lens,
                   float* __restrict__ out, int32_t* counters) {
  extern __shared__ float smf[];
  float* s_q = smf;                                  // [d]
  float* s_o = smf + g.d;                            // [warps][d]
  __shared__ float s_m[kScalarWarps], s_l[kScalarWarps];
  const int h = blockIdx.x, t = blockIdx.y, kvh = h / g.G;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cpe = 16 / (int)sizeof(T);
  int S = seq_lens[t];
  if (S < 0) S = 0;
  if ((long long)S > (long long)g.max_pages * g.P) { S = g.max_pages * g.P; if (threadIdx.x == 0) flag_error(counters, STEP_ERR_CAPACITY); }
  for (int k = threadIdx.x; k < g.d; k += blockDim.x) s_q[k] = ld_f32(q + ((size_t)t * g.Hq + h) * g.d + k);
  __syncthreads();
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)g.d);
  float m = -INFINITY, l = 0.f;
  float acc[kMaxDimsPerLane];
#pragma unroll
  for (int i = 0; i < kMaxDimsPerLane; ++i) acc[i] = 0.f;
  for (int j = warp; j < S; j += kScalarWarps) {
    const int page = j / g.P, slot = j % g.P;
    int b = block_table[(size_t)t * g.max_pages + page];
    if (b < 0 || b >= g.num_blocks) { if (lane == 0) flag_error(counters, STEP_ERR_BAD_BLOCK); b = 0; }
    const T* kp = kv + kv_page_base(g, layer, b, kvh, 0);
    const T* vp = kp + (size_t)g.P * g.d;
    float dot = 0.f;
#pragma unroll
    for (int i = 0; i < kMaxDimsPerLane; ++i) {
      const int k = lane + 32 * i;
      if (k < g.d) dot += s_q[k] * ld_f32(kp + kv_in_page(g, slot, k, cpe));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
    const float s = dot * scale_log2;
    const float m_new = fmaxf(m, s);
    const float corr = exp2f(m - m_new), p = exp2f(s - m_new);
    l = l * corr + p;
#pragma unroll
    for (int i = 0; i < kMaxDimsPerLane; ++i) {
      const int k = lane + 32 * i;
      if (k < g.d) acc[i] = acc[i] * corr + p * ld_f32(vp + kv_in_page(g, slot, k, cpe));
    }
    m = m_new;
  }
  if (lane == 0) { s_m[warp] = m; s_l[warp] = l; }
#pragma unroll
  for (int i = 0; i < kMaxDimsPerLane; ++i) {
    const int k = lane + 32 * i;
    if (k < g.d) s_o[warp * g.d + k] = acc[i];
  }
  __syncthreads();
  float M = -INFINITY;
  for (int w = 0; w < kScalarWarps; ++w) M = fmaxf(M, s_m[w]);
  for (int k = threadIdx.x; k < g.d; k += blockDim.x) {
    float num = 0.f, den = 0.f;
    for (int w = 0; w < kScalarWarps; ++w) {
      if (s_m[w] == -INFINITY) continue;           // that warp saw no position
      const float wgt = exp2f(s_m[w] - M);
      num += wgt * s_o[w * g.d + k];
      den += wgt * s_l[w];
    }
    out[((size_t)t * g.Hq + h) * g.d + k] = den > 0.f ? num / den : 0.f;
  }
}

// =============================================================== tensor-core kernel
constexpr int kP = 16, kD = 128;
constexpr int kPageBytes = 2 * kP * kD * 2;        // K rows then V rows of one KV head: 8 KiB
constexpr int kVOffset = kP * kD * 2;              // 4 KiB

struct AttnArgs {
  const __nv_bfloat16* kv_layer;   // kv_storage + layer offset
  const __nv_bfloat16* q;
  const int32_t* block_table;
  const int32_t* seq_lens;
  float* out;
  float* ws_ml;                    // [partition][2][G][2]
  float* ws_o;                     // [partition][2][G][kD]
  int32_t* counters;
  int n, Hq, Hkv, G, max_pages, num_blocks;
  float scale_log2;
  // shared-prefix passes only
  const int32_t* prefix_blocks;    // [pp] block of every shared page
  float* pre_ml;                   // [n][Hq][2]  (max, sum) of the attention over the shared pages, un-normalised
  float* pre_o;                    // [n][Hq][kD] its weighted value sum
  int pp;                          // shared pages
  int tpb, n_bundles;              // prefix pass: traces per 16-row bundle of query rows, number of bundles
  int q_from_primary;              // 1: the launch before this one in the stream writes q (see decode_attention_dependent)
  int32_t* sched;                  // [1] hand-out counter of the chunks, zero between launches; null: equal shares only
  int dyn16, dyn_chunk;            // sixteenths of every sequence handed out as chunks; smallest chunk (pages)
  int n_static;                    // equal shares of the static stream: warps of the attention launch
  int merge_ctas;                  // CTAs of the launch that combines the pieces, at most (one per SM)
  unsigned long long wait_ns;      // limit of the wait for one page copy
};

// kMode of attn_mma_kernel: the plain kernel; the pass over the shared pages, whose 16 query rows are the G heads of
// tpb = 16 / G traces, so that one read of a shared page serves tpb traces, and which leaves (m, l, o) per
// (trace, head) in pre_ml / pre_o; and the pass over every trace's own pages, which folds that result in at the end.
constexpr int kPlain = 0, kPrefixPass = 1, kSuffixPass = 2;

__device__ inline void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ inline void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ inline void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ inline uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Largest t with Hkv * cum[t] <= pos (cum is an exclusive prefix sum over the launch's sequences).
__device__ inline int seek_trace(const int* cum, int n, int Hkv, long long pos) {
  int lo = 0, hi = n - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if ((long long)Hkv * cum[mid] <= pos) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// Position in the launch's KV stream -> (trace, kv head, page).  The stream lists, for every
// trace in order, for every KV head in order, that trace's pages in order.
struct Cursor {
  int t, h, page, np;   // np = pages of trace t
};
__device__ inline void cursor_seek(Cursor& c, const int* cum, int n, int Hkv, long long pos) {
  const int lo = seek_trace(cum, n, Hkv, pos);
  c.t = lo;
  c.np = cum[lo + 1] - cum[lo];
  const long long r = pos - (long long)Hkv * cum[lo];
  c.h = (int)(r / c.np);
  c.page = (int)(r % c.np);
}
__device__ inline void cursor_next(Cursor& c, const int* cum, int n, int Hkv) {
  if (++c.page < c.np) return;
  c.page = 0;
  if (++c.h < Hkv) return;
  c.h = 0;
  do { ++c.t; } while (c.t < n && cum[c.t + 1] == cum[c.t]);
  c.np = c.t < n ? cum[c.t + 1] - cum[c.t] : 1;
}

constexpr int kDynSlotBase = 2 * kMaxPartitions;       // partial slots of the chunks follow those of the equal shares

// ---- the partition of a launch, as both the attention kernel and the kernel that combines the pieces derive it
// from the launch's lengths.
// Pages of sequence t of the KV stream (kMode as for attn_mma_kernel); `flag` records what is wrong with a length.
template <int kMode>
__device__ inline int seq_pages(const AttnArgs& a, int t, bool flag) {
  if constexpr (kMode == kPrefixPass) {
    // a bundle is read if one of its traces holds the whole prefix
    int pages = 0;
    for (int u = t * a.tpb; u < (t + 1) * a.tpb && u < a.n; ++u)
      if (a.seq_lens[u] >= a.pp * kP) pages = a.pp;
    return pages;
  } else {
    int S = a.seq_lens[t];
    if (S < 0) S = 0;
    int pages = (S + kP - 1) / kP;
    if (pages > a.max_pages) { pages = a.max_pages; if (flag) flag_error(a.counters, STEP_ERR_CAPACITY); }
    if constexpr (kMode == kSuffixPass) {
      // own pages only; a trace shorter than the prefix it is said to share is flagged and gets zeros
      if (S >= a.pp * kP) pages -= a.pp;
      else { pages = 0; if (flag && S > 0) flag_error(a.counters, STEP_ERR_INVALID_ARG); }
    }
    return pages;
  }
}
// Pages of sequence t that may go into chunks (before it is known whether the launch has chunks at all).
__device__ inline int tail_pages(const AttnArgs& a, int pages) { return pages * a.dyn16 / 16; }
// Pages per chunk, from the sum of tail_pages over the launch's sequences (per KV head); 0: the launch has no chunks.
// The smallest allowed size, or larger if the chunks would outnumber their partial slots (every sequence's last
// chunk may be short, hence the 2 * sequences); launches with very many sequences do without the hand-out.
__device__ inline int chunk_pages(const AttnArgs& a, int n_seq, long long tails) {
  const long long seqs = (long long)a.Hkv * n_seq;
  if (!a.sched || a.dyn16 <= 0 || 4 * seqs > kMaxDynChunks) return 0;
  const long long by_cap = ((long long)a.Hkv * tails + (kMaxDynChunks - 2 * seqs) - 1) / (kMaxDynChunks - 2 * seqs);
  return (int)(by_cap > a.dyn_chunk ? by_cap : a.dyn_chunk);
}
// A sequence of `pages` pages: pa pages in the static stream, ch chunk numbers.  A sequence with a tail has one
// number per chunk and one more that stands for no pages - its partial slot takes the sequence's static part when
// that part lies inside a single share.
__device__ inline void split_seq(const AttnArgs& a, int pages, int C, int& pa, int& ch) {
  const int tail = C ? tail_pages(a, pages) : 0;
  pa = pages - tail;
  ch = tail > 0 ? (tail + C - 1) / C + 1 : 0;
}

// The whole partition, by one warp, into shared memory: np[n] pages of every sequence, cum[n + 1] its pages in the
// static stream (prefix sum), cumc[n + 1] its chunk numbers per KV head (prefix sum), *chunk the pages per chunk.
template <int kMode>
__device__ inline void build_partition(const AttnArgs& a, int n, int lane, bool flag, int* np, int* cum, int* cumc, int* chunk) {
  long long tails = 0;
  for (int base = 0; base < n; base += 32) {
    const int t = base + lane;
    if (t < n) {
      const int pages = seq_pages<kMode>(a, t, flag);
      np[t] = pages;
      tails += tail_pages(a, pages);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) tails += __shfl_xor_sync(0xffffffffu, tails, o);
  const int C = chunk_pages(a, n, tails);
  int run_a = 0, run_c = 0;
  for (int base = 0; base < n; base += 32) {
    const int t = base + lane;
    int pa = 0, ch = 0;
    if (t < n) split_seq(a, np[t], C, pa, ch);
    int ia = pa, ic = ch;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int va = __shfl_up_sync(0xffffffffu, ia, o), vc = __shfl_up_sync(0xffffffffu, ic, o);
      if (lane >= o) { ia += va; ic += vc; }
    }
    if (t < n) { cum[t] = run_a + ia - pa; cumc[t] = run_c + ic - ch; }
    run_a += __shfl_sync(0xffffffffu, ia, 31);
    run_c += __shfl_sync(0xffffffffu, ic, 31);
  }
  if (lane == 0) { cum[n] = run_a; cumc[n] = run_c; *chunk = C; }
}

// How a launch's pages are spread over the SMs.
//
// Every (trace, KV head) sequence is cut in two: its first pages - all but dyn16 sixteenths - belong to the "static"
// stream (for every trace in order, for every KV head in order, those pages in order), which is cut into one equal
// contiguous share per warp; its last pages, the "tail", are cut into chunks of C pages, and the chunks of all
// sequences are handed out at run time, by an atomic counter, to whichever warp has finished what it had.  SMs do
// not all stream at the same rate (measured: up to 20 % apart), and with equal shares alone a launch lasts as long
// as its slowest SM while the others idle; the chunks even that out.
// Which warp processes a chunk is decided at run time, but the pieces themselves - and with them every partial
// result and the order in which partials are combined - are fixed by the launch's lengths alone, so the outputs do
// not depend on the hand-out.  This kernel only leaves the partial (max, sum, weighted values) of every piece in
// the piece's slot; a second launch (attn_merge_kernel, a programmatic dependent of this one) combines the pieces
// of every sequence.  (An earlier form combined them in this kernel, by tickets: the fence and the atomic round trip
// at the end of every chunk cost more, in a saturated memory system, than the hand-out gained.)
template <int kWarps, int kStages, bool kRows16, int kMode>
__global__ void __launch_bounds__(kWarps * 32, 1) attn_mma_kernel(AttnArgs a) {
  static_assert(kMode != kPrefixPass || kRows16, "the prefix pass uses all 16 rows of the tile");
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* s_pages = smem;                                              // [kWarps][kStages][8 KiB]
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(smem + (size_t)kWarps * kStages * kPageBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // n = sequences of the KV stream: traces, or (prefix pass) bundles of tpb traces that share the prefix pages
  const int n = kMode == kPrefixPass ? a.n_bundles : a.n, Hkv = a.Hkv, G = a.G;
  int* s_np = reinterpret_cast<int*>(s_bar + kWarps * kStages);               // [n]     pages of sequence t
  int* s_cum = s_np + n;                                                      // [n + 1] its pages in the static stream, prefix sum
  int* s_cumc = s_cum + n + 1;                                                // [n + 1] chunk numbers of its tail (per KV head), prefix sum
  int* s_chunk = s_cumc + n + 1;                                              // [1]     pages per chunk (0: no chunks)

  // ---- pages per sequence, the chunk size, prefix sums (warp 0), barrier init (lane 0 of each warp)
  if (warp == 0) build_partition<kMode>(a, n, lane, true, s_np, s_cum, s_cumc, s_chunk);
  if (lane == 0) {
    for (int s = 0; s < kStages; ++s) mbar_init(smem_u32(&s_bar[warp * kStages + s]), 1);
    mbar_init_fence();
  }
  __syncthreads();

  // Nothing has been written yet, and nothing read so far is written by another launch of this kernel: when this
  // launch was scheduled ahead of the completion of such a launch before it (a layer-by-layer sequence of calls made
  // by the library itself), it may run up to its first write - of an output, a partial or a claim on the
  // chunk counter - and must then wait for that launch, whose scratch it shares.  A no-op for a launch made the
  // plain way.  When the launch before this one is the caller's own kernel that produces q (q_from_primary), the
  // wait moves up to the first read of q: what precedes it - the prefix sums above, the barriers, and every warp's
  // first kStages page copies - depends only on the lengths, the block table and the cache, and overlaps that
  // kernel's tail.
  dependents_may_launch();
  bool waited = false;
  auto before_first_write = [&]() { if (!waited) { wait_for_primary(); waited = true; } };
  // traces without any position get zeros (CTAs take the traces round-robin, every thread its share); in the suffix
  // pass a trace that holds the prefix and nothing else gets the normalised prefix result
  auto fill_empty_traces = [&]() {
    if constexpr (kMode != kPrefixPass) {
      for (int t = blockIdx.x; t < n; t += gridDim.x)
        if (s_np[t] == 0) {
          const bool prefix_only = kMode == kSuffixPass && a.seq_lens[t] >= a.pp * kP;
          for (int k = threadIdx.x; k < a.Hq * kD; k += blockDim.x) {
            float v = 0.f;
            if (prefix_only) v = a.pre_o[(size_t)t * a.Hq * kD + k] / a.pre_ml[((size_t)t * a.Hq + k / kD) * 2 + 1];
            a.out[(size_t)t * a.Hq * kD + k] = v;
          }
        }
    }
  };

  const int C = *s_chunk;
  const long long total = (long long)Hkv * s_cum[n];          // pages of the static stream
  const int n_static = a.n_static;                            // = gridDim.x * kWarps
  const long long W = total > 0 ? (total + n_static - 1) / n_static : 1;
  const int n_dyn = Hkv * s_cumc[n];                          // chunks to hand out
  const int part = blockIdx.x * kWarps + warp;

  const uint32_t my_pages_u32 = smem_u32(s_pages + (size_t)warp * kStages * kPageBytes);
  const uint32_t my_bar_u32 = smem_u32(&s_bar[warp * kStages]);

  // A unit of work: this warp's share of the static stream (idx = its partition, `cnt` pages from stream position
  // pos0 on), or a chunk (idx = chunk number: pages p0 .. p0 + cnt - 1 of sequence (t, h)).
  struct Unit { long long pos0; int cnt, idx, t, h, p0; bool chunk; };
  Unit cur, nxt;
  cur.chunk = false; cur.idx = part; cur.pos0 = (long long)part * W; cur.t = cur.h = cur.p0 = 0;
  cur.cnt = cur.pos0 < total ? (int)((cur.pos0 + W <= total ? cur.pos0 + W : total) - cur.pos0) : 0;
  nxt = cur;
  bool have_nxt = false, dyn_done = n_dyn == 0;

  // ---- producer side: cursor, block-id window (lane i holds the id of page win_base + i)
  Cursor pc;
  bool p_chunk = false;
  if (cur.cnt > 0) cursor_seek(pc, s_cum, n, Hkv, cur.pos0);
  int win_t = -1, win_base = 0, win_ids = 0;
  int p_left = cur.cnt, p_stage = 0, in_flight = 0;
  // the next chunk into nxt; false when none is left.  The counter is shared with the launch before this one (if
  // this launch was scheduled ahead of that one's completion); the kernel that combines a launch's pieces puts it
  // back to zero.
  auto claim = [&]() -> bool {
    if (dyn_done) return false;
    before_first_write();
    for (;;) {
      int c = 0;
      if (lane == 0) c = atomicAdd(&a.sched[0], 1);
      c = __shfl_sync(0xffffffffu, c, 0);
      if (c >= n_dyn) { dyn_done = true; return false; }
      const int t = seek_trace(s_cumc, n, Hkv, c);
      const int r = c - Hkv * s_cumc[t], ch = s_cumc[t + 1] - s_cumc[t];
      const int j = r % ch;
      if (j == ch - 1) continue;                       // the number that stands for no pages
      nxt.chunk = true; nxt.idx = c; nxt.t = t; nxt.h = r / ch;
      nxt.p0 = (s_cum[t + 1] - s_cum[t]) + j * C;
      nxt.cnt = min(C, s_np[t] - nxt.p0);
      nxt.pos0 = 0;
      return true;
    }
  };
  // one more page copy into the ring, if a slot is free and a page is left to fetch
  auto issue_one = [&]() -> bool {
    if (in_flight == kStages) return false;
    if (p_left == 0) {
      if (have_nxt || !claim()) return false;          // (the consumer has yet to enter the chunk claimed last)
      have_nxt = true;
      p_chunk = true;
      pc.t = nxt.t; pc.h = nxt.h; pc.page = nxt.p0; pc.np = s_np[nxt.t];
      p_left = nxt.cnt;
      win_t = -1;
    }
    if (pc.t != win_t || pc.page < win_base || pc.page >= win_base + 32) {
      win_t = pc.t; win_base = pc.page;
      const int pg = win_base + lane;
      if constexpr (kMode == kPrefixPass) win_ids = pg < pc.np ? a.prefix_blocks[pg] : 0;
      else if constexpr (kMode == kSuffixPass) win_ids = pg < pc.np ? a.block_table[(size_t)pc.t * a.max_pages + a.pp + pg] : 0;
      else win_ids = pg < pc.np ? a.block_table[(size_t)pc.t * a.max_pages + pg] : 0;
    }
    int b = __shfl_sync(0xffffffffu, win_ids, pc.page - win_base);
    if (lane == 0) {
      if (b < 0 || b >= a.num_blocks) { flag_error(a.counters, STEP_ERR_BAD_BLOCK); b = 0; }
      const __nv_bfloat16* src = a.kv_layer + ((size_t)b * Hkv + pc.h) * (size_t)(2 * kP * kD);
      const uint32_t bar = my_bar_u32 + p_stage * 8;
      mbar_expect_tx(bar, kPageBytes);
      bulk_load(my_pages_u32 + p_stage * kPageBytes, src, kPageBytes, bar);
    }
    if (p_chunk) ++pc.page; else cursor_next(pc, s_cum, n, Hkv);
    --p_left; ++in_flight;
    if (++p_stage == kStages) p_stage = 0;
    return true;
  };
  while (issue_one()) {}

  // ---- consumer side
  Cursor cc;
  if (cur.cnt > 0) cursor_seek(cc, s_cum, n, Hkv, cur.pos0);
  int c_left = cur.cnt;
  const int g_row = lane >> 2, tq = lane & 3;
  uint32_t qa[8][4];                 // A fragments of Q for the 8 k-steps over head_dim
  float o_acc[16][4];                // O fragments: 16 n-tiles over head_dim
  float m_run[2], l_run[2];          // rows g_row and g_row + 8
  int seg_first_page = 0, seq_last_page = 0;
  bool seg_open = false, seg_is_first = true;
  int stage = 0;
  uint32_t parity = 0;
  bool alive = true;
  const int R = kMode == kPrefixPass ? 16 : G;         // rows of a partial slot

  // ldmatrix lane addressing inside a page (swizzled 16-byte chunks: chunk' = chunk ^ (row & 7))
  const int mi = lane >> 3, r8 = lane & 7;
  const int k_row = ((mi >> 1) << 3) + r8;             // K: matrices 0,1 -> tokens 0-7; 2,3 -> tokens 8-15
  const int k_csel = mi & 1;                           //    matrix parity picks the low/high 8 dims of the k-step
  const int v_row = ((mi & 1) << 3) + r8;              // V: matrices 0,2 -> tokens 0-7; 1,3 -> tokens 8-15
  const int v_csel = mi >> 1;                          //    matrices 2,3 belong to the next 8-wide dim tile

  for (;;) {
    if (c_left == 0) {
      // this unit is done: on to the chunk the producer has claimed (it claims one now if it had no reason to yet)
      while (issue_one()) {}
      if (!have_nxt) break;
      cur = nxt; have_nxt = false;
      cc.t = cur.t; cc.h = cur.h; cc.page = cur.p0; cc.np = s_np[cur.t];
      c_left = cur.cnt;
      seg_open = false; seg_is_first = true;
    }
    if (!seg_open) {
      seq_last_page = s_np[cc.t] - 1;
      // new (trace, head) segment: Q fragments of the G heads of this group, fresh softmax state
      if (a.q_from_primary) before_first_write();
      const uint32_t *q0, *q1;
      bool r0, r1;
      if constexpr (kMode == kPrefixPass) {
        // row r of the tile is head (r % G) of the group of trace cc.t * tpb + r / G
        const int ta = cc.t * a.tpb + g_row / G, tb = cc.t * a.tpb + (g_row + 8) / G;
        r0 = g_row < a.tpb * G && ta < a.n;
        r1 = g_row + 8 < a.tpb * G && tb < a.n;
        q0 = reinterpret_cast<const uint32_t*>(a.q + ((size_t)(r0 ? ta : 0) * a.Hq + (size_t)cc.h * G + g_row % G) * kD);
        q1 = reinterpret_cast<const uint32_t*>(a.q + ((size_t)(r1 ? tb : 0) * a.Hq + (size_t)cc.h * G + (g_row + 8) % G) * kD);
      } else {
        const __nv_bfloat16* qbase = a.q + ((size_t)cc.t * a.Hq + (size_t)cc.h * G) * kD;
        q0 = reinterpret_cast<const uint32_t*>(qbase + (size_t)g_row * kD);
        q1 = reinterpret_cast<const uint32_t*>(qbase + (size_t)(g_row + 8) * kD);
        r0 = g_row < G; r1 = kRows16 && (g_row + 8 < G);
      }
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        qa[ks][0] = r0 ? q0[ks * 8 + tq] : 0u;
        qa[ks][2] = r0 ? q0[ks * 8 + 4 + tq] : 0u;
        qa[ks][1] = r1 ? q1[ks * 8 + tq] : 0u;
        qa[ks][3] = r1 ? q1[ks * 8 + 4 + tq] : 0u;
      }
#pragma unroll
      for (int dt = 0; dt < 16; ++dt) { o_acc[dt][0] = o_acc[dt][1] = o_acc[dt][2] = o_acc[dt][3] = 0.f; }
      m_run[0] = m_run[1] = -INFINITY;
      l_run[0] = l_run[1] = 0.f;
      seg_first_page = cc.page;
      seg_open = true;
    }

    if (!mbar_wait_bounded(my_bar_u32 + stage * 8, parity, a.wait_ns)) {
      if (lane == 0) flag_error(a.counters, STEP_ERR_TIMEOUT);
      alive = false;
      break;
    }
    const uint32_t kpage = my_pages_u32 + stage * kPageBytes;
    const uint32_t vpage = kpage + kVOffset;

    // tokens of this page that exist (only the last page of a sequence can be short)
    int valid = kP;
    if (kMode != kPrefixPass && cc.page == seq_last_page) {     // shared pages are full
      int S = a.seq_lens[cc.t];
      const int cap = a.max_pages * kP;
      if (S > cap) S = cap;
      valid = S - (cc.page + (kMode == kSuffixPass ? a.pp : 0)) * kP;
      if (valid < kP) {
        // unused V rows may hold anything (even NaN bit patterns): zero them so 0 * V stays 0
        for (int idx = lane; idx < (kP - valid) * 16; idx += 32) {
          const int row = valid + (idx >> 4), chunk = idx & 15;
          asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(vpage + row * 256 + chunk * 16), "r"(0u) : "memory");
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
      }
    }

    // ---- S = Q K^T for 16 tokens: two n-tiles of 8 tokens
    float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      const int chunk = ks * 2 + k_csel;
      const uint32_t addr = kpage + k_row * 256 + ((((chunk & 8) | ((chunk ^ k_row) & 7))) << 4);
      uint32_t b0, b1, b2, b3;
      ldsm_x4(addr, b0, b1, b2, b3);
      mma_bf16(s0, qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b0, b1);
      mma_bf16(s1, qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b2, b3);
    }
    // thread holds, for row g_row (and g_row+8): tokens 2tq, 2tq+1 (s0) and 8+2tq, 9+2tq (s1)
    {
      const int j0 = 2 * tq;
      const bool v00 = j0 < valid, v01 = j0 + 1 < valid, v10 = j0 + 8 < valid, v11 = j0 + 9 < valid;
      s0[0] = v00 ? s0[0] * a.scale_log2 : -INFINITY; s0[1] = v01 ? s0[1] * a.scale_log2 : -INFINITY;
      s1[0] = v10 ? s1[0] * a.scale_log2 : -INFINITY; s1[1] = v11 ? s1[1] * a.scale_log2 : -INFINITY;
      if (kRows16) {
        s0[2] = v00 ? s0[2] * a.scale_log2 : -INFINITY; s0[3] = v01 ? s0[3] * a.scale_log2 : -INFINITY;
        s1[2] = v10 ? s1[2] * a.scale_log2 : -INFINITY; s1[3] = v11 ? s1[3] * a.scale_log2 : -INFINITY;
      }
    }
    float mx0 = fmaxf(fmaxf(s0[0], s0[1]), fmaxf(s1[0], s1[1]));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    const float mn0 = fmaxf(m_run[0], mx0);          // finite: token 0 of a page always exists
    const float corr0 = exp2f(m_run[0] - mn0);
    m_run[0] = mn0;
    const float p00 = exp2f(s0[0] - mn0), p01 = exp2f(s0[1] - mn0), p10 = exp2f(s1[0] - mn0), p11 = exp2f(s1[1] - mn0);
    l_run[0] = l_run[0] * corr0 + (p00 + p01) + (p10 + p11);
    uint32_t pa0 = pack_bf16(p00, p01), pa2 = pack_bf16(p10, p11), pa1 = 0u, pa3 = 0u;
    float corr1 = 1.f;
    if (kRows16) {
      float mx1 = fmaxf(fmaxf(s0[2], s0[3]), fmaxf(s1[2], s1[3]));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      const float mn1 = fmaxf(m_run[1], mx1);
      corr1 = exp2f(m_run[1] - mn1);
      m_run[1] = mn1;
      const float q00 = exp2f(s0[2] - mn1), q01 = exp2f(s0[3] - mn1), q10 = exp2f(s1[2] - mn1), q11 = exp2f(s1[3] - mn1);
      l_run[1] = l_run[1] * corr1 + (q00 + q01) + (q10 + q11);
      pa1 = pack_bf16(q00, q01); pa3 = pack_bf16(q10, q11);
    }
    // rescale O only when some row's maximum moved (warp-uniform branch)
    const bool moved = (corr0 != 1.f) || (kRows16 && corr1 != 1.f);
    if (__any_sync(0xffffffffu, moved)) {
#pragma unroll
      for (int dt = 0; dt < 16; ++dt) {
        o_acc[dt][0] *= corr0; o_acc[dt][1] *= corr0;
        if (kRows16) { o_acc[dt][2] *= corr1; o_acc[dt][3] *= corr1; }
      }
    }
    // ---- O += P V : 16 n-tiles over head_dim, k = 16 tokens
#pragma unroll
    for (int dp = 0; dp < 8; ++dp) {
      const int chunk = dp * 2 + v_csel;
      const uint32_t addr = vpage + v_row * 256 + ((((chunk & 8) | ((chunk ^ v_row) & 7))) << 4);
      uint32_t b0, b1, b2, b3;
      ldsm_x4_t(addr, b0, b1, b2, b3);
      mma_bf16(o_acc[2 * dp], pa0, pa1, pa2, pa3, b0, b1);
      mma_bf16(o_acc[2 * dp + 1], pa0, pa1, pa2, pa3, b2, b3);
    }
    __syncwarp();
    --in_flight;
    issue_one();                                       // refill the stage just consumed

    // ---- end of this (trace, head) segment?
    // (in a share cc.np counts the sequence's pages in the static stream: a segment ends there at the latest)
    const bool seq_static_end = !cur.chunk && cc.page + 1 == cc.np;
    const bool seg_end = seq_static_end || c_left == 1;
    if (seg_end) {
      float l0 = l_run[0];
      l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
      l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
      float l1 = l_run[1];
      if (kRows16) {
        l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
      }
      // the whole sequence in this one segment: it has no tail, and its static pages lie in this share
      const bool complete = seq_static_end && seg_first_page == 0 && cc.page == seq_last_page;
      before_first_write();
      if (complete && kMode == kPrefixPass) {
        // the bundle's whole prefix was read by this warp: (m, l, o) of every (trace, head) row, un-normalised
        const int ta = cc.t * a.tpb + g_row / G, tb = cc.t * a.tpb + (g_row + 8) / G;
        if (g_row < a.tpb * G && ta < a.n) {
          const size_t idx = (size_t)ta * a.Hq + (size_t)cc.h * G + g_row % G;
          if (tq == 0) { a.pre_ml[idx * 2] = m_run[0]; a.pre_ml[idx * 2 + 1] = l0; }
#pragma unroll
          for (int dt = 0; dt < 16; ++dt)
            *reinterpret_cast<float2*>(a.pre_o + idx * kD + dt * 8 + 2 * tq) = make_float2(o_acc[dt][0], o_acc[dt][1]);
        }
        if (g_row + 8 < a.tpb * G && tb < a.n) {
          const size_t idx = (size_t)tb * a.Hq + (size_t)cc.h * G + (g_row + 8) % G;
          if (tq == 0) { a.pre_ml[idx * 2] = m_run[1]; a.pre_ml[idx * 2 + 1] = l1; }
#pragma unroll
          for (int dt = 0; dt < 16; ++dt)
            *reinterpret_cast<float2*>(a.pre_o + idx * kD + dt * 8 + 2 * tq) = make_float2(o_acc[dt][2], o_acc[dt][3]);
        }
      } else if (complete) {
        float* ob = a.out + ((size_t)cc.t * a.Hq + (size_t)cc.h * G) * kD;
        if (g_row < G) {
          float ws = 1.f, wp = 0.f, lp = 0.f;
          const float* po = nullptr;
          if constexpr (kMode == kSuffixPass) {          // fold in the shared pages' result
            const size_t idx = (size_t)cc.t * a.Hq + (size_t)cc.h * G + g_row;
            const float mp = a.pre_ml[idx * 2];
            lp = a.pre_ml[idx * 2 + 1];
            const float Mn = fmaxf(m_run[0], mp);
            ws = exp2f(m_run[0] - Mn); wp = exp2f(mp - Mn);
            po = a.pre_o + idx * kD;
          }
          const float inv = 1.f / (l0 * ws + lp * wp);
#pragma unroll
          for (int dt = 0; dt < 16; ++dt) {
            float x = o_acc[dt][0] * ws, y = o_acc[dt][1] * ws;
            if constexpr (kMode == kSuffixPass) {
              const float2 pv = *reinterpret_cast<const float2*>(po + dt * 8 + 2 * tq);
              x += wp * pv.x; y += wp * pv.y;
            }
            *reinterpret_cast<float2*>(ob + (size_t)g_row * kD + dt * 8 + 2 * tq) = make_float2(x * inv, y * inv);
          }
        }
        if (kRows16 && g_row + 8 < G) {
          float ws = 1.f, wp = 0.f, lp = 0.f;
          const float* po = nullptr;
          if constexpr (kMode == kSuffixPass) {
            const size_t idx = (size_t)cc.t * a.Hq + (size_t)cc.h * G + g_row + 8;
            const float mp = a.pre_ml[idx * 2];
            lp = a.pre_ml[idx * 2 + 1];
            const float Mn = fmaxf(m_run[1], mp);
            ws = exp2f(m_run[1] - Mn); wp = exp2f(mp - Mn);
            po = a.pre_o + idx * kD;
          }
          const float inv = 1.f / (l1 * ws + lp * wp);
#pragma unroll
          for (int dt = 0; dt < 16; ++dt) {
            float x = o_acc[dt][2] * ws, y = o_acc[dt][3] * ws;
            if constexpr (kMode == kSuffixPass) {
              const float2 pv = *reinterpret_cast<const float2*>(po + dt * 8 + 2 * tq);
              x += wp * pv.x; y += wp * pv.y;
            }
            *reinterpret_cast<float2*>(ob + (size_t)(g_row + 8) * kD + dt * 8 + 2 * tq) = make_float2(x * inv, y * inv);
          }
        }
      } else {
        // ---- a piece of a sequence: leave its (m, l, o) in this piece's slot.
        // The sequence's chunk numbers are cbase .. cbase + n_ch (n_ch chunks, then the number that stands for no
        // pages); its static part lies in shares s0p .. s1p.  A static piece that reaches an
        // edge of its share uses one of the share's two slots (every share has at most one piece at each edge); a
        // static part that lies inside a single share - there may be many of those in one share - uses the slot of
        // the sequence's spare chunk number.  (A sequence without a tail whose static part lies inside one share
        // was complete and never gets here.)
        const int np_static = s_cum[cc.t + 1] - s_cum[cc.t];
        const int n_nums = s_cumc[cc.t + 1] - s_cumc[cc.t];
        const int n_ch = n_nums > 0 ? n_nums - 1 : 0;
        const int cbase = Hkv * s_cumc[cc.t] + cc.h * n_nums;
        const long long seg_start = (long long)Hkv * s_cum[cc.t] + (long long)cc.h * np_static;
        const int s0p = (int)(seg_start / W), s1p = (int)((seg_start + np_static - 1) / W);
        const int n_s = s1p - s0p + 1;
        const size_t spare = (size_t)kDynSlotBase + cbase + n_ch;
        const size_t slot = cur.chunk ? (size_t)kDynSlotBase + cur.idx
                                      : (n_s == 1 ? spare : (size_t)cur.idx * 2 + (seg_is_first ? 0 : 1));
        float* ml = a.ws_ml + slot * R * 2;
        float* ob = a.ws_o + slot * R * kD;
        if (g_row < R) {
          if (tq == 0) { ml[g_row * 2] = m_run[0]; ml[g_row * 2 + 1] = l0; }
#pragma unroll
          for (int dt = 0; dt < 16; ++dt)
            *reinterpret_cast<float2*>(ob + (size_t)g_row * kD + dt * 8 + 2 * tq) = make_float2(o_acc[dt][0], o_acc[dt][1]);
        }
        if (kRows16 && g_row + 8 < R) {
          if (tq == 0) { ml[(g_row + 8) * 2] = m_run[1]; ml[(g_row + 8) * 2 + 1] = l1; }
#pragma unroll
          for (int dt = 0; dt < 16; ++dt)
            *reinterpret_cast<float2*>(ob + (size_t)(g_row + 8) * kD + dt * 8 + 2 * tq) = make_float2(o_acc[dt][2], o_acc[dt][3]);
        }
      }
      seg_open = false;
      seg_is_first = false;
    }
    if (cur.chunk) ++cc.page; else cursor_next(cc, s_cum, n, Hkv);
    --c_left;
    if (++stage == kStages) { stage = 0; parity ^= 1; }
  }

  before_first_write();
  fill_empty_traces();
  if (!alive) {
    // A wait ran out.  The in_flight copies issued last still target this CTA's shared memory (ring positions stage,
    // stage + 1, ... in the consumer's order): each gets one more wait, with the full limit, before the warp
    // leaves; nothing else is touched.
    for (int k = 0; k < in_flight; ++k) {
      const int st = stage + k;
      mbar_wait_bounded(my_bar_u32 + (st % kStages) * 8, parity ^ (uint32_t)(st >= kStages));
    }
  }
}

// Combines, for every (sequence, KV head) of the launch that was cut into pieces, the pieces' partials into the
// output (or, for the shared pages' pass, into that pass's result).  Work item = one query row of one sequence's
// tile, taken by one warp (items are dealt round-robin to all warps of the grid): the warp takes the row's pieces in
// stream order - static pieces, then chunks - eight at a time (all their loads issued together: one round trip to
// memory for most sequences), lanes over the 128 dims, and keeps a running (max, sum, weighted values) across the
// batches; a fixed order, so the same bits whatever ran where.
// Launched as a programmatic dependent of the attention kernel, with at most one small CTA per SM and few enough
// registers that it is resident BESIDE the attention kernel's CTA: it works out where the pieces are from the
// launch's lengths - the same functions the attention kernel uses - while that kernel is still running, then waits
// for it.  (A launch chained behind this one is scheduled only when every CTA of this one has started, so CTAs that
// had to queue for an SM would hold back the next layer's launch until this layer is over.)
constexpr int kMergeBatch = 8, kMergeWarps = 4;

template <int kMode>
__global__ void __launch_bounds__(kMergeWarps * 32, 5) attn_merge_kernel(AttnArgs a) {
  extern __shared__ int s_part[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int Hkv = a.Hkv, G = a.G;
  const int R = kMode == kPrefixPass ? 16 : G;                    // rows of a partial slot
  const int rows = kMode == kPrefixPass ? a.tpb * G : G;          // rows in use
  dependents_may_launch();
  const int n = kMode == kPrefixPass ? a.n_bundles : a.n;
  int* s_np = s_part;
  int* s_cum = s_np + n;
  int* s_cumc = s_cum + n + 1;
  int* s_chunk = s_cumc + n + 1;
  if (warp == 0) build_partition<kMode>(a, n, lane, false, s_np, s_cum, s_cumc, s_chunk);
  __syncthreads();
  const long long total = (long long)Hkv * s_cum[n];
  const long long W = total > 0 ? (total + a.n_static - 1) / a.n_static : 1;

  wait_for_primary();
  if (blockIdx.x == 0 && threadIdx.x == 0 && a.sched) a.sched[0] = 0;   // the chunk counter, for the next launch

  const int n_items = n * Hkv * rows;
  for (int item = blockIdx.x * kMergeWarps + warp; item < n_items; item += gridDim.x * kMergeWarps) {
    const int g = item % rows, th = item / rows;
    const int t = th / Hkv, h = th - t * Hkv;
    const int np_static = s_cum[t + 1] - s_cum[t];
    if (np_static == 0) continue;                                 // no pages: the attention kernel wrote zeros
    const int n_nums = s_cumc[t + 1] - s_cumc[t];
    const int n_ch = n_nums > 0 ? n_nums - 1 : 0;
    const int cbase = Hkv * s_cumc[t] + h * n_nums;
    const long long seg_start = (long long)Hkv * s_cum[t] + (long long)h * np_static;
    const int s0p = (int)(seg_start / W), s1p = (int)((seg_start + np_static - 1) / W);
    const int n_s = s1p - s0p + 1;
    const int n_pieces = n_s + n_ch;
    if (n_pieces == 1) continue;                                  // one piece: the attention kernel wrote the output itself
    const size_t spare = (size_t)kDynSlotBase + cbase + n_ch;
    auto slot_of = [&](int k) -> size_t {
      if (k < n_s) {
        if (n_s == 1) return spare;
        const int w = s0p + k;
        return (size_t)w * 2 + (seg_start <= (long long)w * W ? 0 : 1);
      }
      return (size_t)kDynSlotBase + cbase + (k - n_s);
    };
    size_t idx = 0;                                               // (trace, head) row of pre_ml / pre_o
    if constexpr (kMode == kPrefixPass) {
      const int tt = t * a.tpb + g / G;
      if (tt >= a.n) continue;
      idx = (size_t)tt * a.Hq + (size_t)h * G + g % G;
    } else if constexpr (kMode == kSuffixPass) {
      idx = (size_t)t * a.Hq + (size_t)h * G + g;
    }

    float M = -INFINITY, den = 0.f;
    float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int k0 = 0; k0 < n_pieces; k0 += kMergeBatch) {
      float2 ml[kMergeBatch];
      float4 o4[kMergeBatch];
#pragma unroll
      for (int j = 0; j < kMergeBatch; ++j) {
        if (k0 + j < n_pieces) {
          const size_t sl = slot_of(k0 + j);
          ml[j] = __ldcg(reinterpret_cast<const float2*>(a.ws_ml + (sl * R + g) * 2));
          o4[j] = __ldcg(reinterpret_cast<const float4*>(a.ws_o + (sl * R + g) * kD) + lane);
        }
      }
      float Mb = M;
#pragma unroll
      for (int j = 0; j < kMergeBatch; ++j)
        if (k0 + j < n_pieces) Mb = fmaxf(Mb, ml[j].x);
      const float keep = exp2f(M - Mb);                           // 0 on the first batch (M = -inf)
      den *= keep; num.x *= keep; num.y *= keep; num.z *= keep; num.w *= keep;
      M = Mb;
#pragma unroll
      for (int j = 0; j < kMergeBatch; ++j) {
        if (k0 + j < n_pieces) {
          const float wgt = exp2f(ml[j].x - M);
          den += wgt * ml[j].y;
          num.x += wgt * o4[j].x; num.y += wgt * o4[j].y; num.z += wgt * o4[j].z; num.w += wgt * o4[j].w;
        }
      }
    }
    if constexpr (kMode == kSuffixPass) {                         // the shared pages count as one more partial
      const float mp = a.pre_ml[idx * 2], lp = a.pre_ml[idx * 2 + 1];
      const float4 o4 = reinterpret_cast<const float4*>(a.pre_o + idx * kD)[lane];
      const float Mb = fmaxf(M, mp);
      const float keep = exp2f(M - Mb), wgt = exp2f(mp - Mb);
      den = den * keep + wgt * lp;
      num.x = num.x * keep + wgt * o4.x; num.y = num.y * keep + wgt * o4.y;
      num.z = num.z * keep + wgt * o4.z; num.w = num.w * keep + wgt * o4.w;
    }
    if constexpr (kMode == kPrefixPass) {
      if (lane == 0) { a.pre_ml[idx * 2] = M; a.pre_ml[idx * 2 + 1] = den; }
      reinterpret_cast<float4*>(a.pre_o + idx * kD)[lane] = num;
    } else {
      float* og = a.out + ((size_t)t * a.Hq + (size_t)h * G + g) * kD;
      const float inv = 1.f / den;
      reinterpret_cast<float4*>(og)[lane] = make_float4(num.x * inv, num.y * inv, num.z * inv, num.w * inv);
    }
  }
}

constexpr int kWarpsDefault = 8, kStagesDefault = 3;

// The attention kernel, then the kernel that combines its pieces as its programmatic dependent.
// dependent: the attention launch itself may be scheduled before the kernel ahead of it in the stream has completed
// (see the kernel's note on its first write).
template <int kWarps, int kStages, bool kRows16, int kMode>
int launch_one(AttnArgs a, int grid, cudaStream_t s, bool dependent = false) {
  const int n_seq = kMode == kPrefixPass ? a.n_bundles : a.n;
  const size_t smem = (size_t)kWarps * kStages * kPageBytes + (size_t)kWarps * kStages * 8 + (size_t)(3 * n_seq + 3) * 4;
  a.n_static = grid * kWarps;
  auto kern = attn_mma_kernel<kWarps, kStages, kRows16, kMode>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return STEP_ERR_CUDA;
  if (dependent) {
    if (launch_dependent(kern, dim3(grid), dim3(kWarps * 32), smem, s, a) != cudaSuccess) return STEP_ERR_CUDA;
  } else {
    kern<<<grid, kWarps * 32, smem, s>>>(a);
    if (launch_ok() != STEP_OK) return STEP_ERR_CUDA;
  }
  const int rows = kMode == kPrefixPass ? a.tpb * a.G : a.G;
  long long mgrid = ((long long)n_seq * a.Hkv * rows + kMergeWarps - 1) / kMergeWarps;
  if (mgrid > a.merge_ctas) mgrid = a.merge_ctas;
  if (launch_dependent(attn_merge_kernel<kMode>, dim3((int)mgrid), dim3(kMergeWarps * 32), (size_t)(3 * n_seq + 3) * 4, s, a) != cudaSuccess) return STEP_ERR_CUDA;
  return launch_ok();
}

template <int kWarps, int kStages, int kMode>
int launch_mma(const step_pool* pool, const AttnArgs& a, cudaStream_t s, bool dependent = false) {
  int grid = pool->attn_grid;
  if (grid * kWarps > kMaxPartitions) grid = kMaxPartitions / kWarps;
  if (grid < 1) grid = 1;
  return a.G > 8 ? launch_one<kWarps, kStages, true, kMode>(a, grid, s, dependent)
                 : launch_one<kWarps, kStages, false, kMode>(a, grid, s, dependent);
}

void fill_args(AttnArgs& a, const step_pool* pool, const Geo& g, int layer, const void* q, const int32_t* block_table,
               const int32_t* seq_lens, int n, void* out) {
  a.kv_layer = (const __nv_bfloat16*)pool->cfg.kv_storage + (size_t)layer * g.num_blocks * g.Hkv * 2 * kP * kD;
  a.q = (const __nv_bfloat16*)q;
  a.block_table = block_table; a.seq_lens = seq_lens; a.out = (float*)out;
  a.ws_ml = pool->v.attn_ml; a.ws_o = pool->v.attn_o; a.counters = pool->v.counters;
  a.n = n; a.Hq = g.Hq; a.Hkv = g.Hkv; a.G = g.G; a.max_pages = g.max_pages; a.num_blocks = g.num_blocks;
  a.scale_log2 = 1.4426950408889634f / sqrtf((float)g.d);
  a.prefix_blocks = nullptr; a.pre_ml = nullptr; a.pre_o = nullptr; a.pp = 0; a.tpb = 1; a.n_bundles = 0;
  a.q_from_primary = 0;
  a.sched = pool->attn_dyn16 > 0 ? pool->v.attn_sched : nullptr;
  a.dyn16 = pool->attn_dyn16; a.dyn_chunk = pool->attn_dyn_chunk;
  a.n_static = 0;                                      // set by the launcher
  a.merge_ctas = pool->num_sms;
  a.wait_ns = pool->wait_limit_ns;
}

bool mma_shape(const step_pool* pool, const Geo& g, int n) {
  return pool->cfg.dtype == STEP_BF16 && g.d == kD && g.P == kP && g.G <= 16 && n <= kMaxTracesFast && pool->swizzle;
}

}  // namespace

// How a launch relates to the kernel before it in the stream: an ordinary launch; a programmatic dependent of
// another launch of this kernel on the same pool (waits in front of its first write); a programmatic dependent of
// the caller's kernel that writes q (waits in front of its first read of q).
enum LaunchMode { kOrdinary = 0, kAfterOwnKind = 1, kAfterQProducer = 2 };

static int decode_attention_launch(step_pool* pool, int layer, const void* q, const int32_t* block_table,
                                   const int32_t* seq_lens, int n, void* out, void* stream, LaunchMode mode);

extern "C" int decode_attention(step_pool* pool, int layer, const void* q, const int32_t* block_table,
                                const int32_t* seq_lens, int n, void* out, void* stream) {
  return decode_attention_launch(pool, layer, q, block_table, seq_lens, n, out, stream, kOrdinary);
}

// decode_attention for a caller that runs the layers one by one (the query of layer l + 1 is computed from the
// output of layer l, so it cannot hand over all layers' queries at once): the launch is made a programmatic dependent
// of whatever kernel precedes it in the stream - the caller's kernel that produces q.  The CTAs are scheduled as
// soon as that kernel's CTAs have exited (or have announced that dependents may start), set themselves up, start
// their first page copies, and wait for that kernel's completion only in front of their first read of q.
extern "C" int decode_attention_dependent(step_pool* pool, int layer, const void* q, const int32_t* block_table,
                                          const int32_t* seq_lens, int n, void* out, void* stream) {
  return decode_attention_launch(pool, layer, q, block_table, seq_lens, n, out, stream, kAfterQProducer);
}

// decode_attention of several consecutive layers whose queries the caller has at hand.  The first layer's launch is an
// ordinary one; every later launch directly follows the launch of the layer before it, reads nothing that one writes,
// and is therefore made its programmatic dependent: an SM that has finished its share of layer l starts on layer l + 1
// at once instead of idling until the whole of layer l is done, and the stream of KV reads never drains at a layer
// boundary (the kernel holds its first write back until the launch before it has completed).
extern "C" int decode_attention_layers(step_pool* pool, int layer0, int n_layers, const void* q,
                                       const int32_t* block_table, const int32_t* seq_lens, int n, void* out,
                                       void* stream) {
  if (!pool || n < 0 || n_layers < 0 || layer0 < 0) return STEP_ERR_INVALID_ARG;
  if (n == 0 || n_layers == 0) return STEP_OK;
  if (layer0 + n_layers > pool->cfg.num_layers) return STEP_ERR_INVALID_ARG;
  const size_t q_layer = (size_t)n * pool->cfg.num_q_heads * pool->cfg.head_dim * pool->elem_bytes;
  const size_t o_layer = (size_t)n * pool->cfg.num_q_heads * pool->cfg.head_dim * sizeof(float);
  for (int l = 0; l < n_layers; ++l) {
    const int st = decode_attention_launch(pool, layer0 + l, q ? (const char*)q + l * q_layer : nullptr, block_table, seq_lens, n,
                                           out ? (char*)out + l * o_layer : nullptr, stream, l > 0 ? kAfterOwnKind : kOrdinary);
    if (st != STEP_OK) return st;
  }
  return STEP_OK;
}

static int decode_attention_launch(step_pool* pool, int layer, const void* q, const int32_t* block_table,
                                   const int32_t* seq_lens, int n, void* out, void* stream, LaunchMode mode) {
  if (!pool || n < 0) return STEP_ERR_INVALID_ARG;
  if (n == 0) return STEP_OK;
  if (!q || !block_table || !seq_lens || !out) return STEP_ERR_INVALID_ARG;
  Geo g = geo_of(pool);
  if (layer < 0 || layer >= g.L) return STEP_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  if (pool->fast_path > 0 && mma_shape(pool, g, n)) {
    AttnArgs a;
    fill_args(a, pool, g, layer, q, block_table, seq_lens, n, out);
    a.q_from_primary = mode == kAfterQProducer;
    return launch_mma<kWarpsDefault, kStagesDefault, kPlain>(pool, a, s, mode != kOrdinary);
  }
  // the scalar kernel is always launched the ordinary way (same results, no overlap)
  if (n > 65535) return STEP_ERR_INVALID_ARG;
  const size_t smem = (size_t)(g.d + kScalarWarps * g.d) * sizeof(float);
  if (pool->cfg.dtype == STEP_BF16)
    attn_scalar_kernel<__nv_bfloat16><<<dim3(g.Hq, n), kScalarWarps * 32, smem, s>>>(
        g, (const __nv_bfloat16*)pool->cfg.kv_storage, layer, (const __nv_bfloat16*)q, block_table, seq_lens,
        (float*)out, pool->v.counters);
  else
    attn_scalar_kernel<float><<<dim3(g.Hq, n), kScalarWarps * 32, smem, s>>>(
        g, (const float*)pool->cfg.kv_storage, layer, (const float*)q, block_table, seq_lens, (float*)out,
        pool->v.counters);
  return launch_ok();
}

// decode_attention when the first prefix_pages pages of every listed trace are the same blocks (the prompt pages
// kv_pool_fork_prefix shares between the traces of one problem).  Two launches: the shared pages are read once per
// bundle of 16 / G traces instead of once per trace, then every trace's own pages are read as usual and the two
// results combined by the usual (max, sum) rule.  HBM traffic is the same as decode_attention's (the L2 absorbs
// the repeated reads there); what shrinks is the L2 -> SM traffic, which is what bounds the step when the prompt
// is long against the generated suffixes.
extern "C" int decode_attention_shared_prefix(step_pool* pool, int layer, const void* q, const int32_t* block_table,
                                              const int32_t* seq_lens, int n, const int32_t* prefix_blocks,
                                              int prefix_pages, void* out, void* stream) {
  if (!pool || n < 0 || prefix_pages < 0) return STEP_ERR_INVALID_ARG;
  if (prefix_pages == 0) return decode_attention(pool, layer, q, block_table, seq_lens, n, out, stream);
  if (n == 0) return STEP_OK;
  if (!q || !block_table || !seq_lens || !out || !prefix_blocks) return STEP_ERR_INVALID_ARG;
  Geo g = geo_of(pool);
  if (layer < 0 || layer >= g.L || prefix_pages > g.max_pages) return STEP_ERR_INVALID_ARG;
  if (!mma_shape(pool, g, n) || n > g.max_traces || !pool->v.pre_o) return STEP_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  AttnArgs a;
  fill_args(a, pool, g, layer, q, block_table, seq_lens, n, out);
  a.prefix_blocks = prefix_blocks; a.pre_ml = pool->v.pre_ml; a.pre_o = pool->v.pre_o; a.pp = prefix_pages;
  a.tpb = 16 / g.G; a.n_bundles = (n + a.tpb - 1) / a.tpb;
  // pass 1: about eight pages per warp, at most one CTA per SM and kPrefixPartitions partitions
  AttnArgs p1 = a;
  p1.ws_ml = pool->v.pre_ws_ml; p1.ws_o = pool->v.pre_ws_o;
  p1.sched = nullptr;                                  // its scratch holds equal shares only
  const long long pages1 = (long long)a.n_bundles * g.Hkv * prefix_pages;
  long long grid1 = (pages1 + kWarpsDefault * 8 - 1) / (kWarpsDefault * 8);
  const int cap1 = pool->attn_grid < kPrefixPartitions / kWarpsDefault ? pool->attn_grid : kPrefixPartitions / kWarpsDefault;
  if (grid1 > cap1) grid1 = cap1;
  if (grid1 < 1) grid1 = 1;
  const int st = launch_one<kWarpsDefault, kStagesDefault, true, kPrefixPass>(p1, (int)grid1, s);
  if (st != STEP_OK) return st;
  // pass 2, a programmatic dependent of pass 1: it reads pass 1's result only where it writes its own outputs, which
  // is behind its wait for the launch before it
  return launch_mma<kWarpsDefault, kStagesDefault, kSuffixPass>(pool, a, s, true);
}

// =============================================================== allocation-free variant
// decode_attention_static: the tensor-core kernel above with its (m, l, o) partials kept in a
// fixed array that is part of the library image instead of in caller-provided metadata.
//
// Who needs it: code that must run attention but is not allowed to obtain device memory at that
// point - e.g. a plug-in called inside someone else's memory-pool-managed region, a real-time loop
// that forbids allocator calls after start-up, or a host that hands this library buffers it cannot
// grow.  Such a caller passes only inputs and the output; nothing here calls cudaMalloc, cudaFree
// or any allocating routine.
//
// The scratch is a file-scope __device__ array of a fixed, modest size (kStaticScratchFloats
// floats, about 9.9 MB); every GPU that loads the library carries it until the process exits.
// In host code the array's NAME is only a stand-in symbol, not a device address, so the launcher
// asks the runtime for the real address once per device (cudaGetSymbolAddress, with that device
// current, return code checked) and passes that pointer to the kernels.
namespace {

constexpr int kStaticMaxPartitions = 1184;   // 148 SMs x 8 warps
constexpr int kStaticMaxG = 8;               // query heads per KV head
constexpr size_t kStaticMlFloats = (size_t)kStaticMaxPartitions * 2 * kStaticMaxG * 2;
constexpr size_t kStaticOFloats = (size_t)kStaticMaxPartitions * 2 * kStaticMaxG * kD;
constexpr int kStaticMaxSegs = 16384;        // (trace, KV head) sequences of one call
constexpr size_t kStaticScratchFloats = kStaticMlFloats + kStaticOFloats;

static __device__ __align__(256) float g_static_scratch[kStaticScratchFloats];

constexpr int kMaxDevices = 64;
float* g_static_scratch_addr[kMaxDevices];   // device address of g_static_scratch, per device; null until set up

// Set-up, once per device: resolve the device address of the scratch symbol.
int static_scratch_for_current_device(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return STEP_ERR_CUDA;
  float* p = __atomic_load_n(&g_static_scratch_addr[dev], __ATOMIC_ACQUIRE);
  if (!p) {
    if (cudaGetSymbolAddress((void**)&p, g_static_scratch) != cudaSuccess || !p) return STEP_ERR_CUDA;
    __atomic_store_n(&g_static_scratch_addr[dev], p, __ATOMIC_RELEASE);   // same value whoever wins
  }
  *out = p;
  return STEP_OK;
}

}  // namespace

extern "C" int decode_attention_static(step_pool* pool, int layer, const void* q, const int32_t* block_table,
                                       const int32_t* seq_lens, int n, void* out, void* stream) {
  if (!pool || n < 0) return STEP_ERR_INVALID_ARG;
  if (n == 0) return STEP_OK;
  if (!q || !block_table || !seq_lens || !out) return STEP_ERR_INVALID_ARG;
  Geo g = geo_of(pool);
  if (layer < 0 || layer >= g.L) return STEP_ERR_INVALID_ARG;
  // only the shape the tensor-core kernel covers
  if (pool->cfg.dtype != STEP_BF16 || g.d != kD || g.P != kP || !pool->swizzle) return STEP_ERR_INVALID_ARG;
  // sizes beyond what the fixed scratch holds, and the entry point's bound on the sequences of one call
  if (g.G > kStaticMaxG || n > kMaxTracesFast || (long long)n * g.Hkv > kStaticMaxSegs) return STEP_ERR_CAPACITY;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return STEP_ERR_CUDA;
  if (dev != pool->device) return STEP_ERR_INVALID_ARG;   // the pool's device must be current
  float* scratch = nullptr;
  const int st = static_scratch_for_current_device(&scratch);
  if (st != STEP_OK) return st;
  int grid = pool->attn_grid;
  if (grid * kWarpsDefault > kStaticMaxPartitions) grid = kStaticMaxPartitions / kWarpsDefault;
  if (grid < 1) grid = 1;
  AttnArgs a;
  fill_args(a, pool, g, layer, q, block_table, seq_lens, n, out);
  // the same kernels, the partials in the library's own array instead of the pool's metadata
  a.ws_ml = scratch; a.ws_o = scratch + kStaticMlFloats;
  a.sched = nullptr;                                   // the fixed array holds the partials of equal shares only
  cudaStream_t s = (cudaStream_t)stream;
  return launch_one<kWarpsDefault, kStagesDefault, false, kPlain>(a, grid, s);
}
