// Tensor-core form of the step scorer's first layer for launches with many boundary rows
// (Sec. 3.1 "Model Architecture": y = sigmoid(w2 . ReLU(W1 h + b1) + b2)).
//
// For up to 256 listed rows r (two halves of 128; launches too small to fill the SMs that way use 128) and a slice [n0, n0 + N) of the m hidden units one work item computes
//     z_slice[r] = sum_{j in slice} w2[j] * ReLU(sum_k h[r][k] * W1[j][k] + b1[j])
// as a 256 x N x D bf16 GEMM on the 5th-generation tensor cores with the whole second layer fused into
// the read-out of the accumulators:
//   * two accumulators (128 rows x N columns each, fp32) live in tensor memory (2 x 256 columns); both row
//     halves multiply the same W1 tile, which halves the W1 bytes fetched per product - operand delivery from
//     L2, not the tensor pipe, is what limits this kernel;
//   * A = the hidden rows named by the row list.  The rows are scattered in the caller's [M, D]
//     array, so eight warps gather them with 16-byte cp.async copies straight into the 128-byte-swizzled
//     K-major arrangement the MMA unit reads (row r of a tile at (r / 8) * 1024 + (r % 8) * 128,
//     16-byte chunk c stored at chunk c ^ (r % 8)); no compacted copy of the rows is ever made;
//     when every candidate row is listed (the list is 0, 1, 2, ...) the rows of an item are contiguous in the
//     caller's array and the TMA thread fetches them as 128-row tiles instead - same arrangement, no gather;
//   * B = W1[n0 .. n0 + N, k .. k + 64): TMA tiled loads (one 64 x 64 box per 64 units, 128-byte
//     swizzle) signalling the stage's mbarrier with their byte count;
//   * the operand ring is 192 KiB; a stage holds exactly what the launch's item shape needs (24 KiB for 128 rows x
//     64 units ... 64 KiB for 256 x 256), so small launches, which are latency-bound, get up to 8 stages in flight;
//   * one thread issues tcgen05.mma (M 128, N 64 | 128 | 256, K 16) four times per row half and 64-wide k-chunk and
//     commits the stage back to the producers;
//   * eight warps read the finished accumulators with tcgen05.ld - a thread owns one row, so
//     + b1, ReLU, * w2 and the sum over the slice's units are plain per-thread fp32 arithmetic on
//     un-rounded activations - and store one partial per (row, slice) for the finishing kernel.
// The kernel is persistent (one CTA per SM, items handed out round-robin).  N is picked on the device
// from the number of boundary rows so that small launches still spread over many SMs.
// Every wait is bounded; a wait that runs out raises STEP_ERR_TIMEOUT and the CTA winds down,
// releasing its tensor memory.
#include "step_internal.cuh"
#include "async_copy.cuh"

#include <cuda.h>
#include <string.h>

using namespace stepk;

namespace {

constexpr int kHalfRows = 128;                    // UMMA M
constexpr int kBK = 64;                           // bf16 elements per k-chunk (one 128-byte swizzle row)
constexpr int kMaxN = 256;                        // UMMA N limit
constexpr int kMaxStages = 8;
constexpr int kHalfBytes = kHalfRows * kBK * 2;   // 16 KiB
constexpr int kRingBytes = 192 * 1024;            // shared memory of the operand ring; a stage is as large as the
                                                  // launch's item shape needs, so small shapes get more stages
constexpr int kBoxRows = 64;                      // hidden units per TMA box
constexpr int kBoxBytes = kBoxRows * kBK * 2;     // 8 KiB
constexpr int kEpiWarps = 8, kGatherWarps = 8;    // read-out: warp w takes TMEM lanes 32 (w % 4) of accumulator w / 4
constexpr int kWarpTma = kEpiWarps + kGatherWarps, kWarpMma = kWarpTma + 1;
constexpr int kThreads = (kWarpMma + 1) * 32;     // 576
constexpr int kTmemCols = 512;                    // two accumulators (row halves) of up to 256 columns
constexpr int kMaxUnits = 1024;                   // b1 / w2 staged in shared memory as fp32
constexpr unsigned long long kDrainNs = 100000000ull;

struct TcArgs {
  const __nv_bfloat16* hidden;
  const __nv_bfloat16* b1;
  const __nv_bfloat16* w2;
  const int32_t* idx;
  float* z;
  int32_t* counters;
  int D, m;
  int Mc;          // candidate rows of the launch
  int dense_ok;    // the second tensor map describes `hidden` ([Mc, D]): usable when every candidate row is listed
};

__device__ inline void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
// The mbarrier gets one arrival from this thread once all its earlier cp.async copies have landed; the thread
// itself does not wait.  (The barrier's expected count includes these arrivals: "noinc".)
__device__ inline void cp_async_arrive_when_done(uint32_t bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ inline void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ inline void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ inline void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ inline void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ inline void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ inline void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, both operands K-major bf16, fp32 accumulate.
__device__ inline void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ inline void tc_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes (64 bf16) stored with the
// 128-byte swizzle: groups of 8 rows are 1024 bytes apart (stride byte offset), the leading byte offset is
// unused by swizzled K-major layouts (1), descriptor version 1, layout type 2 = SWIZZLE_128B.
__device__ inline uint64_t umma_desc_sw128(uint32_t smem_addr) {
  const uint32_t lo = ((smem_addr >> 4) & 0x3FFFu) | (1u << 16);
  const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
  return ((uint64_t)hi << 32) | lo;
}
// The k-chunk an item starts its reduction at.  Every item walks all D / 64 chunks once, cyclically; starting
// them at different chunks keeps the CTAs that run side by side from all asking for the same few lines of
// W1 (and the same byte offset of every hidden row) at the same moment.
__device__ inline int first_chunk(int item, int KC) { return (int)(((unsigned)item * 7u) % (unsigned)KC); }

// Instruction descriptor of kind::f16: fp32 accumulator, bf16 A and B, both K-major, M = 128, N = n.
__device__ inline uint32_t umma_idesc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kHalfRows >> 4) << 24);
}

__global__ void __launch_bounds__(kThreads, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap map_w1, const __grid_constant__ CUtensorMap map_h, TcArgs a) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;                 // swizzled tiles want 1024-byte alignment
  unsigned char* sm = smem_raw + (base - raw);
  float* s_b1 = reinterpret_cast<float*>(sm + kRingBytes);
  float* s_w2 = s_b1 + kMaxUnits;
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(s_w2 + kMaxUnits);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_bar + 2 * kMaxStages + 2);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
  const uint32_t bar_full = smem_u32(s_bar), bar_empty = bar_full + 8 * kMaxStages;
  const uint32_t bar_tfull = bar_empty + 8 * kMaxStages, bar_tempty = bar_tfull + 8;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kMaxStages; ++s) {
      mbar_init(bar_full + 8 * s, kGatherWarps * 32 + 1);       // one arrival per gather thread + the TMA thread
      mbar_init(bar_empty + 8 * s, 1);                          // tcgen05.commit
    }
    mbar_init(bar_tfull, 1);                                    // tcgen05.commit
    mbar_init(bar_tempty, kEpiWarps);                           // one arrival per read-out warp
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kWarpMma) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  for (int j = threadIdx.x; j < a.m; j += kThreads) {
    s_b1[j] = __bfloat162float(a.b1[j]);
    s_w2[j] = __bfloat162float(a.w2[j]);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;

  // Everything above touched only this CTA's own shared and tensor memory and the weights; the row list and the
  // launch's shape come from the compaction kernel, whose completion this kernel may have been scheduled ahead of.
  dependents_may_launch();
  wait_for_primary();
  // the launch decided on the device whether this kernel or the CUDA-core kernel scores its rows
  const int n_units = a.counters[C_SCORE_TC];
  const bool active = n_units != 0;   // 0: the CUDA-core kernel scored this launch's rows (or there were none)
  const int N = active ? n_units : kBoxRows;
  const int nb = active ? a.counters[C_SCORE_NB] : 0;
  const int slices = a.m / N;
  const int R = active ? a.counters[C_SCORE_TILE] : kHalfRows;  // rows per item: 256, or 128 for launches too small to
  const int tiles = (nb + R - 1) / R;                           // fill the SMs with 256-row items
  // operand ring: a stage holds R x 64 of the hidden rows and N x 64 of W1 (24 - 64 KiB), 3 to 8 stages
  const int a_bytes = R / kHalfRows * kHalfBytes;
  const int stage_bytes = a_bytes + N * kBK * 2;
  const int n_stages = min(kMaxStages, kRingBytes / stage_bytes);
  // Items are handed out round-robin, so a launch takes as long as the CTA with the most items.  With 256-row
  // items the last round can be nearly empty; the rows that would make it up are cut into 128-row items instead,
  // which spreads that last bit of work over twice as many CTAs.  (The ring keeps the 256-row stage layout.)
  int n_big = tiles * slices, n_big_tiles = tiles, n_small = 0;
  if (R > kHalfRows && n_big > (int)gridDim.x && n_big % (int)gridDim.x != 0) {
    n_big_tiles = n_big / (int)gridDim.x * (int)gridDim.x / slices;
    n_big = n_big_tiles * slices;
    n_small = (nb - n_big_tiles * R + kHalfRows - 1) / kHalfRows * slices;
  }
  const int items = n_big + n_small;
  // item -> first listed row, rows (256 or 128), slice of hidden units
  auto item_rows = [&](int item, int& row0, int& slice) -> int {
    if (item < n_big) { const int t = item / slices; slice = item - t * slices; row0 = t * R; return R; }
    const int j = item - n_big, t = j / slices;
    slice = j - t * slices; row0 = n_big_tiles * R + t * kHalfRows;
    return kHalfRows;
  };
  const int KC = a.D / kBK;
  // Every candidate row ends a step (scoring collected step-end states offline): the list is 0, 1, 2, ..., the rows
  // of an item are contiguous in the caller's array, and the TMA thread fetches them as tiles - same arrangement in
  // shared memory, none of the gather warps' instructions.
  const bool dense = a.dense_ok && nb == a.Mc;

  if (!active) {
    // nothing to do but give the tensor memory back below
  } else if (warp < kEpiWarps) {
    // ------------------------------------------------ read-out: second layer on the accumulators
    const int quarter = warp & 3, half = warp >> 2;
    int li = 0;
    for (int item = blockIdx.x; item < items; item += gridDim.x, ++li) {
      int row0, slice;
      const int rows = item_rows(item, row0, slice);
      const int n0 = slice * N;
      if (*s_abort) break;
      if (!mbar_wait_bounded(bar_tfull, li & 1)) {
        if (lane == 0) flag_error(a.counters, STEP_ERR_TIMEOUT);
        *s_abort = 1;
        break;
      }
      tc_fence_after();
      const int row = row0 + half * kHalfRows + quarter * 32 + lane;
      const bool used = half * kHalfRows < rows && row0 + half * kHalfRows < nb;    // did this half get any products?
      float z = 0.f;
      if (used) {
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(half * kMaxN);
        for (int c0 = 0; c0 < N; c0 += 32) {
          float v[32];
          tc_ld32(taddr + c0, v);
#pragma unroll
          for (int j = 0; j < 32; ++j) z = fmaf(s_w2[n0 + c0 + j], fmaxf(v[j] + s_b1[n0 + c0 + j], 0.f), z);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty);
      if (used && row < nb) a.z[(size_t)row * kScoreSplits + slice] = z;
    }
  } else if (warp < kWarpTma) {
    // ------------------------------------------------ gather of the listed hidden rows into A
    const int tg = threadIdx.x - kEpiWarps * 32;                // 0 .. 255
    const int c = tg & 7, rb = tg >> 3;                         // 16-byte chunk of the row; rows rb + 32 i
    const uint32_t dst0 = base + (uint32_t)((rb >> 3) * 1024 + (rb & 7) * 128 + ((c ^ (rb & 7)) << 4));
    int s = 0;                                                  // ring position and its phase, kept incrementally
    uint32_t ph = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < items && ok; item += gridDim.x) {
      int row0, slice;
      const int rows = item_rows(item, row0, slice);
      const __nv_bfloat16* src[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int gr = row0 + rb + 32 * i;
        // rows past the end of the list are not fetched: each output row depends on its own operand row only, so
        // whatever the shared memory holds there ends up in accumulator rows that nobody reads out
        src[i] = !dense && gr < nb && 32 * i < rows ? a.hidden + (size_t)a.idx[gr] * a.D + c * 8 : nullptr;
      }
      int kr = first_chunk(item, KC);
      for (int kc = 0; kc < KC; ++kc) {
        if (*s_abort || !mbar_wait_bounded(bar_empty + 8 * s, ph ^ 1)) { ok = false; break; }
        const uint32_t dst = dst0 + (uint32_t)(s * stage_bytes);
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (src[i]) cp_async16(dst + i * 4096, src[i] + kr * kBK);
        if (++kr == KC) kr = 0;
        // the stage's barrier hears from this thread when these copies have landed; the thread moves on at once,
        // so the copies of all stages can be in flight and nothing here waits for data
        cp_async_arrive_when_done(bar_full + 8 * s);
        if (++s == n_stages) { s = 0; ph ^= 1; }
      }
    }
    cp_async_wait_all();                                        // nothing of this thread is in flight when it leaves
    if (!ok) {
      if (lane == 0) flag_error(a.counters, STEP_ERR_TIMEOUT);
      *s_abort = 1;
    }
  } else if (warp == kWarpTma) {
    // ------------------------------------------------ TMA loads of the W1 slice into B
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      const int boxes = N / kBoxRows;
      for (int item = blockIdx.x; item < items && ok; item += gridDim.x) {
        int row0, slice;
        const int rows = item_rows(item, row0, slice);
        const int n0 = slice * N;
        // row halves fetched as tiles (rows past the end of the array arrive as zeros, and count as bytes)
        const int halves_a = !dense ? 0 : (rows > kHalfRows && row0 + kHalfRows < nb ? 2 : 1);
        int kr = first_chunk(item, KC);
        for (int kc = 0; kc < KC; ++kc) {
          if (*s_abort || !mbar_wait_bounded(bar_empty + 8 * s, ph ^ 1)) { ok = false; break; }
          const uint32_t bar = bar_full + 8 * s;
          mbar_expect_tx(bar, (uint32_t)(boxes * kBoxBytes + halves_a * kHalfBytes));
          for (int h = 0; h < halves_a; ++h)
            tma_load_2d(base + (uint32_t)(s * stage_bytes + h * kHalfBytes), &map_h, kr * kBK, row0 + h * kHalfRows, bar);
          const uint32_t dst = base + (uint32_t)(s * stage_bytes + a_bytes);
          for (int j = 0; j < boxes; ++j) tma_load_2d(dst + j * kBoxBytes, &map_w1, kr * kBK, n0 + j * kBoxRows, bar);
          if (++kr == KC) kr = 0;
          if (++s == n_stages) { s = 0; ph ^= 1; }
        }
      }
      if (!ok) {
        flag_error(a.counters, STEP_ERR_TIMEOUT);
        *s_abort = 1;
        // loads already issued still target this CTA's shared memory: give them a moment to land
        for (int q = 0; q < n_stages; ++q) {
          mbar_wait_bounded(bar_full + 8 * q, 0, kDrainNs);
          mbar_wait_bounded(bar_full + 8 * q, 1, kDrainNs);
        }
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------ MMA issue
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(N);
      int s = 0, li = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < items && ok; item += gridDim.x, ++li) {
        int row0, slice;
        const int rows = item_rows(item, row0, slice);
        const int halves = rows > kHalfRows && row0 + kHalfRows < nb ? 2 : 1;
        // the read-out of the previous item must have drained the accumulators
        if (*s_abort || !mbar_wait_bounded(bar_tempty, (li & 1) ^ 1)) { ok = false; break; }
        tc_fence_after();
        for (int kc = 0; kc < KC; ++kc) {
          if (*s_abort || !mbar_wait_bounded(bar_full + 8 * s, ph)) { ok = false; break; }
          fence_async_smem();                                   // the gathered rows were written through the generic proxy
          tc_fence_after();
          const uint64_t bdesc = umma_desc_sw128(base + (uint32_t)(s * stage_bytes + a_bytes));
          for (int h = 0; h < halves; ++h) {                    // both row halves multiply the same W1 tile
            const uint64_t adesc = umma_desc_sw128(base + (uint32_t)(s * stage_bytes + h * kHalfBytes));
            const uint32_t d_tmem = tmem_base + (uint32_t)(h * kMaxN);
#pragma unroll
            for (int kk = 0; kk < kBK / 16; ++kk)                // 16 bf16 = 32 bytes further along the swizzled row
              tc_mma_bf16(d_tmem, adesc + 2 * kk, bdesc + 2 * kk, idesc, (kc | kk) != 0);
          }
          tc_commit(bar_empty + 8 * s);                         // the stage is free once these products have read it
          if (++s == n_stages) { s = 0; ph ^= 1; }
        }
        if (ok) tc_commit(bar_tfull);                           // the accumulators are complete
      }
      if (!ok) {
        flag_error(a.counters, STEP_ERR_TIMEOUT);
        *s_abort = 1;
      }
    }
    __syncwarp();
  }

  tc_fence_before();
  __syncthreads();
  if (warp == kWarpMma) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

constexpr size_t kSmemBytes = 1024 + (size_t)kRingBytes + 2 * kMaxUnits * sizeof(float) +
                              (2 * kMaxStages + 2) * sizeof(uint64_t) + 16;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
    tried = true;
  }
  return fn;
}

}  // namespace

namespace stepk {

bool score_tc_supported(const scorer_weights* w, const void* hidden) {
  if (w->dtype != STEP_BF16) return false;
  if (w->D < kBK || w->D % kBK != 0) return false;                       // whole 64-wide k-chunks
  if (w->m < kBoxRows || w->m % kBoxRows != 0 || w->m > kMaxUnits) return false;
  if (w->m / kMaxN > kScoreSplits) return false;
  if (((uintptr_t)w->W1 | (uintptr_t)hidden) & 15) return false;         // 16-byte copies and TMA base
  return encode_tiled_fn() != nullptr;
}

int score_tc_launch(step_pool* pool, const void* hidden, int Mc, const scorer_weights* w, cudaStream_t s) {
  static_assert(sizeof(CUtensorMap) <= sizeof(pool->tmap_bytes), "tensor map cache too small");
  if (pool->tmap_w1 != w->W1 || pool->tmap_D != w->D || pool->tmap_m != w->m) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return STEP_ERR_CUDA;
    CUtensorMap fresh;
    const cuuint64_t dims[2] = {(cuuint64_t)w->D, (cuuint64_t)w->m};       // innermost first
    const cuuint64_t strides[1] = {(cuuint64_t)w->D * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)kBoxRows};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&fresh, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(w->W1), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return STEP_ERR_CUDA;
    memcpy(pool->tmap_bytes, &fresh, sizeof(fresh));
    pool->tmap_w1 = w->W1; pool->tmap_D = w->D; pool->tmap_m = w->m;
  }
  CUtensorMap map;
  memcpy(&map, pool->tmap_bytes, sizeof(map));
  // the candidate rows as a [Mc, D] array of 128-row tiles, for launches in which every row ends a step
  if (pool->tmap_h_ptr != hidden || pool->tmap_h_D != w->D || pool->tmap_h_M != Mc) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return STEP_ERR_CUDA;
    CUtensorMap fresh;
    const cuuint64_t dims[2] = {(cuuint64_t)w->D, (cuuint64_t)Mc};
    const cuuint64_t strides[1] = {(cuuint64_t)w->D * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)kHalfRows};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&fresh, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(hidden), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return STEP_ERR_CUDA;
    memcpy(pool->tmap_h_bytes, &fresh, sizeof(fresh));
    pool->tmap_h_ptr = hidden; pool->tmap_h_D = w->D; pool->tmap_h_M = Mc;
  }
  CUtensorMap map_h;
  memcpy(&map_h, pool->tmap_h_bytes, sizeof(map_h));
  if (!pool->tc_smem_set) {
    if (cudaFuncSetAttribute(score_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes) != cudaSuccess)
      return STEP_ERR_CUDA;
    pool->tc_smem_set = true;
  }
  TcArgs a;
  a.hidden = (const __nv_bfloat16*)hidden;
  a.b1 = (const __nv_bfloat16*)w->b1; a.w2 = (const __nv_bfloat16*)w->w2;
  a.idx = pool->v.score_idx; a.z = pool->v.score_z; a.counters = pool->v.counters;
  a.D = w->D; a.m = w->m;
  a.Mc = Mc; a.dense_ok = 1;
  long long max_items = (long long)((Mc + kHalfRows - 1) / kHalfRows) * (w->m / kBoxRows);
  int grid = pool->num_sms;
  if (max_items < grid) grid = (int)max_items;
  if (grid < 1) grid = 1;
  // a dependent launch: the CTAs set themselves up while the compaction kernel is still running
  if (launch_dependent(score_tc_kernel, dim3(grid), dim3(kThreads), kSmemBytes, s, map, map_h, a) != cudaSuccess) return STEP_ERR_CUDA;
  return launch_ok();
}

}  // namespace stepk
