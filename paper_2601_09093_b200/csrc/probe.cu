// step_read_stream_probe: what the device's HBM delivers to the copy structure decode_attention uses, with no
// attention arithmetic attached - a measured ceiling to put beside the attention kernel's own bandwidth.
//
// The kernel is the attention kernel's data path and nothing else: one CTA per SM, eight warps, every warp owns
// an equal contiguous run of 8 KiB pieces of the buffer and keeps a ring of three bulk async copies
// (cp.async.bulk + mbarrier complete_tx) in flight into its own shared memory; a piece that has landed is
// dropped.  Launched n times in a row it can be chained the way decode_attention_layers chains its layers
// (every launch after the first a programmatic dependent of the one before it, the wait for that launch held
// back to the kernel's end), or launched the ordinary way.
#include "step_internal.cuh"
#include "async_copy.cuh"

using namespace stepk;

namespace {

constexpr int kWarps = 8, kStages = 3, kPiece = 8192;

__global__ void __launch_bounds__(kWarps * 32, 1)
read_stream_kernel(const unsigned char* __restrict__ buf, long long pieces, int32_t* __restrict__ err) {
  extern __shared__ __align__(1024) unsigned char smem[];
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(smem + (size_t)kWarps * kStages * kPiece);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) {
    for (int s = 0; s < kStages; ++s) mbar_init(smem_u32(&s_bar[warp * kStages + s]), 1);
    mbar_init_fence();
  }
  __syncthreads();
  dependents_may_launch();
  const long long n_part = (long long)gridDim.x * kWarps;
  const long long W = (pieces + n_part - 1) / n_part;
  const long long p0 = ((long long)blockIdx.x * kWarps + warp) * W;
  const long long cnt = p0 >= pieces ? 0 : (p0 + W <= pieces ? W : pieces - p0);
  const uint32_t ring = smem_u32(smem + (size_t)warp * kStages * kPiece);
  const uint32_t bars = smem_u32(&s_bar[warp * kStages]);
  long long issued = 0;
  auto produce = [&](int stage) {
    if (lane == 0) {
      mbar_expect_tx(bars + stage * 8, kPiece);
      bulk_load(ring + stage * kPiece, buf + (size_t)(p0 + issued) * kPiece, kPiece, bars + stage * 8);
    }
    ++issued;
  };
  for (int s = 0; s < kStages && issued < cnt; ++s) produce(s);
  int stage = 0;
  uint32_t parity = 0;
  bool alive = true;
  for (long long i = 0; i < cnt; ++i) {
    if (!mbar_wait_bounded(bars + stage * 8, parity)) { alive = false; break; }
    __syncwarp();
    if (issued < cnt) produce(stage);
    if (++stage == kStages) { stage = 0; parity ^= 1; }
  }
  if (!alive) {
    if (lane == 0) atomicExch(err, 1);
    for (int s = 0; s < kStages; ++s) {                // copies in flight still target this CTA's shared memory
      mbar_wait_bounded(bars + s * 8, 0);
      mbar_wait_bounded(bars + s * 8, 1);
    }
  }
  wait_for_primary();                                  // where the attention kernel would make its first write
}

}  // namespace

extern "C" int step_read_stream_probe(const void* buf, size_t bytes, int n_launches, int chained, int32_t* err_flag,
                                      void* stream) {
  if (!buf || !err_flag || n_launches < 1 || bytes < (size_t)kPiece || ((uintptr_t)buf & 15)) return STEP_ERR_INVALID_ARG;
  int dev = 0, sms = 0;
  STEP_CUDA_OK(cudaGetDevice(&dev));
  STEP_CUDA_OK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const size_t smem = (size_t)kWarps * kStages * kPiece + (size_t)kWarps * kStages * 8;
  STEP_CUDA_OK(cudaFuncSetAttribute(read_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  cudaStream_t s = (cudaStream_t)stream;
  const long long pieces = (long long)(bytes / kPiece);
  for (int i = 0; i < n_launches; ++i) {
    if (chained && i > 0) {
      STEP_CUDA_OK(launch_dependent(read_stream_kernel, dim3(sms), dim3(kWarps * 32), smem, s,
                                    (const unsigned char*)buf, pieces, err_flag));
    } else {
      read_stream_kernel<<<sms, kWarps * 32, smem, s>>>((const unsigned char*)buf, pieces, err_flag);
    }
  }
  return launch_ok();
}
