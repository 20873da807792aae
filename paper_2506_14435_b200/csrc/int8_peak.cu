// Speed of light of the int8 tensor pipe, measured: every SM issues tcgen05.mma.kind::i8
// (M128 x N256 x K32, s8 x u8 -> s32, the instruction shape of the routed expert GEMMs) back to
// back on operands that never leave shared memory.  No TMA, no unpacking, no epilogue: what is
// timed is the MMA issue rate alone, the ceiling the expert GEMM kernels are measured against.
#include <algorithm>

#include "mote_common.cuh"
#include "mote_internal.h"
#include "ptx_sm100.cuh"

namespace mote {

using namespace ptx;

constexpr int kPeakMmasPerBatch = 64;            // one commit per batch
constexpr int kPeakA = 128 * 128, kPeakB = 256 * 128;

__global__ void __launch_bounds__(128, 1) int8_mma_peak_kernel(uint32_t* status, int n_batches) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t bar[2];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_word;
  volatile int* abort_flag = &abort_word;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  // operands: pseudo-random int8 tokens and ternary codes stored as code+1, as in the real GEMM
  // (constant data would toggle fewer wires and run cooler than the workload does)
  uint32_t h = 0x9E3779B9u * (blockIdx.x + 1) + threadIdx.x;
  for (int i = threadIdx.x; i < (kPeakA + kPeakB) / 4; i += blockDim.x) {
    h = h * 1664525u + 1013904223u;
    uint32_t w = h ^ (h >> 15);
    if (i >= kPeakA / 4) {                       // four codes in {0, 1, 2}
      const uint32_t two = w & 0x02020202u;
      w = two | ((w & 0x01010101u) & ~(two >> 1));
    }
    reinterpret_cast<uint32_t*>(gen)[i] = w;
  }
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar[0]), 1);
    mbar_init(smem_u32(&bar[1]), 1);
    abort_word = 0;
    fence_barrier_init();
  }
  fence_proxy_async_smem();
  if (threadIdx.x < 32) {
    tmem_alloc(smem_u32(&tmem_slot), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_slot;
  if (threadIdx.x == 0) {
    const uint32_t idesc = make_idesc(2, 1, 0, 128, 256);
    const uint64_t da = smem_desc_sw128(base), db = smem_desc_sw128(base + kPeakA);
    bool ok = true;
    for (int b = 0; ok && b < n_batches; ++b) {
      // two batches in flight: before reusing an accumulator, wait for the batch that last wrote it
      if (b >= 2) ok = mbar_wait(smem_u32(&bar[b & 1]), ((b >> 1) - 1) & 1, abort_flag);
      if (!ok) break;
      const uint32_t d_tmem = tmem + (b & 1) * 256;
#pragma unroll 8
      for (int j = 0; j < kPeakMmasPerBatch; ++j) mma_i8(d_tmem, da + 2 * (j & 3), db + 2 * (j & 3), idesc, j > 0);
      mma_commit(smem_u32(&bar[b & 1]));
    }
    // drain: the last commit of each accumulator
    for (int b = (n_batches > 2 ? n_batches - 2 : 0); ok && b < n_batches; ++b)
      ok = mbar_wait(smem_u32(&bar[b & 1]), (b >> 1) & 1, abort_flag);
  }
  __syncthreads();
  if (*abort_flag) {
    const uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x < 32) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
  if (threadIdx.x == 0 && *abort_flag) atomicExch(status, 1u);
}

}  // namespace mote

extern "C" mote_status_t mote_int8_mma_peak(void* ws, int n_batches, double* ops_host, void* stream_) {
  using namespace mote;
  if (!ws || !ops_host) return MOTE_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return MOTE_ERR_ALIGN;
  if (n_batches < 1 || n_batches > 100000) return MOTE_ERR_SHAPE;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  constexpr int kSmem = 1024 + kPeakA + kPeakB;
  static PerDeviceOnce attr_once;
  MOTE_CUDA_OK(set_max_dynamic_smem(attr_once, int8_mma_peak_kernel, kSmem));
  const int sms = device_sm_count();
  int8_mma_peak_kernel<<<sms, 128, kSmem, stream>>>(static_cast<uint32_t*>(ws), n_batches);
  MOTE_LAUNCH_OK();
  *ops_host = double(sms) * n_batches * kPeakMmasPerBatch * (2.0 * 128 * 256 * 32);
  return MOTE_OK;
}
