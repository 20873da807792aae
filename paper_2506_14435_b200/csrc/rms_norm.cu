// RMS normalisation of token rows: the LN of Eq. 2 as the Qwen2.5 models the paper builds on
// apply it (no mean subtraction), with unit gain:  y = bf16( x * rsqrt(mean(x^2) + eps) ).
// The layer itself takes an already normalised input; this is for callers that chain layers
// (mote_stack_forward).  One warp per row; fp32 sums in a fixed order, so results do not depend
// on scheduling.  HBM-bound: 2 B read + 2 B written per element.
#include "mote_common.cuh"
#include "mote_internal.h"

namespace mote {

__global__ void __launch_bounds__(256) rms_norm_kernel(const uint16_t* __restrict__ x, int64_t T, int d, float eps,
                                                       uint16_t* __restrict__ y) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t row = int64_t(blockIdx.x) * 8 + warp;
  pdl_wait();                            // x may be the output of the kernel ahead (a layer stack)
  if (row >= T) return;
  const uint4* src = reinterpret_cast<const uint4*>(x + row * int64_t(d));
  uint4* dst = reinterpret_cast<uint4*>(y + row * int64_t(d));
  const int n_vec = d / 8;
  float ss = 0.0f;
  for (int v = lane; v < n_vec; v += 32) {
    const uint4 r = src[v];
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float a = bf16_lo(w[j]), b = bf16_hi(w[j]);
      ss = fmaf(a, a, ss);
      ss = fmaf(b, b, ss);
    }
  }
  ss = warp_sum(ss);
  const float inv = rsqrtf(ss / float(d) + eps);
  for (int v = lane; v < n_vec; v += 32) {
    const uint4 r = src[v];                              // second read of the row hits L1/L2
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) o[j] = pack_bf16x2(bf16_lo(w[j]) * inv, bf16_hi(w[j]) * inv);
    dst[v] = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

mote_status_t launch_rms_norm(const void* x, int64_t T, int d, float eps, void* y, cudaStream_t stream) {
  if (T == 0) return MOTE_OK;
  MOTE_CUDA_OK(launch_pdl(rms_norm_kernel, dim3((unsigned)((T + 7) / 8)), dim3(256), 0, stream,
                          static_cast<const uint16_t*>(x), T, d, eps, static_cast<uint16_t*>(y)));
  ++g_launch_count;
  MOTE_LAUNCH_OK();
  return MOTE_OK;
}

}  // namespace mote

extern "C" mote_status_t mote_rms_norm(const void* x_bf16, int64_t T, int64_t d, float eps, void* y_bf16, void* stream) {
  using namespace mote;
  if (T < 0 || d <= 0 || (d % 8) != 0 || d > (1 << 20) || !(eps >= 0.0f)) return MOTE_ERR_SHAPE;
  if (T == 0) return MOTE_OK;
  if (!x_bf16 || !y_bf16) return MOTE_ERR_NULL;
  if (!aligned16(x_bf16) || !aligned16(y_bf16)) return MOTE_ERR_ALIGN;
  return launch_rms_norm(x_bf16, T, (int)d, eps, y_bf16, static_cast<cudaStream_t>(stream));
}
