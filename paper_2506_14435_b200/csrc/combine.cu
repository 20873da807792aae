// Gate-weighted combine and un-permute (Eq. 2, Eq. 4), gather form (no atomics, deterministic):
//   out[t,:] = bf16( [residual[t,:] +] s[t,:] + sum_{j<k} w[t,j] * y[perm[t*k+j], :] )
// (s may arrive as the partial sums of a K-split down projection, added here in ascending order)
// fp32 arithmetic, slots added in ascending j, one bf16 rounding at the end.
// HBM-bound: per output element 4 B (s) + 4k B (y) [+ 2 B residual] read, 2 B written.
#include "mote_common.cuh"
#include "mote_internal.h"

namespace mote {

__global__ void __launch_bounds__(256) combine_kernel(const float* __restrict__ s, const float* __restrict__ y,
                                                      const float* __restrict__ w, const int32_t* __restrict__ perm,
                                                      const uint16_t* residual, int64_t T, int d, int k,
                                                      uint16_t* out, int n_partials) {
  const int vec_per_row = d / 8;
  const int64_t total = T * vec_per_row;
  pdl_wait();                            // no-op unless launched as a programmatic dependent
  const int64_t stride = int64_t(gridDim.x) * blockDim.x;
  for (int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += stride) {
    const int64_t t = i / vec_per_row;
    const int v = (int)(i - t * vec_per_row);
    float acc[8];
    {
      const float4* sp = reinterpret_cast<const float4*>(s + t * d + v * 8);
      const float4 a = sp[0], b = sp[1];
      acc[0] = a.x; acc[1] = a.y; acc[2] = a.z; acc[3] = a.w;
      acc[4] = b.x; acc[5] = b.y; acc[6] = b.z; acc[7] = b.w;
    }
    for (int p = 1; p < n_partials; ++p) {           // partial sums of a K-split projection, in order
      const float4* sp = reinterpret_cast<const float4*>(s + (int64_t(p) * T + t) * d + v * 8);
      const float4 a = sp[0], b = sp[1];
      acc[0] += a.x; acc[1] += a.y; acc[2] += a.z; acc[3] += a.w;
      acc[4] += b.x; acc[5] += b.y; acc[6] += b.z; acc[7] += b.w;
    }
    for (int j = 0; j < k; ++j) {
      const float wj = w[t * k + j];
      const int64_t r = perm[t * k + j];
      const float4* yp = reinterpret_cast<const float4*>(y + r * d + v * 8);
      const float4 a = yp[0], b = yp[1];
      acc[0] = fmaf(wj, a.x, acc[0]); acc[1] = fmaf(wj, a.y, acc[1]);
      acc[2] = fmaf(wj, a.z, acc[2]); acc[3] = fmaf(wj, a.w, acc[3]);
      acc[4] = fmaf(wj, b.x, acc[4]); acc[5] = fmaf(wj, b.y, acc[5]);
      acc[6] = fmaf(wj, b.z, acc[6]); acc[7] = fmaf(wj, b.w, acc[7]);
    }
    if (residual) {
      const uint4 r = *reinterpret_cast<const uint4*>(residual + t * d + v * 8);
      const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
      for (int q = 0; q < 4; ++q) { acc[2 * q] += bf16_lo(rw[q]); acc[2 * q + 1] += bf16_hi(rw[q]); }
    }
    uint32_t o[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) o[q] = f32_to_bf16_bits(acc[2 * q]) | (f32_to_bf16_bits(acc[2 * q + 1]) << 16);
    *reinterpret_cast<uint4*>(out + t * d + v * 8) = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

mote_status_t launch_combine(const float* s, const float* y, const float* w, const int32_t* perm,
                             const void* residual, int64_t T, int d, int k, void* out_bf16, cudaStream_t stream,
                             bool pdl, int n_partials) {
  if (T == 0) return MOTE_OK;
  const int64_t total = T * (d / 8);
  const unsigned blocks = (unsigned)std::min<int64_t>((total + 255) / 256, 148 * 16);
  if (pdl)
    MOTE_CUDA_OK(launch_pdl(combine_kernel, dim3(blocks), dim3(256), 0, stream, s, y, w, perm,
                            static_cast<const uint16_t*>(residual), T, d, k, static_cast<uint16_t*>(out_bf16),
                            n_partials));
  else
    combine_kernel<<<blocks, 256, 0, stream>>>(s, y, w, perm, static_cast<const uint16_t*>(residual), T, d, k,
                                               static_cast<uint16_t*>(out_bf16), n_partials);
  ++g_launch_count;
  MOTE_LAUNCH_OK();
  return MOTE_OK;
}

}  // namespace mote
