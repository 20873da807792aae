// RTN absmax weight quantizer of the shared expert (Section 4.3): one scale per output row,
// INT8 or INT4 codes.  Offline step: one CTA per row, two passes over the row (absmax, codes).
#include "mote_common.cuh"
#include "mote_internal.h"

namespace mote {

// 8 consecutive elements of a row as fp32
template <bool kBf16>
__device__ __forceinline__ void load8(const void* row, int j, float (&v)[8]) {
  if (kBf16) {
    const uint4 r = *reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(row) + j);
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) { v[2 * i] = bf16_lo(w[i]); v[2 * i + 1] = bf16_hi(w[i]); }
  } else {
    const float4 a = *reinterpret_cast<const float4*>(static_cast<const float*>(row) + j);
    const float4 b = *reinterpret_cast<const float4*>(static_cast<const float*>(row) + j + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  }
}

template <bool kBf16>
__global__ void __launch_bounds__(256) rtn_quant_kernel(const void* __restrict__ W, int64_t m, int n, int bits,
                                                        uint8_t* __restrict__ q, float* __restrict__ scale) {
  __shared__ float s_max[8];
  const int64_t r = blockIdx.x;
  const void* row = static_cast<const char*>(W) + r * n * (kBf16 ? 2 : 4);
  float amax = 0.0f;
  for (int j = threadIdx.x * 8; j < n; j += 256 * 8) {
    float v[8];
    load8<kBf16>(row, j, v);
#pragma unroll
    for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(v[i]));
  }
  amax = warp_max(amax);
  if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = amax;
  __syncthreads();
  amax = s_max[0];
#pragma unroll
  for (int w = 1; w < 8; ++w) amax = fmaxf(amax, s_max[w]);
  const float beta = fmaxf(amax, kEpsScale);
  const float qmax = bits == 8 ? 127.0f : 7.0f;
  if (threadIdx.x == 0) scale[r] = __fdiv_rn(beta, qmax);
  for (int j = threadIdx.x * 8; j < n; j += 256 * 8) {
    float v[8];
    load8<kBf16>(row, j, v);
    int c[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float t = rintf(__fdiv_rn(__fmul_rn(qmax, v[i]), beta));
      c[i] = (int)fminf(fmaxf(t, -qmax), qmax);
    }
    if (bits == 8) {
      uint2 o;
      o.x = (uint32_t)(c[0] & 0xFF) | ((uint32_t)(c[1] & 0xFF) << 8) | ((uint32_t)(c[2] & 0xFF) << 16) |
            ((uint32_t)(c[3] & 0xFF) << 24);
      o.y = (uint32_t)(c[4] & 0xFF) | ((uint32_t)(c[5] & 0xFF) << 8) | ((uint32_t)(c[6] & 0xFF) << 16) |
            ((uint32_t)(c[7] & 0xFF) << 24);
      *reinterpret_cast<uint2*>(q + r * n + j) = o;
    } else {
      uint32_t word = 0u;
#pragma unroll
      for (int p = 0; p < 4; ++p) {
        word |= (uint32_t)(c[2 * p] + 8) << (4 * p);
        word |= (uint32_t)(c[2 * p + 1] + 8) << (16 + 4 * p);
      }
      *reinterpret_cast<uint32_t*>(q + r * (n / 2) + j / 2) = word;
    }
  }
}

}  // namespace mote

using namespace mote;

extern "C" mote_status_t mote_rtn_quant(const void* W, int w_dtype, int64_t m, int64_t n, int bits, void* q,
                                        float* scale, void* stream_) {
  if (!W || !q || !scale) return MOTE_ERR_NULL;
  if (w_dtype != MOTE_DTYPE_F32 && w_dtype != MOTE_DTYPE_BF16) return MOTE_ERR_DTYPE;
  if (m <= 0 || n <= 0 || n % 16 != 0 || n > 65536 || m > (int64_t(1) << 31) - 1 || (bits != 8 && bits != 4))
    return MOTE_ERR_SHAPE;
  if (!aligned16(W) || !aligned16(q)) return MOTE_ERR_ALIGN;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (w_dtype == MOTE_DTYPE_BF16)
    rtn_quant_kernel<true><<<(unsigned)m, 256, 0, stream>>>(W, m, (int)n, bits, static_cast<uint8_t*>(q), scale);
  else
    rtn_quant_kernel<false><<<(unsigned)m, 256, 0, stream>>>(W, m, (int)n, bits, static_cast<uint8_t*>(q), scale);
  MOTE_LAUNCH_OK();
  return MOTE_OK;
}
