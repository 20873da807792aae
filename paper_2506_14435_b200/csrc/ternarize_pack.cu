// Absmean ternary weight quantizer with INT2 packing (Eq. 7, 9, 10; storage per Section 3.1).
//
// Three launches per matrix:
//   1. abs_sum_bins    exact accumulation of sum |w|: each fp32 magnitude is split into its
//                      24-bit integer significand and its exponent; significands are added (shifted
//                      to a common unit, as integers) into 64-bit integer bins indexed by exponent.
//                      Integer adds commute, so the bins' total does not depend on thread order.
//   2. alpha_finalize  one thread adds the bins into a 384-bit integer (exact), rounds it to
//                      fp64 (nearest even), divides by m*n in fp64 and rounds once to fp32.
//   3. pack_codes      code = clamp(rint(w / alpha), -1, 1), four codes per byte.
#include <algorithm>
#include <mutex>

#include "mote_common.cuh"

namespace mote {

constexpr int kBins = 256;

// Exact sum of |w| without a warp vote per element: every thread keeps ONE 64-bit fixed-point
// accumulator in units of 2^(base - 150), where `base` is an exponent it picks from its first
// non-zero element (16 binades below it).  An element with exponent e in [base, base + 31] adds
// significand << (e - base), below 2^55, so some five hundred elements fit before a flush is needed;
// the grid gives a thread far fewer, and the flush is made anyway every 256 additions (and when a larger element moves the window up).  A flush adds
// the low 32 bits to bin `base` and the high 32 bits to bin `base + 32` (whose unit is 2^32 times
// larger): exact, and every bin stays far below 2^64.  The rare element outside the window goes
// straight to the bin of its own exponent.  All of it is integer addition, so neither the choice of
// base nor the order of threads changes the bins' total.
struct AbsAcc {
  unsigned long long acc;
  int base, count;
};

__device__ __forceinline__ void abs_acc_flush(AbsAcc& st, unsigned long long* sbins) {
  if (st.acc) {
    atomicAdd(&sbins[st.base], st.acc & 0xFFFFFFFFull);
    if (st.acc >> 32) atomicAdd(&sbins[st.base + 32], st.acc >> 32);
  }
  st.acc = 0ull;
  st.count = 0;
}

__device__ __forceinline__ void abs_acc_add(AbsAcc& st, uint32_t bits, unsigned long long* sbins) {
  const uint32_t a = bits & 0x7FFFFFFFu;
  if (a == 0u) return;
  const uint32_t e_raw = a >> 23;
  const uint32_t mant = e_raw ? ((a & 0x7FFFFFu) | 0x800000u) : a;   // subnormals: no hidden bit
  const int e = e_raw ? (int)e_raw : 1;                              // ... and the unit of exponent 1
  if (st.base < 0 || e > st.base + 31) {                             // first element, or one above the window:
    if (st.base >= 0) abs_acc_flush(st, sbins);                      // move the window up to it
    st.base = min(max(e - 16, 1), 222);                              // base + 32 must be a valid bin
  }
  const unsigned sh = (unsigned)(e - st.base);
  if (sh < 32u) {
    st.acc += (unsigned long long)mant << sh;
    if (++st.count == 256) abs_acc_flush(st, sbins);
  } else {
    atomicAdd(&sbins[e_raw], (unsigned long long)mant);              // outside the window: its own bin
  }
}

template <bool kBf16>
__global__ void __launch_bounds__(256) abs_sum_bins_kernel(const void* __restrict__ W, int64_t n_vec,
                                                           unsigned long long* __restrict__ bins) {
  __shared__ unsigned long long sbins[kBins];
  for (int i = threadIdx.x; i < kBins; i += blockDim.x) sbins[i] = 0ull;
  __syncthreads();

  // one "vec" = 4 elements (a float4, or 4 bf16 = uint2); two vecs in flight per thread
  const int64_t stride = int64_t(gridDim.x) * blockDim.x;
  AbsAcc st{0ull, -1, 0};
  for (int64_t v = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; v < n_vec; v += 2 * stride) {
    uint32_t bits[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int64_t vv = v + u * stride;
      if (vv < n_vec) {
        if (kBf16) {
          const uint2 r = reinterpret_cast<const uint2*>(W)[vv];
          bits[4 * u] = r.x << 16; bits[4 * u + 1] = r.x & 0xFFFF0000u;
          bits[4 * u + 2] = r.y << 16; bits[4 * u + 3] = r.y & 0xFFFF0000u;
        } else {
          const uint4 r = reinterpret_cast<const uint4*>(W)[vv];
          bits[4 * u] = r.x; bits[4 * u + 1] = r.y; bits[4 * u + 2] = r.z; bits[4 * u + 3] = r.w;
        }
      }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) abs_acc_add(st, bits[j], sbins);
  }
  abs_acc_flush(st, sbins);
  __syncthreads();
  for (int i = threadIdx.x; i < kBins; i += blockDim.x)
    if (sbins[i]) atomicAdd(&bins[i], sbins[i]);
}

// bins[e] counts units of 2^(max(e,1) - 150).  total = sum_e bins[e] << (max(e,1) - 1) in units
// of 2^-149.
__global__ void alpha_finalize_kernel(const unsigned long long* __restrict__ bins, double count,
                                      float* __restrict__ alpha) {
  // the warp fetches the bins together (one round trip instead of 255 dependent ones) ...
  __shared__ unsigned long long s_bins[kBins];
  for (int i = threadIdx.x; i < kBins; i += blockDim.x) s_bins[i] = bins[i];
  __syncthreads();
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  // ... and one thread adds them up
  constexpr int kLimbs = 12;
  uint32_t L[kLimbs];
  for (int i = 0; i < kLimbs; ++i) L[i] = 0u;
  for (int e = 0; e < 255; ++e) {            // e = 255 (inf/nan) is undefined input, ignored
    const unsigned long long v = s_bins[e];
    if (!v) continue;
    const int s = (e ? e : 1) - 1;
    const int wo = s >> 5, bo = s & 31;
    const unsigned __int128 sv = (unsigned __int128)v << bo;   // < 2^95
    uint32_t part[3] = {(uint32_t)sv, (uint32_t)(sv >> 32), (uint32_t)(sv >> 64)};
    unsigned long long carry = 0ull;
    for (int i = 0; i < 3; ++i) {
      unsigned long long t = (unsigned long long)L[wo + i] + part[i] + carry;
      L[wo + i] = (uint32_t)t;
      carry = t >> 32;
    }
    for (int i = wo + 3; carry && i < kLimbs; ++i) {
      unsigned long long t = (unsigned long long)L[i] + carry;
      L[i] = (uint32_t)t;
      carry = t >> 32;
    }
  }
  int top = kLimbs - 1;
  while (top >= 0 && L[top] == 0u) --top;
  double sum = 0.0;
  if (top >= 0) {
    const int msb = top * 32 + (31 - __clz(L[top]));
    auto bit = [&](int i) -> unsigned long long { return i < 0 ? 0ull : ((L[i >> 5] >> (i & 31)) & 1u); };
    if (msb <= 52) {
      unsigned long long m = 0ull;
      for (int i = msb; i >= 0; --i) m = (m << 1) | bit(i);
      sum = scalbn((double)m, -149);
    } else {
      const int sh = msb - 52;
      unsigned long long m = 0ull;
      for (int i = msb; i >= sh; --i) m = (m << 1) | bit(i);
      const unsigned long long round_bit = bit(sh - 1);
      unsigned long long sticky = 0ull;
      for (int i = sh - 2; i >= 0 && !sticky; --i) sticky |= bit(i);
      if (round_bit && (sticky || (m & 1ull))) ++m;     // nearest, ties to even
      sum = scalbn((double)m, sh - 149);
    }
  }
  const float a = (float)(sum / count);                  // fp64 divide, one rounding to fp32
  *alpha = fmaxf(a, kEpsScale);
}

template <bool kBf16>
__global__ void __launch_bounds__(256) pack_codes_kernel(const void* __restrict__ W, int64_t n_words,
                                                         const float* __restrict__ alpha_ptr,
                                                         uint32_t* __restrict__ packed) {
  const float alpha = *alpha_ptr;
  const int64_t stride = int64_t(gridDim.x) * blockDim.x;
  for (int64_t w = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; w < n_words; w += stride) {
    float v[16];
    if (kBf16) {
      const uint4* src = reinterpret_cast<const uint4*>(W) + w * 2;
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        uint4 r = src[i];
        uint32_t u[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) { v[i * 8 + 2 * j] = bf16_lo(u[j]); v[i * 8 + 2 * j + 1] = bf16_hi(u[j]); }
      }
    } else {
      const float4* src = reinterpret_cast<const float4*>(W) + w * 4;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float4 r = src[i];
        v[4 * i] = r.x; v[4 * i + 1] = r.y; v[4 * i + 2] = r.z; v[4 * i + 3] = r.w;
      }
    }
    uint32_t out = 0u;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      float c = rintf(__fdiv_rn(v[j], alpha));
      c = fminf(fmaxf(c, -1.0f), 1.0f);
      out |= uint32_t(__float2int_rn(c) + 1) << (2 * j);
    }
    packed[w] = out;
  }
}

}  // namespace mote

namespace mote {

// The quantizer's launch sequence on exponent bins that the caller owns (a workspace, or the
// library's built-in array): clear the bins, exact sum of |w|, alpha, codes.
static mote_status_t ternarize_with_bins(const void* W, int w_dtype, int64_t total, uint8_t* packed, float* alpha,
                                         unsigned long long* bins, cudaStream_t stream) {
  const int64_t n_vec = total / 4, n_words = total / 16;
  // whatever the bins held before (an earlier call's sums, or nothing defined) must go
  MOTE_CUDA_OK(cudaMemsetAsync(bins, 0, kBins * sizeof(unsigned long long), stream));
  const int threads = 256;
  const int blocks_a = (int)std::min<int64_t>((n_vec + threads - 1) / threads, 148 * 8);
  const int blocks_c = (int)std::min<int64_t>((n_words + threads - 1) / threads, 148 * 16);
  if (w_dtype == MOTE_DTYPE_BF16)
    abs_sum_bins_kernel<true><<<blocks_a, threads, 0, stream>>>(W, n_vec, bins);
  else
    abs_sum_bins_kernel<false><<<blocks_a, threads, 0, stream>>>(W, n_vec, bins);
  MOTE_LAUNCH_OK();
  alpha_finalize_kernel<<<1, 32, 0, stream>>>(bins, (double)total, alpha);
  MOTE_LAUNCH_OK();
  if (w_dtype == MOTE_DTYPE_BF16)
    pack_codes_kernel<true><<<blocks_c, threads, 0, stream>>>(W, n_words, alpha, reinterpret_cast<uint32_t*>(packed));
  else
    pack_codes_kernel<false><<<blocks_c, threads, 0, stream>>>(W, n_words, alpha, reinterpret_cast<uint32_t*>(packed));
  MOTE_LAUNCH_OK();
  return MOTE_OK;
}

}  // namespace mote

extern "C" size_t mote_ternarize_workspace_bytes(void) { return mote::kBins * sizeof(unsigned long long); }

extern "C" mote_status_t mote_ternarize_pack(const void* W, int w_dtype, int64_t m, int64_t n,
                                             uint8_t* packed, float* alpha, void* ws, size_t ws_bytes,
                                             void* stream_) {
  using namespace mote;
  if (!W || !packed || !alpha || !ws) return MOTE_ERR_NULL;
  if (w_dtype != MOTE_DTYPE_F32 && w_dtype != MOTE_DTYPE_BF16) return MOTE_ERR_DTYPE;
  if (m <= 0 || n <= 0 || (n % 16) != 0) return MOTE_ERR_SHAPE;
  if (m >= (int64_t(1) << 38) / n) return MOTE_ERR_SHAPE;
  if (!aligned16(W) || !aligned16(packed) || !aligned16(ws)) return MOTE_ERR_ALIGN;
  if (ws_bytes < mote_ternarize_workspace_bytes()) return MOTE_ERR_WORKSPACE;
  return ternarize_with_bins(W, w_dtype, m * n, packed, alpha, static_cast<unsigned long long*>(ws),
                             static_cast<cudaStream_t>(stream_));
}

// ---------------------------------------------------------------------------------------------
// mote_ternarize_pack_static: the same quantizer for callers that have no scratch buffer to give.
// The exponent bins live in a device array that is part of the loaded library image.
// ---------------------------------------------------------------------------------------------
namespace mote {

// 256 bins x 8 bytes.  One copy per GPU that loads the library, held until the process exits.
static __device__ __align__(256) unsigned long long g_static_bins[kBins];

static unsigned long long* g_static_bins_ptr[kMaxDevices];   // device address of g_static_bins, per device
static std::mutex g_static_bins_mutex;

// In host code `g_static_bins` is only a handle; the kernels need the address the array has on the
// device that is current.  It is looked up on the first call made on each device.
static mote_status_t static_bins_address(unsigned long long** out) {
  int dev = -1;
  MOTE_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return MOTE_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_static_bins_mutex);
  if (!g_static_bins_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_bins) != cudaSuccess || !p) return MOTE_ERR_CUDA;
    g_static_bins_ptr[dev] = static_cast<unsigned long long*>(p);
  }
  *out = g_static_bins_ptr[dev];
  return MOTE_OK;
}

}  // namespace mote

extern "C" mote_status_t mote_ternarize_pack_static(const void* W, int w_dtype, int64_t m, int64_t n,
                                                    uint8_t* packed, float* alpha, void* stream_) {
  using namespace mote;
  if (!W || !packed || !alpha) return MOTE_ERR_NULL;
  if (w_dtype != MOTE_DTYPE_F32 && w_dtype != MOTE_DTYPE_BF16) return MOTE_ERR_DTYPE;
  if (m <= 0 || n <= 0 || (n % 16) != 0) return MOTE_ERR_SHAPE;
  if (m > MOTE_STATIC_MAX_ELEMENTS / n) return MOTE_ERR_TOO_LARGE;
  if (!aligned16(W) || !aligned16(packed)) return MOTE_ERR_ALIGN;
  unsigned long long* bins = nullptr;
  const mote_status_t st = static_bins_address(&bins);
  if (st != MOTE_OK) return st;
  return ternarize_with_bins(W, w_dtype, m * n, packed, alpha, bins, static_cast<cudaStream_t>(stream_));
}
