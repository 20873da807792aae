// CUDA-core expert GEMMs: the shape-agnostic path (any d, f that are multiples of 16) used for
// small or odd layers and as the cross-check of the tensor-core path.
//
//   ternary gate/up (Eq. 6):  acc_g, acc_u = codes . q  (dp4a, exact int32)
//                             h = bf16(u * silu(g)),  g = fl32(acc_g)*alpha_g*(beta/127), u likewise
//   ternary down    (Eq. 5):  y = fl32(acc_d) * alpha_d*(beta_h/127)
//   shared gate/up, down (Eq. 2): bf16 operands (or RTN codes, Section 4.3), fp32 FMA accumulation
//
// Rows are in expert-sorted order; a CTA owns a 32-row x 64-column tile of one expert.
#include "mote_common.cuh"
#include "mote_internal.h"

namespace mote {

constexpr int kTM = 32;      // rows per tile
constexpr int kTN = 64;      // output columns per tile
constexpr int kTK = 64;      // reduction elements per step (int8 path)

// Finds the (expert, first row, row count) of row-tile `tile` in the ragged expert segments.
__device__ __forceinline__ bool locate_tile(const int32_t* __restrict__ offsets, int E, int tile, int tm,
                                            int& expert, int& row0, int& rows) {
  int t = tile;
  for (int e = 0; e < E; ++e) {
    const int a = offsets[e], b = offsets[e + 1];
    const int nt = (b - a + tm - 1) / tm;
    if (t < nt) {
      expert = e;
      row0 = a + t * tm;
      rows = min(tm, b - row0);
      return true;
    }
    t -= nt;
  }
  return false;
}

// 16 two-bit codes (stored code+1) -> four words of signed int8 in canonical order
__device__ __forceinline__ void unpack16_signed(uint32_t w, uint32_t out[4]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint32_t b = (w >> (8 * i)) & 0xFFu;
    const uint32_t spread = (b & 3u) | ((b & 0xCu) << 6) | ((b & 0x30u) << 12) | ((b & 0xC0u) << 18);
    out[i] = __vsub4(spread, 0x01010101u);
  }
}

template <bool kGateUp>
__global__ void __launch_bounds__(256) ternary_gemm_simt_kernel(TernaryGemmArgs a) {
  constexpr int kMats = kGateUp ? 2 : 1;
  __shared__ uint32_t As[kTM][kTK / 4 + 1];
  __shared__ uint32_t Bs[kMats * kTN][kTK / 4 + 1];

  int expert, row0, rows;
  if (!locate_tile(a.offsets, a.E, blockIdx.y, kTM, expert, row0, rows)) return;
  const int col0 = blockIdx.x * kTN;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int K = a.K, N = a.N;
  const int kw_row = K / 16;                       // packed u32 words per weight row
  const uint32_t* W0 = reinterpret_cast<const uint32_t*>(a.w0) + int64_t(expert) * N * kw_row;
  const uint32_t* W1 = kGateUp ? reinterpret_cast<const uint32_t*>(a.w1) + int64_t(expert) * N * kw_row : nullptr;

  int acc[kMats][2][4];
#pragma unroll
  for (int m = 0; m < kMats; ++m)
#pragma unroll
    for (int r = 0; r < 2; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[m][r][c] = 0;

  for (int k0 = 0; k0 < K; k0 += kTK) {
    // activations: 32 rows x 4 units of 16 bytes
    if (tid < kTM * 4) {
      const int r = tid >> 2, u = tid & 3;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (r < rows && k0 + u * 16 < K)
        v = *reinterpret_cast<const uint4*>(a.qa + int64_t(row0 + r) * K + k0 + u * 16);
      As[r][u * 4 + 0] = v.x; As[r][u * 4 + 1] = v.y; As[r][u * 4 + 2] = v.z; As[r][u * 4 + 3] = v.w;
    }
    // weights: kMats*64 rows x 4 packed words -> 16 int8 words each
    for (int i = tid; i < kMats * kTN * 4; i += 256) {
      const int wr = i >> 2, u = i & 3;
      const int m = wr / kTN, c = wr % kTN;
      uint32_t pw = 0x55555555u;                   // code 0 everywhere
      if (col0 + c < N && k0 + u * 16 < K) {
        const uint32_t* src = (m == 0 ? W0 : W1) + int64_t(col0 + c) * kw_row + (k0 / 16 + u);
        pw = *src;
      }
      uint32_t o[4];
      unpack16_signed(pw, o);
#pragma unroll
      for (int j = 0; j < 4; ++j) Bs[wr][u * 4 + j] = o[j];
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kTK / 4; ++kk) {
      const int a0 = (int)As[ty * 2][kk], a1 = (int)As[ty * 2 + 1][kk];
#pragma unroll
      for (int m = 0; m < kMats; ++m)
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int b = (int)Bs[m * kTN + tx + 16 * c][kk];
          acc[m][0][c] = __dp4a(a0, b, acc[m][0][c]);
          acc[m][1][c] = __dp4a(a1, b, acc[m][1][c]);
        }
    }
    __syncthreads();
  }

  const float al0 = a.alpha0[expert];
  const float al1 = kGateUp ? a.alpha1[expert] : 0.0f;
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int lr = ty * 2 + r;
    if (lr >= rows) continue;
    const int64_t row = row0 + lr;
    const float beta = a.beta[row];
    const float c0 = dequant_scale(al0, beta);
    const float c1 = kGateUp ? dequant_scale(al1, beta) : 0.0f;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int col = col0 + tx + 16 * c;
      if (col >= N) continue;
      if (a.acc0_tap) a.acc0_tap[row * N + col] = acc[0][r][c];
      if (kGateUp) {
        if (a.acc1_tap) a.acc1_tap[row * N + col] = acc[1][r][c];
        const float h = glu_h(acc[0][r][c], acc[1][r][c], c0, c1);
        reinterpret_cast<uint16_t*>(a.h_bf16)[row * N + col] = (uint16_t)f32_to_bf16_bits(h);
      } else {
        a.y[row * N + col] = __fmul_rn(__int2float_rn(acc[0][r][c]), c0);
      }
    }
  }
}

static mote_status_t launch_ternary_simt(const TernaryGemmArgs& a, bool gateup, cudaStream_t stream) {
  if (a.P == 0) return MOTE_OK;
  const unsigned tiles_y = (unsigned)((a.P + kTM - 1) / kTM + a.E);
  dim3 grid((a.N + kTN - 1) / kTN, tiles_y);
  if (gateup) ternary_gemm_simt_kernel<true><<<grid, 256, 0, stream>>>(a);
  else ternary_gemm_simt_kernel<false><<<grid, 256, 0, stream>>>(a);
  ++g_launch_count;
  MOTE_LAUNCH_OK();
  return MOTE_OK;
}
mote_status_t launch_ternary_gateup_simt(const TernaryGemmArgs& a, cudaStream_t s) { return launch_ternary_simt(a, true, s); }
mote_status_t launch_ternary_down_simt(const TernaryGemmArgs& a, cudaStream_t s) { return launch_ternary_simt(a, false, s); }

// ---------------------------------------------------------------------------------------------
// Shared expert, bf16 operands, fp32 accumulation.
// ---------------------------------------------------------------------------------------------
constexpr int kSK = 32;      // reduction elements per step (bf16 path)

// kBits: 16 = bf16 weights; 8 / 4 = RTN codes (Section 4.3), expanded here and scaled per output
// column after the sum.
template <int kBits>
__device__ __forceinline__ void load_w8(const void* W, int64_t row, int K, int k, float (&v)[8]) {
  if (kBits == 16) {
    const uint4 r = *reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(W) + row * K + k);
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) { v[2 * j] = bf16_lo(w[j]); v[2 * j + 1] = bf16_hi(w[j]); }
  } else if (kBits == 8) {
    const uint2 r = *reinterpret_cast<const uint2*>(static_cast<const int8_t*>(W) + row * K + k);
    const uint32_t w[2] = {r.x, r.y};
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = (float)(int8_t)((w[j >> 2] >> (8 * (j & 3))) & 0xFFu);
  } else {
    const uint32_t word = *reinterpret_cast<const uint32_t*>(static_cast<const uint8_t*>(W) + row * (K / 2) + k / 2);
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      v[2 * p] = (float)((int)((word >> (4 * p)) & 15u) - 8);
      v[2 * p + 1] = (float)((int)((word >> (16 + 4 * p)) & 15u) - 8);
    }
  }
}

template <bool kGateUp, int kBits>
__global__ void __launch_bounds__(256) shared_gemm_simt_kernel(const uint16_t* __restrict__ A, int64_t M, int K,
                                                               const void* __restrict__ W0,
                                                               const void* __restrict__ W1,
                                                               const float* __restrict__ scale0,
                                                               const float* __restrict__ scale1, int N,
                                                               uint16_t* __restrict__ h_out,
                                                               float* __restrict__ s_out) {
  constexpr int kMats = kGateUp ? 2 : 1;
  __shared__ float As[kTM][kSK + 1];
  __shared__ float Bs[kMats * kTN][kSK + 1];
  const int64_t row0 = int64_t(blockIdx.y) * kTM;
  const int col0 = blockIdx.x * kTN;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;

  float acc[kMats][2][4];
#pragma unroll
  for (int m = 0; m < kMats; ++m)
#pragma unroll
    for (int r = 0; r < 2; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[m][r][c] = 0.0f;

  for (int k0 = 0; k0 < K; k0 += kSK) {
    // A: 32 rows x 4 units of 8 bf16
    if (tid < kTM * 4) {
      const int r = tid >> 2, u = tid & 3;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (row0 + r < M && k0 + u * 8 < K)
        v = *reinterpret_cast<const uint4*>(A + (row0 + r) * K + k0 + u * 8);
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) { As[r][u * 8 + 2 * j] = bf16_lo(w[j]); As[r][u * 8 + 2 * j + 1] = bf16_hi(w[j]); }
    }
    for (int i = tid; i < kMats * kTN * 4; i += 256) {
      const int wr = i >> 2, u = i & 3;
      const int m = wr / kTN, c = wr % kTN;
      float v[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      if (col0 + c < N && k0 + u * 8 < K) load_w8<kBits>(m == 0 ? W0 : W1, col0 + c, K, k0 + u * 8, v);
#pragma unroll
      for (int j = 0; j < 8; ++j) Bs[wr][u * 8 + j] = v[j];
    }
    __syncthreads();
#pragma unroll 8
    for (int kk = 0; kk < kSK; ++kk) {
      const float a0 = As[ty * 2][kk], a1 = As[ty * 2 + 1][kk];
#pragma unroll
      for (int m = 0; m < kMats; ++m)
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const float b = Bs[m * kTN + tx + 16 * c][kk];
          acc[m][0][c] = fmaf(a0, b, acc[m][0][c]);
          acc[m][1][c] = fmaf(a1, b, acc[m][1][c]);
        }
    }
    __syncthreads();
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int64_t row = row0 + ty * 2 + r;
    if (row >= M) continue;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int col = col0 + tx + 16 * c;
      if (col >= N) continue;
      const float s0 = kBits == 16 ? 1.0f : scale0[col];
      if (kGateUp) {
        const float s1 = kBits == 16 ? 1.0f : scale1[col];
        const float g = acc[0][r][c] * s0, u = acc[1][r][c] * s1;
        const float h = u * (g / (1.0f + expf(-g)));
        h_out[row * N + col] = (uint16_t)f32_to_bf16_bits(h);
      } else {
        s_out[row * N + col] = acc[0][r][c] * s0;
      }
    }
  }
}

template <bool kGateUp>
static void launch_shared_simt(dim3 grid, cudaStream_t stream, int bits, const uint16_t* A, int64_t M, int K,
                               const void* W0, const void* W1, const float* s0, const float* s1, int N,
                               uint16_t* h_out, float* s_out) {
  if (bits == 8) shared_gemm_simt_kernel<kGateUp, 8><<<grid, 256, 0, stream>>>(A, M, K, W0, W1, s0, s1, N, h_out, s_out);
  else if (bits == 4) shared_gemm_simt_kernel<kGateUp, 4><<<grid, 256, 0, stream>>>(A, M, K, W0, W1, s0, s1, N, h_out, s_out);
  else shared_gemm_simt_kernel<kGateUp, 16><<<grid, 256, 0, stream>>>(A, M, K, W0, W1, s0, s1, N, h_out, s_out);
}

mote_status_t launch_shared_gateup_simt(const void* x, const SharedMat& Wg, const SharedMat& Wu, int bits, int64_t T,
                                        int d, int f, void* h_bf16, cudaStream_t stream) {
  if (T == 0) return MOTE_OK;
  dim3 grid((f + kTN - 1) / kTN, (unsigned)((T + kTM - 1) / kTM));
  launch_shared_simt<true>(grid, stream, bits, static_cast<const uint16_t*>(x), T, d, Wg.w, Wu.w, Wg.scale, Wu.scale,
                           f, static_cast<uint16_t*>(h_bf16), nullptr);
  ++g_launch_count;
  MOTE_LAUNCH_OK();
  return MOTE_OK;
}

mote_status_t launch_shared_down_simt(const void* h, const SharedMat& Wd, int bits, int64_t T, int d, int f, float* s,
                                      cudaStream_t stream) {
  if (T == 0) return MOTE_OK;
  dim3 grid((d + kTN - 1) / kTN, (unsigned)((T + kTM - 1) / kTM));
  launch_shared_simt<false>(grid, stream, bits, static_cast<const uint16_t*>(h), T, f, Wd.w, nullptr, Wd.scale, nullptr,
                            d, nullptr, s);
  ++g_launch_count;
  MOTE_LAUNCH_OK();
  return MOTE_OK;
}

}  // namespace mote
