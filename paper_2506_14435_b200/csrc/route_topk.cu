// Router of Eq. 3: fp32 logits, top-k selection, gate weights.
//
// Two kernels.  route_topk_mma_kernel (d % 32 == 0) computes the logits of 16 tokens per CTA on
// the tensor cores; route_topk_simt_kernel covers every other width.
//
// CUDA-core kernel: one warp owns kRouteTok consecutive tokens; its lanes split the hidden dimension in units of 8
// elements.  Every router-weight vector a lane loads is used for all of the warp's tokens, which
// cuts the L1 traffic of the (L2-resident) router matrix by that factor; x is read once from HBM
// (the second pass of a row, for more than kRouteChunk experts, hits L1).  Products bf16 x
// bf16-representable weight are exact in fp32; only the additions round.
#include "mote_common.cuh"
#include "mote_internal.h"

namespace mote {

constexpr int kRouteChunk = 8;   // experts accumulated per pass over the rows
constexpr int kRouteTok = 4;     // tokens per warp
constexpr int kRouteWarps = 4;   // warps per CTA

__global__ void __launch_bounds__(kRouteWarps * 32) route_topk_simt_kernel(const uint16_t* __restrict__ x, int64_t T, int d,
                                                                    const float* __restrict__ Wr,
                                                                    const float* __restrict__ bias, int E, int k,
                                                                    int norm_topk, int32_t* __restrict__ idx_out,
                                                                    float* __restrict__ w_out,
                                                                    float* __restrict__ logits_out) {
  __shared__ float s_logits[kRouteWarps][kRouteTok][MOTE_MAX_EXPERTS];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t t0 = (int64_t(blockIdx.x) * kRouteWarps + warp) * kRouteTok;
  if (t0 >= T) return;                     // whole warp leaves together; no block-wide barrier below
  const uint4* xr[kRouteTok];
#pragma unroll
  for (int i = 0; i < kRouteTok; ++i)      // rows past the end alias the last row; their results are dropped
    xr[i] = reinterpret_cast<const uint4*>(x + min(t0 + i, T - 1) * int64_t(d));
  const int n_vec = d / 8;

  for (int e0 = 0; e0 < E; e0 += kRouteChunk) {
    float acc[kRouteTok][kRouteChunk];
#pragma unroll
    for (int i = 0; i < kRouteTok; ++i)
#pragma unroll
      for (int c = 0; c < kRouteChunk; ++c) acc[i][c] = 0.0f;
    for (int v = lane; v < n_vec; v += 32) {
      float xv[kRouteTok][8];
#pragma unroll
      for (int i = 0; i < kRouteTok; ++i) {
        const uint4 r = xr[i][v];
        xv[i][0] = bf16_lo(r.x); xv[i][1] = bf16_hi(r.x); xv[i][2] = bf16_lo(r.y); xv[i][3] = bf16_hi(r.y);
        xv[i][4] = bf16_lo(r.z); xv[i][5] = bf16_hi(r.z); xv[i][6] = bf16_lo(r.w); xv[i][7] = bf16_hi(r.w);
      }
#pragma unroll
      for (int c = 0; c < kRouteChunk; ++c) {
        if (e0 + c < E) {
          const float4* wp = reinterpret_cast<const float4*>(Wr + int64_t(e0 + c) * d + v * 8);
          const float4 a = wp[0], b = wp[1];
#pragma unroll
          for (int i = 0; i < kRouteTok; ++i) {
            float s = acc[i][c];
            s = fmaf(xv[i][0], a.x, s); s = fmaf(xv[i][1], a.y, s); s = fmaf(xv[i][2], a.z, s); s = fmaf(xv[i][3], a.w, s);
            s = fmaf(xv[i][4], b.x, s); s = fmaf(xv[i][5], b.y, s); s = fmaf(xv[i][6], b.z, s); s = fmaf(xv[i][7], b.w, s);
            acc[i][c] = s;
          }
        }
      }
    }
#pragma unroll
    for (int i = 0; i < kRouteTok; ++i)
#pragma unroll
      for (int c = 0; c < kRouteChunk; ++c) {
        const float s = warp_sum(acc[i][c]);
        if (lane == 0 && e0 + c < E) s_logits[warp][i][e0 + c] = s + (bias ? bias[e0 + c] : 0.0f);
      }
  }
  __syncwarp();

  for (int i = 0; i < kRouteTok; ++i) {
    const int64_t t = t0 + i;
    if (t >= T) break;
    // each lane owns experts lane and lane+32
    float l0 = lane < E ? s_logits[warp][i][lane] : -INFINITY;
    float l1 = lane + 32 < E ? s_logits[warp][i][lane + 32] : -INFINITY;
    if (logits_out) {
      if (lane < E) logits_out[t * E + lane] = l0;
      if (lane + 32 < E) logits_out[t * E + lane + 32] = l1;
    }
    const float lmax = warp_max(fmaxf(l0, l1));
    float denom_all = 0.0f;
    if (!norm_topk) {
      float part = (lane < E ? expf(l0 - lmax) : 0.0f) + (lane + 32 < E ? expf(l1 - lmax) : 0.0f);
      denom_all = warp_sum(part);
    }

    float sel_l[MOTE_MAX_TOPK];
    int sel_i[MOTE_MAX_TOPK];
#pragma unroll
    for (int j = 0; j < MOTE_MAX_TOPK; ++j) {
      if (j < k) {
        // arg-max over the warp; equal logits resolve to the lower expert index
        float bv = l0; int bi = lane;
        if (l1 > bv) { bv = l1; bi = lane + 32; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
          const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
          if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
        }
        sel_l[j] = bv; sel_i[j] = bi;
        if (bi == lane) l0 = -INFINITY;
        if (bi == lane + 32) l1 = -INFINITY;
      }
    }
    if (lane == 0) {
      float ex[MOTE_MAX_TOPK];
      float denom = 0.0f;
#pragma unroll
      for (int j = 0; j < MOTE_MAX_TOPK; ++j)
        if (j < k) { ex[j] = expf(sel_l[j] - lmax); denom += ex[j]; }
      if (!norm_topk) denom = denom_all;
#pragma unroll
      for (int j = 0; j < MOTE_MAX_TOPK; ++j)
        if (j < k) {
          idx_out[t * k + j] = sel_i[j];
          w_out[t * k + j] = ex[j] / denom;
        }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Tensor-core logits.  logits[16 tokens, E] = x[16, d] * Wr[E, d]^T as warp-level bf16 MMAs
// (m16n8k16, fp32 accumulation).  x is bf16 already.  A router weight w (fp32) is split exactly
// into three bf16 terms, w = hi + mid + lo (hi = w with the low 16 bits cleared, mid the same of
// w - hi, lo the rest: 8 + 8 + 8 significand bits), each term feeding its own MMA, so nothing of w
// is lost; for weights that are bf16 values to begin with mid = lo = 0.
// The 8 warps of a CTA split d; lane (g, t) loads elements [32*step + 8*t, +8) of token rows g
// and g+8 and of weight row 8*n + g (the reduction index may be permuted freely as long as both
// operands use the same permutation).  Partial sums are added across warps in warp order.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// upper halves of two floats -> bf16x2 (first in the low half)
__device__ __forceinline__ uint32_t hi16_pair(float a, float b) {
  return __byte_perm(__float_as_uint(a), __float_as_uint(b), 0x7632);
}

constexpr int kRmWarps = 8;

template <int NE>   // 8-expert column tiles: ceil(E / 8) rounded up to 1, 2, 4 or 8
__global__ void __launch_bounds__(kRmWarps * 32, NE <= 2 ? 4 : 0) route_topk_mma_kernel(const uint16_t* __restrict__ x, int64_t T, int d,
                                                                     const float* __restrict__ Wr,
                                                                     const float* __restrict__ bias, int E, int k,
                                                                     int norm_topk, int32_t* __restrict__ idx_out,
                                                                     float* __restrict__ w_out,
                                                                     float* __restrict__ logits_out,
                                                                     int32_t* __restrict__ blk_hist,
                                                                     uint32_t* __restrict__ zero_word) {
  __shared__ float s_part[kRmWarps][NE * 4][32];
  __shared__ float s_logits[16][NE * 8];
  __shared__ int s_hist[NE * 8];                      // pairs per expert among this CTA's 16 tokens
  if (threadIdx.x < NE * 8) s_hist[threadIdx.x] = 0;
  // first kernel of a layer call on the tensor path: clears the call's device status word
  if (zero_word && blockIdx.x == 0 && threadIdx.x == 0) *zero_word = 0u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int64_t t0 = int64_t(blockIdx.x) * 16;
  const uint16_t* xa = x + min(t0 + g, T - 1) * int64_t(d) + t * 8;       // rows past the end alias the last row
  const uint16_t* xb = x + min(t0 + g + 8, T - 1) * int64_t(d) + t * 8;
  const float* wrow[NE];
#pragma unroll
  for (int n = 0; n < NE; ++n) wrow[n] = Wr + int64_t(min(n * 8 + g, E - 1)) * d + t * 8;

  float acc[NE][4];
#pragma unroll
  for (int n = 0; n < NE; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.0f;

  const int n_steps = d / 32;
  const int base = n_steps / kRmWarps, rem = n_steps % kRmWarps;
  const int sb = warp * base + min(warp, rem), se = sb + base + (warp < rem ? 1 : 0);
  // token loads in flight per lane; two for E > 8 keep the kernel at 64 registers, i.e. four CTAs per
  // SM, so that the 512 CTAs of an 8192-token prefill are resident at once (router 38 -> 24 us there)
  constexpr int kAhead = (NE >= 2) ? 2 : 4;
  uint4 ra[kAhead], rb[kAhead];
#pragma unroll
  for (int i = 0; i < kAhead; ++i) {
    const bool in = sb + i < se;
    ra[i] = in ? *reinterpret_cast<const uint4*>(xa + (sb + i) * 32) : make_uint4(0u, 0u, 0u, 0u);
    rb[i] = in ? *reinterpret_cast<const uint4*>(xb + (sb + i) * 32) : make_uint4(0u, 0u, 0u, 0u);
  }
  for (int s0 = sb; s0 < se; s0 += kAhead) {
#pragma unroll
    for (int i = 0; i < kAhead; ++i) {
      const int s = s0 + i;
      if (s < se) {
        const uint4 ca = ra[i], cb = rb[i];
        if (s + kAhead < se) {
          ra[i] = *reinterpret_cast<const uint4*>(xa + (s + kAhead) * 32);
          rb[i] = *reinterpret_cast<const uint4*>(xb + (s + kAhead) * 32);
        }
#pragma unroll
        for (int n = 0; n < NE; ++n) {
          const float4 w0 = *reinterpret_cast<const float4*>(wrow[n] + s * 32);
          const float4 w1 = *reinterpret_cast<const float4*>(wrow[n] + s * 32 + 4);
          const float w[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
          float hi[8], mid[8], lo[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            hi[j] = __uint_as_float(__float_as_uint(w[j]) & 0xFFFF0000u);
            const float r1 = __fsub_rn(w[j], hi[j]);
            mid[j] = __uint_as_float(__float_as_uint(r1) & 0xFFFF0000u);
            lo[j] = __fsub_rn(r1, mid[j]);
          }
          mma_bf16_16816(acc[n], ca.x, cb.x, ca.y, cb.y, hi16_pair(hi[0], hi[1]), hi16_pair(hi[2], hi[3]));
          mma_bf16_16816(acc[n], ca.z, cb.z, ca.w, cb.w, hi16_pair(hi[4], hi[5]), hi16_pair(hi[6], hi[7]));
          mma_bf16_16816(acc[n], ca.x, cb.x, ca.y, cb.y, hi16_pair(mid[0], mid[1]), hi16_pair(mid[2], mid[3]));
          mma_bf16_16816(acc[n], ca.z, cb.z, ca.w, cb.w, hi16_pair(mid[4], mid[5]), hi16_pair(mid[6], mid[7]));
          mma_bf16_16816(acc[n], ca.x, cb.x, ca.y, cb.y, hi16_pair(lo[0], lo[1]), hi16_pair(lo[2], lo[3]));
          mma_bf16_16816(acc[n], ca.z, cb.z, ca.w, cb.w, hi16_pair(lo[4], lo[5]), hi16_pair(lo[6], lo[7]));
        }
      }
    }
  }
#pragma unroll
  for (int n = 0; n < NE; ++n)
#pragma unroll
    for (int i = 0; i < 4; ++i) s_part[warp][n * 4 + i][lane] = acc[n][i];
  __syncthreads();
  // fragment: value i of column tile n at lane (g, t) is token row g + 8*(i/2), expert 8n + 2t + (i&1)
  for (int v = warp; v < NE * 4; v += kRmWarps) {
    float z = s_part[0][v][lane];
#pragma unroll
    for (int w = 1; w < kRmWarps; ++w) z += s_part[w][v][lane];
    const int n = v >> 2, i = v & 3;
    const int e = n * 8 + 2 * t + (i & 1);
    s_logits[g + 8 * (i >> 1)][e] = z + ((bias && e < E) ? bias[e] : 0.0f);
  }
  __syncthreads();

  for (int r = warp; r < 16; r += kRmWarps) {
    const int64_t tok = t0 + r;
    if (tok >= T) break;
    // each lane owns experts lane and lane+32
    float l0 = lane < E ? s_logits[r][lane] : -INFINITY;
    float l1 = (NE > 4 && lane + 32 < E) ? s_logits[r][(lane + 32) % (NE * 8)] : -INFINITY;
    if (logits_out) {
      if (lane < E) logits_out[tok * E + lane] = l0;
      if (lane + 32 < E) logits_out[tok * E + lane + 32] = l1;
    }
    const float lmax = warp_max(fmaxf(l0, l1));
    float denom_all = 0.0f;
    if (!norm_topk) {
      float part = (lane < E ? expf(l0 - lmax) : 0.0f) + (lane + 32 < E ? expf(l1 - lmax) : 0.0f);
      denom_all = warp_sum(part);
    }
    float sel_l[MOTE_MAX_TOPK];
    int sel_i[MOTE_MAX_TOPK];
#pragma unroll
    for (int j = 0; j < MOTE_MAX_TOPK; ++j) {
      if (j < k) {
        float bv = l0; int bi = lane;                  // equal logits resolve to the lower expert index
        if (l1 > bv) { bv = l1; bi = lane + 32; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
          const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
          if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
        }
        sel_l[j] = bv; sel_i[j] = bi;
        if (bi == lane) l0 = -INFINITY;
        if (bi == lane + 32) l1 = -INFINITY;
      }
    }
    if (lane == 0) {
      float ex[MOTE_MAX_TOPK];
      float denom = 0.0f;
#pragma unroll
      for (int j = 0; j < MOTE_MAX_TOPK; ++j)
        if (j < k) { ex[j] = expf(sel_l[j] - lmax); denom += ex[j]; }
      if (!norm_topk) denom = denom_all;
#pragma unroll
      for (int j = 0; j < MOTE_MAX_TOPK; ++j)
        if (j < k) {
          idx_out[tok * k + j] = sel_i[j];
          w_out[tok * k + j] = ex[j] / denom;
          atomicAdd(&s_hist[sel_i[j]], 1);
        }
    }
  }
  if (blk_hist) {                                      // input of the block-wise dispatch (dispatch.cu)
    __syncthreads();
    if (threadIdx.x < E) blk_hist[int64_t(threadIdx.x) * blk_stride((int)gridDim.x) + blockIdx.x] = s_hist[threadIdx.x];
  }
}

mote_status_t launch_route_topk(const void* x, int64_t T, int d, const float* Wr, const float* bias, int E,
                                int k, int norm_topk, int32_t* idx, float* w, float* logits, int32_t* blk_hist,
                                cudaStream_t stream, uint32_t* zero_word) {
  if (T == 0) return MOTE_OK;
  const uint16_t* xp = static_cast<const uint16_t*>(x);
  if (d % 32 == 0) {
    const unsigned blocks = (unsigned)((T + 15) / 16);
    const int ne = (E + 7) / 8;
    if (ne <= 1) route_topk_mma_kernel<1><<<blocks, kRmWarps * 32, 0, stream>>>(xp, T, d, Wr, bias, E, k, norm_topk, idx, w, logits, blk_hist, zero_word);
    else if (ne <= 2) route_topk_mma_kernel<2><<<blocks, kRmWarps * 32, 0, stream>>>(xp, T, d, Wr, bias, E, k, norm_topk, idx, w, logits, blk_hist, zero_word);
    else if (ne <= 4) route_topk_mma_kernel<4><<<blocks, kRmWarps * 32, 0, stream>>>(xp, T, d, Wr, bias, E, k, norm_topk, idx, w, logits, blk_hist, zero_word);
    else route_topk_mma_kernel<8><<<blocks, kRmWarps * 32, 0, stream>>>(xp, T, d, Wr, bias, E, k, norm_topk, idx, w, logits, blk_hist, zero_word);
  } else {
    const int per_cta = kRouteWarps * kRouteTok;
    const unsigned blocks = (unsigned)((T + per_cta - 1) / per_cta);
    route_topk_simt_kernel<<<blocks, kRouteWarps * 32, 0, stream>>>(xp, T, d, Wr, bias, E, k, norm_topk, idx, w, logits);
  }
  ++g_launch_count;
  MOTE_LAUNCH_OK();
  return MOTE_OK;
}

}  // namespace mote

namespace mote {

// Per-expert factors of the load-balancing loss (Eq. 12): one CTA per expert walks the batch in a
// fixed order (thread-strided partial sums, then a fixed tree), so the sums are reproducible.
__global__ void __launch_bounds__(256) route_stats_kernel(const float* __restrict__ logits,
                                                          const int32_t* __restrict__ idx, int64_t T, int E, int k,
                                                          int32_t* __restrict__ tokens_per_expert,
                                                          float* __restrict__ prob_sum) {
  __shared__ float s_p[8];
  __shared__ int s_c[8];
  const int e = blockIdx.x;
  float p = 0.0f;
  int c = 0;
  for (int64_t t = threadIdx.x; t < T; t += blockDim.x) {
    const float* l = logits + t * E;
    float m = l[0];
    for (int j = 1; j < E; ++j) m = fmaxf(m, l[j]);
    float den = 0.0f;
    for (int j = 0; j < E; ++j) den += expf(l[j] - m);
    p += expf(l[e] - m) / den;
    for (int j = 0; j < k; ++j) c += (idx[t * k + j] == e) ? 1 : 0;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    p += __shfl_xor_sync(0xffffffffu, p, o);
    c += __shfl_xor_sync(0xffffffffu, c, o);
  }
  if ((threadIdx.x & 31) == 0) { s_p[threadIdx.x >> 5] = p; s_c[threadIdx.x >> 5] = c; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float ps = 0.0f;
    int cs = 0;
    for (int w = 0; w < 8; ++w) { ps += s_p[w]; cs += s_c[w]; }
    prob_sum[e] = ps;
    tokens_per_expert[e] = cs;
  }
}

}  // namespace mote

extern "C" mote_status_t mote_route_stats(const float* logits, const int32_t* topk_idx, int64_t T, int E, int k,
                                          int32_t* tokens_per_expert, float* prob_sum, void* stream) {
  using namespace mote;
  if (T < 0 || E < 1 || E > MOTE_MAX_EXPERTS || k < 1 || k > E || k > MOTE_MAX_TOPK) return MOTE_ERR_SHAPE;
  if (!tokens_per_expert || !prob_sum) return MOTE_ERR_NULL;
  if (T > 0 && (!logits || !topk_idx)) return MOTE_ERR_NULL;
  route_stats_kernel<<<E, 256, 0, static_cast<cudaStream_t>(stream)>>>(logits, topk_idx, T, E, k, tokens_per_expert,
                                                                       prob_sum);
  MOTE_LAUNCH_OK();
  return MOTE_OK;
}

extern "C" mote_status_t mote_route_topk(const void* x_bf16, int64_t T, int64_t d, const float* Wr,
                                         const float* bias, int E, int k, int norm_topk, int32_t* topk_idx,
                                         float* topk_w, float* logits, void* stream) {
  using namespace mote;
  if (T < 0 || d <= 0 || (d % 8) != 0 || d > (1 << 20)) return MOTE_ERR_SHAPE;
  if (E < 1 || E > MOTE_MAX_EXPERTS || k < 1 || k > E || k > MOTE_MAX_TOPK) return MOTE_ERR_SHAPE;
  if (T == 0) return MOTE_OK;
  if (!x_bf16 || !Wr || !topk_idx || !topk_w) return MOTE_ERR_NULL;
  if (!aligned16(x_bf16) || !aligned16(Wr)) return MOTE_ERR_ALIGN;
  return launch_route_topk(x_bf16, T, (int)d, Wr, bias, E, k, norm_topk, topk_idx, topk_w, logits, nullptr,
                           static_cast<cudaStream_t>(stream));
}
