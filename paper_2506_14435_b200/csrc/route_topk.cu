// Router of Eq. 3: fp32 logits, top-k selection, gate weights.
//
// One warp owns kRouteTok consecutive tokens; its lanes split the hidden dimension in units of 8
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

__global__ void __launch_bounds__(kRouteWarps * 32) route_topk_kernel(const uint16_t* __restrict__ x, int64_t T, int d,
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

mote_status_t launch_route_topk(const void* x, int64_t T, int d, const float* Wr, const float* bias, int E,
                                int k, int norm_topk, int32_t* idx, float* w, float* logits,
                                cudaStream_t stream) {
  if (T == 0) return MOTE_OK;
  const int per_cta = kRouteWarps * kRouteTok;
  const unsigned blocks = (unsigned)((T + per_cta - 1) / per_cta);
  route_topk_kernel<<<blocks, kRouteWarps * 32, 0, stream>>>(static_cast<const uint16_t*>(x), T, d, Wr, bias, E, k,
                                                norm_topk, idx, w, logits);
  ++g_launch_count;
  MOTE_LAUNCH_OK();
  return MOTE_OK;
}

}  // namespace mote

extern "C" mote_status_t mote_route_topk(const void* x_bf16, int64_t T, int64_t d, const float* Wr,
                                         const float* bias, int E, int k, int norm_topk, int32_t* topk_idx,
                                         float* topk_w, float* logits, void* stream) {
  using namespace mote;
  if (T < 0 || d <= 0 || (d % 8) != 0 || d > (1 << 20)) return MOTE_ERR_SHAPE;
  if (E < 1 || E > MOTE_MAX_EXPERTS || k < 1 || k > E || k > MOTE_MAX_TOPK) return MOTE_ERR_SHAPE;
  if (T == 0) return MOTE_OK;
  if (!x_bf16 || !Wr || !topk_idx || !topk_w) return MOTE_ERR_NULL;
  if (!aligned16(x_bf16) || !aligned16(Wr)) return MOTE_ERR_ALIGN;
  return launch_route_topk(x_bf16, T, (int)d, Wr, bias, E, k, norm_topk, topk_idx, topk_w, logits,
                           static_cast<cudaStream_t>(stream));
}
