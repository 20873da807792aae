// Decode path (up to 64 tokens): the layer as a weight stream.
//
// With a handful of tokens every expert matrix is read once and used for a few dot products
// per row: the layer is bound by HBM, by the 2-bit codes of the experts that were selected
// (3*d*f/4 bytes each) and the bf16 weights of the shared expert (6*d*f bytes).  The kernels here
// never stage weights in shared memory: each lane loads 16 bytes of one weight row straight from
// global memory into registers, expands the 2-bit codes there (one shift and one mask per four
// codes) and feeds them to warp-level tensor-core MMAs (mma.sync m16n8k32 u8 x s8 -> s32 for the
// ternary experts, m16n8k16 bf16 for the shared expert -- whose weights are bf16, or RTN INT8/INT4
// codes (Section 4.3) expanded to bf16 in registers) as the A operand, with the tokens as the
// 8-wide B operand.  The reduction index of an integer dot product can be permuted freely, so a
// lane's 64 consecutive codes need no shuffling: the token operand is stored in the matching
// ("k-interleaved") order by the quantizer.
//
//   decode_prologue   one CTA per token: Q_a(x) (Eq. 8), router logits, top-k and gate weights
//                     (Eq. 3); the last CTA to finish builds the dispatch tables
//   decode_gateup     routed gate/up (Eq. 6) + shared gate/up (Eq. 2): h, row maxima of h, h_shared
//   (Q_a(h): quant_rows_known_beta_kernel of quant_act.cu)
//   decode_down       routed down (Eq. 5) + shared down: y, s; the CTA that finishes the last item
//                     of a 16-column tile combines it (Eq. 2, Eq. 4) and writes the layer output
#include <algorithm>

#include "mote_common.cuh"
#include "mote_internal.h"

namespace mote {

constexpr int kDecodeMaxTokens = 64;
constexpr int kDecodeMaxPairs = kDecodeMaxTokens * MOTE_MAX_TOPK;

// ------------------------------------------------------------------------------------------------
// small device helpers
// ------------------------------------------------------------------------------------------------
// weights are read exactly once: keep them out of L1, which serves the token operand
__device__ __forceinline__ uint4 ldg_stream16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// D(16x8, s32) += A(16x32, u8, row) * B(32x8, s8, col)
__device__ __forceinline__ void mma_u8s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// D(16x8, f32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// ------------------------------------------------------------------------------------------------
// decode_prologue: Q_a(x), router, dispatch
// ------------------------------------------------------------------------------------------------
struct DecodePrologueArgs {
  const uint16_t* x;      // [T, d] bf16
  int T, d, E, k, norm_topk;
  const float* Wr;        // [E, d]
  const float* bias;      // [E] or null
  int32_t* topk_idx;      // [T*k]
  float* topk_w;          // [T*k]
  int8_t* qx;             // [T, d] token order, k-interleaved units
  float* beta_x;          // [T]
  int32_t* rowsum_x;      // [T]
  uint32_t* beta_h_bits;  // [T*k] zeroed here
  int32_t* rowsum_h;      // [T*k] zeroed here
  uint32_t* counter;      // zero on entry; left at zero
  int zero_head_words;    // single-token call: words to zero from (counter - 1) on, see below; else 0
  int32_t* offsets;       // [E+1]
  int32_t* perm;          // [T*k]
  int32_t* inv;           // [T*k]
};

__global__ void __launch_bounds__(256) decode_prologue_kernel(DecodePrologueArgs a) {
  extern __shared__ uint4 s_x4[];                      // the token row, bf16
  __shared__ float s_red[8];
  __shared__ int s_redi[8];
  __shared__ float s_logits[MOTE_MAX_EXPERTS];
  __shared__ float s_part[8][8];
  __shared__ int s_last;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int t = blockIdx.x;
  const int d = a.d, n_vec = d / 8, n_units = d / 16;
  const uint4* src = reinterpret_cast<const uint4*>(a.x + int64_t(t) * d);

  // The router weights do not depend on the token: the first pass's rows for this thread's first
  // unit are requested now, and the later passes' rows are pulled into L2, so that their latency
  // runs under the absmax / Q_a(x) phase instead of after it.
  float4 wp0[8], wq0[8];
  if (tid < n_vec) {
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const float4* wr = reinterpret_cast<const float4*>(a.Wr + int64_t(min(c, a.E - 1)) * d) + 2 * tid;
      wp0[c] = wr[0]; wq0[c] = wr[1];
    }
    for (int e = 8; e < a.E; ++e)
      asm volatile("prefetch.global.L2 [%0];" ::"l"(a.Wr + int64_t(e) * d + 8 * tid));
  }
  // x may be the output of the kernel ahead (the RMS norm of a layer stack, launched as this kernel's
  // programmatic predecessor).  Only then may the gate/up kernel start on the shared expert, which
  // reads x too.
  pdl_wait();
  pdl_trigger();
  // A single-token call has one prologue CTA and does not use the arrival counter, so this CTA can
  // zero the head of the workspace (status word, counter, the down kernel's tile counters: first
  // touched by the down kernel, which starts after this kernel has completed) instead of a memset
  // ahead of the launch.
  for (int i = tid; i < a.zero_head_words; i += 256) (a.counter - 1)[i] = 0u;

  float amax = 0.0f;
  for (int v = tid; v < n_vec; v += 256) {
    const uint4 r = src[v];
    s_x4[v] = r;
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) amax = fmaxf(amax, fmaxf(fabsf(bf16_lo(w[j])), fabsf(bf16_hi(w[j]))));
  }
  amax = warp_max(amax);
  if (lane == 0) s_red[warp] = amax;
  __syncthreads();
  amax = s_red[0];
#pragma unroll
  for (int i = 1; i < 8; ++i) amax = fmaxf(amax, s_red[i]);
  const float beta = fmaxf(amax, kEpsScale);
  const QaScale qs = qa_scale(beta);

  // Q_a(x): units of 16 elements, stored k-interleaved
  int local_sum = 0;
  uint4* qdst = reinterpret_cast<uint4*>(a.qx + int64_t(t) * d);
  for (int u = tid; u < n_units; u += 256) {
    const uint4 r0 = s_x4[2 * u], r1 = s_x4[2 * u + 1];
    const uint32_t w[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
    uint32_t q[16];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      q[2 * j] = quant_byte(bf16_lo(w[j]), qs);
      q[2 * j + 1] = quant_byte(bf16_hi(w[j]), qs);
    }
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      o[i] = pack_low_bytes(q[i], q[4 + i], q[8 + i], q[12 + i]);
      local_sum = __dp4a((int)o[i], 0x01010101, local_sum);
    }
    qdst[u] = make_uint4(o[0], o[1], o[2], o[3]);
  }
  local_sum = warp_sum(local_sum);
  if (lane == 0) s_redi[warp] = local_sum;

  // router logits: every thread takes units of 8 elements, 8 experts per pass; the 16 weight loads
  // of a pass are independent, so a pass costs one memory round trip
  for (int e0 = 0; e0 < a.E; e0 += 8) {
    float acc[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[c] = 0.0f;
    for (int v = tid; v < n_vec; v += 256) {
      const uint4 r = s_x4[v];
      const float xv[8] = {bf16_lo(r.x), bf16_hi(r.x), bf16_lo(r.y), bf16_hi(r.y),
                           bf16_lo(r.z), bf16_hi(r.z), bf16_lo(r.w), bf16_hi(r.w)};
      float4 wp[8], wq[8];
      if (e0 == 0 && v == tid) {
#pragma unroll
        for (int c = 0; c < 8; ++c) { wp[c] = wp0[c]; wq[c] = wq0[c]; }
      } else {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const float4* wr = reinterpret_cast<const float4*>(a.Wr + int64_t(min(e0 + c, a.E - 1)) * d) + 2 * v;
          wp[c] = wr[0]; wq[c] = wr[1];
        }
      }
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        float z = acc[c];
        z = fmaf(xv[0], wp[c].x, z); z = fmaf(xv[1], wp[c].y, z); z = fmaf(xv[2], wp[c].z, z); z = fmaf(xv[3], wp[c].w, z);
        z = fmaf(xv[4], wq[c].x, z); z = fmaf(xv[5], wq[c].y, z); z = fmaf(xv[6], wq[c].z, z); z = fmaf(xv[7], wq[c].w, z);
        acc[c] = z;
      }
    }
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const float z = warp_sum(acc[c]);
      if (lane == 0) s_part[warp][c] = z;
    }
    __syncthreads();
    if (tid < 8 && e0 + tid < a.E) {
      float z = s_part[0][tid];
#pragma unroll
      for (int w = 1; w < 8; ++w) z += s_part[w][tid];
      s_logits[e0 + tid] = z + (a.bias ? a.bias[e0 + tid] : 0.0f);
    }
    __syncthreads();
  }

  if (tid == 0) {
    int s = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) s += s_redi[i];
    a.beta_x[t] = beta;
    a.rowsum_x[t] = s;
  }
  if (tid < a.k) {
    a.beta_h_bits[t * a.k + tid] = 0u;
    a.rowsum_h[t * a.k + tid] = 0;
  }
  if (warp == 0) {
    const int E = a.E, k = a.k;
    float l0 = lane < E ? s_logits[lane] : -INFINITY;
    float l1 = lane + 32 < E ? s_logits[lane + 32] : -INFINITY;
    const float lmax = warp_max(fmaxf(l0, l1));
    float denom_all = 0.0f;
    if (!a.norm_topk) {
      const float part = (lane < E ? expf(l0 - lmax) : 0.0f) + (lane + 32 < E ? expf(l1 - lmax) : 0.0f);
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
      if (!a.norm_topk) denom = denom_all;
#pragma unroll
      for (int j = 0; j < MOTE_MAX_TOPK; ++j)
        if (j < k) {
          a.topk_idx[t * k + j] = sel_i[j];
          a.topk_w[t * k + j] = ex[j] / denom;
        }
    }
    if (a.T == 1) {
      // one token: its k pairs are grouped right here (every lane holds the selection), without
      // the round trips of the arrival counter
      int mine = 0;
#pragma unroll
      for (int j = 0; j < MOTE_MAX_TOPK; ++j)
        if (j < k && lane == j) mine = sel_i[j];
      int rank = 0;
      for (int e = lane; e <= E; e += 32) {
        int c = 0;
#pragma unroll
        for (int j = 0; j < MOTE_MAX_TOPK; ++j)
          if (j < k) c += sel_i[j] < e ? 1 : 0;
        a.offsets[e] = c;
      }
#pragma unroll
      for (int j = 0; j < MOTE_MAX_TOPK; ++j)
        if (j < k) rank += sel_i[j] < mine ? 1 : 0;
      if (lane < k) {
        a.perm[lane] = rank;
        a.inv[rank] = lane;
      }
    }
  }
  if (a.T == 1) return;

  // the CTA that finishes last sees every token's selection and groups the pairs by expert
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = (atomicAdd(a.counter, 1u) == (unsigned)(a.T - 1));
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  if (warp == 0) {
    const int P = a.T * a.k;
    int mine[kDecodeMaxPairs / 32];
#pragma unroll
    for (int c = 0; c < kDecodeMaxPairs / 32; ++c) {
      const int p = c * 32 + lane;
      mine[c] = p < P ? __ldcg(a.topk_idx + p) : -1;
    }
    int running = 0;
    for (int e = 0; e < a.E; ++e) {
      if (lane == 0) a.offsets[e] = running;
#pragma unroll
      for (int c = 0; c < kDecodeMaxPairs / 32; ++c) {
        if (c * 32 < P) {
          const unsigned m = __ballot_sync(0xffffffffu, mine[c] == e);
          if (mine[c] == e) {
            const int pos = running + __popc(m & ((1u << lane) - 1u));
            a.perm[c * 32 + lane] = pos;
            a.inv[pos] = c * 32 + lane;
          }
          running += __popc(m);
        }
      }
    }
    if (lane == 0) {
      a.offsets[a.E] = running;
      *a.counter = 0u;
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Warp-level streaming products.  Lane (g, t) = (lane / 4, lane % 4).
// ------------------------------------------------------------------------------------------------
// Ternary rows: one step covers 256 reduction elements (64 packed bytes) of two weight rows:
// lane (g, t) loads bytes [64*step + 16*t, +16) of row A (fragment rows 0-7) and of row B
// (fragment rows 8-15).  Word w of the 16 bytes, shifted by 2*i and masked, holds the codes of
// elements 16*w + i + {0, 4, 8, 12} of the lane's 64: exactly word i of unit w of the
// k-interleaved token operand, which is what the lane loads as the B fragment.
constexpr int kTernaryAhead = 3;   // steps of both rows kept in flight per lane (6 x 16 bytes)
constexpr int kBf16Ahead = 4;      // 8 x 16 bytes

template <int NT>
__device__ __forceinline__ void ternary_rows_steps(const uint8_t* __restrict__ row_a, const uint8_t* __restrict__ row_b,
                                                   const int8_t* const (&tok)[NT], int step_begin, int step_end,
                                                   int k_bytes, int lane, int (&acc)[NT][4]) {
  const int t = lane & 3;
  // packed bytes per row = k_bytes; a lane past the end of a short last step contributes zeros
  // (stored code 1 = weight 0, token bytes 0)
  const uint4 kZero = make_uint4(0x55555555u, 0x55555555u, 0x55555555u, 0x55555555u);
  uint4 ra[kTernaryAhead], rb[kTernaryAhead];
#pragma unroll
  for (int i = 0; i < kTernaryAhead; ++i) {
    const int off = (step_begin + i) * 64 + t * 16;
    const bool ok = step_begin + i < step_end && off < k_bytes;
    ra[i] = ok ? ldg_stream16(row_a + off) : kZero;
    rb[i] = ok ? ldg_stream16(row_b + off) : kZero;
  }
  for (int s0 = step_begin; s0 < step_end; s0 += kTernaryAhead) {
#pragma unroll
    for (int i = 0; i < kTernaryAhead; ++i) {
      const int s = s0 + i;
      if (s < step_end) {
        const uint32_t wa[4] = {ra[i].x, ra[i].y, ra[i].z, ra[i].w};
        const uint32_t wb[4] = {rb[i].x, rb[i].y, rb[i].z, rb[i].w};
        {
          const int off = (s + kTernaryAhead) * 64 + t * 16;
          const bool ok = s + kTernaryAhead < step_end && off < k_bytes;
          ra[i] = ok ? ldg_stream16(row_a + off) : kZero;
          rb[i] = ok ? ldg_stream16(row_b + off) : kZero;
        }
        const int q_off = s * 256 + t * 64;           // this lane's 64 token bytes of the step
        const bool q_ok = (s * 64 + t * 16) < k_bytes;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          uint32_t fa[4], fb[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            fa[j] = (wa[w] >> (2 * j)) & 0x03030303u;
            fb[j] = (wb[w] >> (2 * j)) & 0x03030303u;
          }
          // the token fragments of up to four column tiles first (independent loads), then their MMAs
          constexpr int kG = NT < 4 ? NT : 4;
#pragma unroll
          for (int n0 = 0; n0 < NT; n0 += kG) {
            uint4 q[kG];
#pragma unroll
            for (int n = 0; n < kG; ++n) {
              q[n] = make_uint4(0u, 0u, 0u, 0u);
              if (tok[n0 + n] && q_ok) q[n] = *reinterpret_cast<const uint4*>(tok[n0 + n] + q_off + w * 16);
            }
#pragma unroll
            for (int n = 0; n < kG; ++n) {
              mma_u8s8(acc[n0 + n], fa[0], fb[0], fa[1], fb[1], q[n].x, q[n].y);
              mma_u8s8(acc[n0 + n], fa[2], fb[2], fa[3], fb[3], q[n].z, q[n].w);
            }
          }
        }
      }
    }
  }
}

// bf16 rows: one step covers 32 reduction elements: lane (g, t) loads elements [32*step + 8*t, +8)
// of row A and row B, and the same elements of its token column.
template <int NT>
__device__ __forceinline__ void bf16_rows_steps(const uint16_t* __restrict__ row_a, const uint16_t* __restrict__ row_b,
                                                const uint16_t* const (&tok)[NT], int step_begin, int step_end,
                                                int lane, float (&acc)[NT][4]) {
  const int t = lane & 3;
  const uint4 kZero = make_uint4(0u, 0u, 0u, 0u);
  uint4 qa[kBf16Ahead], qb[kBf16Ahead];
#pragma unroll
  for (int i = 0; i < kBf16Ahead; ++i) {
    const bool ok = step_begin + i < step_end;
    qa[i] = ok ? ldg_stream16(row_a + (step_begin + i) * 32 + t * 8) : kZero;
    qb[i] = ok ? ldg_stream16(row_b + (step_begin + i) * 32 + t * 8) : kZero;
  }
  for (int s0 = step_begin; s0 < step_end; s0 += kBf16Ahead) {
#pragma unroll
    for (int i = 0; i < kBf16Ahead; ++i) {
      const int s = s0 + i;
      if (s < step_end) {
        const uint4 ca = qa[i], cb = qb[i];
        if (s + kBf16Ahead < step_end) {
          qa[i] = ldg_stream16(row_a + (s + kBf16Ahead) * 32 + t * 8);
          qb[i] = ldg_stream16(row_b + (s + kBf16Ahead) * 32 + t * 8);
        }
        constexpr int kG = NT < 4 ? NT : 4;
#pragma unroll
        for (int n0 = 0; n0 < NT; n0 += kG) {
          uint4 q[kG];
#pragma unroll
          for (int n = 0; n < kG; ++n) {
            q[n] = kZero;
            if (tok[n0 + n]) q[n] = *reinterpret_cast<const uint4*>(tok[n0 + n] + s * 32 + t * 8);
          }
#pragma unroll
          for (int n = 0; n < kG; ++n) {
            mma_bf16(acc[n0 + n], ca.x, cb.x, ca.y, cb.y, q[n].x, q[n].y);
            mma_bf16(acc[n0 + n], ca.z, cb.z, ca.w, cb.w, q[n].z, q[n].w);
          }
        }
      }
    }
  }
}

// RTN-coded rows (Section 4.3): one step covers 64 bytes of each row (64 int8 or 128 4-bit codes):
// lane (g, t) loads bytes [64*step + 16*t, +16) of row A and row B, expands them to bf16 pairs in
// registers and multiplies them with the same elements of its token column.  A lane past the end
// of a short last step contributes zeros.
template <int NT, int kBits>
__device__ __forceinline__ void rtn_rows_steps(const uint8_t* __restrict__ row_a, const uint8_t* __restrict__ row_b,
                                               const uint16_t* const (&tok)[NT], int step_begin, int step_end,
                                               int k_bytes, int lane, float (&acc)[NT][4]) {
  constexpr int kElems = kBits == 8 ? 16 : 32;        // elements in 16 bytes
  const int t = lane & 3;
  const uint32_t z = kBits == 8 ? 0u : 0x88888888u;   // codes of weight 0
  const uint4 kZero = make_uint4(z, z, z, z);
  uint4 qa[kBf16Ahead], qb[kBf16Ahead];
#pragma unroll
  for (int i = 0; i < kBf16Ahead; ++i) {
    const int off = (step_begin + i) * 64 + t * 16;
    const bool ok = step_begin + i < step_end && off < k_bytes;
    qa[i] = ok ? ldg_stream16(row_a + off) : kZero;
    qb[i] = ok ? ldg_stream16(row_b + off) : kZero;
  }
  for (int s0 = step_begin; s0 < step_end; s0 += kBf16Ahead) {
#pragma unroll
    for (int i = 0; i < kBf16Ahead; ++i) {
      const int s = s0 + i;
      if (s < step_end) {
        const uint32_t wa[4] = {qa[i].x, qa[i].y, qa[i].z, qa[i].w};
        const uint32_t wb[4] = {qb[i].x, qb[i].y, qb[i].z, qb[i].w};
        {
          const int off = (s + kBf16Ahead) * 64 + t * 16;
          const bool ok = s + kBf16Ahead < step_end && off < k_bytes;
          qa[i] = ok ? ldg_stream16(row_a + off) : kZero;
          qb[i] = ok ? ldg_stream16(row_b + off) : kZero;
        }
        const bool q_ok = (s * 64 + t * 16) < k_bytes;
        const int e0 = (s * 4 + t) * kElems;          // first element of this lane's 16 bytes
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          if (kBits == 8) {
            uint32_t a01, a23, b01, b23;
            s8x4_to_bf16x2(wa[w], a01, a23);
            s8x4_to_bf16x2(wb[w], b01, b23);
            constexpr int kG = NT < 4 ? NT : 4;
#pragma unroll
            for (int n0 = 0; n0 < NT; n0 += kG) {
              uint2 q[kG];
#pragma unroll
              for (int n = 0; n < kG; ++n) {
                q[n] = make_uint2(0u, 0u);
                if (tok[n0 + n] && q_ok) q[n] = *reinterpret_cast<const uint2*>(tok[n0 + n] + e0 + 4 * w);
              }
#pragma unroll
              for (int n = 0; n < kG; ++n) mma_bf16(acc[n0 + n], a01, b01, a23, b23, q[n].x, q[n].y);
            }
          } else {
            uint32_t ea[4], eb[4];
            u4x8_to_bf16x2(wa[w], ea);
            u4x8_to_bf16x2(wb[w], eb);
            constexpr int kG = NT < 4 ? NT : 4;
#pragma unroll
            for (int n0 = 0; n0 < NT; n0 += kG) {
              uint4 q[kG];
#pragma unroll
              for (int n = 0; n < kG; ++n) {
                q[n] = make_uint4(0u, 0u, 0u, 0u);
                if (tok[n0 + n] && q_ok) q[n] = *reinterpret_cast<const uint4*>(tok[n0 + n] + e0 + 8 * w);
              }
#pragma unroll
              for (int n = 0; n < kG; ++n) {
                mma_bf16(acc[n0 + n], ea[0], eb[0], ea[1], eb[1], q[n].x, q[n].y);
                mma_bf16(acc[n0 + n], ea[2], eb[2], ea[3], eb[3], q[n].z, q[n].w);
              }
            }
          }
        }
      }
    }
  }
}

// splits n_steps as evenly as possible over n_parts; part p gets [begin, end)
__device__ __forceinline__ void split_steps(int n_steps, int n_parts, int p, int& begin, int& end) {
  const int base = n_steps / n_parts, rem = n_steps % n_parts;
  begin = p * base + min(p, rem);
  end = begin + base + (p < rem ? 1 : 0);
}

// Two rows of one shared-expert matrix against the token columns: bf16 values or RTN codes.
// K = reduction length in elements; warp `part` of `n_parts` takes its share of the steps.
template <int NT, int kShBits>
__device__ __forceinline__ void shared_rows(const void* W, int64_t row_a, int64_t row_b, int K,
                                            const uint16_t* const (&tok)[NT], int n_parts, int part, int lane,
                                            float (&acc)[NT][4]) {
  int sb, se;
  if (kShBits == 16) {
    const uint16_t* w = static_cast<const uint16_t*>(W);
    split_steps(K / 32, n_parts, part, sb, se);
    bf16_rows_steps<NT>(w + row_a * K, w + row_b * K, tok, sb, se, lane, acc);
  } else {
    const uint8_t* w = static_cast<const uint8_t*>(W);
    const int k_bytes = kShBits == 8 ? K : K / 2;
    split_steps((k_bytes + 63) / 64, n_parts, part, sb, se);
    rtn_rows_steps<NT, kShBits == 16 ? 8 : kShBits>(w + row_a * k_bytes, w + row_b * k_bytes, tok, sb, se, k_bytes,
                                                    lane, acc);
  }
}

// ------------------------------------------------------------------------------------------------
// Work list shared by the two streaming kernels: the shared expert's tiles first, then the tiles of
// every expert that received tokens.
// ------------------------------------------------------------------------------------------------
struct DecodeCommon {
  int T, d, f, E, k;
  const int32_t* offsets;   // [E+1]
  const int32_t* inv;       // [P] sorted row -> pair
  const int8_t* qx;         // [T, d] token order
  const float* beta_x;      // [T]
  const int32_t* rowsum_x;  // [T]
};

struct ExpertList {
  int n;                               // experts with at least one token
  int id[MOTE_MAX_EXPERTS];
};

__device__ __forceinline__ void build_expert_list(const int32_t* __restrict__ offsets, int E, ExpertList* list) {
  // called by one warp
  const int lane = threadIdx.x & 31;
  int n = 0;
  for (int e0 = 0; e0 < E; e0 += 32) {
    const int e = e0 + lane;
    const bool has = e < E && offsets[e + 1] > offsets[e];
    const unsigned m = __ballot_sync(0xffffffffu, has);
    if (has) list->id[n + __popc(m & ((1u << lane) - 1u))] = e;
    n += __popc(m);
  }
  if (lane == 0) list->n = n;
}

// ------------------------------------------------------------------------------------------------
// decode_gateup: 4 warps per CTA.
//   shared item  = 8 rows of f (gate rows in fragment rows 0-7, up rows in 8-15), the 4 warps split d
//   routed item  = 4 consecutive 8-row tiles of one expert, one per warp, whole d
// ------------------------------------------------------------------------------------------------
struct DecodeGateUpArgs {
  DecodeCommon c;
  const uint8_t* gate_packed; const uint8_t* up_packed;   // [E][f, d/4]
  const float* alpha_gate; const float* alpha_up;
  SharedMat sh_gate, sh_up; int sh_bits;                   // [f, d] bf16, or RTN codes + row scales
  const uint16_t* x;                                       // [T, d] bf16
  uint16_t* h;              // [P, f] bf16, sorted rows
  uint32_t* beta_h_bits;    // [P]
  uint16_t* hs;             // [T, f] bf16
  int32_t* tap_gate; int32_t* tap_up;                      // optional [P, f]
};

constexpr int kGuWarps = 4;

template <int NT>
__device__ __forceinline__ void gateup_routed_tile(const DecodeGateUpArgs& a, int e, int tile, int lane) {
  const int d = a.c.d, f = a.c.f, k = a.c.k;
  const int g = lane >> 2, t = lane & 3;
  const int row0 = a.c.offsets[e], n_e = a.c.offsets[e + 1] - row0;
  const int k_bytes = d / 4;
  const int frow = tile * 8 + g;
  const uint8_t* gate_row = a.gate_packed + (int64_t(e) * f + frow) * k_bytes;
  const uint8_t* up_row = a.up_packed + (int64_t(e) * f + frow) * k_bytes;
  const int8_t* tok[NT];
#pragma unroll
  for (int n = 0; n < NT; ++n) {
    const int slot = n * 8 + g;
    tok[n] = slot < n_e ? a.c.qx + int64_t(a.c.inv[row0 + slot] / k) * d : nullptr;
  }
  int acc[NT][4];
#pragma unroll
  for (int n = 0; n < NT; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0;
  ternary_rows_steps<NT>(gate_row, up_row, tok, 0, (k_bytes + 63) / 64, k_bytes, lane, acc);

  // fragment: acc[n][0..1] = gate row g for token slots 8n+2t, 8n+2t+1; acc[n][2..3] = up, same slots
  const float ag = a.alpha_gate[e], au = a.alpha_up[e];
#pragma unroll
  for (int n = 0; n < NT; ++n) {
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int slot = n * 8 + 2 * t + j;
      float habs = 0.0f;
      const bool ok = slot < n_e;
      const int row = row0 + (ok ? slot : 0);
      if (ok) {
        const int token = a.c.inv[row] / k;
        const float beta = a.c.beta_x[token];
        const int rs = a.c.rowsum_x[token];
        const int ig = acc[n][j] - rs, iu = acc[n][2 + j] - rs;   // stored codes are code+1
        const float hv = glu_h(ig, iu, dequant_scale(ag, beta), dequant_scale(au, beta));
        const uint32_t hb = f32_to_bf16_bits(hv);
        a.h[int64_t(row) * f + frow] = (uint16_t)hb;
        habs = __uint_as_float((hb & 0x7FFFu) << 16);
        if (a.tap_gate) {
          a.tap_gate[int64_t(row) * f + frow] = ig;
          a.tap_up[int64_t(row) * f + frow] = iu;
        }
      }
      // max over the 8 rows of the tile (lanes with equal t), one atomic per (tile, token)
      habs = fmaxf(habs, __shfl_xor_sync(0xffffffffu, habs, 4));
      habs = fmaxf(habs, __shfl_xor_sync(0xffffffffu, habs, 8));
      habs = fmaxf(habs, __shfl_xor_sync(0xffffffffu, habs, 16));
      if (ok && g == 0 && habs > 0.0f) atomicMax(a.beta_h_bits + row, __float_as_uint(habs));
    }
  }
}

template <int NT, int kShBits>
__device__ __forceinline__ void gateup_shared_tile(const DecodeGateUpArgs& a, int tile, int warp, int lane,
                                                   float* s_part) {
  const int d = a.c.d, f = a.c.f, T = a.c.T;
  const int g = lane >> 2, t = lane & 3;
  const int frow = tile * 8 + g;
  const uint16_t* tok[NT];
#pragma unroll
  for (int n = 0; n < NT; ++n) tok[n] = (n * 8 + g) < T ? a.x + int64_t(n * 8 + g) * d : nullptr;
  float acc[NT][4];
#pragma unroll
  for (int n = 0; n < NT; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.0f;
  // gate row in fragment rows 0-7, up row in 8-15: two different matrices, one call each half
  if (kShBits == 16) {
    int sb, se;
    split_steps(d / 32, kGuWarps, warp, sb, se);
    bf16_rows_steps<NT>(static_cast<const uint16_t*>(a.sh_gate.w) + int64_t(frow) * d,
                        static_cast<const uint16_t*>(a.sh_up.w) + int64_t(frow) * d, tok, sb, se, lane, acc);
  } else {
    const int k_bytes = kShBits == 8 ? d : d / 2;
    const uint8_t* rg = static_cast<const uint8_t*>(a.sh_gate.w) + int64_t(frow) * k_bytes;
    const uint8_t* ru = static_cast<const uint8_t*>(a.sh_up.w) + int64_t(frow) * k_bytes;
    int sb, se;
    split_steps((k_bytes + 63) / 64, kGuWarps, warp, sb, se);
    rtn_rows_steps<NT, kShBits == 16 ? 8 : kShBits>(rg, ru, tok, sb, se, k_bytes, lane, acc);
  }
  // partial sums of the 4 warps are added in warp order
#pragma unroll
  for (int n = 0; n < NT; ++n)
#pragma unroll
    for (int i = 0; i < 4; ++i) s_part[(warp * NT * 4 + n * 4 + i) * 32 + lane] = acc[n][i];
  __syncthreads();
  const float sc_g = kShBits == 16 ? 1.0f : a.sh_gate.scale[frow];
  const float sc_u = kShBits == 16 ? 1.0f : a.sh_up.scale[frow];
  for (int n = warp; n < NT; n += kGuWarps) {
    float v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float s = s_part[(n * 4 + i) * 32 + lane];
#pragma unroll
      for (int w = 1; w < kGuWarps; ++w) s += s_part[(w * NT * 4 + n * 4 + i) * 32 + lane];
      v[i] = s;
    }
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int token = n * 8 + 2 * t + j;
      if (token < T) {
        const float gv = v[j] * sc_g, uv = v[2 + j] * sc_u;
        const float hv = uv * __fdividef(gv, 1.0f + __expf(-gv));
        a.hs[int64_t(token) * f + frow] = (uint16_t)f32_to_bf16_bits(hv);
      }
    }
  }
  __syncthreads();
}

// NTB = number of 8-token column tiles the launch is built for (1, 2, 4 or 8): ceil(T / 8) rounded up
// kShBits = storage of the shared expert (16, 8 or 4): a kernel of its own per width, so that the
// code expansion of the RTN widths costs the bf16 kernel no registers
// The bf16 kernel for 9..16 tokens is held to 72 registers (it takes 80 left alone): seven CTAs per SM
// instead of six, 8 % off the gate/up stream at T = 16.  (96 registers for 17..32 tokens: no gain.)
// The other instantiations must stay without a minimum (0): a minimum of one CTA is not the same
// to the compiler as none (it then plans for all 512 registers a thread could have, and the
// streams of 1..8 and 17..32 tokens came out 9-50 % slower).
template <int NTB, int kShBits>
__global__ void __launch_bounds__(kGuWarps * 32, (NTB == 2 && kShBits == 16) ? 7 : 0) decode_gateup_kernel(DecodeGateUpArgs a) {
  __shared__ ExpertList s_list;
  __shared__ float s_part[kGuWarps * NTB * 4 * 32];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tiles = a.c.f / 8;
  const int quads = (tiles + kGuWarps - 1) / kGuWarps;
  const int n_shared = tiles;
  // The shared expert needs nothing from the prologue kernel, so its items run before the wait on
  // that kernel; the routing tables are read only when the CTA reaches its first routed item.
  bool routed_ready = false;
  int n_items = n_shared;
  for (int item = blockIdx.x;; item += gridDim.x) {
    if (item >= n_shared && !routed_ready) {
      pdl_wait();
      if (warp == 0) build_expert_list(a.c.offsets, a.c.E, &s_list);
      __syncthreads();
      n_items = n_shared + s_list.n * quads;
      routed_ready = true;
    }
    if (item >= n_items) break;
    if (item < n_shared) {
      gateup_shared_tile<NTB, kShBits>(a, item, warp, lane, s_part);
    } else {
      const int r = item - n_shared;
      const int e = s_list.id[r / quads];
      const int tile = (r % quads) * kGuWarps + warp;
      if (tile < tiles) {
        const int nt = (a.c.offsets[e + 1] - a.c.offsets[e] + 7) / 8;
        if (NTB == 1 || nt <= 1) gateup_routed_tile<1>(a, e, tile, lane);
        else if (NTB == 2 || nt <= 2) gateup_routed_tile<(NTB >= 2 ? 2 : 1)>(a, e, tile, lane);
        else if (NTB == 4 || nt <= 4) gateup_routed_tile<(NTB >= 4 ? 4 : 1)>(a, e, tile, lane);
        else gateup_routed_tile<(NTB >= 8 ? 8 : 1)>(a, e, tile, lane);
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// decode_down: kDownWarps warps per CTA split the reduction dimension f of one 16-row tile of d.
// ------------------------------------------------------------------------------------------------
struct DecodeDownArgs {
  DecodeCommon c;
  const uint8_t* down_packed;   // [E][d, f/4]
  const float* alpha_down;
  SharedMat sh_down; int sh_bits;   // [d, f] bf16, or RTN codes + row scales
  const int8_t* qh;             // [P, f] sorted rows, k-interleaved
  const float* beta_h;          // [P]
  const int32_t* rowsum_h;      // [P]
  const uint16_t* hs;           // [T, f] bf16
  float* y;                     // [P, d]
  float* s;                     // [T, d]
  int32_t* tap_down;            // optional [P, d]
  // combine of Eq. 2 / Eq. 4, done per 16-column tile by the CTA that finishes the tile's last item
  const float* topk_w;          // [T, k]
  const int32_t* perm;          // [T*k] pair -> sorted row
  const uint16_t* residual;     // [T, d] bf16 or null; may alias out
  uint16_t* out;                // [T, d] bf16
  uint32_t* tile_count;         // [d/16] zero on entry
};

constexpr int kDownWarps = 16;

template <int NT>
__device__ __forceinline__ void down_routed_tile(const DecodeDownArgs& a, int e, int tile, int warp, int lane,
                                                 int* s_part) {
  const int d = a.c.d, f = a.c.f;
  const int g = lane >> 2, t = lane & 3;
  const int row0 = a.c.offsets[e], n_e = a.c.offsets[e + 1] - row0;
  const int k_bytes = f / 4;
  const int drow = tile * 16 + g;
  const uint8_t* wa = a.down_packed + (int64_t(e) * d + drow) * k_bytes;
  const uint8_t* wb = wa + int64_t(8) * k_bytes;
  const int8_t* tok[NT];
#pragma unroll
  for (int n = 0; n < NT; ++n) tok[n] = (n * 8 + g) < n_e ? a.qh + int64_t(row0 + n * 8 + g) * f : nullptr;
  int acc[NT][4];
#pragma unroll
  for (int n = 0; n < NT; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0;
  int sb, se;
  split_steps((k_bytes + 63) / 64, kDownWarps, warp, sb, se);
  ternary_rows_steps<NT>(wa, wb, tok, sb, se, k_bytes, lane, acc);
#pragma unroll
  for (int n = 0; n < NT; ++n)
#pragma unroll
    for (int i = 0; i < 4; ++i) s_part[(warp * NT * 4 + n * 4 + i) * 32 + lane] = acc[n][i];
  __syncthreads();
  const float al = a.alpha_down[e];
  for (int n = warp; n < NT; n += kDownWarps) {
    int v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int s = 0;
#pragma unroll
      for (int w = 0; w < kDownWarps; ++w) s += s_part[(w * NT * 4 + n * 4 + i) * 32 + lane];
      v[i] = s;
    }
    // fragment: v[0..1] = row g for slots 8n+2t, +1; v[2..3] = row g+8
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int slot = n * 8 + 2 * t + j;
      if (slot < n_e) {
        const int row = row0 + slot;
        const int rs = a.rowsum_h[row];
        const float c0 = dequant_scale(al, a.beta_h[row]);
        const int lo = v[j] - rs, hi = v[2 + j] - rs;
        a.y[int64_t(row) * d + drow] = __fmul_rn(i2f_small(lo), c0);
        a.y[int64_t(row) * d + drow + 8] = __fmul_rn(i2f_small(hi), c0);
        if (a.tap_down) {
          a.tap_down[int64_t(row) * d + drow] = lo;
          a.tap_down[int64_t(row) * d + drow + 8] = hi;
        }
      }
    }
  }
  __syncthreads();
}

template <int NT, int kShBits>
__device__ __forceinline__ void down_shared_tile(const DecodeDownArgs& a, int tile, int warp, int lane, float* s_part) {
  const int d = a.c.d, f = a.c.f, T = a.c.T;
  const int g = lane >> 2, t = lane & 3;
  const int drow = tile * 16 + g;
  const uint16_t* tok[NT];
#pragma unroll
  for (int n = 0; n < NT; ++n) tok[n] = (n * 8 + g) < T ? a.hs + int64_t(n * 8 + g) * f : nullptr;
  float acc[NT][4];
#pragma unroll
  for (int n = 0; n < NT; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.0f;
  shared_rows<NT, kShBits>(a.sh_down.w, drow, drow + 8, f, tok, kDownWarps, warp, lane, acc);
#pragma unroll
  for (int n = 0; n < NT; ++n)
#pragma unroll
    for (int i = 0; i < 4; ++i) s_part[(warp * NT * 4 + n * 4 + i) * 32 + lane] = acc[n][i];
  __syncthreads();
  const float sc_lo = kShBits == 16 ? 1.0f : a.sh_down.scale[drow];
  const float sc_hi = kShBits == 16 ? 1.0f : a.sh_down.scale[drow + 8];
  for (int n = warp; n < NT; n += kDownWarps) {
    float v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float s = s_part[(n * 4 + i) * 32 + lane];
#pragma unroll
      for (int w = 1; w < kDownWarps; ++w) s += s_part[(w * NT * 4 + n * 4 + i) * 32 + lane];
      v[i] = s;
    }
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int token = n * 8 + 2 * t + j;
      if (token < T) {
        a.s[int64_t(token) * d + drow] = v[j] * sc_lo;
        a.s[int64_t(token) * d + drow + 8] = v[2 + j] * sc_hi;
      }
    }
  }
  __syncthreads();
}

// The CTA that completes the last of a tile's items (the shared expert's and one per expert that
// received tokens) adds them up: out[t, c] = bf16( s[t, c] + sum_j w[t, j] * y[perm[t*k+j], c] [+ residual] ),
// fp32, slots in ascending j -- the arithmetic of combine_kernel.  Every thread calls this after
// its stores of the item; the count is kept per tile, so the combines of different tiles run in
// parallel on whichever CTAs arrive last.
__device__ __forceinline__ void down_tile_done(const DecodeDownArgs& a, int tile, int n_producers, int* s_last) {
  __threadfence();                                   // this thread's y / s values are visible device-wide
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint32_t old = atomicAdd(a.tile_count + tile, 1u);
    *s_last = (old == (uint32_t)n_producers - 1u);
    if (*s_last) a.tile_count[tile] = 0u;            // left clean for the next call
  }
  __syncthreads();
  if (!*s_last) return;
  __threadfence();
  const int d = a.c.d, k = a.c.k, T = a.c.T;
  for (int i = threadIdx.x; i < T * 16; i += blockDim.x) {
    const int t = i >> 4, col = tile * 16 + (i & 15);
    float acc = __ldcg(a.s + int64_t(t) * d + col);
    for (int j = 0; j < k; ++j)
      acc = fmaf(a.topk_w[t * k + j], __ldcg(a.y + int64_t(a.perm[t * k + j]) * d + col), acc);
    if (a.residual) acc += __uint_as_float(uint32_t(a.residual[int64_t(t) * d + col]) << 16);
    a.out[int64_t(t) * d + col] = (uint16_t)f32_to_bf16_bits(acc);
  }
  __syncthreads();
}

// up to 16 tokens: two CTAs per SM (at most 64 registers; at 78 registers the 16-token kernel had
// one CTA per SM and was 8-15 % slower; every one-tile kernel is capped too: left alone the bf16 one
// takes 106 registers, one CTA per SM, and the step is 5-10 % slower.  The 16-token 4-bit expansion
// would spill too much under that cap.)
template <int NTB, int kShBits>
__global__ void __launch_bounds__(kDownWarps * 32,
                                  (NTB == 1 || (NTB == 2 && kShBits != 4)) ? 2 : 1)
decode_down_kernel(DecodeDownArgs a) {
  __shared__ ExpertList s_list;
  __shared__ int s_last;
  extern __shared__ float s_part[];                       // kDownWarps * NTB * 4 * 32 floats
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // This kernel is let in as soon as Q_a(h) has STARTED (which is after the gate/up kernel and
  // the prologue have completed): the dispatch tables and h_shared are there, and the shared
  // expert's slices are streamed while Q_a(h) runs.  The routed items wait for it.
  if (warp == 0) build_expert_list(a.c.offsets, a.c.E, &s_list);
  __syncthreads();
  const int tiles = a.c.d / 16;
  const int n_shared = tiles;
  const int n_items = n_shared + s_list.n * tiles;
  int* ip = reinterpret_cast<int*>(s_part);
  bool waited = false;
  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
    if (item >= n_shared && !waited) {
      pdl_wait();                          // Q_a(h) has completed
      waited = true;
    }
    if (item < n_shared) {
      down_shared_tile<NTB, kShBits>(a, item, warp, lane, s_part);
      down_tile_done(a, item, 1 + s_list.n, &s_last);
    } else {
      const int r = item - n_shared;
      const int e = s_list.id[r / tiles];
      const int tile = r % tiles;
      const int nt = (a.c.offsets[e + 1] - a.c.offsets[e] + 7) / 8;
      if (NTB == 1 || nt <= 1) down_routed_tile<1>(a, e, tile, warp, lane, ip);
      else if (NTB == 2 || nt <= 2) down_routed_tile<(NTB >= 2 ? 2 : 1)>(a, e, tile, warp, lane, ip);
      else if (NTB == 4 || nt <= 4) down_routed_tile<(NTB >= 4 ? 4 : 1)>(a, e, tile, warp, lane, ip);
      else down_routed_tile<(NTB >= 8 ? 8 : 1)>(a, e, tile, warp, lane, ip);
      down_tile_done(a, tile, 1 + s_list.n, &s_last);
    }
  }
  if (!waited) pdl_wait();                 // no CTA leaves before the kernels ahead of it are complete
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
bool decode_stream_supported(int d, int f, int E, int k, int64_t T) {
  // rows of packed codes (d/4, f/4 bytes) are read 16 bytes at a time
  return T >= 1 && T <= kDecodeMaxTokens && T * k <= kDecodeMaxPairs && d % 64 == 0 && f % 64 == 0 && d <= 16384 &&
         E <= MOTE_MAX_EXPERTS;
}

// phase 0: prologue, 1: gate/up, 2: down
mote_status_t launch_decode_stream(const DecodeStreamArgs& p, int phase, cudaStream_t stream) {
  const int T = (int)p.T, d = p.d, f = p.f, E = p.E, k = p.k;
  const int sms = device_sm_count();
  const int ntb = T <= 8 ? 1 : T <= 16 ? 2 : T <= 32 ? 4 : 8;

  if (phase == 0) {
    DecodePrologueArgs pa{};
    pa.x = static_cast<const uint16_t*>(p.x); pa.T = T; pa.d = d; pa.E = E; pa.k = k; pa.norm_topk = p.norm_topk;
    pa.Wr = p.Wr; pa.bias = p.router_bias; pa.topk_idx = p.topk_idx; pa.topk_w = p.topk_w; pa.qx = p.qx;
    pa.beta_x = p.beta_x; pa.rowsum_x = p.rowsum_x; pa.beta_h_bits = reinterpret_cast<uint32_t*>(p.beta_h);
    pa.rowsum_h = p.rowsum_h; pa.counter = p.counter; pa.zero_head_words = (T == 1) ? p.zero_head_words : 0; pa.offsets = p.offsets; pa.perm = p.perm; pa.inv = p.inv;
    static PerDeviceOnce prologue_attr;
    MOTE_CUDA_OK(set_max_dynamic_smem(prologue_attr, decode_prologue_kernel, 32768));
    MOTE_CUDA_OK(launch_pdl(decode_prologue_kernel, dim3(T), dim3(256), size_t(d) * 2, stream, pa));
    ++g_launch_count;
    MOTE_LAUNCH_OK();
    return MOTE_OK;
  }

  DecodeCommon c{};
  c.T = T; c.d = d; c.f = f; c.E = E; c.k = k; c.offsets = p.offsets; c.inv = p.inv; c.qx = p.qx;
  c.beta_x = p.beta_x; c.rowsum_x = p.rowsum_x;

  if (phase == 1) {
    DecodeGateUpArgs ga{};
    ga.c = c; ga.gate_packed = p.gate_packed; ga.up_packed = p.up_packed; ga.alpha_gate = p.alpha_gate;
    ga.alpha_up = p.alpha_up; ga.sh_gate = p.sh_gate;
    ga.sh_up = p.sh_up; ga.sh_bits = p.shared_bits; ga.x = static_cast<const uint16_t*>(p.x);
    ga.h = static_cast<uint16_t*>(p.h); ga.beta_h_bits = reinterpret_cast<uint32_t*>(p.beta_h);
    ga.hs = static_cast<uint16_t*>(p.hs); ga.tap_gate = p.tap_gate; ga.tap_up = p.tap_up;
    const int tiles = f / 8, quads = (tiles + kGuWarps - 1) / kGuWarps;
    const int max_items = tiles + std::min<int>(E, T * k) * quads;
    const int grid = std::min(max_items, sms * 12);
#define MOTE_GU_LAUNCH(NTB_, BITS_) \
  MOTE_CUDA_OK(launch_pdl(decode_gateup_kernel<NTB_, BITS_>, dim3(grid), dim3(kGuWarps * 32), 0, stream, ga))
#define MOTE_GU_BITS(NTB_)                                 \
  do {                                                     \
    if (p.shared_bits == 8) MOTE_GU_LAUNCH(NTB_, 8);       \
    else if (p.shared_bits == 4) MOTE_GU_LAUNCH(NTB_, 4);  \
    else MOTE_GU_LAUNCH(NTB_, 16);                         \
  } while (0)
    if (ntb == 1) MOTE_GU_BITS(1);
    else if (ntb == 2) MOTE_GU_BITS(2);
    else if (ntb == 4) MOTE_GU_BITS(4);
    else MOTE_GU_BITS(8);
#undef MOTE_GU_BITS
#undef MOTE_GU_LAUNCH
    ++g_launch_count;
    MOTE_LAUNCH_OK();
    return MOTE_OK;
  }

  DecodeDownArgs da{};
  da.c = c; da.down_packed = p.down_packed; da.alpha_down = p.alpha_down;
  da.topk_w = p.topk_w; da.perm = p.perm; da.residual = static_cast<const uint16_t*>(p.residual);
  da.out = static_cast<uint16_t*>(p.out); da.tile_count = p.tile_count;
  da.sh_down = p.sh_down; da.sh_bits = p.shared_bits; da.qh = p.qh; da.beta_h = p.beta_h; da.rowsum_h = p.rowsum_h;
  da.hs = static_cast<const uint16_t*>(p.hs); da.y = p.y; da.s = p.s; da.tap_down = p.tap_down;
  const int tiles = d / 16;
  const int max_items = tiles + std::min<int>(E, T * k) * tiles;
  const int grid = std::min(max_items, sms * 3);
  const size_t smem = size_t(kDownWarps) * ntb * 4 * 32 * sizeof(float);
  static PerDeviceOnce down_attr16, down_attr8, down_attr4;
  MOTE_CUDA_OK(set_max_dynamic_smem(down_attr16, decode_down_kernel<8, 16>, 65536));
  MOTE_CUDA_OK(set_max_dynamic_smem(down_attr8, decode_down_kernel<8, 8>, 65536));
  MOTE_CUDA_OK(set_max_dynamic_smem(down_attr4, decode_down_kernel<8, 4>, 65536));
#define MOTE_DN_LAUNCH(NTB_, BITS_) \
  MOTE_CUDA_OK(launch_pdl(decode_down_kernel<NTB_, BITS_>, dim3(grid), dim3(kDownWarps * 32), smem, stream, da))
#define MOTE_DN_BITS(NTB_)                                 \
  do {                                                     \
    if (p.shared_bits == 8) MOTE_DN_LAUNCH(NTB_, 8);       \
    else if (p.shared_bits == 4) MOTE_DN_LAUNCH(NTB_, 4);  \
    else MOTE_DN_LAUNCH(NTB_, 16);                         \
  } while (0)
  if (ntb == 1) MOTE_DN_BITS(1);
  else if (ntb == 2) MOTE_DN_BITS(2);
  else if (ntb == 4) MOTE_DN_BITS(4);
  else MOTE_DN_BITS(8);
#undef MOTE_DN_BITS
#undef MOTE_DN_LAUNCH
  ++g_launch_count;
  MOTE_LAUNCH_OK();
  return MOTE_OK;
}

}  // namespace mote
