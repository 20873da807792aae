// Per-token absmax int8 activation quantizer (Eq. 8-10).
//
// One group of G threads (G = 32..256, a power of two) owns one token row and keeps it in
// registers between the absmax pass and the quantisation pass, so x is read from HBM once.
// Each thread handles units of 16 consecutive elements: two 128-bit loads in, one 128-bit store
// out.  HBM-bound: 2 B read + 1 B written per element.
//
// The layer-internal variant writes the row to the k expert-sorted positions of its token and
// can store each unit of 16 codes in the "k-interleaved" order the tensor-core GEMM wants
// (stored[4*i + b] = q[4*b + i]): the GEMM's 2-bit weight unpacker yields weights in the same
// order, and an integer dot product does not depend on the order of its terms.
#include <algorithm>

#include "mote_common.cuh"
#include "mote_internal.h"
#include "ptx_sm100.cuh"

namespace mote {

template <int kUnits, bool kScatter>
__global__ void __launch_bounds__(256, kUnits <= 2 ? 4 : 0) quant_act_kernel(QuantActArgs a) {
  __shared__ float s_max[8];
  __shared__ int s_sum[8];
  const int G = a.group;                          // threads per row
  const int rows_per_cta = blockDim.x / G;
  const int g = threadIdx.x / G;                  // row slot inside the CTA
  const int tg = threadIdx.x % G;                 // thread inside the group
  const int64_t row = int64_t(blockIdx.x) * rows_per_cta + g;
  const bool row_ok = row < a.T;
  const int n_units = a.d / 16;

  uint4 raw[kUnits][2];
  float amax = 0.0f;
  const uint4* src = reinterpret_cast<const uint4*>(
      reinterpret_cast<const uint16_t*>(a.x) + (row_ok ? row : 0) * a.ldx);
#pragma unroll
  for (int u = 0; u < kUnits; ++u) {
    const int unit = tg + u * G;
    if (row_ok && unit < n_units) {
      raw[u][0] = src[unit * 2];
      raw[u][1] = src[unit * 2 + 1];
    } else {
      raw[u][0] = make_uint4(0, 0, 0, 0);
      raw[u][1] = make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const uint32_t w[4] = {raw[u][h].x, raw[u][h].y, raw[u][h].z, raw[u][h].w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        amax = fmaxf(amax, fabsf(bf16_lo(w[j])));
        amax = fmaxf(amax, fabsf(bf16_hi(w[j])));
      }
    }
  }
  // group-wide max
  amax = warp_max(amax);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (G > 32) {
    if (lane == 0) s_max[warp] = amax;
    __syncthreads();
    const int w0 = (g * G) >> 5, nw = G >> 5;
    float m = s_max[w0];
    for (int i = 1; i < nw; ++i) m = fmaxf(m, s_max[w0 + i]);
    amax = m;
  }
  const float beta = fmaxf(amax, kEpsScale);
  const QaScale qs = qa_scale(beta);

  int local_sum = 0;
  uint4 outw[kUnits];
#pragma unroll
  for (int u = 0; u < kUnits; ++u) {
    uint32_t q[16];                                // low byte of each word = the int8 code
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const uint32_t w[4] = {raw[u][h].x, raw[u][h].y, raw[u][h].z, raw[u][h].w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        q[h * 8 + 2 * j] = quant_byte(bf16_lo(w[j]), qs);
        q[h * 8 + 2 * j + 1] = quant_byte(bf16_hi(w[j]), qs);
      }
    }
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      o[i] = a.interleave ? pack_low_bytes(q[i], q[4 + i], q[8 + i], q[12 + i])
                          : pack_low_bytes(q[4 * i], q[4 * i + 1], q[4 * i + 2], q[4 * i + 3]);
      local_sum = __dp4a((int)o[i], 0x01010101, local_sum);
    }
    outw[u] = make_uint4(o[0], o[1], o[2], o[3]);
  }
  local_sum = warp_sum(local_sum);
  if (G > 32) {
    if (lane == 0) s_sum[warp] = local_sum;
    __syncthreads();
    const int w0 = (g * G) >> 5, nw = G >> 5;
    int s = 0;
    for (int i = 0; i < nw; ++i) s += s_sum[w0 + i];
    local_sum = s;
  }
  if (!row_ok) return;

  // everything above depends on x only; the routing of the kernels before this one is needed from here on
  if (kScatter) pdl_wait();
  const int n_dst = kScatter ? a.k : 1;
  for (int j = 0; j < n_dst; ++j) {
    int64_t dst = row;
    if (kScatter) {
      if (a.blk_base) {
        // sorted row = first row of (block, expert) + number of earlier pairs of the block with that
        // expert; a row group is made of whole warps, so the ballots below see converged warps
        const int pair = (int)row * a.k + j;
        const int e = a.topk_idx[pair];
        const int blk = (int)(row / kRouteBlockTokens);
        const int p0 = blk * kRouteBlockTokens * a.k;
        int rank = 0;
        for (int off = 0; off < kRouteBlockTokens * a.k; off += 32) {
          const int pp = p0 + off + lane;
          const bool m = pp < pair && a.topk_idx[pp] == e;
          rank += __popc(__ballot_sync(0xffffffffu, m));
        }
        dst = a.blk_base[e * blk_stride(a.n_blk) + blk] + rank;
        if (tg == 0) {
          a.perm_out[pair] = (int32_t)dst;
          a.inv_out[dst] = pair;
          if (a.zero_u32) {                              // targets of the gate/up epilogue's atomics
            a.zero_u32[dst] = 0u;
            a.zero_i32[dst] = 0;
          }
        }
      } else {
        dst = a.perm[row * a.k + j];
      }
    }
    uint4* out = reinterpret_cast<uint4*>(a.q + dst * int64_t(a.d));
#pragma unroll
    for (int u = 0; u < kUnits; ++u) {
      const int unit = tg + u * G;
      if (unit < n_units) out[unit] = outw[u];
    }
    if (tg == 0) {
      a.beta[dst] = beta;
      if (a.rowsum) a.rowsum[dst] = local_sum;
    }
  }
}

// The stand-alone entry point's kernel (mote_quant_act): one warp owns one token row at a time and
// keeps it in shared memory between the absmax pass and the quantisation pass.  No block-wide
// barrier and few registers, so many warps are resident and each keeps up to 128 bytes per lane in
// flight on its way in: 1.2-1.5 times the group-per-row kernel above on rows of 1536 elements and
// more (3.4 TB/s at d = 2048).  (Inside the layer the rows are scattered to expert-sorted positions
// that are known only after the kernels ahead; there the kernel above, which has all its arithmetic
// done before it waits for them, stays ahead at small d and level at large d.)
__global__ void __launch_bounds__(256, 4) quant_act_rows_kernel(QuantActArgs a) {
  extern __shared__ uint4 s_rows[];               // [warps][d / 8]: the warp's row, bf16
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
  const int n_units = a.d / 16;
  uint4* my = s_rows + size_t(warp) * (a.d / 8);
  for (int64_t row = int64_t(blockIdx.x) * n_warps + warp; row < a.T; row += int64_t(gridDim.x) * n_warps) {
    const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(a.x) + row * a.ldx);
    // pass 1: the row into shared memory, four units (128 bytes) per lane requested at a time
    float amax = 0.0f;
    for (int u0 = lane; u0 < n_units; u0 += 32 * 4) {
      uint4 r[4][2];
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int unit = u0 + b * 32;
        if (unit < n_units) {
          r[b][0] = src[unit * 2];
          r[b][1] = src[unit * 2 + 1];
        }
      }
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int unit = u0 + b * 32;
        if (unit < n_units) {
          my[unit * 2] = r[b][0];
          my[unit * 2 + 1] = r[b][1];
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const uint32_t w[4] = {r[b][h].x, r[b][h].y, r[b][h].z, r[b][h].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) amax = fmaxf(amax, fmaxf(fabsf(bf16_lo(w[j])), fabsf(bf16_hi(w[j]))));
          }
        }
      }
    }
    amax = warp_max(amax);
    const float beta = fmaxf(amax, kEpsScale);
    const QaScale qs = qa_scale(beta);
    __syncwarp();
    // pass 2: codes
    int local_sum = 0;
    for (int unit = lane; unit < n_units; unit += 32) {
      const uint4 r0 = my[unit * 2], r1 = my[unit * 2 + 1];
      const uint32_t w[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
      uint32_t q[16];                                // low byte of each word = the int8 code
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        q[2 * j] = quant_byte(bf16_lo(w[j]), qs);
        q[2 * j + 1] = quant_byte(bf16_hi(w[j]), qs);
      }
      uint32_t o[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        o[i] = a.interleave ? pack_low_bytes(q[i], q[4 + i], q[8 + i], q[12 + i])
                            : pack_low_bytes(q[4 * i], q[4 * i + 1], q[4 * i + 2], q[4 * i + 3]);
        local_sum = __dp4a((int)o[i], 0x01010101, local_sum);
      }
      reinterpret_cast<uint4*>(a.q + row * int64_t(a.d))[unit] = make_uint4(o[0], o[1], o[2], o[3]);
    }
    local_sum = warp_sum(local_sum);
    if (lane == 0) {
      a.beta[row] = beta;
      if (a.rowsum) a.rowsum[row] = local_sum;
    }
    __syncwarp();                                    // the next row overwrites the staging area
  }
}

// Q_a(h) when the row maxima are already known (the gate/up GEMM epilogue accumulates them with
// atomicMax): a pure streaming pass.  A work item is a run of `seg_units` 16-element units of one
// row; a warp takes items round-robin and its lanes take the run's units 32 bytes at a time, two
// loads in flight per lane.  Row, scale and the row sum are handled once per item, not per unit.
//
// Eq. 8 for one unit of 16 elements: the division-free form (r = x * c, c = fl(127 * fl(1/beta)))
// per element, which needs the division only where r is within 2^-14 of a
// half-integer: |r - 127x/beta| <= 127 * 3 * 2^-24 and |fl(fl(127x)/beta) - 127x/beta| <= 127 * 2^-24
// add up to 3.03e-5 < 2^-14, so outside that band both round to the same integer.  A unit with such
// an element (one in 500) is redone by an out-of-line function, so that the streaming loop holds
// neither the division's instructions nor a branch per element: 13 instead of 18 instructions per
// element on rows of 4864, 9.4 on rows of 11008.  (The two kernels above keep the branch per element: with the out-of-line call the
// row-staging kernel spills and drops from 3.5 to 2.9 TB/s, and the scatter kernel gains at
// T = 8192 what it loses at T <= 4096, under 0.4 % of the layer either way.)
constexpr float kQaFastBand = 0.49993896484375f;   // 0.5 - 2^-14

__device__ __forceinline__ uint4 pack_unit(const uint32_t (&qv)[16], int interleave) {
  uint32_t o[4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
    o[i] = interleave ? pack_low_bytes(qv[i], qv[4 + i], qv[8 + i], qv[12 + i])
                      : pack_low_bytes(qv[4 * i], qv[4 * i + 1], qv[4 * i + 2], qv[4 * i + 3]);
  return make_uint4(o[0], o[1], o[2], o[3]);
}

// `band` is kQaFastBand, or a negative number for a row whose scale is outside the range in which
// the division-free form is valid (every element then takes the division).
__device__ __forceinline__ float qa_band(const QaScale& s) { return s.fast ? kQaFastBand : -1.0f; }

__device__ __noinline__ uint4 quant_unit_exact(uint4 wa, uint4 wb, float beta, float c, float band, int interleave) {
  const uint32_t w[8] = {wa.x, wa.y, wa.z, wa.w, wb.x, wb.y, wb.z, wb.w};
  uint32_t qv[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const float x = (j & 1) ? bf16_hi(w[j >> 1]) : bf16_lo(w[j >> 1]);
    const float r = __fmul_rn(x, c);
    const float m = __fadd_rn(r, kMagic);
    const float frac = __fsub_rn(r, __fsub_rn(m, kMagic));
    qv[j] = (fabsf(frac) < band) ? __float_as_uint(m) : (uint32_t)quant_one(x, beta);
  }
  return pack_unit(qv, interleave);
}

// The unit's 16 codes, packed (plain or interleaved byte order).
__device__ __forceinline__ uint4 quant_unit(uint4 wa, uint4 wb, float beta, float c, float band, int interleave) {
  const uint32_t w[8] = {wa.x, wa.y, wa.z, wa.w, wb.x, wb.y, wb.z, wb.w};
  uint32_t qv[16];
  bool exact = false;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const float r0 = __fmul_rn(bf16_lo(w[j]), c), r1 = __fmul_rn(bf16_hi(w[j]), c);
    const float m0 = __fadd_rn(r0, kMagic), m1 = __fadd_rn(r1, kMagic);
    const float f0 = __fsub_rn(r0, __fsub_rn(m0, kMagic)), f1 = __fsub_rn(r1, __fsub_rn(m1, kMagic));
    qv[2 * j] = __float_as_uint(m0);
    qv[2 * j + 1] = __float_as_uint(m1);
    exact = exact || !(fabsf(f0) < band) || !(fabsf(f1) < band);
  }
  uint4 o = pack_unit(qv, interleave);
  if (exact) o = quant_unit_exact(wa, wb, beta, c, band, interleave);
  return o;
}

// sum of the 16 codes of a packed unit
__device__ __forceinline__ int unit_sum(uint4 o) {
  int sum = __dp4a((int)o.x, 0x01010101, 0);
  sum = __dp4a((int)o.y, 0x01010101, sum);
  sum = __dp4a((int)o.z, 0x01010101, sum);
  return __dp4a((int)o.w, 0x01010101, sum);
}

__global__ void __launch_bounds__(256) quant_rows_known_beta_kernel(const uint4* __restrict__ h, int64_t n_items,
                                                                    int units_per_row, int seg_units, int nseg,
                                                                    uint4* __restrict__ q, float* beta,
                                                                    int32_t* __restrict__ rowsum, int interleave,
                                                                    int early_trigger) {
  const int lane = threadIdx.x & 31;
  const int64_t n_warps = (int64_t(gridDim.x) * blockDim.x) >> 5;
  pdl_wait();                            // no-op unless launched as a programmatic dependent
  // decode path: the down kernel may start on work that does not need this kernel's output.  (Not
  // for the tensor path: its persistent GEMM CTAs would take this kernel's registers away.)
  if (early_trigger) pdl_trigger();
  for (int64_t item = (int64_t(blockIdx.x) * blockDim.x + threadIdx.x) >> 5; item < n_items; item += n_warps) {
    const int row = (int)(item / nseg);
    const int seg = (int)(item - int64_t(row) * nseg);
    const int u_end = min((seg + 1) * seg_units, units_per_row);
    const float b = fmaxf(beta[row], kEpsScale);
    const QaScale qs = qa_scale(b);
    const float band = qa_band(qs);
    const uint4* hr = h + int64_t(row) * units_per_row * 2;
    uint4* qr = q + int64_t(row) * units_per_row;
    int sum = 0;
    for (int u = seg * seg_units + lane; u < u_end; u += 64) {
      const bool second = u + 32 < u_end;
      uint32_t w0[8], w1[8];
      ptx::ld_global_v8(hr + u * 2, w0);            // a unit's 16 bf16 values: one 32-byte load
      if (second) ptx::ld_global_v8(hr + (u + 32) * 2, w1);
      const uint4 o0 = quant_unit(make_uint4(w0[0], w0[1], w0[2], w0[3]), make_uint4(w0[4], w0[5], w0[6], w0[7]), b,
                                  qs.c, band, interleave);
      qr[u] = o0;
      sum += unit_sum(o0);
      if (second) {
        const uint4 o1 = quant_unit(make_uint4(w1[0], w1[1], w1[2], w1[3]), make_uint4(w1[4], w1[5], w1[6], w1[7]), b,
                                    qs.c, band, interleave);
        qr[u + 32] = o1;
        sum += unit_sum(o1);
      }
    }
    sum = __reduce_add_sync(0xffffffffu, sum);
    if (lane == 0) {
      atomicAdd(rowsum + row, sum);
      if (seg == 0) beta[row] = b;                  // publish the clamped scale
    }
  }
}

mote_status_t launch_quant_rows_known_beta(const void* h_bf16, int64_t rows, int n, int8_t* q, float* beta,
                                           int32_t* rowsum, int interleave, cudaStream_t stream, bool pdl,
                                           bool early_trigger) {
  if (rows == 0) return MOTE_OK;
  const int units_per_row = n / 16;
  // Runs of equal length, 32 units at least, and about four times as many warps as are resident at
  // once, two runs each: measured against one resident wave of longer-lived warps (8 % slower at
  // T = 8192, f = 11008) and against shorter runs (one load round per run: 5-25 % slower).
  const int64_t target_warps = int64_t(device_sm_count()) * 256;
  const int max_seg = (units_per_row + 31) / 32;
  int nseg = (int)std::min<int64_t>(std::max<int64_t>((target_warps + rows - 1) / rows, 1), max_seg);
  const int seg_units = (units_per_row + nseg - 1) / nseg;
  nseg = (units_per_row + seg_units - 1) / seg_units;
  const int64_t items = rows * nseg;
  const int64_t per_warp = (items + target_warps - 1) / target_warps;
  const int64_t warps = (items + per_warp - 1) / per_warp;
  const unsigned blocks = (unsigned)((warps + 7) / 8);
  if (pdl)
    MOTE_CUDA_OK(launch_pdl(quant_rows_known_beta_kernel, dim3(blocks), dim3(256), 0, stream,
                            static_cast<const uint4*>(h_bf16), items, units_per_row, seg_units, nseg,
                            reinterpret_cast<uint4*>(q), beta, rowsum, interleave, early_trigger ? 1 : 0));
  else
    quant_rows_known_beta_kernel<<<blocks, 256, 0, stream>>>(static_cast<const uint4*>(h_bf16), items, units_per_row,
                                                             seg_units, nseg, reinterpret_cast<uint4*>(q), beta,
                                                             rowsum, interleave, 0);
  ++g_launch_count;
  MOTE_LAUNCH_OK();
  return MOTE_OK;
}

mote_status_t launch_quant_act(const QuantActArgs& a, bool scatter, cudaStream_t stream) {
  if (a.T == 0) return MOTE_OK;
  if (!scatter && a.d >= 1024) {
    // warp per row: eight warps per CTA, fewer where eight staged rows (2 * d bytes each) would not fit
    const size_t row_bytes = size_t(a.d) * 2;
    const int warps = (int)std::max<size_t>(1, std::min<size_t>(8, (200 * 1024) / row_bytes));
    const int64_t ctas_needed = (a.T + warps - 1) / warps;
    const unsigned blocks = (unsigned)std::min<int64_t>(ctas_needed, int64_t(device_sm_count()) * 32);
    static PerDeviceOnce attr_once;
    MOTE_CUDA_OK(set_max_dynamic_smem(attr_once, quant_act_rows_kernel, 200 * 1024));
    quant_act_rows_kernel<<<blocks, warps * 32, warps * row_bytes, stream>>>(a);
    ++g_launch_count;
    MOTE_LAUNCH_OK();
    return MOTE_OK;
  }
  const int n_units = a.d / 16;
  // smallest power-of-two group with at most 2 units per thread (up to 8 for the widest rows): with
  // two the kernel fits four CTAs per SM, and it is the rows in flight per SM that set its time
  int G = 32;
  while (G < 256 && n_units > G * 2) G <<= 1;
  const int upt = (n_units + G - 1) / G;
  QuantActArgs args = a;
  args.group = G;
  const int threads = 256;
  const int rows_per_cta = threads / G;
  const unsigned blocks = (unsigned)((a.T + rows_per_cta - 1) / rows_per_cta);
#define MOTE_QA_LAUNCH(U)                                                          \
  do {                                                                             \
    if (scatter && args.blk_base)                                                   \
      MOTE_CUDA_OK(launch_pdl(quant_act_kernel<U, true>, dim3(blocks), dim3(threads), 0, stream, args)); \
    else if (scatter) quant_act_kernel<U, true><<<blocks, threads, 0, stream>>>(args);  \
    else quant_act_kernel<U, false><<<blocks, threads, 0, stream>>>(args);         \
  } while (0)
  if (upt <= 1) MOTE_QA_LAUNCH(1);
  else if (upt <= 2) MOTE_QA_LAUNCH(2);
  else if (upt <= 4) MOTE_QA_LAUNCH(4);
  else MOTE_QA_LAUNCH(8);
#undef MOTE_QA_LAUNCH
  ++g_launch_count;
  MOTE_LAUNCH_OK();
  return MOTE_OK;
}

}  // namespace mote

extern "C" mote_status_t mote_quant_act(const void* x_bf16, int64_t T, int64_t d, int64_t ldx,
                                        int8_t* q, float* beta, int32_t* rowsum, void* stream) {
  using namespace mote;
  if (T < 0 || d <= 0 || (d % 16) != 0 || d > 32768 || ldx < d || (ldx % 8) != 0) return MOTE_ERR_SHAPE;
  if (T == 0) return MOTE_OK;
  if (!x_bf16 || !q || !beta) return MOTE_ERR_NULL;
  if (!aligned16(x_bf16) || !aligned16(q)) return MOTE_ERR_ALIGN;
  QuantActArgs a{};
  a.x = x_bf16; a.T = T; a.d = (int)d; a.ldx = ldx; a.q = q; a.beta = beta; a.rowsum = rowsum;
  a.perm = nullptr; a.k = 1; a.interleave = 0;
  return launch_quant_act(a, false, static_cast<cudaStream_t>(stream));
}
