// Host-side declarations shared by the translation units of libmote (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "mote.h"

namespace mote {

struct QuantActArgs {
  const void* x;        // bf16 [T, ldx]
  int64_t T;
  int d;
  int64_t ldx;
  int8_t* q;            // [rows, d]
  float* beta;          // [rows]
  int32_t* rowsum;      // [rows] or null
  const int32_t* perm;  // scatter variant: pair (t*k+j) -> destination row (when blk_base is null)
  // scatter variant with the block-wise dispatch: the destination row is derived here from the
  // top-k indices and the per-block bases, and written to perm_out / inv_out
  const int32_t* topk_idx; const int32_t* blk_base; int E; int n_blk;
  int32_t* perm_out; int32_t* inv_out;
  uint32_t* zero_u32; int32_t* zero_i32;   // optional [rows] arrays cleared at every destination row
  int k;
  int interleave;       // 1: store each unit of 16 codes k-interleaved
  int group;            // threads per row (set by the launcher)
};
mote_status_t launch_quant_act(const QuantActArgs& a, bool scatter, cudaStream_t stream);

// Router (Eq. 3).  Arguments as mote_route_topk.
// blk_hist (optional, written only by the tensor-core kernel, i.e. when d % 32 == 0):
// [E][blk_stride(n_blk)] pairs per expert of every block of kRouteBlockTokens tokens, n_blk =
// ceil(T / kRouteBlockTokens); expert-major, so that the scan reads an expert's counts contiguously.
constexpr int kRouteBlockTokens = 16;
#ifdef __CUDACC__
__host__ __device__
#endif
constexpr int blk_stride(int n_blk) { return (n_blk + 3) & ~3; }   // rows start on 16-byte boundaries
mote_status_t launch_route_topk(const void* x, int64_t T, int d, const float* Wr, const float* bias,
                                int E, int k, int norm_topk, int32_t* idx, float* w, float* logits,
                                int32_t* blk_hist, cudaStream_t stream, uint32_t* zero_word = nullptr);
// zero_word (optional, tensor-core kernel only): a word the kernel's first thread sets to zero.

// Stable grouping of the T*k pairs by expert: offsets[E+1], perm[P] (pair -> row), inv[P] (row -> pair).
// Optionally also writes the 128-row tile tables of the tensor-core GEMMs ([0] = {count},
// [1+i] = {expert, first row, rows}); tiles_routed needs 1 + P/128 + E entries, tiles_shared
// 1 + ceil(T/128).
mote_status_t launch_dispatch(const int32_t* idx, int64_t P, int E, int32_t* offsets, int32_t* perm,
                              int32_t* inv, int4* tiles_routed, int4* tiles_shared, int64_t T,
                              cudaStream_t stream);

// Block-wise variant: offsets, per-block bases and the tile tables from the router's block histograms.
mote_status_t launch_dispatch_scan(const int32_t* blk_hist, int n_blk, int E, int32_t* offsets, int32_t* blk_base,
                                   int4* tiles_routed, int4* tiles_shared, int64_t T, cudaStream_t stream);

// CUDA-core (dp4a) grouped ternary GEMMs.  qa rows are in expert-sorted order, canonical k order.
struct TernaryGemmArgs {
  const int8_t* qa;          // [P, K] int8 activations, sorted rows
  const float* beta;         // [P]
  const int32_t* offsets;    // [E+1]
  const uint8_t* w0;         // [E][N, K/4] packed (gate, or down)
  const uint8_t* w1;         // [E][N, K/4] packed up (gate/up mode) or null
  const float* alpha0;       // [E]
  const float* alpha1;       // [E] or null
  int E, N, K;
  int64_t P;
  // outputs
  void* h_bf16;              // gate/up mode: [P, N] bf16
  float* y;                  // down mode: [P, N] fp32
  int32_t* acc0_tap;         // optional [P, N]
  int32_t* acc1_tap;         // optional [P, N]
};
mote_status_t launch_ternary_gateup_simt(const TernaryGemmArgs& a, cudaStream_t stream);
mote_status_t launch_ternary_down_simt(const TernaryGemmArgs& a, cudaStream_t stream);

// Tensor-core (tcgen05) versions.  qa must be stored k-interleaved (see quant_act.cu); needs
// K % 128 == 0 and N % 128 == 0.
// beta_out_bits (gate/up only, may be null): per row, atomicMax of the bits of |h| (must be zeroed).
mote_status_t launch_ternary_umma(const TernaryGemmArgs& a, bool gateup, const int4* tiles, int max_mtiles,
                                  const int32_t* rowsum, uint32_t* beta_out_bits, uint32_t* status,
                                  cudaStream_t stream, bool pdl = false);

// Q_a(h) for rows whose absmax is already known: beta_bits holds max |h| per row (raw bits);
// writes q (k-interleaved if asked), the clamped beta in place, and accumulates rowsum (zeroed).
// pdl: launch as a programmatic dependent of the kernel before it on the stream (decode path)
mote_status_t launch_quant_rows_known_beta(const void* h_bf16, int64_t rows, int n, int8_t* q, float* beta,
                                           int32_t* rowsum, int interleave, cudaStream_t stream, bool pdl = false,
                                           bool early_trigger = false);
// One matrix of the shared expert: bf16 values (bits = 16, scale unused) or the codes of
// mote_rtn_quant (bits = 8 or 4: int8 rows, or 4-bit codes in the pair-split word order) with one
// scale per row.
struct SharedMat { const void* w; const float* scale; };

// comb (down projection only, may be null): fold the combine of Eq. 2 / Eq. 4 into the epilogue and
// write the layer output directly; `out` (fp32 s) may then be null.
struct CombineArgs {
  const float* y; const float* w; const int32_t* perm; const void* residual; void* out; int k;
};
// k_splits > 1 (down projection only, no comb): `out` receives k_splits partial outputs of T x N
// floats each, to be added in ascending order (see shared_down_k_splits).
mote_status_t launch_shared_umma(const void* act, const SharedMat& w0, const SharedMat& w1, int bits, bool gateup,
                                 int64_t T, int K, int N, void* out, const int4* tiles, int max_mtiles,
                                 uint32_t* status, const CombineArgs* comb, cudaStream_t stream, bool pdl = false,
                                 int k_splits = 1);
// Diagnostic: one CTA waits on an mbarrier that nothing arrives at, with the GEMM kernels' bounded
// wait and teardown; after limit_ns it raises *status and returns.
mote_status_t launch_bounded_wait_selftest(uint32_t* status, uint64_t limit_ns, cudaStream_t stream);
constexpr int64_t kMaxPartialRows = 4096;
int shared_down_k_splits(int64_t T, int N, int K);

// CUDA-core GEMMs of the shared expert.
mote_status_t launch_shared_gateup_simt(const void* x, const SharedMat& Wg, const SharedMat& Wu, int bits, int64_t T,
                                        int d, int f, void* h_bf16, cudaStream_t stream);
mote_status_t launch_shared_down_simt(const void* h, const SharedMat& Wd, int bits, int64_t T, int d, int f, float* s,
                                      cudaStream_t stream);

// Decode path (T <= 64): prologue (Q_a(x), router, dispatch), streamed gate/up, Q_a(h), streamed
// down with the combine.  Fills topk_*, offsets/perm/inv, qx (TOKEN order, k-interleaved),
// beta_x/rowsum_x (token order), h, beta_h, qh, rowsum_h, y, hs, s and the layer output.
struct DecodeStreamArgs {
  const void* x; int64_t T; int d, f, E, k, norm_topk;
  const float* Wr; const float* router_bias;
  const uint8_t* gate_packed; const uint8_t* up_packed; const uint8_t* down_packed;
  const float* alpha_gate; const float* alpha_up; const float* alpha_down;
  SharedMat sh_gate, sh_up, sh_down; int shared_bits;      // 16, 8 or 4
  int32_t* topk_idx; float* topk_w; int32_t* offsets; int32_t* perm; int32_t* inv;
  int8_t* qx; float* beta_x; int32_t* rowsum_x;
  void* h; int8_t* qh; float* beta_h; int32_t* rowsum_h; float* y; void* hs; float* s;
  uint32_t* counter;                       // one zeroed word
  int zero_head_words;                     // T = 1: the prologue zeroes this many words from (counter - 1) on
                                           // itself (status word, counter, tile counters); else 0
  uint32_t* tile_count;                    // d/16 zeroed words
  const void* residual; void* out;         // [T, d] bf16 (residual may be null, may alias out)
  int32_t* tap_gate; int32_t* tap_up; int32_t* tap_down;   // optional
};
bool decode_stream_supported(int d, int f, int E, int k, int64_t T);
// phase 0: prologue, 1: gate/up (routed + shared), 2: down (routed + shared); Q_a(h) runs between 1 and 2
mote_status_t launch_decode_stream(const DecodeStreamArgs& a, int phase, cudaStream_t stream);

// y = bf16(x * rsqrt(mean(x^2) + eps)) per row (the LN of Eq. 2, unit gain)
mote_status_t launch_rms_norm(const void* x, int64_t T, int d, float eps, void* y, cudaStream_t stream);

// out = [residual +] s + sum_j w_j * y[perm[t*k+j]]
// s may hold n_partials partial outputs of T x d floats each; they are added in ascending order.
mote_status_t launch_combine(const float* s, const float* y, const float* w, const int32_t* perm,
                             const void* residual, int64_t T, int d, int k, void* out_bf16,
                             cudaStream_t stream, bool pdl = false, int n_partials = 1);

}  // namespace mote
