// Host side of mote_moe_forward: argument checks, workspace plan, launch sequence (Eq. 2-8).
//
//   S1 route -> S2 dispatch -> S3 Q_a(x) scattered to expert-sorted rows -> S4 gate/up ternary
//   GEMM (+dequant, SwiGLU) -> S5 Q_a(h) -> S6 down ternary GEMM -> S7 shared bf16 FFN ->
//   S8 combine.  Everything is enqueued on the caller's stream; nothing synchronises.
#include <algorithm>

#include "mote_common.cuh"
#include "mote_internal.h"

namespace mote {

thread_local int g_launch_count = 0;

// Set while mote_stack_forward runs its layers: the stack clears the device status word once, at
// its start, and the layer calls inside it leave the word alone, so that a bounded wait that ran
// out in ANY layer is still there when the caller reads mote_device_status after the stack.
static thread_local bool g_keep_status = false;

// Head of a workspace: the status word, the decode prologue's arrival counter and the decode down
// kernel's tile counters (one per 16 output columns, from byte 256 on).
static inline size_t status_region_bytes(int d) { return 256 + size_t(d / 16) * 4; }

// Optional per-stage CUDA events (mote_moe_forward_profile): event i is recorded on the launch
// stream after stage i has been enqueued, event 0 before the first stage.
struct StageTimer {
  cudaEvent_t ev[MOTE_N_STAGES + 1];
  bool active = false;
};
static thread_local StageTimer g_timer;
static inline void stage_mark(int i, cudaStream_t stream) {
  if (g_timer.active) cudaEventRecord(g_timer.ev[i], stream);
}

// Head of the workspace: [0] device status word (cleared at the start of every top-level call),
// [1] arrival counter of the decode prologue, from byte 256 on the per-tile arrival counters of the
// decode path's down kernel (d / 16 <= 2048 words); the counters are cleared by every layer call.
constexpr size_t kStatusBytes = 256 + 2048 * 4;

struct Plan {
  size_t status, topk_idx, topk_w, offsets, perm, inv;
  size_t qx, beta_x, rowsum_x, h, qh, beta_h, rowsum_h, y, hs, s, tiles_routed, tiles_shared, blk_hist, blk_base;
  size_t total;
  size_t sh_codes_bf16;   // the three RTN-coded shared matrices expanded to bf16 (prefill); after `total`
  size_t total_expanded;
};

// From this many tokens on, a prefill with an RTN-coded shared expert first expands the codes of the
// layer to bf16 in the workspace (one streaming pass) and runs the plain bf16 GEMMs on them; below,
// the GEMM expands the codes tile by tile in shared memory (less weight traffic, more work per row tile).
constexpr int64_t kExpandMinTokens = 768;
constexpr int64_t kStreamAutoMaxTokens = 32;

static Plan make_plan(int d, int f, int E, int k, int64_t T) {
  Plan p{};
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += round_up(std::max<size_t>(bytes, 1), 256); return o; };
  const size_t P = size_t(T) * k;
  p.status = take(kStatusBytes);
  p.topk_idx = take(P * 4);
  p.topk_w = take(P * 4);
  p.offsets = take(size_t(E + 1) * 4);
  p.perm = take(P * 4);
  p.inv = take(P * 4);
  p.qx = take(P * size_t(d));
  p.beta_x = take(P * 4);
  p.rowsum_x = take(P * 4);
  p.h = take(P * size_t(f) * 2);
  p.qh = take(P * size_t(f));
  p.beta_h = take(P * 4);
  p.rowsum_h = take(P * 4);
  p.y = take(P * size_t(d) * 4);
  p.hs = take(size_t(T) * f * 2);
  // room for the partial outputs of a K-split shared down projection (short prefills)
  p.s = take(size_t(std::max<int64_t>(T, std::min<int64_t>(kMaxPartialRows, 16 * T))) * d * 4);
  p.tiles_routed = take((1 + P / 128 + E) * 16);
  p.tiles_shared = take((1 + (size_t(T) + 127) / 128) * 16);
  const size_t n_blk = (size_t(T) + kRouteBlockTokens - 1) / kRouteBlockTokens;
  p.blk_hist = take(size_t(blk_stride((int)n_blk)) * E * 4);
  p.blk_base = take(size_t(blk_stride((int)n_blk)) * E * 4);
  p.total = off;
  p.sh_codes_bf16 = take(T >= kExpandMinTokens ? size_t(3) * d * f * 2 : 1);
  p.total_expanded = T >= kExpandMinTokens ? off : p.total;
  return p;
}

// RTN codes (int8, or 4-bit in the pair-split word order) -> the same integers as bf16, 16 code
// bytes per thread and step.
struct ExpandArgs { const uint4* codes[3]; uint4* out[3]; };
__global__ void __launch_bounds__(256) expand_codes_kernel(ExpandArgs a, int64_t n_chunks, int bits) {
  const uint4* __restrict__ codes = a.codes[blockIdx.y];     // blockIdx.y: gate, up, down
  uint4* __restrict__ out = a.out[blockIdx.y];
  const int64_t stride = int64_t(gridDim.x) * blockDim.x;
  for (int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n_chunks; i += stride) {
    const uint4 w = codes[i];
    const uint32_t pw[4] = {w.x, w.y, w.z, w.w};
    if (bits == 8) {
      uint32_t e[8];
#pragma unroll
      for (int j = 0; j < 4; ++j) s8x4_to_bf16x2(pw[j], e[2 * j], e[2 * j + 1]);
      out[2 * i] = make_uint4(e[0], e[1], e[2], e[3]);
      out[2 * i + 1] = make_uint4(e[4], e[5], e[6], e[7]);
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        uint32_t e[4];
        u4x8_to_bf16x2(pw[j], e);
        out[4 * i + j] = make_uint4(e[0], e[1], e[2], e[3]);
      }
    }
  }
}

static mote_status_t launch_expand_codes(const ExpandArgs& a, int64_t elements, int bits, cudaStream_t stream) {
  const int64_t n_chunks = elements / (bits == 8 ? 16 : 32);
  const unsigned grid = (unsigned)std::min<int64_t>((n_chunks + 255) / 256, 148 * 8);
  expand_codes_kernel<<<dim3(grid, 3), 256, 0, stream>>>(a, n_chunks, bits);
  ++g_launch_count;
  MOTE_LAUNCH_OK();
  return MOTE_OK;
}

static bool shape_ok(int d, int f, int E, int k) {
  return d > 0 && f > 0 && d % 16 == 0 && f % 16 == 0 && d <= 32768 && f <= 32768 && E >= 1 &&
         E <= MOTE_MAX_EXPERTS && k >= 1 && k <= E && k <= MOTE_MAX_TOPK;
}

// Copies int8 rows, undoing the k-interleaved storage of each 16-code unit when asked, with an
// optional row map (dst row r <- src row map[r * map_stride]).
__global__ void copy_q_rows_kernel(const int8_t* __restrict__ src, int8_t* __restrict__ dst, int64_t rows,
                                   int n_units, const int32_t* __restrict__ map, int map_stride, int deinterleave) {
  const int64_t total = rows * n_units;
  const int64_t stride = int64_t(gridDim.x) * blockDim.x;
  for (int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; i < total; i += stride) {
    const int64_t r = i / n_units;
    const int u = (int)(i - r * n_units);
    const int64_t sr = map ? int64_t(map[r * map_stride]) : r;
    uint4 v = reinterpret_cast<const uint4*>(src)[sr * n_units + u];
    if (deinterleave) {
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
      uint32_t o[4];
#pragma unroll
      for (int b = 0; b < 4; ++b)
        o[b] = ((w[0] >> (8 * b)) & 0xFFu) | (((w[1] >> (8 * b)) & 0xFFu) << 8) |
               (((w[2] >> (8 * b)) & 0xFFu) << 16) | (((w[3] >> (8 * b)) & 0xFFu) << 24);
      v = make_uint4(o[0], o[1], o[2], o[3]);
    }
    reinterpret_cast<uint4*>(dst)[r * n_units + u] = v;
  }
}

// dst[i] = sum_p src[p * n + i], p ascending (the partial outputs of a K-split projection; tap only)
__global__ void sum_partials_kernel(const float* __restrict__ src, int n_partials, int64_t n, float* __restrict__ dst) {
  const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float acc = src[i];
  for (int p = 1; p < n_partials; ++p) acc += src[int64_t(p) * n + i];
  dst[i] = acc;
}

__global__ void gather_f32_kernel(const float* __restrict__ src, float* __restrict__ dst, int64_t n,
                                  const int32_t* __restrict__ map, int map_stride) {
  const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = src[map[i * map_stride]];
}

}  // namespace mote

using namespace mote;

extern "C" const char* mote_status_string(mote_status_t st) {
  switch (st) {
    case MOTE_OK: return "ok";
    case MOTE_ERR_NULL: return "null pointer";
    case MOTE_ERR_SHAPE: return "unsupported shape";
    case MOTE_ERR_ALIGN: return "misaligned pointer or stride";
    case MOTE_ERR_WORKSPACE: return "workspace missing or too small";
    case MOTE_ERR_DTYPE: return "unknown dtype";
    case MOTE_ERR_CUDA: return "CUDA error";
    case MOTE_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case MOTE_ERR_TOO_LARGE: return "input larger than this entry point's fixed capacity";
  }
  return "unknown status";
}

extern "C" size_t mote_workspace_bytes(int d, int f, int E, int k, int64_t T_max) {
  if (!shape_ok(d, f, E, k) || T_max < 0 || T_max > (int64_t(1) << 24)) return 0;
  return make_plan(d, f, E, k, T_max).total;
}

extern "C" size_t mote_layer_workspace_bytes(const mote_layer_t* L, int64_t T_max) {
  if (!L || !shape_ok(L->d, L->f, L->E, L->k) || T_max < 0 || T_max > (int64_t(1) << 24)) return 0;
  const Plan pl = make_plan(L->d, L->f, L->E, L->k, T_max);
  const bool rtn = L->shared_bits == MOTE_SHARED_INT8 || L->shared_bits == MOTE_SHARED_INT4;
  return rtn ? pl.total_expanded : pl.total;
}

extern "C" size_t mote_host_staging_bytes(int d, int64_t T_max) {
  if (d <= 0 || T_max < 0) return 0;
  return 3 * round_up(size_t(T_max) * d * 2, 256);
}

extern "C" int mote_last_launch_count(void) { return g_launch_count; }

extern "C" mote_status_t mote_device_status(void* ws, void* stream_) {
  if (!ws) return MOTE_ERR_NULL;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  uint32_t word = 0;
  MOTE_CUDA_OK(cudaMemcpyAsync(&word, ws, sizeof(word), cudaMemcpyDeviceToHost, stream));
  MOTE_CUDA_OK(cudaStreamSynchronize(stream));
  if (word != 0) {
    MOTE_CUDA_OK(cudaMemsetAsync(ws, 0, sizeof(word), stream));
    return MOTE_ERR_DEVICE_TIMEOUT;
  }
  return MOTE_OK;
}

extern "C" mote_status_t mote_selftest_bounded_wait(void* ws, uint64_t limit_ns, void* stream_) {
  if (!ws) return MOTE_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return MOTE_ERR_ALIGN;
  if (limit_ns < 1000ull || limit_ns > 100000000ull) return MOTE_ERR_SHAPE;
  return launch_bounded_wait_selftest(static_cast<uint32_t*>(ws), limit_ns, static_cast<cudaStream_t>(stream_));
}

extern "C" mote_status_t mote_moe_forward(const mote_layer_t* L, const void* x, const void* residual, int64_t T,
                                          void* out, const mote_taps_t* taps, void* ws, size_t ws_bytes,
                                          void* stream_) {
  g_launch_count = 0;
  if (!L) return MOTE_ERR_NULL;
  const int d = L->d, f = L->f, E = L->E, k = L->k;
  if (!shape_ok(d, f, E, k) || T < 0 || T > (int64_t(1) << 24)) return MOTE_ERR_SHAPE;
  if (L->path < MOTE_PATH_AUTO || L->path > MOTE_PATH_STREAM) return MOTE_ERR_SHAPE;
  if (T == 0) return MOTE_OK;
  if (!x || !out || !ws || !L->Wr || !L->gate_packed || !L->up_packed || !L->down_packed || !L->alpha_gate ||
      !L->alpha_up || !L->alpha_down || !L->sh_gate || !L->sh_up || !L->sh_down)
    return MOTE_ERR_NULL;
  if (x == out) return MOTE_ERR_SHAPE;
  const int sh_bits = L->shared_bits == 0 ? MOTE_SHARED_BF16 : L->shared_bits;
  if (sh_bits != MOTE_SHARED_BF16 && sh_bits != MOTE_SHARED_INT8 && sh_bits != MOTE_SHARED_INT4) return MOTE_ERR_SHAPE;
  const bool sh_rtn = sh_bits != MOTE_SHARED_BF16;
  if (sh_rtn && (!L->sh_gate_scale || !L->sh_up_scale || !L->sh_down_scale)) return MOTE_ERR_NULL;
  const SharedMat sh_gate{L->sh_gate, sh_rtn ? L->sh_gate_scale : nullptr};
  const SharedMat sh_up{L->sh_up, sh_rtn ? L->sh_up_scale : nullptr};
  const SharedMat sh_down{L->sh_down, sh_rtn ? L->sh_down_scale : nullptr};
  const void* ptrs[] = {x, out, residual, L->Wr, L->gate_packed, L->up_packed, L->down_packed,
                        L->sh_gate, L->sh_up, L->sh_down, sh_gate.scale, sh_up.scale, sh_down.scale};
  for (const void* p : ptrs)
    if (p && !aligned16(p)) return MOTE_ERR_ALIGN;
  if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return MOTE_ERR_ALIGN;
  const Plan pl = make_plan(d, f, E, k, T);
  if (ws_bytes < pl.total) return MOTE_ERR_WORKSPACE;
  const int64_t P = T * k;
  if ((P + 31) / 32 + E > 65535) return MOTE_ERR_SHAPE;

  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  char* base = static_cast<char*>(ws);
  auto* topk_idx = reinterpret_cast<int32_t*>(base + pl.topk_idx);
  auto* topk_w = reinterpret_cast<float*>(base + pl.topk_w);
  auto* offsets = reinterpret_cast<int32_t*>(base + pl.offsets);
  auto* perm = reinterpret_cast<int32_t*>(base + pl.perm);
  auto* inv = reinterpret_cast<int32_t*>(base + pl.inv);
  auto* qx = reinterpret_cast<int8_t*>(base + pl.qx);
  auto* beta_x = reinterpret_cast<float*>(base + pl.beta_x);
  auto* rowsum_x = reinterpret_cast<int32_t*>(base + pl.rowsum_x);
  void* h = base + pl.h;
  auto* qh = reinterpret_cast<int8_t*>(base + pl.qh);
  auto* beta_h = reinterpret_cast<float*>(base + pl.beta_h);
  auto* rowsum_h = reinterpret_cast<int32_t*>(base + pl.rowsum_h);
  auto* y = reinterpret_cast<float*>(base + pl.y);
  void* hs = base + pl.hs;
  auto* s = reinterpret_cast<float*>(base + pl.s);

  auto* status = reinterpret_cast<uint32_t*>(base + pl.status);
  auto* tiles_routed = reinterpret_cast<int4*>(base + pl.tiles_routed);
  auto* tiles_shared = reinterpret_cast<int4*>(base + pl.tiles_shared);
  const int max_mtiles_routed = (int)(P / 128 + E);
  const int max_mtiles_shared = (int)((T + 127) / 128);

  const bool tensor_ok = (d % 128 == 0) && (f % 128 == 0);
  const bool stream_ok = decode_stream_supported(d, f, E, k, T);
  int path = L->path;
  // AUTO: the weight stream up to 32 tokens (beyond that its eight-column-tile kernels run at low
  // occupancy and the tcgen05 GEMMs, with the shared down projection split along K, are faster)
  if (path == MOTE_PATH_AUTO)
    path = (stream_ok && (T <= kStreamAutoMaxTokens || !tensor_ok)) ? MOTE_PATH_STREAM
           : tensor_ok ? MOTE_PATH_TENSOR : MOTE_PATH_SIMT;
  if (path == MOTE_PATH_STREAM && !stream_ok) return MOTE_ERR_SHAPE;
  if (path == MOTE_PATH_TENSOR && !tensor_ok) return MOTE_ERR_SHAPE;
  const bool tensor = (path == MOTE_PATH_TENSOR);
  const int interleave = (tensor || path == MOTE_PATH_STREAM) ? 1 : 0;

  if (path == MOTE_PATH_STREAM) {
    // status word, the prologue's arrival counter, the down kernel's tile counters
    // (the kernels leave their counters at zero, so inside a stack the stack's one memset is enough)
    // (a single-token call lets its prologue kernel do it: one operation less on the stream)
    const bool prologue_zeroes = !g_keep_status && T == 1;
    if (!g_keep_status && !prologue_zeroes) MOTE_CUDA_OK(cudaMemsetAsync(status, 0, status_region_bytes(d), stream));
    stage_mark(0, stream);
    DecodeStreamArgs ds{};
    ds.zero_head_words = prologue_zeroes ? int(status_region_bytes(d) / 4) : 0;
    ds.x = x; ds.T = T; ds.d = d; ds.f = f; ds.E = E; ds.k = k; ds.norm_topk = L->norm_topk;
    ds.Wr = L->Wr; ds.router_bias = L->router_bias;
    ds.gate_packed = L->gate_packed; ds.up_packed = L->up_packed; ds.down_packed = L->down_packed;
    ds.alpha_gate = L->alpha_gate; ds.alpha_up = L->alpha_up; ds.alpha_down = L->alpha_down;
    ds.sh_gate = sh_gate; ds.sh_up = sh_up; ds.sh_down = sh_down; ds.shared_bits = sh_bits;
    ds.topk_idx = topk_idx; ds.topk_w = topk_w; ds.offsets = offsets; ds.perm = perm; ds.inv = inv;
    ds.qx = qx; ds.beta_x = beta_x; ds.rowsum_x = rowsum_x; ds.h = h; ds.qh = qh; ds.beta_h = beta_h;
    ds.rowsum_h = rowsum_h; ds.y = y; ds.hs = hs; ds.s = s; ds.counter = status + 1;
    ds.tile_count = status + 64; ds.residual = residual; ds.out = out;
    ds.tap_gate = taps ? taps->acc_gate : nullptr; ds.tap_up = taps ? taps->acc_up : nullptr;
    ds.tap_down = taps ? taps->acc_down : nullptr;
    if (taps && (!taps->acc_gate != !taps->acc_up)) return MOTE_ERR_NULL;
    mote_status_t st = launch_decode_stream(ds, 0, stream);   // Q_a(x), router, dispatch in one kernel
    if (st) return st;
    stage_mark(1, stream); stage_mark(2, stream); stage_mark(3, stream);
    st = launch_decode_stream(ds, 1, stream);                 // routed and shared gate/up
    if (st) return st;
    stage_mark(4, stream);
    st = launch_quant_rows_known_beta(h, P, f, qh, beta_h, rowsum_h, 1, stream, true, true);
    if (st) return st;
    stage_mark(5, stream);
    st = launch_decode_stream(ds, 2, stream);                 // routed and shared down, combine
    if (st) return st;
    stage_mark(6, stream); stage_mark(7, stream); stage_mark(8, stream); stage_mark(9, stream);
    if (taps) {
      auto d2d = [&](void* dst, const void* src, size_t bytes) -> bool {
        return !dst || cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, stream) == cudaSuccess;
      };
      bool ok = d2d(taps->topk_idx, topk_idx, P * 4) && d2d(taps->topk_w, topk_w, P * 4) &&
                d2d(taps->offsets, offsets, size_t(E + 1) * 4) && d2d(taps->perm, perm, P * 4) &&
                d2d(taps->beta_x, beta_x, size_t(T) * 4) && d2d(taps->h_bf16, h, size_t(P) * f * 2) &&
                d2d(taps->beta_h, beta_h, P * 4) && d2d(taps->y, y, size_t(P) * d * 4) &&
                d2d(taps->shared_out, s, size_t(T) * d * 4);
      if (!ok) return MOTE_ERR_CUDA;
      if (taps->qx) {   // token order already; undo the k-interleave
        copy_q_rows_kernel<<<148, 256, 0, stream>>>(qx, taps->qx, T, d / 16, nullptr, 0, 1);
        MOTE_LAUNCH_OK();
      }
      if (taps->qh) {
        copy_q_rows_kernel<<<148, 256, 0, stream>>>(qh, taps->qh, P, f / 16, nullptr, 0, 1);
        MOTE_LAUNCH_OK();
      }
    }
    return MOTE_OK;
  }

  mote_status_t st;
  // device status word: cleared by the router kernel where the tensor-core router runs (one
  // operation less on the stream), else by a memset
  const bool router_clears = !g_keep_status && tensor && (d % 32 == 0);
  if (!g_keep_status && !router_clears) MOTE_CUDA_OK(cudaMemsetAsync(status, 0, 4, stream));
  stage_mark(0, stream);
  // S1 router, S2 dispatch
  // block-wise dispatch: the tensor-core router (d % 32 == 0) leaves per-block expert counts, a small
  // scan turns them into bases, and Q_a(x) derives every pair's sorted row itself
  const bool blockwise = tensor && (d % 32 == 0);
  auto* blk_hist = reinterpret_cast<int32_t*>(base + pl.blk_hist);
  auto* blk_base = reinterpret_cast<int32_t*>(base + pl.blk_base);
  const int n_blk = (int)((T + kRouteBlockTokens - 1) / kRouteBlockTokens);
  st = launch_route_topk(x, T, d, L->Wr, L->router_bias, E, k, L->norm_topk, topk_idx, topk_w, nullptr,
                         blockwise ? blk_hist : nullptr, stream, router_clears ? status : nullptr);
  if (st) return st;
  stage_mark(1, stream);
  st = blockwise ? launch_dispatch_scan(blk_hist, n_blk, E, offsets, blk_base, tiles_routed, tiles_shared, T, stream)
                 : launch_dispatch(topk_idx, P, E, offsets, perm, inv, tensor ? tiles_routed : nullptr,
                                   tensor ? tiles_shared : nullptr, T, stream);
  if (st) return st;
  stage_mark(2, stream);
  // S3 Q_a(x), written once per selected expert into the expert-sorted rows
  QuantActArgs qa{};
  qa.x = x; qa.T = T; qa.d = d; qa.ldx = d; qa.q = qx; qa.beta = beta_x; qa.rowsum = rowsum_x;
  qa.perm = perm; qa.k = k; qa.interleave = interleave;
  if (blockwise) {
    qa.topk_idx = topk_idx; qa.blk_base = blk_base; qa.E = E; qa.n_blk = n_blk; qa.perm_out = perm; qa.inv_out = inv;
    qa.zero_u32 = reinterpret_cast<uint32_t*>(beta_h); qa.zero_i32 = rowsum_h;
  }
  const bool pdl = blockwise;    // from here on every kernel is a programmatic dependent of the one before
  st = launch_quant_act(qa, true, stream);
  if (st) return st;
  stage_mark(3, stream);
  // S4 gate/up
  TernaryGemmArgs g1{};
  g1.qa = qx; g1.beta = beta_x; g1.offsets = offsets; g1.w0 = L->gate_packed; g1.w1 = L->up_packed;
  g1.alpha0 = L->alpha_gate; g1.alpha1 = L->alpha_up; g1.E = E; g1.N = f; g1.K = d; g1.P = P;
  g1.h_bf16 = h; g1.acc0_tap = taps ? taps->acc_gate : nullptr; g1.acc1_tap = taps ? taps->acc_up : nullptr;
  if (tensor && !blockwise)   // beta_h (atomicMax target) and rowsum_h (atomicAdd target) are adjacent
    MOTE_CUDA_OK(cudaMemsetAsync(beta_h, 0, (pl.rowsum_h - pl.beta_h) + size_t(P) * 4, stream));
  st = tensor ? launch_ternary_umma(g1, true, tiles_routed, max_mtiles_routed, rowsum_x,
                                    reinterpret_cast<uint32_t*>(beta_h), status, stream, pdl)
              : launch_ternary_gateup_simt(g1, stream);
  if (st) return st;
  stage_mark(4, stream);
  // S5 Q_a(h)
  QuantActArgs qb{};
  qb.x = h; qb.T = P; qb.d = f; qb.ldx = f; qb.q = qh; qb.beta = beta_h; qb.rowsum = rowsum_h;
  qb.perm = nullptr; qb.k = 1; qb.interleave = interleave;
  st = tensor ? launch_quant_rows_known_beta(h, P, f, qh, beta_h, rowsum_h, interleave, stream, pdl)
              : launch_quant_act(qb, false, stream);
  if (st) return st;
  stage_mark(5, stream);
  // S6 down
  TernaryGemmArgs g2{};
  g2.qa = qh; g2.beta = beta_h; g2.offsets = offsets; g2.w0 = L->down_packed; g2.alpha0 = L->alpha_down;
  g2.E = E; g2.N = d; g2.K = f; g2.P = P; g2.y = y; g2.acc0_tap = taps ? taps->acc_down : nullptr;
  st = tensor ? launch_ternary_umma(g2, false, tiles_routed, max_mtiles_routed, rowsum_h, nullptr, status, stream, pdl)
              : launch_ternary_down_simt(g2, stream);
  if (st) return st;
  stage_mark(6, stream);
  // S7 shared expert
  // prefill with an RTN-coded shared expert and room in the workspace: expand the codes to bf16 once
  SharedMat xg = sh_gate, xu = sh_up, xd = sh_down;
  int x_bits = sh_bits;
  if (sh_rtn && tensor && T >= kExpandMinTokens && ws_bytes >= pl.total_expanded) {
    char* e0 = base + pl.sh_codes_bf16;
    const size_t mat = size_t(d) * f * 2;
    ExpandArgs ea{};
    for (int i = 0; i < 3; ++i) {
      ea.codes[i] = static_cast<const uint4*>(i == 0 ? sh_gate.w : i == 1 ? sh_up.w : sh_down.w);
      ea.out[i] = reinterpret_cast<uint4*>(e0 + i * mat);
    }
    st = launch_expand_codes(ea, int64_t(d) * f, sh_bits, stream);
    if (st) return st;
    xg.w = e0; xu.w = e0 + mat; xd.w = e0 + 2 * mat;
    x_bits = MOTE_SHARED_BF16;                     // bf16 operands; the row scales still apply
  }
  st = tensor ? launch_shared_umma(x, xg, xu, x_bits, true, T, d, f, hs, tiles_shared, max_mtiles_shared,
                                   status, nullptr, stream, pdl)
              : launch_shared_gateup_simt(x, sh_gate, sh_up, sh_bits, T, d, f, hs, stream);
  if (st) return st;
  stage_mark(7, stream);
  const int k_splits = tensor ? shared_down_k_splits(T, d, f) : 1;
  if (tensor && k_splits > 1) {
    // few row tiles: the shared down projection is cut along K, its partial outputs are added by the combine
    st = launch_shared_umma(hs, xd, SharedMat{nullptr, nullptr}, x_bits, false, T, f, d, s, tiles_shared,
                            max_mtiles_shared, status, nullptr, stream, pdl, k_splits);
    if (st) return st;
    stage_mark(8, stream);
    st = launch_combine(s, y, topk_w, perm, residual, T, d, k, out, stream, pdl, k_splits);
    if (st) return st;
  } else if (tensor) {
    // shared down projection with S8 (combine, residual, bf16 rounding) in its epilogue; the fp32
    // shared output is written only when a tap asks for it
    CombineArgs cb{y, topk_w, perm, residual, out, k};
    st = launch_shared_umma(hs, xd, SharedMat{nullptr, nullptr}, x_bits, false, T, f, d,
                            (taps && taps->shared_out) ? s : nullptr, tiles_shared, max_mtiles_shared, status, &cb,
                            stream, pdl);
    if (st) return st;
    stage_mark(8, stream);
  } else {
    st = launch_shared_down_simt(hs, sh_down, sh_bits, T, d, f, s, stream);
    if (st) return st;
    stage_mark(8, stream);
    // S8 combine
    st = launch_combine(s, y, topk_w, perm, residual, T, d, k, out, stream);
    if (st) return st;
  }
  stage_mark(9, stream);

  if (taps) {
    auto d2d = [&](void* dst, const void* src, size_t bytes) -> bool {
      return !dst || cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, stream) == cudaSuccess;
    };
    bool ok = d2d(taps->topk_idx, topk_idx, P * 4) && d2d(taps->topk_w, topk_w, P * 4) &&
              d2d(taps->offsets, offsets, size_t(E + 1) * 4) && d2d(taps->perm, perm, P * 4) &&
              d2d(taps->h_bf16, h, size_t(P) * f * 2) && d2d(taps->beta_h, beta_h, P * 4) &&
              d2d(taps->y, y, size_t(P) * d * 4) &&
              (k_splits > 1 || d2d(taps->shared_out, s, size_t(T) * d * 4));
    if (!ok) return MOTE_ERR_CUDA;
    if (k_splits > 1 && taps->shared_out) {
      const int64_t n = T * d;
      sum_partials_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(s, k_splits, n, taps->shared_out);
      MOTE_LAUNCH_OK();
    }
    if (taps->qx) {
      copy_q_rows_kernel<<<148 * 4, 256, 0, stream>>>(qx, taps->qx, T, d / 16, perm, k, interleave);
      MOTE_LAUNCH_OK();
    }
    if (taps->beta_x) {
      gather_f32_kernel<<<(unsigned)((T + 255) / 256), 256, 0, stream>>>(beta_x, taps->beta_x, T, perm, k);
      MOTE_LAUNCH_OK();
    }
    if (taps->qh) {
      copy_q_rows_kernel<<<148 * 4, 256, 0, stream>>>(qh, taps->qh, P, f / 16, nullptr, 0, interleave);
      MOTE_LAUNCH_OK();
    }
  }
  return MOTE_OK;
}

extern "C" size_t mote_stack_workspace_bytes(const mote_layer_t* layers, int n_layers, int64_t T_max) {
  if (!layers || n_layers < 1 || T_max < 0) return 0;
  size_t core = 0;
  for (int l = 0; l < n_layers; ++l) {
    const size_t b = mote_layer_workspace_bytes(&layers[l], T_max);
    if (b == 0 || layers[l].d != layers[0].d) return 0;
    core = std::max(core, b);
  }
  return core + 3 * round_up(size_t(T_max) * layers[0].d * 2, 256);   // two residual-stream slabs + LN output
}

extern "C" mote_status_t mote_stack_forward(const mote_layer_t* layers, int n_layers, float rms_eps, const void* x,
                                            int64_t T, void* out, void* layer_inputs, void* ws, size_t ws_bytes,
                                            void* stream_) {
  if (!layers) return MOTE_ERR_NULL;
  if (n_layers < 1 || T < 0 || !(rms_eps >= 0.0f)) return MOTE_ERR_SHAPE;
  if (T == 0) return MOTE_OK;
  if (!x || !out || !ws) return MOTE_ERR_NULL;
  if (x == out) return MOTE_ERR_SHAPE;
  const size_t need = mote_stack_workspace_bytes(layers, n_layers, T);
  if (need == 0) return MOTE_ERR_SHAPE;
  if (ws_bytes < need) return MOTE_ERR_WORKSPACE;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const int d = layers[0].d;
  const size_t row_bytes = size_t(T) * d * 2;
  const size_t slab = round_up(row_bytes, 256);
  const size_t core = need - 3 * slab;
  char* ping = static_cast<char*>(ws) + core;
  void* normed = ping + 2 * slab;
  int launches = 0;
  const void* res = x;                                 // residual stream x_{l-1}
  // device status word and the decode kernels' counters: once for the whole stack
  MOTE_CUDA_OK(cudaMemsetAsync(ws, 0, status_region_bytes(d), stream));
  struct KeepStatus { KeepStatus() { g_keep_status = true; } ~KeepStatus() { g_keep_status = false; } } keep_status;
  for (int l = 0; l < n_layers; ++l) {
    void* dst = (l == n_layers - 1) ? out : static_cast<void*>(ping + size_t(l & 1) * slab);
    if (layer_inputs)
      MOTE_CUDA_OK(cudaMemcpyAsync(static_cast<char*>(layer_inputs) + size_t(l) * row_bytes, res, row_bytes,
                                   cudaMemcpyDeviceToDevice, stream));
    const void* in = res;
    if (rms_eps > 0.0f) {
      g_launch_count = 0;
      const mote_status_t sn = launch_rms_norm(res, T, d, rms_eps, normed, stream);
      if (sn) return sn;
      launches += g_launch_count;
      in = normed;
    }
    const mote_status_t st = mote_moe_forward(&layers[l], in, res, T, dst, nullptr, ws, core, stream);
    if (st) return st;
    launches += g_launch_count;
    res = dst;
  }
  g_launch_count = launches;
  return MOTE_OK;
}

// Copy streams and events of the pipelined host call below: made on a thread's first long call on a
// device and kept for the thread's life time.
struct HostPipe {
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t start = nullptr, copied[2] = {nullptr, nullptr}, computed[2] = {nullptr, nullptr}, done = nullptr;
  bool ready = false;
};
static thread_local HostPipe g_host_pipe[kMaxDevices];

static HostPipe* host_pipe() {
  const int dev = current_device();
  if (dev < 0 || dev >= kMaxDevices) return nullptr;
  HostPipe& p = g_host_pipe[dev];
  if (p.ready) return &p;
  bool ok = cudaStreamCreateWithFlags(&p.in, cudaStreamNonBlocking) == cudaSuccess &&
            cudaStreamCreateWithFlags(&p.out, cudaStreamNonBlocking) == cudaSuccess;
  cudaEvent_t* evs[] = {&p.start, &p.copied[0], &p.copied[1], &p.computed[0], &p.computed[1], &p.done};
  for (cudaEvent_t* e : evs) ok = ok && cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess;
  if (!ok) return nullptr;                             // the caller falls back to the plain sequence
  p.ready = true;
  return &p;
}

// Prefills of this many tokens or more go through the device as two halves: the second half's input
// copy runs beside the first half's layer, the first half's output copy beside the second half's
// layer (tokens are independent of one another, Eq. 2-4, so the halves are too).
constexpr int64_t kHostPipelineMinTokens = 4096;

extern "C" mote_status_t mote_moe_forward_host(const mote_layer_t* L, const void* x_host, const void* residual_host,
                                               int64_t T, void* out_host, void* ws, size_t ws_bytes, void* stream_) {
  if (!L) return MOTE_ERR_NULL;
  if (T < 0) return MOTE_ERR_SHAPE;
  if (T == 0) return MOTE_OK;
  if (!x_host || !out_host || !ws) return MOTE_ERR_NULL;
  const size_t core = mote_layer_workspace_bytes(L, T);
  if (core == 0) return MOTE_ERR_SHAPE;
  const size_t slab = round_up(size_t(T) * L->d * 2, 256);
  if (ws_bytes < core + 3 * slab) return MOTE_ERR_WORKSPACE;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  char* stage = static_cast<char*>(ws) + core;
  char* x_dev = stage;
  char* res_dev = residual_host ? stage + slab : nullptr;
  char* out_dev = stage + 2 * slab;
  const size_t row = size_t(L->d) * 2;
  const size_t bytes = size_t(T) * row;
  HostPipe* pipe = T >= kHostPipelineMinTokens ? host_pipe() : nullptr;
  if (!pipe) {
    MOTE_CUDA_OK(cudaMemcpyAsync(x_dev, x_host, bytes, cudaMemcpyHostToDevice, stream));
    if (residual_host) MOTE_CUDA_OK(cudaMemcpyAsync(res_dev, residual_host, bytes, cudaMemcpyHostToDevice, stream));
    mote_status_t st = mote_moe_forward(L, x_dev, res_dev, T, out_dev, nullptr, ws, core, stream);
    if (st) return st;
    MOTE_CUDA_OK(cudaMemcpyAsync(out_host, out_dev, bytes, cudaMemcpyDeviceToHost, stream));
    MOTE_CUDA_OK(cudaStreamSynchronize(stream));
    return MOTE_OK;
  }
  const int64_t t0[3] = {0, (T / 2 + 127) / 128 * 128, T};       // the halves: whole row tiles in the first
  MOTE_CUDA_OK(cudaEventRecord(pipe->start, stream));             // the copies start after the stream's earlier work
  MOTE_CUDA_OK(cudaStreamWaitEvent(pipe->in, pipe->start, 0));
  for (int c = 0; c < 2; ++c) {
    const size_t off = size_t(t0[c]) * row, n = size_t(t0[c + 1] - t0[c]) * row;
    MOTE_CUDA_OK(cudaMemcpyAsync(x_dev + off, static_cast<const char*>(x_host) + off, n, cudaMemcpyHostToDevice, pipe->in));
    if (residual_host)
      MOTE_CUDA_OK(cudaMemcpyAsync(res_dev + off, static_cast<const char*>(residual_host) + off, n, cudaMemcpyHostToDevice,
                                   pipe->in));
    MOTE_CUDA_OK(cudaEventRecord(pipe->copied[c], pipe->in));
  }
  MOTE_CUDA_OK(cudaMemsetAsync(ws, 0, status_region_bytes(L->d), stream));   // status word, counters: once for both halves
  mote_status_t st = MOTE_OK;
  {
    struct KeepStatus { KeepStatus() { g_keep_status = true; } ~KeepStatus() { g_keep_status = false; } } keep_status;
    for (int c = 0; c < 2 && st == MOTE_OK; ++c) {
      const size_t off = size_t(t0[c]) * row;
      if (cudaStreamWaitEvent(stream, pipe->copied[c], 0) != cudaSuccess) { st = MOTE_ERR_CUDA; break; }
      st = mote_moe_forward(L, x_dev + off, res_dev ? res_dev + off : nullptr, t0[c + 1] - t0[c], out_dev + off, nullptr,
                            ws, core, stream);
      if (st) break;
      if (cudaEventRecord(pipe->computed[c], stream) != cudaSuccess ||
          cudaStreamWaitEvent(pipe->out, pipe->computed[c], 0) != cudaSuccess ||
          cudaMemcpyAsync(static_cast<char*>(out_host) + off, out_dev + off, size_t(t0[c + 1] - t0[c]) * row,
                          cudaMemcpyDeviceToHost, pipe->out) != cudaSuccess)
        st = MOTE_ERR_CUDA;
    }
  }
  // whatever happened, leave none of the helper streams' work behind
  const bool drained = cudaEventRecord(pipe->done, pipe->out) == cudaSuccess &&
                       cudaStreamWaitEvent(stream, pipe->done, 0) == cudaSuccess;
  const bool in_ok = cudaStreamSynchronize(pipe->in) == cudaSuccess;
  const bool out_ok = cudaStreamSynchronize(pipe->out) == cudaSuccess;
  const bool main_ok = cudaStreamSynchronize(stream) == cudaSuccess;
  if (st) return st;
  return (drained && in_ok && out_ok && main_ok) ? MOTE_OK : MOTE_ERR_CUDA;
}

extern "C" mote_status_t mote_moe_forward_profile(const mote_layer_t* L, const void* x, const void* residual,
                                                  int64_t T, void* out, void* ws, size_t ws_bytes, void* stream_,
                                                  float* stage_ms_host) {
  if (!stage_ms_host) return MOTE_ERR_NULL;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  for (int i = 0; i < MOTE_N_STAGES; ++i) stage_ms_host[i] = 0.0f;
  for (int i = 0; i <= MOTE_N_STAGES; ++i) MOTE_CUDA_OK(cudaEventCreate(&g_timer.ev[i]));
  g_timer.active = true;
  mote_status_t st = mote_moe_forward(L, x, residual, T, out, nullptr, ws, ws_bytes, stream);
  g_timer.active = false;
  if (st == MOTE_OK && T > 0) {
    if (cudaStreamSynchronize(stream) != cudaSuccess) st = MOTE_ERR_CUDA;
    for (int i = 0; st == MOTE_OK && i < MOTE_N_STAGES; ++i)
      if (cudaEventElapsedTime(&stage_ms_host[i], g_timer.ev[i], g_timer.ev[i + 1]) != cudaSuccess) st = MOTE_ERR_CUDA;
  }
  for (int i = 0; i <= MOTE_N_STAGES; ++i) cudaEventDestroy(g_timer.ev[i]);
  return st;
}
