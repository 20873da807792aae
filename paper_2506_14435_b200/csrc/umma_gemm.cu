// Tensor-core expert GEMMs for sm_100a: tcgen05.mma with TMEM accumulators, operands staged in
// shared memory by TMA, warp-specialised persistent CTAs (one per SM).
//
//   T_GATEUP  routed gate/up (Eq. 6): int8 tokens x 2-bit weights -> int32; epilogue applies
//             the dequantisation scales, SiLU and the gate*up product, writes h as bf16
//   T_DOWN    routed down (Eq. 5): int8 Q_a(h) x 2-bit weights -> int32 -> y fp32
//   B_GATEUP  shared expert gate/up (Eq. 2): bf16 x bf16 -> fp32 -> h_shared bf16
//   B_DOWN    shared expert down -> s fp32
//   Q8_*, Q4_* the same two with RTN INT8 / INT4 weight codes (Section 4.3): the codes travel to
//             shared memory as stored, the unpacker warps expand them to bf16 (exact: |q| <= 127)
//             in the swizzled operand layout, the MMA is the bf16 one and the epilogue multiplies
//             every output column by its row scale
//
// Tile: 128 token rows (UMMA M, one TMEM lane per row) x BN weight rows (UMMA N = 256; for a down
// projection the largest multiple of 32 up to 256 that divides its width, e.g. 224 for 896); K advances 128 bytes of the token
// operand per pipeline stage (128 int8 or 64 bf16), four K=32-byte MMAs per stage.
//
// Ternary weights travel as 2-bit codes all the way into shared memory (TMA box of 32 bytes per
// weight row and stage) and are expanded there to int8 by four unpacker warps, directly into the
// 128-byte-swizzled operand layout the MMA reads.  The stored code is code+1 in {0,1,2}, so the
// expansion is a shift and a mask ((w >> 2i) & 0x03030303); the weights enter the MMA as
// UNSIGNED int8 and the epilogue subtracts the token's row sum (sum_k q_k) to recover
// sum_k q_k * code_k exactly.  The shift/mask yields the 16 codes of a word in the order
// 0,4,8,12,1,5,...; the token operand is stored in the same order by the activation quantizer,
// and an integer dot product does not depend on the order of its terms.
//
// Warp roles (640 threads): 0 TMA producer of the token operand (and of bf16 weights),
// 1 TMA producer of packed weights, 2 MMA issuer + TMEM owner, 4-11 two groups of unpackers
// that take alternate pipeline stages, 12-19 epilogue (two warps per TMEM lane quarter, each
// owning half of the tile's columns).
// Two accumulator buffers of 256 TMEM columns let the epilogue of one tile overlap the MMAs of
// the next.  Every mbarrier wait is bounded; on expiry the CTA raises a status word and leaves.
#include <cuda.h>

#include <algorithm>
#include <mutex>

#include "mote_common.cuh"
#include "mote_internal.h"
#include "ptx_sm100.cuh"

namespace mote {

using namespace ptx;

enum { MODE_T_GATEUP = 0, MODE_T_DOWN = 1, MODE_B_GATEUP = 2, MODE_B_DOWN = 3,
       MODE_Q8_GATEUP = 4, MODE_Q8_DOWN = 5, MODE_Q4_GATEUP = 6, MODE_Q4_DOWN = 7 };

constexpr int kBM = 128;
constexpr int kStageA = kBM * 128;             // 16 KB: 128 rows x 128 B
constexpr int kStageB = 256 * 128;             // 32 KB: up to 256 rows x 128 B
constexpr int kStagesTernary = 3, kStagesBf16 = 4, kStagesRtn = 3;
constexpr int kThreads = 640;
constexpr int kTmemCols = 512;

struct UmmaArgs {
  const int4* tiles;        // [0] = {n_mtiles,0,0,0}; [1+i] = {expert, row0, rows, 0}
  int n_ntiles;             // tiles along the output columns
  int k_steps;              // pipeline stages along K (128 bytes of the token operand each)
  int k_splits;             // down projections: items per output tile, each over 1/k_splits of K (>= 1)
  int64_t split_stride;     // elements between the partial outputs of consecutive splits
  int bn;                   // weight rows per tile (UMMA N)
  int split_tail;           // down projections with bn = 256, k_splits = 1: see plan_items
  int n_out;                // output row length (f for gate/up, d for down)
  int b_rows_per_expert;    // rows of the weight tensor map per expert (0: shared expert)
  const float* beta;        // [rows]   (ternary modes)
  const int32_t* rowsum;    // [rows]
  const float* alpha0;      // [E]; RTN modes: [n_out] scale of every output column
  const float* alpha1;      // [E] (gate/up: alpha_up); RTN gate/up: [n_out] scales of the up matrix
  void* out;                // bf16 [rows, n_out] (gate/up) or fp32 [rows, n_out] (down)
  int32_t* tap0;            // optional int32 [rows, n_out]
  int32_t* tap1;
  uint32_t* beta_out_bits;  // gate/up of the routed experts: running max |h| per row (atomicMax on the bits)
  uint32_t* status;
  // shared down projection with the combine of Eq. 2 and Eq. 4 folded into its epilogue (comb_out != null):
  //   comb_out[t, :] = bf16( s[t, :] + sum_j comb_w[t, j] * comb_y[comb_perm[t*k + j], :] [+ comb_res[t, :]] )
  const float* comb_y; const float* comb_w; const int32_t* comb_perm; const uint16_t* comb_res; uint16_t* comb_out;
  int comb_k;
  int comb_wide;            // comb_res and comb_out are 32-byte aligned (the caller only promises 16): 32-byte accesses
};

struct __align__(8) PipeBarriers {
  uint64_t full_a[4], empty[4], full_u[4], full_p[4], empty_p[4], tmem_full[2], tmem_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};

template <int MODE>
struct ModeTraits {
  static constexpr bool kTernary = (MODE == MODE_T_GATEUP || MODE == MODE_T_DOWN);
  static constexpr int kRtnBits = MODE >= MODE_Q4_GATEUP ? 4 : MODE >= MODE_Q8_GATEUP ? 8 : 0;
  static constexpr bool kRtn = kRtnBits != 0;
  static constexpr bool kUnpack = kTernary || kRtn;       // weights reach shared memory as codes
  static constexpr bool kGateUp = (MODE % 2 == 0);
  static constexpr int kStages = kTernary ? kStagesTernary : kRtn ? kStagesRtn : kStagesBf16;
  // code bytes per weight row and pipeline stage: 128 2-bit codes, 64 int8 codes or 64 4-bit codes
  static constexpr int kCodeRowBytes = kRtnBits == 8 ? 64 : 32;
  static constexpr int kStageP = 256 * kCodeRowBytes;     // up to 256 rows
  static constexpr int kStagesP = kRtnBits == 8 ? 3 : 4;
  // gate/up epilogue: every epilogue warp stages 32 rows x kEpiCols bf16 (row pitch padded by 16 B)
  // and writes them out as whole row segments
  // (bf16 gate/up only.  For the ternary gate/up, whose epilogue competes with the unpackers for
  // issue slots, staging -- with plain stores or with a TMA store -- measured slower than letting
  // every thread write its own 32 bytes.)
  static constexpr int kEpiCols = 32;
  static constexpr int kEpiPitch = kEpiCols * 2 + 16;
  static constexpr size_t kEpiStage = (kGateUp && !kTernary) ? size_t(8) * 32 * kEpiPitch : 0;
  static constexpr size_t kSmem = 1024 + size_t(kStages) * (kStageA + kStageB) +
                                  (kUnpack ? size_t(kStagesP) * kStageP : 0) + kEpiStage + sizeof(PipeBarriers);
};

// Item order.  The CTAs of the grid work on neighbouring items at the same time, and the operand
// those items share is the one L2 serves to all of them from a single HBM read.
//   gate/up: row tile fastest -- concurrent items share the (small) weight tile; the token operand
//            (T x d) stays in L2 across column tiles;
//   down:    column tile fastest -- concurrent items share the token operand (P x f, larger than
//            L2 for long prefills), which is then read from HBM once instead of once per column tile.
// A down projection with few row tiles may split K over k_splits items per output tile (each
// writes its partial sums; the caller adds them in a fixed order): item = (row tile, split, column tile).
//
// The items of the last, partial round of the persistent grid would leave most SMs idle for a whole
// tile time (512 tiles on 148 CTAs: 3.46 rounds cost 4).  Where at most half of the CTAs have a
// tile left in that round, a down projection with 256-column tiles cuts each of those tiles into its
// two 128-column halves, one item each: the round then takes 0.57 of a tile time (the MMA pipe runs
// N = 128 at 0.87 of its N = 256 rate).  Items [0, n_whole) are whole tiles, [n_whole, n_items) halves.
struct ItemPlan { int n_items, n_whole; };
template <bool kGateUp>
__device__ __forceinline__ ItemPlan plan_items(const UmmaArgs& a, int n_mtiles) {
  ItemPlan p;
  p.n_items = p.n_whole = n_mtiles * a.n_ntiles * (kGateUp ? 1 : a.k_splits);
  if (!kGateUp && a.split_tail) {
    const int tail = p.n_items % (int)gridDim.x;
    if (tail > 0 && 2 * tail <= (int)gridDim.x) { p.n_whole = p.n_items - tail; p.n_items += tail; }
  }
  return p;
}
// half: -1 for a whole tile, else which 128-column half of tile (m_tile, n_tile) the item is
template <bool kGateUp>
__device__ __forceinline__ void decode_item(const UmmaArgs& a, int item, int n_mtiles, int n_whole, int4& tile,
                                            int& n_tile, int& half) {
  half = -1;
  if (!kGateUp && item >= n_whole) {
    const int j = item - n_whole;
    item = n_whole + (j >> 1);
    half = j & 1;
  }
  int m_tile;
  if (kGateUp) { m_tile = item % n_mtiles; n_tile = item / n_mtiles; }
  else { m_tile = item / (a.n_ntiles * a.k_splits); n_tile = item % a.n_ntiles; }
  tile = a.tiles[1 + m_tile];
}
// pipeline steps [kb, ke) of an item, and which split it is
template <bool kGateUp>
__device__ __forceinline__ int item_k_range(const UmmaArgs& a, int item, int& kb, int& ke) {
  if (kGateUp || a.k_splits <= 1) { kb = 0; ke = a.k_steps; return 0; }
  const int split = (item / a.n_ntiles) % a.k_splits;
  kb = split * a.k_steps / a.k_splits;
  ke = (split + 1) * a.k_steps / a.k_splits;
  return split;
}

// What a CTA does after one of its bounded waits has run out (abort flag raised in shared memory):
// give copies and MMAs still in flight time to land before shared memory and TMEM go away ...
__device__ __forceinline__ void drain_after_abort(volatile int* abort_flag) {
  if (*abort_flag) {
    const uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
  }
}
// ... and raise the device status word the host reads with mote_device_status.
__device__ __forceinline__ void report_abort(volatile int* abort_flag, uint32_t* status) {
  if (*abort_flag) atomicExch(status, 1u);
}

// glu_h as ONE copy of code.  The gate/up epilogue recomputes about one element in a thousand with
// the pinned sequence, from a loop unrolled over sixteen elements: sixteen inlined copies of the
// division and the polynomial cost it instruction cache and scheduling freedom for nothing
// (8 % of the kernel at K = 896).
static __device__ __noinline__ float glu_h_rare(int acc_g, int acc_u, float c_g, float c_u) {
  return glu_h(acc_g, acc_u, c_g, c_u);
}

// ------------------------------------------------------------------------------------------------
template <int MODE>
__global__ void __launch_bounds__(kThreads, 1)
umma_gemm_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b0,
                 const __grid_constant__ CUtensorMap tm_b1, const UmmaArgs a) {
  using TR = ModeTraits<MODE>;
  constexpr int S = TR::kStages;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t sA = smem_base;
  const uint32_t sB = sA + S * kStageA;
  const uint32_t sP = sB + S * kStageB;
  uint8_t* genB = smem_gen + S * kStageA;
  uint8_t* genP = genB + S * kStageB;
  uint8_t* genE = genP + (TR::kUnpack ? TR::kStagesP * TR::kStageP : 0);
  PipeBarriers* bars = reinterpret_cast<PipeBarriers*>(genE + TR::kEpiStage);
  volatile int* abort_flag = &bars->abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < 4; ++s) {
      mbar_init(smem_u32(&bars->full_a[s]), 1);
      mbar_init(smem_u32(&bars->empty[s]), 1);
      mbar_init(smem_u32(&bars->full_u[s]), 4);
      mbar_init(smem_u32(&bars->full_p[s]), 1);
      mbar_init(smem_u32(&bars->empty_p[s]), 4);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bars->tmem_full[b]), 1);
      mbar_init(smem_u32(&bars->tmem_empty[b]), 8);
    }
    bars->abort_flag = 0;
    fence_barrier_init();
    prefetch_tensormap(&tm_a);
    prefetch_tensormap(&tm_b0);
    prefetch_tensormap(&tm_b1);
  }
  if (warp == 2) {
    tmem_alloc(smem_u32(&bars->tmem_base), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  pdl_wait();                              // set-up above overlaps the tail of the kernel before this one
  const int n_mtiles = a.tiles[0].x;
  const ItemPlan plan = plan_items<TR::kGateUp>(a, n_mtiles);
  const int n_items = plan.n_items, n_whole = plan.n_whole;

  if (warp == 0) {
    // ---------------------------------------------------------------- token-operand producer
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
        int4 tile; int n_tile, half;
        decode_item<TR::kGateUp>(a, item, n_mtiles, n_whole, tile, n_tile, half);
        const int width = half < 0 ? a.bn : 128;
        const int b_row = (a.b_rows_per_expert ? tile.x * a.b_rows_per_expert : 0) +
                          n_tile * (TR::kGateUp ? a.bn / 2 : a.bn) + (half > 0 ? 128 : 0);
        int kb, ke;
        item_k_range<TR::kGateUp>(a, item, kb, ke);
        for (int ks = kb; ks < ke; ++ks) {
          if (!(ok = mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1, abort_flag))) break;
          const uint32_t bar = smem_u32(&bars->full_a[stage]);
          if (TR::kTernary) {
            mbar_expect_tx(bar, kStageA);
            tma_load_2d(sA + stage * kStageA, &tm_a, ks * 128, tile.y, bar);
          } else if (TR::kRtn) {
            mbar_expect_tx(bar, kStageA);
            tma_load_2d(sA + stage * kStageA, &tm_a, ks * 64, tile.y, bar);
          } else {
            mbar_expect_tx(bar, kStageA + width * 128);
            tma_load_2d(sA + stage * kStageA, &tm_a, ks * 64, tile.y, bar);
            if (TR::kGateUp) {
              tma_load_2d(sB + stage * kStageB, &tm_b0, ks * 64, b_row, bar);
              tma_load_2d(sB + stage * kStageB + 128 * 128, &tm_b1, ks * 64, b_row, bar);
            } else {
              tma_load_2d(sB + stage * kStageB, &tm_b0, ks * 64, b_row, bar);
              if (width > 128) tma_load_2d(sB + stage * kStageB + 128 * 128, &tm_b1, ks * 64, b_row + 128, bar);
            }
          }
          if (++stage == S) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- packed-weight producer
    if (TR::kUnpack && lane == 0) {
      constexpr int kRB = TR::kCodeRowBytes;
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
        int4 tile; int n_tile, half;
        decode_item<TR::kGateUp>(a, item, n_mtiles, n_whole, tile, n_tile, half);
        const int width = half < 0 ? a.bn : 128;
        const int b_row = tile.x * a.b_rows_per_expert + n_tile * (TR::kGateUp ? a.bn / 2 : a.bn) + (half > 0 ? 128 : 0);
        int kb, ke;
        item_k_range<TR::kGateUp>(a, item, kb, ke);
        for (int ks = kb; ks < ke; ++ks) {
          if (!(ok = mbar_wait(smem_u32(&bars->empty_p[stage]), phase ^ 1, abort_flag))) break;
          const uint32_t bar = smem_u32(&bars->full_p[stage]);
          mbar_expect_tx(bar, width * kRB);
          const uint32_t dst = sP + stage * TR::kStageP;
          if (TR::kGateUp) {
            tma_load_2d(dst, &tm_b0, ks * kRB, b_row, bar);
            tma_load_2d(dst + 128 * kRB, &tm_b1, ks * kRB, b_row, bar);
          } else {
            tma_load_2d(dst, &tm_b0, ks * kRB, b_row, bar);
            if (width > 128) tma_load_2d(dst + 128 * kRB, &tm_b1, ks * kRB, b_row + 128, bar);
          }
          if (++stage == TR::kStagesP) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 2) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc_whole = TR::kTernary ? make_idesc(2, 1, 0, kBM, (uint32_t)a.bn)     // s32 += s8 * u8
                                                : make_idesc(1, 1, 1, kBM, (uint32_t)a.bn);    // f32 += bf16 * bf16
      const uint32_t idesc_half = TR::kTernary ? make_idesc(2, 1, 0, kBM, 128u) : make_idesc(1, 1, 1, kBM, 128u);
      uint32_t stage = 0, phase = 0;
      int local = 0;
      bool ok = true;
      for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x, ++local) {
        const int buf = local & 1;
        const uint32_t use = (uint32_t)(local >> 1);
        if (!(ok = mbar_wait(smem_u32(&bars->tmem_empty[buf]), (use & 1) ^ 1, abort_flag))) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * 256;
        const uint32_t idesc = (!TR::kGateUp && item >= n_whole) ? idesc_half : idesc_whole;
        int kb, ke;
        item_k_range<TR::kGateUp>(a, item, kb, ke);
        for (int ks = kb; ks < ke; ++ks) {
          if (!(ok = mbar_wait(smem_u32(&bars->full_a[stage]), phase, abort_flag))) break;
          if (TR::kUnpack)
            if (!(ok = mbar_wait(smem_u32(&bars->full_u[stage]), phase, abort_flag))) break;
          tc_fence_after();
          const uint64_t da = smem_desc_sw128(sA + stage * kStageA);
          const uint64_t db = smem_desc_sw128(sB + stage * kStageB);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t acc = (ks > kb || j > 0) ? 1u : 0u;
            if (TR::kTernary) mma_i8(d_tmem, da + 2 * j, db + 2 * j, idesc, acc);
            else mma_f16(d_tmem, da + 2 * j, db + 2 * j, idesc, acc);
          }
          mma_commit(smem_u32(&bars->empty[stage]));
          if (++stage == S) { stage = 0; phase ^= 1; }
        }
        if (ok) mma_commit(smem_u32(&bars->tmem_full[buf]));
      }
    }
  } else if (warp >= 4 && warp < 12) {
    // ---------------------------------------------------------------- code unpackers
    // (2-bit -> int8 for the ternary experts; int8 / 4-bit -> bf16 for an RTN-coded shared expert)
    // group 0 (warps 4-7) expands the even pipeline steps, group 1 (warps 8-11) the odd ones
    if (TR::kUnpack) {
      const int group = (warp - 4) >> 2;
      const int tid = (threadIdx.x - 128) & 127;
      uint32_t stage = 0, phase = 0, pstage = 0, pphase = 0, step = 0;
      bool ok = true;
      for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
        // chunks of 16 code bytes, spread over 128 threads
        const int n_chunks = ((!TR::kGateUp && item >= n_whole) ? 128 : a.bn) * (TR::kCodeRowBytes / 16);
        int kb, ke;
        item_k_range<TR::kGateUp>(a, item, kb, ke);
        for (int ks = kb; ks < ke; ++ks, ++step) {
          if ((step & 1u) == (uint32_t)group) {
            ok = mbar_wait(smem_u32(&bars->full_p[pstage]), pphase, abort_flag) &&
                 mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const uint8_t* src = genP + pstage * TR::kStageP;
            uint8_t* dst = genB + stage * kStageB;
            // batches of four chunks per thread, all loads of a batch ahead of its conversions
            for (int c0 = tid; c0 < n_chunks; c0 += 128 * 4) {
              uint4 wv[4];
#pragma unroll
              for (int b = 0; b < 4; ++b) {
                const int c = c0 + b * 128;
                if (c < n_chunks) wv[b] = *reinterpret_cast<const uint4*>(src + c * 16);
              }
#pragma unroll
              for (int b = 0; b < 4; ++b) {
                const int c = c0 + b * 128;
                if (c >= n_chunks) break;
                const uint32_t pw[4] = {wv[b].x, wv[b].y, wv[b].z, wv[b].w};
                if (TR::kRtnBits == 8) {
                  // 16 int8 codes -> two 16-byte pieces of 8 bf16 each
                  const int r = c >> 2, quarter = c & 3;
                  uint8_t* row = dst + (r >> 3) * 1024 + (r & 7) * 128;
                  uint32_t e[8];
#pragma unroll
                  for (int j = 0; j < 4; ++j) s8x4_to_bf16x2(pw[j], e[2 * j], e[2 * j + 1]);
                  *reinterpret_cast<uint4*>(row + (((quarter * 2) ^ (r & 7)) << 4)) = make_uint4(e[0], e[1], e[2], e[3]);
                  *reinterpret_cast<uint4*>(row + (((quarter * 2 + 1) ^ (r & 7)) << 4)) = make_uint4(e[4], e[5], e[6], e[7]);
                } else {
                  const int r = c >> 1, half = c & 1;
                  uint8_t* row = dst + (r >> 3) * 1024 + (r & 7) * 128;
#pragma unroll
                  for (int j = 0; j < 4; ++j) {
                    uint4 o;
                    if (TR::kRtnBits == 4) {
                      // 8 four-bit codes -> one 16-byte piece of 8 bf16
                      uint32_t e[4];
                      u4x8_to_bf16x2(pw[j], e);
                      o = make_uint4(e[0], e[1], e[2], e[3]);
                    } else {
                      o.x = pw[j] & 0x03030303u;
                      o.y = (pw[j] >> 2) & 0x03030303u;
                      o.z = (pw[j] >> 4) & 0x03030303u;
                      o.w = (pw[j] >> 6) & 0x03030303u;
                    }
                    *reinterpret_cast<uint4*>(row + (((half * 4 + j) ^ (r & 7)) << 4)) = o;
                  }
                }
              }
            }
            fence_proxy_async_smem();                // generic-proxy writes -> visible to the MMA
            __syncwarp();
            if (lane == 0) {
              mbar_arrive(smem_u32(&bars->full_u[stage]));
              mbar_arrive(smem_u32(&bars->empty_p[pstage]));
            }
          }
          if (++stage == S) { stage = 0; phase ^= 1; }
          if (++pstage == TR::kStagesP) { pstage = 0; pphase ^= 1; }
        }
      }
    }
  } else if (warp >= 12) {
    // ---------------------------------------------------------------- epilogue
    const int q = warp & 3;                          // TMEM lane quarter this warp may read
    const int chalf = (warp - 12) >> 2;              // which half of the tile's columns
    const int r_in_tile = q * 32 + lane;
    int local = 0;
    bool ok = true;
    for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x, ++local) {
      int4 tile; int n_tile, half;
      decode_item<TR::kGateUp>(a, item, n_mtiles, n_whole, tile, n_tile, half);
      int kb_, ke_;
      const int split = item_k_range<TR::kGateUp>(a, item, kb_, ke_);
      const int buf = local & 1;
      const uint32_t use = (uint32_t)(local >> 1);
      ok = mbar_wait(smem_u32(&bars->tmem_full[buf]), use & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const bool row_ok = r_in_tile < tile.z;
      const int64_t row = int64_t(tile.y) + r_in_tile;
      const uint32_t t_row = tmem_base + (uint32_t(q * 32) << 16) + buf * 256;
      float c0 = 0.f, c1 = 0.f;
      int rs = 0;
      if (TR::kTernary && row_ok) {
        const float beta = fmaxf(a.beta[row], kEpsScale);
        rs = a.rowsum[row];
        c0 = dequant_scale(a.alpha0[tile.x], beta);
        if (TR::kGateUp) c1 = dequant_scale(a.alpha1[tile.x], beta);
      }
      if (TR::kGateUp) {
        const int col0 = n_tile * 128;
        const bool row_fast = __fmul_rn(c0, c1) > 1e-12f;
        const uint32_t acc_bias = 0x4B400000u - (uint32_t)rs;
        float hmax = 0.0f;                           // max |h| (before the bf16 rounding, which is monotonic)
        constexpr int kCols = TR::kEpiCols, kPitch = TR::kEpiPitch;
        constexpr int kLanesPerRow = kCols * 2 / 16, kRowsPerStore = 32 / kLanesPerRow;
        uint8_t* stg = genE + (warp - 12) * 32 * kPitch;
#pragma unroll 1
        for (int cr = chalf * 64; cr < chalf * 64 + 64; cr += kCols) {
#pragma unroll 1
          for (int c = cr; c < cr + kCols; c += 16) {
            uint32_t rg[16], ru[16];
            tmem_ld_32x32b_x16(t_row + c, rg);
            tmem_ld_32x32b_x16(t_row + 128 + c, ru);
            tmem_wait_ld();
            if (row_ok) {
              float hv[16];
              if (TR::kTernary) {
                uint32_t redo_mask = 0u;
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                  bool redo;
                  hv[j] = glu_h_fast_biased(rg[j], ru[j], acc_bias, c0, c1, redo);
                  if (redo) redo_mask |= 1u << j;
                }
                if (!row_fast) redo_mask = 0xFFFFu;
                if (redo_mask) {                     // mostly one element: look at four at a time
#pragma unroll
                  for (int j0 = 0; j0 < 16; j0 += 4)
                    if ((redo_mask >> j0) & 0xFu) {
#pragma unroll
                      for (int j = j0; j < j0 + 4; ++j)
                        if ((redo_mask >> j) & 1u) hv[j] = glu_h_rare((int)rg[j] - rs, (int)ru[j] - rs, c0, c1);
                    }
                }
#pragma unroll
                for (int j = 0; j < 16; ++j) hmax = fmaxf(hmax, fabsf(hv[j]));
              } else if (TR::kRtn || a.alpha0 != nullptr) {
                // RTN-coded shared expert (codes expanded here, or beforehand): row scales of the
                // gate and up matrices = scales of this tile's output columns
                const float4* sgp = reinterpret_cast<const float4*>(a.alpha0 + col0 + c);
                const float4* sup = reinterpret_cast<const float4*>(a.alpha1 + col0 + c);
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                  const float4 sg = __ldg(sgp + v), su = __ldg(sup + v);
                  const float sgv[4] = {sg.x, sg.y, sg.z, sg.w}, suv[4] = {su.x, su.y, su.z, su.w};
#pragma unroll
                  for (int u = 0; u < 4; ++u) {
                    const float g = __uint_as_float(rg[4 * v + u]) * sgv[u];
                    hv[4 * v + u] = __uint_as_float(ru[4 * v + u]) * suv[u] * silu_fast(g);
                  }
                }
              } else {
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                  const float g = __uint_as_float(rg[j]);
                  hv[j] = __uint_as_float(ru[j]) * silu_fast(g);
                }
              }
              uint32_t packed[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) packed[j] = pack_bf16x2(hv[2 * j], hv[2 * j + 1]);
              if (TR::kTernary) {
                // the thread's 16 bf16 values are one 32-byte sector of its row: one store
                st_global_v8(reinterpret_cast<uint16_t*>(a.out) + row * a.n_out + col0 + c, packed[0], packed[1], packed[2],
                             packed[3], packed[4], packed[5], packed[6], packed[7]);
              } else {
                uint4* sdst = reinterpret_cast<uint4*>(stg + lane * kPitch + (c - cr) * 2);
                sdst[0] = make_uint4(packed[0], packed[1], packed[2], packed[3]);
                sdst[1] = make_uint4(packed[4], packed[5], packed[6], packed[7]);
              }
              if (TR::kTernary && a.tap0) {
                int4* t0 = reinterpret_cast<int4*>(a.tap0 + row * a.n_out + col0 + c);
                int4* t1 = reinterpret_cast<int4*>(a.tap1 + row * a.n_out + col0 + c);
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                  t0[v] = make_int4((int)rg[4 * v] - rs, (int)rg[4 * v + 1] - rs, (int)rg[4 * v + 2] - rs, (int)rg[4 * v + 3] - rs);
                  t1[v] = make_int4((int)ru[4 * v] - rs, (int)ru[4 * v + 1] - rs, (int)ru[4 * v + 2] - rs, (int)ru[4 * v + 3] - rs);
                }
              }
            }
          }
          if (!TR::kTernary) {
            __syncwarp();
            // the warp's 32 rows x kCols columns leave as whole row segments (kCols * 2 bytes each)
#pragma unroll
            for (int r0 = 0; r0 < 32; r0 += kRowsPerStore) {
              const int r = r0 + lane / kLanesPerRow, piece = lane % kLanesPerRow;
              if (q * 32 + r < tile.z) {
                const uint4 v = *reinterpret_cast<const uint4*>(stg + r * kPitch + piece * 16);
                uint16_t* orow = reinterpret_cast<uint16_t*>(a.out) + (int64_t(tile.y) + q * 32 + r) * a.n_out + col0 + cr;
                reinterpret_cast<uint4*>(orow)[piece] = v;
              }
            }
            __syncwarp();
          }
        }
        // bits of non-negative floats order like unsigned integers; bf16_rn(max) = max(bf16_rn)
        if (TR::kTernary && row_ok && a.beta_out_bits) {
          const uint32_t hb = f32_to_bf16_bits(hmax) << 16;
          if (hb) atomicMax(a.beta_out_bits + row, hb);
        }
      } else {
        const uint32_t acc_bias = 0x4B400000u - (uint32_t)rs;   // see glu_h_fast_biased
        const int width = half < 0 ? a.bn : 128;
        const int col0 = n_tile * a.bn + (half > 0 ? 128 : 0);
        const int cbeg = chalf * (width / 2), cend = cbeg + width / 2;
        const bool combine = !TR::kTernary && a.comb_out != nullptr;
        float cw[MOTE_MAX_TOPK];
        const float* cy[MOTE_MAX_TOPK];
        if (combine && row_ok) {
#pragma unroll
          for (int j = 0; j < MOTE_MAX_TOPK; ++j)
            if (j < a.comb_k) {
              cw[j] = a.comb_w[row * a.comb_k + j];
              cy[j] = a.comb_y + int64_t(a.comb_perm[row * a.comb_k + j]) * a.n_out + col0;
            }
        }
#pragma unroll 1
        for (int c = cbeg; c < cend; c += 16) {
          uint32_t ra[16];
          tmem_ld_32x32b_x16(t_row + c, ra);
          tmem_wait_ld();
          if (row_ok) {
            float o[16];
#pragma unroll
            for (int v = 0; v < 16; ++v)
              o[v] = TR::kTernary ? __fmul_rn(__fsub_rn(__uint_as_float(ra[v] + acc_bias), kMagic), c0)   // fl32(acc - rs) * c0
                                  : __uint_as_float(ra[v]);
            if (TR::kRtn || (!TR::kTernary && a.alpha0 != nullptr)) {
              const float4* sp = reinterpret_cast<const float4*>(a.alpha0 + col0 + c);
#pragma unroll
              for (int v = 0; v < 4; ++v) {
                const float4 sc = __ldg(sp + v);
                o[4 * v] *= sc.x; o[4 * v + 1] *= sc.y; o[4 * v + 2] *= sc.z; o[4 * v + 3] *= sc.w;
              }
            }
            if (a.out) {
              float* dst = reinterpret_cast<float*>(a.out) + split * a.split_stride + row * a.n_out + col0 + c;
#pragma unroll
              for (int v = 0; v < 2; ++v)
                st_global_v8(dst + 8 * v, __float_as_uint(o[8 * v]), __float_as_uint(o[8 * v + 1]), __float_as_uint(o[8 * v + 2]),
                             __float_as_uint(o[8 * v + 3]), __float_as_uint(o[8 * v + 4]), __float_as_uint(o[8 * v + 5]),
                             __float_as_uint(o[8 * v + 6]), __float_as_uint(o[8 * v + 7]));
            }
            if (TR::kTernary && a.tap0) {
              int4* t0 = reinterpret_cast<int4*>(a.tap0 + row * a.n_out + col0 + c);
#pragma unroll
              for (int v = 0; v < 4; ++v)
                t0[v] = make_int4((int)ra[4 * v] - rs, (int)ra[4 * v + 1] - rs, (int)ra[4 * v + 2] - rs, (int)ra[4 * v + 3] - rs);
            }
            if (combine) {
              // fp32, slots in ascending j, then the residual, one bf16 rounding
#pragma unroll
              for (int j = 0; j < MOTE_MAX_TOPK; ++j)
                if (j < a.comb_k) {
#pragma unroll
                  for (int v = 0; v < 2; ++v) {
                    uint32_t yv[8];
                    ld_global_v8(cy[j] + c + 8 * v, yv);
#pragma unroll
                    for (int u = 0; u < 8; ++u) o[8 * v + u] = fmaf(cw[j], __uint_as_float(yv[u]), o[8 * v + u]);
                  }
                }
              if (a.comb_res) {
                uint32_t rw[8];
                if (a.comb_wide) {
                  ld_global_v8(a.comb_res + row * a.n_out + col0 + c, rw);
                } else {
                  const uint4* rp = reinterpret_cast<const uint4*>(a.comb_res + row * a.n_out + col0 + c);
                  const uint4 r0 = rp[0], r1 = rp[1];
                  rw[0] = r0.x; rw[1] = r0.y; rw[2] = r0.z; rw[3] = r0.w; rw[4] = r1.x; rw[5] = r1.y; rw[6] = r1.z; rw[7] = r1.w;
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) { o[2 * u] += bf16_lo(rw[u]); o[2 * u + 1] += bf16_hi(rw[u]); }
              }
              uint32_t pk[8];
#pragma unroll
              for (int v = 0; v < 8; ++v) pk[v] = f32_to_bf16_bits(o[2 * v]) | (f32_to_bf16_bits(o[2 * v + 1]) << 16);
              if (a.comb_wide) {
                st_global_v8(a.comb_out + row * a.n_out + col0 + c, pk[0], pk[1], pk[2], pk[3], pk[4], pk[5], pk[6], pk[7]);
              } else {
                uint4* od = reinterpret_cast<uint4*>(a.comb_out + row * a.n_out + col0 + c);
                od[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                od[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
              }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->tmem_empty[buf]));
    }
  }

  // ------------------------------------------------------------------ teardown
  drain_after_abort(abort_flag);
  tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
  if (threadIdx.x == 0) report_abort(abort_flag, a.status);
}

// One CTA that runs the GEMM kernels' bounded wait to its limit: an mbarrier nothing ever arrives
// at, no copy and no MMA in flight.  The wait gives up after limit_ns, the CTA takes the same
// teardown as the GEMM (drain, status word) and returns normally; the context stays usable.
__global__ void bounded_wait_selftest_kernel(uint32_t* status, uint64_t limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_word;
  volatile int* abort_flag = &abort_word;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_word = 0;
    fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) (void)mbar_wait(smem_u32(&bar), 0, abort_flag, limit_ns);
  __syncthreads();
  drain_after_abort(abort_flag);
  __syncthreads();
  if (threadIdx.x == 0) report_abort(abort_flag, status);
}

mote_status_t launch_bounded_wait_selftest(uint32_t* status, uint64_t limit_ns, cudaStream_t stream) {
  bounded_wait_selftest_kernel<<<1, 32, 0, stream>>>(status, limit_ns);
  MOTE_LAUNCH_OK();
  return MOTE_OK;
}

// ------------------------------------------------------------------------------------------------
// Host side: tensor maps and launches
// ------------------------------------------------------------------------------------------------
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

// 2-D row-major tensor [rows, cols] of elem_bytes-wide elements, box [box_rows, box_cols].
static bool make_map_2d(CUtensorMap* m, const void* base, CUtensorMapDataType dt, int elem_bytes, uint64_t rows,
                        uint64_t cols, uint32_t box_rows, uint32_t box_cols, CUtensorMapSwizzle sw) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * (uint64_t)elem_bytes};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(m, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Width of a down-projection tile: the largest multiple of 32 up to 256 that divides N (N is a
// multiple of 128).  Wider tiles reuse the token operand for more MMA work per byte fetched.
static int pick_bn(int N) {
  for (int bn = 256; bn > 128; bn -= 32)
    if (N % bn == 0) return bn;
  return 128;
}

template <int MODE>
static mote_status_t launch_umma(const CUtensorMap& ta, const CUtensorMap& tb0, const CUtensorMap& tb1,
                                 const UmmaArgs& a, int max_items, cudaStream_t stream, bool pdl) {
  using TR = ModeTraits<MODE>;
  static PerDeviceOnce attr_once;                  // one per MODE (this function is a template)
  MOTE_CUDA_OK(set_max_dynamic_smem(attr_once, umma_gemm_kernel<MODE>, (int)TR::kSmem));
  const int sms = device_sm_count();
  const int grid = std::max(1, std::min(sms, max_items));
  if (pdl) MOTE_CUDA_OK(launch_pdl(umma_gemm_kernel<MODE>, dim3(grid), dim3(kThreads), TR::kSmem, stream, ta, tb0, tb1, a));
  else umma_gemm_kernel<MODE><<<grid, kThreads, TR::kSmem, stream>>>(ta, tb0, tb1, a);
  ++g_launch_count;
  MOTE_LAUNCH_OK();
  return MOTE_OK;
}

mote_status_t launch_ternary_umma(const TernaryGemmArgs& g, bool gateup, const int4* tiles, int max_mtiles,
                                  const int32_t* rowsum, uint32_t* beta_out_bits, uint32_t* status,
                                  cudaStream_t stream, bool pdl) {
  if (g.P == 0) return MOTE_OK;
  CUtensorMap ta, tb0, tb1;
  int bn = gateup ? 256 : pick_bn(g.N);
  // a down projection with few row tiles: 128-wide tiles double the items (the weights are the
  // traffic here, and they are read once either way)
  if (!gateup && bn > 128) {
    const int sms = device_sm_count();
    if (max_mtiles * (g.N / bn) * 2 <= sms) bn = 128;
  }
  if (!make_map_2d(&ta, g.qa, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, (uint64_t)g.P, (uint64_t)g.K, 128, 128,
                   CU_TENSOR_MAP_SWIZZLE_128B))
    return MOTE_ERR_CUDA;
  if (!make_map_2d(&tb0, g.w0, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, (uint64_t)g.E * g.N, (uint64_t)g.K / 4, 128, 32,
                   CU_TENSOR_MAP_SWIZZLE_NONE))
    return MOTE_ERR_CUDA;
  // second map: the up matrix (gate/up), or the rows beyond 128 of a down tile
  if (!make_map_2d(&tb1, gateup ? g.w1 : g.w0, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, (uint64_t)g.E * g.N,
                   (uint64_t)g.K / 4, (gateup || bn <= 128) ? 128 : bn - 128, 32, CU_TENSOR_MAP_SWIZZLE_NONE))
    return MOTE_ERR_CUDA;
  UmmaArgs a{};
  a.tiles = tiles;
  a.n_ntiles = gateup ? g.N / 128 : g.N / bn;
  a.k_steps = g.K / 128;
  a.k_splits = 1;
  a.bn = bn;
  a.split_tail = (!gateup && bn == 256) ? 1 : 0;
  a.n_out = g.N;
  a.b_rows_per_expert = g.N;
  a.beta = g.beta; a.rowsum = rowsum; a.alpha0 = g.alpha0; a.alpha1 = g.alpha1;
  a.out = gateup ? g.h_bf16 : static_cast<void*>(g.y);
  a.tap0 = g.acc0_tap; a.tap1 = g.acc1_tap;
  a.beta_out_bits = gateup ? beta_out_bits : nullptr;
  a.status = status;
  const int max_items = max_mtiles * a.n_ntiles;
  return gateup ? launch_umma<MODE_T_GATEUP>(ta, tb0, tb1, a, max_items, stream, pdl)
                : launch_umma<MODE_T_DOWN>(ta, tb0, tb1, a, max_items, stream, pdl);
}

// K splits of the shared down projection: with few row tiles its T x N output has too few tiles to
// occupy the SMs (one row tile of c3: 6 tiles for 27 MB of weights), so each tile's K range is cut
// into up to 16 items whose partial sums the caller adds.  At most 4096 partial rows in all.
int shared_down_k_splits(int64_t T, int N, int K) {
  const int sms = device_sm_count();
  const int64_t n_tiles = ((T + 127) / 128) * (N / pick_bn(N));
  if (n_tiles * 2 > sms) return 1;
  int64_t splits = std::min<int64_t>(16, sms / n_tiles);
  splits = std::min<int64_t>(splits, (K / 64) / 4);
  splits = std::min<int64_t>(splits, kMaxPartialRows / T);
  return (int)std::max<int64_t>(splits, 1);
}

mote_status_t launch_shared_umma(const void* act, const SharedMat& w0, const SharedMat& w1, int bits, bool gateup,
                                 int64_t T, int K, int N, void* out, const int4* tiles, int max_mtiles,
                                 uint32_t* status, const CombineArgs* comb, cudaStream_t stream, bool pdl,
                                 int k_splits) {
  if (T == 0) return MOTE_OK;
  if (k_splits > 1 && (gateup || comb || !out)) return MOTE_ERR_SHAPE;
  CUtensorMap ta, tb0, tb1;
  const int bn = gateup ? 256 : pick_bn(N);
  const uint32_t rows1 = (gateup || bn <= 128) ? 128 : bn - 128;
  if (!make_map_2d(&ta, act, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)T, (uint64_t)K, 128, 64,
                   CU_TENSOR_MAP_SWIZZLE_128B))
    return MOTE_ERR_CUDA;
  const void* wb1 = gateup ? w1.w : w0.w;
  if (bits == 16) {
    if (!make_map_2d(&tb0, w0.w, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)N, (uint64_t)K, 128, 64,
                     CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_2d(&tb1, wb1, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (uint64_t)N, (uint64_t)K, rows1, 64,
                     CU_TENSOR_MAP_SWIZZLE_128B))
      return MOTE_ERR_CUDA;
  } else {
    // code rows as bytes: K (int8) or K/2 (4-bit) per row, 64 reduction elements per pipeline stage
    const uint64_t row_bytes = bits == 8 ? (uint64_t)K : (uint64_t)K / 2;
    const uint32_t box = bits == 8 ? 64 : 32;
    if (!make_map_2d(&tb0, w0.w, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, (uint64_t)N, row_bytes, 128, box,
                     CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !make_map_2d(&tb1, wb1, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, (uint64_t)N, row_bytes, rows1, box,
                     CU_TENSOR_MAP_SWIZZLE_NONE))
      return MOTE_ERR_CUDA;
  }
  UmmaArgs a{};
  a.tiles = tiles;
  a.n_ntiles = gateup ? N / 128 : N / bn;
  a.k_steps = K / 64;
  a.k_splits = std::max(k_splits, 1);
  a.split_stride = T * N;
  a.bn = bn;
  a.split_tail = (!gateup && bn == 256 && a.k_splits == 1) ? 1 : 0;
  a.n_out = N;
  a.b_rows_per_expert = 0;
  a.out = out;
  a.status = status;
  a.alpha0 = w0.scale; a.alpha1 = w1.scale;     // row scales of an RTN-coded shared expert, else null
  if (comb && !gateup) {
    a.comb_y = comb->y; a.comb_w = comb->w; a.comb_perm = comb->perm;
    a.comb_res = static_cast<const uint16_t*>(comb->residual); a.comb_out = static_cast<uint16_t*>(comb->out);
    a.comb_k = comb->k;
    a.comb_wide = ((reinterpret_cast<uintptr_t>(comb->out) | reinterpret_cast<uintptr_t>(comb->residual)) & 31u) == 0;
  }
  const int max_items = max_mtiles * a.n_ntiles * a.k_splits;
  if (bits == 8)
    return gateup ? launch_umma<MODE_Q8_GATEUP>(ta, tb0, tb1, a, max_items, stream, pdl)
                  : launch_umma<MODE_Q8_DOWN>(ta, tb0, tb1, a, max_items, stream, pdl);
  if (bits == 4)
    return gateup ? launch_umma<MODE_Q4_GATEUP>(ta, tb0, tb1, a, max_items, stream, pdl)
                  : launch_umma<MODE_Q4_DOWN>(ta, tb0, tb1, a, max_items, stream, pdl);
  return gateup ? launch_umma<MODE_B_GATEUP>(ta, tb0, tb1, a, max_items, stream, pdl)
                : launch_umma<MODE_B_DOWN>(ta, tb0, tb1, a, max_items, stream, pdl);
}

}  // namespace mote
