// Expert dispatch: a stable counting sort of the P = T*k (token, slot) pairs by expert.
//   offsets[E+1]  first sorted row of every expert
//   perm[P]       pair p = t*k + j  ->  sorted row
//   inv[P]        sorted row        ->  pair
// Inside an expert the pairs keep their (token, slot) order, so the result does not depend on
// thread scheduling.  One CTA walks the pairs in chunks of 1024; inside a chunk the rank of a
// pair among equal experts comes from a warp-level match/popc prefix plus a per-warp histogram
// that is turned into per-warp bases by a shuffle scan over the warps (one expert per warp).
#include "mote_common.cuh"
#include "mote_internal.h"

namespace mote {

constexpr int kDispatchThreads = 1024;
constexpr int kBatch = 8;                 // chunks whose loads are issued together

__global__ void __launch_bounds__(kDispatchThreads) dispatch_kernel(const int32_t* __restrict__ idx, int P, int E,
                                                                    int32_t* __restrict__ offsets,
                                                                    int32_t* __restrict__ perm,
                                                                    int32_t* __restrict__ inv,
                                                                    int4* __restrict__ tiles_routed,
                                                                    int4* __restrict__ tiles_shared, int T) {
  __shared__ int s_count[MOTE_MAX_EXPERTS];
  __shared__ int s_running[MOTE_MAX_EXPERTS];
  __shared__ int s_warp[32][MOTE_MAX_EXPERTS];
  __shared__ int s_pref[32][MOTE_MAX_EXPERTS];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid < MOTE_MAX_EXPERTS) s_count[tid] = 0;
  for (int i = tid; i < 32 * MOTE_MAX_EXPERTS; i += kDispatchThreads) (&s_warp[0][0])[i] = 0;
  __syncthreads();
  // histogram, one atomic per warp and expert; the loads of a batch are independent of each other
  for (int base = 0; base < P; base += kBatch * kDispatchThreads) {
    int ev[kBatch];
#pragma unroll
    for (int c = 0; c < kBatch; ++c) {
      const int p = base + c * kDispatchThreads + tid;
      ev[c] = p < P ? idx[p] : -1;
    }
#pragma unroll
    for (int c = 0; c < kBatch; ++c) {
      const int e = (ev[c] >= 0 && ev[c] < E) ? ev[c] : -1;
      const unsigned peers = __match_any_sync(0xffffffffu, e);
      if (e >= 0 && lane == __ffs(peers) - 1) atomicAdd(&s_count[e], __popc(peers));
    }
  }
  __syncthreads();
  if (tid == 0) {
    int run = 0;
    for (int e = 0; e < E; ++e) {
      offsets[e] = run;
      s_running[e] = run;
      run += s_count[e];
    }
    offsets[E] = run;
  }
  // row-tile tables of the tensor-core GEMMs: [0] = {count}, [1+i] = {expert, first row, rows}
  if (tid == 32 && tiles_routed) {
    int n = 0, run = 0;
    for (int e = 0; e < E; ++e) {
      const int cnt = s_count[e];
      for (int r = 0; r < cnt; r += 128) tiles_routed[1 + n++] = make_int4(e, run + r, min(128, cnt - r), 0);
      run += cnt;
    }
    tiles_routed[0] = make_int4(n, 0, 0, 0);
  }
  if (tiles_shared) {
    const int n = (T + 127) / 128;
    for (int i = tid; i < n; i += kDispatchThreads) tiles_shared[1 + i] = make_int4(0, i * 128, min(128, T - i * 128), 0);
    if (tid == 0) tiles_shared[0] = make_int4(n, 0, 0, 0);
  }
  __syncthreads();

  // s_warp[w][e]: pairs of expert e held by warp w in the current chunk (zero between chunks)
  for (int base0 = 0; base0 < P; base0 += kBatch * kDispatchThreads) {
    int ev[kBatch];
#pragma unroll
    for (int c = 0; c < kBatch; ++c) {
      const int p = base0 + c * kDispatchThreads + tid;
      ev[c] = p < P ? idx[p] : -1;
    }
#pragma unroll
    for (int c = 0; c < kBatch; ++c) {
      if (base0 + c * kDispatchThreads >= P) break;            // uniform over the CTA
      const int p = base0 + c * kDispatchThreads + tid;
      const int e = (ev[c] >= 0 && ev[c] < E) ? ev[c] : -1;
      const unsigned peers = __match_any_sync(0xffffffffu, e);
      const int rank = __popc(peers & ((1u << lane) - 1u));
      if (e >= 0 && rank == 0) s_warp[warp][e] = __popc(peers);
      __syncthreads();
      // exclusive scan over the 32 warps, one expert per warp and round (lane = warp index)
      for (int ee = warp; ee < E; ee += 32) {
        const int v = s_warp[lane][ee];
        s_warp[lane][ee] = 0;
        int incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int n = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += n;
        }
        const int first = s_running[ee];
        s_pref[lane][ee] = first + incl - v;
        if (lane == 31) s_running[ee] = first + incl;
      }
      __syncthreads();
      if (e >= 0) {
        const int pos = s_pref[warp][e] + rank;
        perm[p] = pos;
        inv[pos] = p;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Block-wise dispatch for long prefills.  The router leaves, for every block of kRouteBlockTokens
// tokens, the number of its pairs per expert (blk_hist[E][blk_stride(n_blk)]).  This kernel turns
// them into
//   offsets[E+1]                      first sorted row of every expert
//   blk_base[E][blk_stride(n_blk)]    first sorted row of the block's pairs of that expert
// (experts outermost, blocks in order: the same stable order as above) and writes the tile tables.
// The rank of a pair inside its block is recomputed by the activation quantizer, which then knows
// the sorted row of every pair without a pass of its own.  One CTA, one warp per expert: lane l
// sums 16 consecutive blocks (four 16-byte loads), a shuffle scan orders the lanes, a second walk
// writes the bases.  (With the counts block-major, every load and store of a warp touched 32
// separate sectors: 18 us at 512 blocks x 16 experts, 11 of them in the second walk.)
// ------------------------------------------------------------------------------------------------
constexpr int kScanPer = 16;                           // blocks per lane and chunk

// the lane's 16 counts of chunk c0, zero beyond n_blk
__device__ __forceinline__ void load_counts(const int32_t* __restrict__ row, int c0, int lane, int n_blk, int (&v)[kScanPer]) {
  const int b0 = c0 + lane * kScanPer;
#pragma unroll
  for (int i = 0; i < kScanPer / 4; ++i) {
    const int b = b0 + 4 * i;
    int4 t = make_int4(0, 0, 0, 0);
    if (b < n_blk) t = *reinterpret_cast<const int4*>(row + b);     // the padded row holds b .. b + 3
    v[4 * i] = t.x;
    v[4 * i + 1] = b + 1 < n_blk ? t.y : 0;
    v[4 * i + 2] = b + 2 < n_blk ? t.z : 0;
    v[4 * i + 3] = b + 3 < n_blk ? t.w : 0;
  }
}

__global__ void __launch_bounds__(kDispatchThreads) dispatch_scan_kernel(const int32_t* __restrict__ blk_hist, int n_blk,
                                                                         int E, int32_t* __restrict__ offsets,
                                                                         int32_t* __restrict__ blk_base,
                                                                         int4* __restrict__ tiles_routed,
                                                                         int4* __restrict__ tiles_shared, int T) {
  __shared__ int s_count[MOTE_MAX_EXPERTS];
  __shared__ int s_first[MOTE_MAX_EXPERTS];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int stride = blk_stride(n_blk);
  pdl_wait();                                          // the router's block counts are complete
  // totals per expert (two rounds of 32 warps cover MOTE_MAX_EXPERTS = 64)
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int e = warp + 32 * r;
    if (e < E) {
      int tot = 0;
      for (int c0 = 0; c0 < n_blk; c0 += 32 * kScanPer) {
        int v[kScanPer];
        load_counts(blk_hist + size_t(e) * stride, c0, lane, n_blk, v);
#pragma unroll
        for (int i = 0; i < kScanPer; ++i) tot += v[i];
      }
      tot = warp_sum(tot);
      if (lane == 0) s_count[e] = tot;
    }
  }
  __syncthreads();
  if (tid == 0) {
    int run = 0;
    for (int e = 0; e < E; ++e) {
      offsets[e] = run;
      s_first[e] = run;
      run += s_count[e];
    }
    offsets[E] = run;
  }
  if (tid == 32 && tiles_routed) {
    int n = 0, run = 0;
    for (int e = 0; e < E; ++e) {
      const int cnt = s_count[e];
      for (int r = 0; r < cnt; r += 128) tiles_routed[1 + n++] = make_int4(e, run + r, min(128, cnt - r), 0);
      run += cnt;
    }
    tiles_routed[0] = make_int4(n, 0, 0, 0);
  }
  if (tiles_shared) {
    const int n = (T + 127) / 128;
    for (int i = tid; i < n; i += kDispatchThreads) tiles_shared[1 + i] = make_int4(0, i * 128, min(128, T - i * 128), 0);
    if (tid == 0) tiles_shared[0] = make_int4(n, 0, 0, 0);
  }
  __syncthreads();
  // bases: blocks in order inside every expert
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int e = warp + 32 * r;
    if (e < E) {
      int carry = s_first[e];
      int32_t* out = blk_base + size_t(e) * stride;
      for (int c0 = 0; c0 < n_blk; c0 += 32 * kScanPer) {
        int v[kScanPer];
        load_counts(blk_hist + size_t(e) * stride, c0, lane, n_blk, v);
        int tot = 0;
#pragma unroll
        for (int i = 0; i < kScanPer; ++i) tot += v[i];
        int incl = tot;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int n = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += n;
        }
        int run = carry + incl - tot;
        const int b0 = c0 + lane * kScanPer;
#pragma unroll
        for (int i = 0; i < kScanPer / 4; ++i) {
          int4 t;
          t.x = run; run += v[4 * i];
          t.y = run; run += v[4 * i + 1];
          t.z = run; run += v[4 * i + 2];
          t.w = run; run += v[4 * i + 3];
          if (b0 + 4 * i < n_blk) *reinterpret_cast<int4*>(out + b0 + 4 * i) = t;   // the padded row has room
        }
        carry += __shfl_sync(0xffffffffu, incl, 31);
      }
    }
  }
}

mote_status_t launch_dispatch_scan(const int32_t* blk_hist, int n_blk, int E, int32_t* offsets, int32_t* blk_base,
                                   int4* tiles_routed, int4* tiles_shared, int64_t T, cudaStream_t stream) {
  MOTE_CUDA_OK(launch_pdl(dispatch_scan_kernel, dim3(1), dim3(kDispatchThreads), 0, stream, blk_hist, n_blk, E, offsets,
                          blk_base, tiles_routed, tiles_shared, (int)T));
  ++g_launch_count;
  MOTE_LAUNCH_OK();
  return MOTE_OK;
}

mote_status_t launch_dispatch(const int32_t* idx, int64_t P, int E, int32_t* offsets, int32_t* perm,
                              int32_t* inv, int4* tiles_routed, int4* tiles_shared, int64_t T,
                              cudaStream_t stream) {
  dispatch_kernel<<<1, kDispatchThreads, 0, stream>>>(idx, (int)P, E, offsets, perm, inv, tiles_routed,
                                                      tiles_shared, (int)T);
  ++g_launch_count;
  MOTE_LAUNCH_OK();
  return MOTE_OK;
}

}  // namespace mote
