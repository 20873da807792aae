// Expert dispatch: a stable counting sort of the P = T*k (token, slot) pairs by expert.
//   offsets[E+1]  first sorted row of every expert
//   perm[P]       pair p = t*k + j  ->  sorted row
//   inv[P]        sorted row        ->  pair
// Inside an expert the pairs keep their (token, slot) order, so the result does not depend on
// thread scheduling.  One CTA walks the pairs in chunks of 1024; inside a chunk the rank of a
// pair among equal experts comes from a warp-level match/popc prefix plus a per-warp histogram.
#include "mote_common.cuh"
#include "mote_internal.h"

namespace mote {

constexpr int kDispatchThreads = 1024;

__global__ void __launch_bounds__(kDispatchThreads) dispatch_kernel(const int32_t* __restrict__ idx, int P, int E,
                                                                    int32_t* __restrict__ offsets,
                                                                    int32_t* __restrict__ perm,
                                                                    int32_t* __restrict__ inv,
                                                                    int4* __restrict__ tiles_routed,
                                                                    int4* __restrict__ tiles_shared, int T) {
  __shared__ int s_count[MOTE_MAX_EXPERTS];
  __shared__ int s_running[MOTE_MAX_EXPERTS];
  __shared__ int s_warp[32][MOTE_MAX_EXPERTS];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid < MOTE_MAX_EXPERTS) s_count[tid] = 0;
  for (int i = tid; i < 32 * MOTE_MAX_EXPERTS; i += kDispatchThreads) (&s_warp[0][0])[i] = 0;
  __syncthreads();
  for (int p = tid; p < P; p += kDispatchThreads) {
    const int e = idx[p];
    if (e >= 0 && e < E) atomicAdd(&s_count[e], 1);
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

  for (int base = 0; base < P; base += kDispatchThreads) {
    const int p = base + tid;
    int e = -1;
    if (p < P) {
      e = idx[p];
      if (e < 0 || e >= E) e = -1;
    }
    const unsigned peers = __match_any_sync(0xffffffffu, e);
    const int rank = __popc(peers & ((1u << lane) - 1u));
    if (e >= 0 && rank == 0) s_warp[warp][e] = __popc(peers);
    __syncthreads();
    if (e >= 0) {
      int pos = s_running[e] + rank;
      for (int w = 0; w < warp; ++w) pos += s_warp[w][e];
      perm[p] = pos;
      inv[pos] = p;
    }
    __syncthreads();
    if (tid < E) {
      int add = 0;
      for (int w = 0; w < 32; ++w) { add += s_warp[w][tid]; s_warp[w][tid] = 0; }
      s_running[tid] += add;
    }
    __syncthreads();
  }
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
