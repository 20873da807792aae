// Shared host/device helpers of the MoTE sm_100a kernels.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "mote.h"

#define MOTE_CUDA_OK(expr)                                   \
  do {                                                       \
    cudaError_t _e = (expr);                                 \
    if (_e != cudaSuccess) return MOTE_ERR_CUDA;             \
  } while (0)

#define MOTE_LAUNCH_OK()                                     \
  do {                                                       \
    if (cudaGetLastError() != cudaSuccess) return MOTE_ERR_CUDA; \
  } while (0)

namespace mote {

// ------------------------------------------------------------------------------------------------
// RTN codes of the shared expert (Section 4.3) -> bf16 operands of the tensor-core MMAs, exactly.
// 0x4300 | m is the bf16 number 128 + m for a 7-bit m, so a code becomes a bf16 bit pattern with
// byte moves and one exact bf16 subtraction.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t sub_bf16x2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
// four int8 codes (one word, memory order) -> bf16x2 of elements (0, 1) and (2, 3):
// q = (q & 127) - 128 * signbit = (128 + (q & 127)) - (128 + 128 * signbit)
__device__ __forceinline__ void s8x4_to_bf16x2(uint32_t w, uint32_t& e01, uint32_t& e23) {
  const uint32_t m = w & 0x7F7F7F7Fu, sg = w & 0x80808080u;
  e01 = sub_bf16x2(__byte_perm(m, 0x43434343u, 0x4140), __byte_perm(sg, 0x43434343u, 0x4140));
  e23 = sub_bf16x2(__byte_perm(m, 0x43434343u, 0x4342), __byte_perm(sg, 0x43434343u, 0x4342));
}
// eight 4-bit codes (one word: nibble p = element 2p, nibble 4+p = element 2p+1, stored q + 8)
// -> bf16x2 of elements (2p, 2p+1), p = 0..3:  q = (128 + u) - 136
__device__ __forceinline__ void u4x8_to_bf16x2(uint32_t w, uint32_t (&e)[4]) {
#pragma unroll
  for (int p = 0; p < 4; ++p) e[p] = sub_bf16x2(((w >> (4 * p)) & 0x000F000Fu) | 0x43004300u, 0x43084308u);
}

// ---------------------------------------------------------------------------------------------
// Programmatic dependent launch: a kernel launched with launch_pdl may start while the kernel
// before it on the stream is still running; it calls pdl_wait() before it touches anything that
// kernel writes (the wait returns once the earlier kernel has completed and its writes are
// visible; in a kernel launched the ordinary way it returns at once).  A kernel calls
// pdl_trigger() to let its successor start early; without it the successor starts as the kernel's
// CTAs exit, which still hides the successor's launch latency.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                     Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

constexpr float kEpsScale = 1e-5f;  // lower clamp of alpha (Eq. 9) and beta (Eq. 8)

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// ---------------------------------------------------------------------------------------------
// Per-device host state.  Function attributes (the dynamic shared memory limit) and the SM count
// belong to a device, not to the process: a process that drives several GPUs must set / query them
// once on each.  Device ordinals beyond kMaxDevices are served without caching.
// ---------------------------------------------------------------------------------------------
constexpr int kMaxDevices = 64;

static inline int current_device() {
  int dev = 0;
  return cudaGetDevice(&dev) == cudaSuccess ? dev : -1;
}

// SM count of the current device (148 if the query fails)
static inline int device_sm_count() {
  static std::atomic<int> cache[kMaxDevices];
  const int dev = current_device();
  if (dev >= 0 && dev < kMaxDevices) {
    const int c = cache[dev].load(std::memory_order_relaxed);
    if (c > 0) return c;
  }
  int n = 148;
  if (dev < 0 || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
  if (dev < kMaxDevices) cache[dev].store(n, std::memory_order_relaxed);
  return n;
}

// One flag per device for a set-up step that must run once on each (setting it twice is harmless,
// so a relaxed flag is enough).  Declare one `static PerDeviceOnce` beside the step it guards.
struct PerDeviceOnce {
  std::atomic<bool> done[kMaxDevices];
  bool needed(int dev) const { return dev < 0 || dev >= kMaxDevices || !done[dev].load(std::memory_order_acquire); }
  void mark(int dev) { if (dev >= 0 && dev < kMaxDevices) done[dev].store(true, std::memory_order_release); }
};

// Raises the dynamic shared memory limit of `kernel` on the current device, once per device.
template <typename K>
static inline cudaError_t set_max_dynamic_smem(PerDeviceOnce& once, K kernel, int bytes) {
  const int dev = current_device();
  if (!once.needed(dev)) return cudaSuccess;
  const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) once.mark(dev);
  return e;
}

// Counts kernel launches of the current forward call (host side, per thread).
extern thread_local int g_launch_count;

// ---------------------------------------------------------------------------------------------
// bf16 helpers (bf16 = upper half of an IEEE binary32)
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float bf16_lo(uint32_t packed2) { return __uint_as_float(packed2 << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t packed2) { return __uint_as_float(packed2 & 0xFFFF0000u); }
__device__ __forceinline__ float bf16_bits_to_f32(uint16_t b) { return __uint_as_float(uint32_t(b) << 16); }

// round-to-nearest-even fp32 -> bf16 bits (finite inputs)
__device__ __forceinline__ uint32_t f32_to_bf16_bits(float x) {
  uint32_t u = __float_as_uint(x);
  u += 0x7FFFu + ((u >> 16) & 1u);
  return u >> 16;
}

// ---------------------------------------------------------------------------------------------
// Eq. 8: q = clamp(rint((127*x)/beta), -128, 127); 127*x is exact for a bf16 x.
// ---------------------------------------------------------------------------------------------
constexpr float kMagic = 12582912.0f;          // 1.5 * 2^23 = bits 0x4B400000

// |127*x/beta| <= 127 whenever beta >= |x|, so the nearest-even integer can be read from the
// low bits of (v + 1.5*2^23); the clamp is applied to that integer.
__device__ __forceinline__ int quant_one(float x, float beta) {
  const float v = __fdiv_rn(__fmul_rn(127.0f, x), beta);
  const int q = __float_as_int(__fadd_rn(fminf(fmaxf(v, -1024.0f), 1024.0f), kMagic)) - 0x4B400000;
  return min(max(q, -128), 127);
}

// The same integer without a division per element.  Per row: c = fl(127 * fl(1/beta)).  Per
// element: r = fl(x*c) differs from 127*x/beta by at most 127 * 3 * 2^-24 < 2^-15, and the
// reference value v = fl(fl(127*x)/beta) by at most 127 * 2^-24 < 2^-17.  If r is farther than
// 2^-12 from every half-integer, no half-integer lies between r and v or equals either, hence
// rint(r) == rint(v).  Otherwise (about 5 elements in 10^4) the division is evaluated.
// Rows whose beta is outside [1e-30, 1e30] (1/beta or x*c could leave the normal range) always
// take the division.
struct QaScale {
  float beta, c;
  bool fast;
};
__device__ __forceinline__ QaScale qa_scale(float beta) {
  QaScale s;
  s.beta = beta;
  s.c = __fmul_rn(127.0f, __fdiv_rn(1.0f, beta));
  s.fast = beta > 1e-30f && beta < 1e30f;
  return s;
}
// Returns a word whose LOW BYTE is q (two's complement); the upper bytes are unspecified.
__device__ __forceinline__ uint32_t quant_byte(float x, const QaScale& s) {
  const float r = __fmul_rn(x, s.c);
  const float m = __fadd_rn(r, kMagic);
  const float frac = __fsub_rn(r, __fsub_rn(m, kMagic));
  if (!(fabsf(frac) < 0.499755859375f) || !s.fast) return (uint32_t)quant_one(x, s.beta);
  return __float_as_uint(m);
}
// low bytes of four words -> one word (a in the lowest byte)
__device__ __forceinline__ uint32_t pack_low_bytes(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  return __byte_perm(__byte_perm(a, b, 0x0040), __byte_perm(c, d, 0x0040), 0x5410);
}

// ---------------------------------------------------------------------------------------------
// SiLU of Eq. 6 as a fixed sequence of single correctly-rounded fp32 operations (no FMA
// contraction: every multiply and add is an explicit _rn intrinsic).
//   t = clamp((-g)*log2(e), -125, 125);  n = rint(t);  r = t - n
//   p = c6;  p = p*r + c_i  (i = 5..0), c_i = fl32(ln2^i / i!)
//   E = p * 2^n;   silu = g / (1 + E)
// ---------------------------------------------------------------------------------------------
//
// Two exact shortcuts keep the instruction count down without changing a single bit:
//   * rint(t) for |t| <= 125 is (t + 1.5*2^23) - 1.5*2^23 in round-to-nearest-even, and the
//     low bits of (t + 1.5*2^23) hold the integer n, so p * 2^n is an integer add of n << 23
//     to the bits of p (p in [0.70, 1.42], n in [-125, 125]: no overflow, no subnormals);
//   * fl32(acc) for |acc| < 2^22 is bits(acc + 0x4B400000) - 1.5*2^23 (an integer add and an
//     exact float subtract) instead of a conversion instruction.
__device__ __forceinline__ float i2f_small(int a) { return __fsub_rn(__int_as_float(a + 0x4B400000), kMagic); }

__device__ __forceinline__ float exp_neg_pinned(float g) {
  float t = __fmul_rn(-g, 1.4426950408889634f);
  t = fminf(fmaxf(t, -125.0f), 125.0f);
  const float tm = __fadd_rn(t, kMagic);
  float n = __fsub_rn(tm, kMagic);
  float r = __fsub_rn(t, n);
  float p = 1.5403530393381609e-4f;                       // ln2^6/720
  p = __fadd_rn(__fmul_rn(p, r), 1.3333558146428443e-3f); // ln2^5/120
  p = __fadd_rn(__fmul_rn(p, r), 9.6181291076284772e-3f); // ln2^4/24
  p = __fadd_rn(__fmul_rn(p, r), 5.5504108664821580e-2f); // ln2^3/6
  p = __fadd_rn(__fmul_rn(p, r), 2.4022650695910071e-1f); // ln2^2/2
  p = __fadd_rn(__fmul_rn(p, r), 6.9314718055994531e-1f); // ln2
  p = __fadd_rn(__fmul_rn(p, r), 1.0f);
  return __int_as_float(__float_as_int(p) + (__float_as_int(tm) << 23));
}

__device__ __forceinline__ float silu_pinned(float g) {
  return __fdiv_rn(g, __fadd_rn(1.0f, exp_neg_pinned(g)));
}

// h = bf16_rn(u * silu(g)),  g = fl32(acc_g) * c_g,  u = fl32(acc_u) * c_u
__device__ __forceinline__ float glu_h(int acc_g, int acc_u, float c_g, float c_u) {
  float g = __fmul_rn(i2f_small(acc_g), c_g);
  float u = __fmul_rn(i2f_small(acc_u), c_u);
  return __fmul_rn(u, silu_pinned(g));
}
// The same h through the special-function unit, with a flag telling when that is not enough.
//   E' = ex2.approx(t), t = fl(-g*log2e) as above (relative error <= 2^-22; the polynomial's E is
//        within 4e-7 of 2^t)                                     -> |E' - E| <= 6.4e-7 * E
//   den' = fl(1 + E')                                            -> relative distance <= 7.6e-7
//   s'  = fl(g * rcp.approx(den'))  (rcp: <= 2^-23, product 2^-24) vs s = fl(g / den) -> <= 1.0e-6
//   h'  = fl(u * s')                                             vs h  -> <= 1.12e-6 < 19 ulp
// bf16_rn(h') == bf16_rn(h) unless h' lies within 19 fp32 ulps of the midpoint between two bf16
// values; the flag is raised within 32 ulps of a midpoint (low 16 bits in [0x7FE0, 0x8020]), and
// for |t| > 64 where the clamp, overflow or gradual underflow could make the two differ more.
// Flagged elements (about 0.1 %) are recomputed with glu_h.  The caller must also send rows with
// c_g * c_u <= 1e-12 to glu_h (h' could be subnormal there).
// It works on raw accumulators that still carry the token's row sum (code + 1 storage): `bias` is
// 0x4B400000 - rowsum, so that fl32(acc - rowsum) costs one integer add and one subtract per value
// ((acc - rowsum) + 0x4B400000 == acc + bias in 32-bit arithmetic; see i2f_small).
__device__ __forceinline__ float glu_h_fast_biased(uint32_t raw_g, uint32_t raw_u, uint32_t bias, float c_g, float c_u,
                                                   bool& redo) {
  const float g = __fmul_rn(__fsub_rn(__uint_as_float(raw_g + bias), kMagic), c_g);
  const float u = __fmul_rn(__fsub_rn(__uint_as_float(raw_u + bias), kMagic), c_u);
  const float t = __fmul_rn(-g, 1.4426950408889634f);
  float e, rc;
  // .ftz: single instructions; with |t| <= 64 neither the operands nor the results are subnormal
  // (a subnormal t is flushed to 0, where 2^t = 1 to well within the error budget)
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(t));
  const float den = __fadd_rn(1.0f, e);
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(rc) : "f"(den));
  const float h = __fmul_rn(u, __fmul_rn(g, rc));
  // low 16 bits in [0x7FE0, 0x8020], tested in the upper half of a word: one shift-and-add, one compare
  redo = ((__float_as_uint(h) << 16) + 0x80200000u) <= 0x00400000u || !(fabsf(t) <= 64.0f);
  return h;
}

// two floats -> packed bf16x2 (round to nearest even), lo in the low half
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}

// SiLU for the shared (bf16, not bit-pinned) expert: g / (1 + 2^(-g*log2e)) on the special-function unit
__device__ __forceinline__ float silu_fast(float g) {
  float e, rc;
  const float t = fminf(fmaxf(g * -1.4426950408889634f, -80.0f), 80.0f);
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(t));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(rc) : "f"(1.0f + e));
  return g * rc;
}

// scale of one ternary linear output row: alpha * (beta / 127)
__device__ __forceinline__ float dequant_scale(float alpha, float beta) {
  return __fmul_rn(alpha, __fdiv_rn(beta, 127.0f));
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

}  // namespace mote
