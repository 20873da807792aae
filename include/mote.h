/*
 * mote.h -- C ABI of the B200 (sm_100a) forward pass of one Mixture-of-Ternary-Experts FFN layer
 * (MoTE, arXiv 2506.14435, Section 3.1).
 *
 *     out = [residual +] FFN(x) + sum_{j<k} w_j * FFN^T_{e_j}(x)            (Eq. 2, Eq. 4)
 *
 * FFN is the bf16 shared SwiGLU expert; FFN^T_e are routed GLU experts whose weights are ternary
 * {-1,0,1} with one absmean scale per matrix (Eq. 7, 9) and whose inputs are per-token absmax int8
 * (Eq. 8).  Ternary weights are stored as INT2 (Section 3.1, last paragraph).  The shared expert
 * may also be held as RTN weight-only INT8 or INT4 codes (post-training quantization, Section 4.3).
 *
 * General rules for every entry point
 *   - Pointers are DEVICE pointers unless an argument name ends in `_host`.  The caller owns all
 *     memory; the library never allocates or frees device memory and never synchronises
 *     (exception: mote_moe_forward_host, documented below).
 *   - All work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = default stream).
 *   - Every function returns a mote_status_t.  Argument errors are detected on the host BEFORE
 *     anything is launched.  A failed launch maps to MOTE_ERR_CUDA.  No exceptions, no exit().
 *   - bf16 tensors are raw 16-bit patterns.  Matrices are row-major; a weight matrix is W[m, n]
 *     with n the reduction ("in") dimension, y = W x.
 *   - Non-finite inputs give undefined results.
 */
#ifndef MOTE_H_
#define MOTE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  MOTE_OK = 0,
  MOTE_ERR_NULL = 1,           /* a required pointer is NULL                                   */
  MOTE_ERR_SHAPE = 2,          /* unsupported size (see each call)                              */
  MOTE_ERR_ALIGN = 3,          /* a pointer or row stride is not 16-byte aligned                */
  MOTE_ERR_WORKSPACE = 4,      /* workspace missing or too small                                */
  MOTE_ERR_DTYPE = 5,          /* unknown dtype code                                            */
  MOTE_ERR_CUDA = 6,           /* a CUDA call or launch failed                                  */
  MOTE_ERR_DEVICE_TIMEOUT = 7, /* a bounded device-side wait expired (see mote_device_status)   */
  MOTE_ERR_TOO_LARGE = 8       /* more elements than a fixed-capacity entry point accepts       */
} mote_status_t;

enum { MOTE_DTYPE_F32 = 0, MOTE_DTYPE_BF16 = 1 };
enum { MOTE_MAX_EXPERTS = 64, MOTE_MAX_TOPK = 8 };
/* storage of the shared expert's three matrices (mote_layer_t.shared_bits; 0 means bf16) */
enum { MOTE_SHARED_BF16 = 16, MOTE_SHARED_INT8 = 8, MOTE_SHARED_INT4 = 4 };

/* Which implementation runs the layer.  AUTO picks per shape; the others force one path (used by
 * the tests to check every path against the oracle).
 *   STREAM  decode, T <= 64 with d % 64 == 0, f % 64 == 0, d <= 16384, T*k <= 512: the weights are
 *           streamed once from HBM through registers into warp-level MMAs
 *   TENSOR  d % 128 == 0 and f % 128 == 0: tcgen05 GEMMs (int8 x 2-bit routed, bf16 shared; an
 *           RTN-coded shared expert is expanded to bf16 on the way, see mote_layer_workspace_bytes)
 *   SIMT    any d, f that are multiples of 16: CUDA-core GEMMs
 * AUTO takes STREAM up to 32 tokens (up to 64 where TENSOR's conditions do not hold), then TENSOR,
 * then SIMT. */
enum { MOTE_PATH_AUTO = 0, MOTE_PATH_SIMT = 1, MOTE_PATH_TENSOR = 2, MOTE_PATH_STREAM = 3 };

const char* mote_status_string(mote_status_t st);

/* ------------------------------------------------------------------------------------------------
 * mote_ternarize_pack -- absmean ternary weight quantizer and INT2 packing (Eq. 7, 9, 10; storage
 * per Section 3.1).  Offline step, once per matrix.
 *
 *   alpha  = max( fl32( fl64(exact sum of |w|) / (m*n) ), 1e-5 )   the sum is exact (integer
 *            accumulation of fp32 significands), so alpha does not depend on thread order; it is
 *            rounded once to fp64, divided in fp64 and the quotient rounded to fp32
 *   code   = clamp( rint( w / alpha ), -1, 1 )                 true fp32 division, ties to even
 *   packed : m * n/4 bytes; stored value u = code + 1; 4 consecutive elements of a row per byte,
 *            element j in bits [2*(j%4), 2*(j%4)+1]
 *
 *   W        in   [m, n] row-major, dtype w_dtype (MOTE_DTYPE_F32 or MOTE_DTYPE_BF16), 16-B aligned
 *   packed   out  [m, n/4] uint8, 16-B aligned
 *   alpha    out  1 float
 *   ws       scratch of at least mote_ternarize_workspace_bytes() bytes, 16-B aligned
 * Errors: NULL -> ERR_NULL; m<=0, n<=0, n%16 != 0, m*n >= 2^38 -> ERR_SHAPE; bad dtype -> ERR_DTYPE.
 */
size_t mote_ternarize_workspace_bytes(void);
mote_status_t mote_ternarize_pack(const void* W, int w_dtype, int64_t m, int64_t n,
                                  uint8_t* packed, float* alpha,
                                  void* ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------------------------------
 * mote_ternarize_pack_static -- mote_ternarize_pack without the `ws` argument.  (The paper has no
 * counterpart: this is a packaging variant of the same quantizer, same results bit for bit.)
 *
 * For callers that cannot hand over device scratch and must not trigger an allocation: code that
 * runs inside a memory pool whose budget is already fully committed, a plug-in loaded into a host
 * process that owns every allocation, or a latency-critical loop that cannot afford the
 * device-wide synchronisation an allocation may imply.
 * The 256 exponent bins (2 KiB) that the exact sum of |w| needs live in a device array inside the
 * library image, so every GPU that loads the library carries those 2 KiB until the process ends.
 * The call itself asks for no device memory; it issues one memset and three kernels.  (The very
 * first use of the library on a device may make the CUDA runtime load the library's code there;
 * that happens once, is not specific to this call, and a caller that must avoid it warms up once
 * at start-up.)
 *
 *   W, w_dtype, m, n, packed, alpha, stream    exactly as mote_ternarize_pack
 *
 * Limits and rules
 *   - m*n <= MOTE_STATIC_MAX_ELEMENTS (2^31, e.g. a 32768 x 65536 matrix); beyond that the call
 *     returns MOTE_ERR_TOO_LARGE and launches nothing.  Use mote_ternarize_pack for larger ones.
 *   - The first call on each device looks up the device address of the array (a host-side query)
 *     and keeps it for the life of the process; make that first call outside any stream capture.
 *     The kept address does not survive cudaDeviceReset.
 *   - All calls on one device share the one array, and it keeps what the last call left in it;
 *     each call clears it on `stream` before use.  Two calls that can overlap on the GPU (issued
 *     on different streams without an ordering between them, or from two host threads) race on
 *     the bins and both give undefined alpha and codes: serialise them.
 * Errors: as mote_ternarize_pack, plus MOTE_ERR_TOO_LARGE; MOTE_ERR_CUDA if the address lookup
 * fails or the device ordinal is 64 or higher.
 */
#define MOTE_STATIC_MAX_ELEMENTS ((int64_t)1 << 31)
mote_status_t mote_ternarize_pack_static(const void* W, int w_dtype, int64_t m, int64_t n,
                                         uint8_t* packed, float* alpha, void* stream);

/* ------------------------------------------------------------------------------------------------
 * mote_rtn_quant -- round-to-nearest absmax weight quantizer for the shared expert (Section 4.3:
 * the shared expert is post-training quantized to INT8, or INT4 under tighter memory budgets).
 * The paper names the method (RTN) and the bit widths only; this library takes one scale per
 * output row, the absmax form of Eq. 8-10 applied to the rows of W.  Offline step, once per matrix.
 *
 *   qmax     = 2^(bits-1) - 1                                   127 or 7
 *   beta_r   = max( max_j |W[r,j]|, 1e-5 )
 *   q[r,j]   = clamp( rint( (qmax * W[r,j]) / beta_r ), -qmax, qmax )   fp32 multiply, true fp32
 *                                                                division, ties to even
 *   scale[r] = beta_r / qmax                                    dequantized weight = scale[r] * q[r,j]
 *
 *   W      in   [m, n] row-major, dtype w_dtype (MOTE_DTYPE_F32 or MOTE_DTYPE_BF16), 16-B aligned
 *   bits   8 or 4
 *   q      out  bits = 8: [m, n] int8.
 *               bits = 4: [m, n/2] bytes; stored nibble u = q + 8 (1..15); every 8 consecutive
 *               elements of a row form one little-endian 32-bit word whose nibble p (bits 4p..4p+3)
 *               holds element 2p and whose nibble 4+p holds element 2p+1, p = 0..3.  (Both halves of
 *               the word then expand to element pairs with one mask each.)
 *               16-B aligned.
 *   scale  out  [m] float
 * Errors: NULL -> ERR_NULL; m<=0, n<=0, n%16 != 0, n > 65536, bits not 8 or 4 -> ERR_SHAPE; ERR_DTYPE; ERR_ALIGN.
 */
mote_status_t mote_rtn_quant(const void* W, int w_dtype, int64_t m, int64_t n, int bits,
                             void* q, float* scale, void* stream);

/* ------------------------------------------------------------------------------------------------
 * mote_quant_act -- per-token absmax int8 activation quantizer (Eq. 8, 9, 10).
 *
 *   beta_t = max( max_j |x[t,j]|, 1e-5 );   q[t,j] = clamp( rint( (127 * x[t,j]) / beta_t ), -128, 127 )
 *   (127*x exact in fp32, true fp32 division, ties to even);  rowsum[t] = sum_j q[t,j]
 *
 *   x_bf16  in   [T, d] bf16, row stride ldx elements (ldx >= d, ldx % 8 == 0), 16-B aligned
 *   q       out  [T, d] int8 contiguous, 16-B aligned
 *   beta    out  [T] float
 *   rowsum  out  [T] int32, may be NULL
 * T = 0 is a no-op.  Errors: d<=0, d%16 != 0, d > 32768, T<0 -> ERR_SHAPE.
 */
mote_status_t mote_quant_act(const void* x_bf16, int64_t T, int64_t d, int64_t ldx,
                             int8_t* q, float* beta, int32_t* rowsum, void* stream);

/* ------------------------------------------------------------------------------------------------
 * mote_route_topk -- router of Eq. 3 with top-k selection (no capacity limit, no token dropping).
 *
 *   logits[t,e] = sum_j x[t,j] * Wr[e,j] (+ bias[e])        fp32 accumulation
 *   selection   : the k largest logits, ties to the lower expert index, listed in descending order
 *   norm_topk=1 : w = softmax over the k selected logits (sums to 1)
 *   norm_topk=0 : w = P(x)_e of Eq. 3 (softmax over all E experts)
 *
 *   x_bf16 [T,d] bf16 contiguous (16-B aligned), Wr [E,d] fp32, bias [E] fp32 or NULL,
 *   topk_idx [T,k] int32, topk_w [T,k] float, logits [T,E] float or NULL.
 * Errors: E<1, E>MOTE_MAX_EXPERTS, k<1, k>E, k>MOTE_MAX_TOPK, d%8 != 0 -> ERR_SHAPE.
 */
mote_status_t mote_route_topk(const void* x_bf16, int64_t T, int64_t d,
                              const float* Wr, const float* bias, int E, int k, int norm_topk,
                              int32_t* topk_idx, float* topk_w, float* logits, void* stream);

/* ------------------------------------------------------------------------------------------------
 * mote_route_stats -- the two per-expert factors of the load-balancing loss (Eq. 12) for a batch,
 * from the router's outputs:
 *     tokens_per_expert[i] = t_i        number of (token, slot) pairs routed to expert i
 *     prob_sum[i]          = sum_x P(x)_i   routing probability of Eq. 3 (softmax over all E experts)
 * so that L_balance = E / T * sum_i t_i * prob_sum[i].  fp32, summed in a fixed order (reproducible).
 *   logits [T,E] float (the optional output of mote_route_topk), topk_idx [T,k] int32,
 *   tokens_per_expert [E] int32, prob_sum [E] float.  T = 0 gives zeros.
 * Errors: E, k out of range -> ERR_SHAPE; NULL -> ERR_NULL.
 */
mote_status_t mote_route_stats(const float* logits, const int32_t* topk_idx, int64_t T, int E, int k,
                               int32_t* tokens_per_expert, float* prob_sum, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Layer description (Eq. 2-6).  All device pointers, immutable while calls are in flight.
 */
typedef struct {
  int32_t d, f, E, k, norm_topk;
  int32_t path;                    /* MOTE_PATH_*                                               */
  const float* Wr;                 /* [E, d] router projection                                  */
  const float* router_bias;        /* [E] or NULL                                               */
  const uint8_t* gate_packed;      /* [E][f, d/4]  packed W_gate of every routed expert          */
  const uint8_t* up_packed;        /* [E][f, d/4]                                               */
  const uint8_t* down_packed;      /* [E][d, f/4]                                               */
  const float* alpha_gate;         /* [E]                                                       */
  const float* alpha_up;           /* [E]                                                       */
  const float* alpha_down;         /* [E]                                                       */
  const void* sh_gate;             /* [f, d]  shared expert: bf16, or the q of mote_rtn_quant   */
  const void* sh_up;               /* [f, d]                                                    */
  const void* sh_down;             /* [d, f]                                                    */
  int32_t shared_bits;             /* MOTE_SHARED_BF16 (or 0), MOTE_SHARED_INT8, MOTE_SHARED_INT4 */
  const float* sh_gate_scale;      /* [f]  scales of mote_rtn_quant when shared_bits is 8 or 4,  */
  const float* sh_up_scale;        /* [f]  16-B aligned; ignored for bf16                        */
  const float* sh_down_scale;      /* [d]                                                       */
} mote_layer_t;

/* Optional copies of intermediates (for parity checks).  Every member may be NULL; a non-NULL
 * member is filled.  Row-indexed taps are in expert-sorted order: row r = perm[t*k + j]. */
typedef struct {
  int32_t* topk_idx;   /* [T, k]                                                                */
  float* topk_w;       /* [T, k]                                                                */
  int32_t* offsets;    /* [E+1]   first sorted row of each expert                               */
  int32_t* perm;       /* [T*k]   pair (t*k+j) -> sorted row                                    */
  int8_t* qx;          /* [T, d]  Q_a(x) codes, token order                                     */
  float* beta_x;       /* [T]                                                                   */
  int32_t* acc_gate;   /* [P, f]  integer accumulators codes_gate . qx                          */
  int32_t* acc_up;     /* [P, f]                                                                */
  void* h_bf16;        /* [P, f]  u * SiLU(g), bf16                                             */
  int8_t* qh;          /* [P, f]  Q_a(h) codes                                                  */
  float* beta_h;       /* [P]                                                                   */
  int32_t* acc_down;   /* [P, d]                                                                */
  float* y;            /* [P, d]  routed expert outputs before gating                           */
  float* shared_out;   /* [T, d]  FFN(x) of the shared expert                                   */
} mote_taps_t;

/* Bytes of scratch mote_moe_forward needs for up to T_max tokens (0 if the shape is invalid). */
size_t mote_workspace_bytes(int d, int f, int E, int k, int64_t T_max);
/* The same for one layer description.  Larger than mote_workspace_bytes only for an RTN-coded shared
 * expert and T_max >= 768: 6*d*f more bytes, in which a prefill expands the shared expert's codes to
 * bf16 once per call (a streaming pass) instead of expanding them inside the GEMM for every row
 * tile.  A call that is given only mote_workspace_bytes() still runs, expanding inside the GEMM. */
size_t mote_layer_workspace_bytes(const mote_layer_t* L, int64_t T_max);

/* ------------------------------------------------------------------------------------------------
 * mote_moe_forward -- the whole layer (Eq. 2-8): route, dispatch, Q_a(x), gate/up ternary GEMM
 * with fused dequantisation and SwiGLU, Q_a(h), down ternary GEMM, shared bf16 FFN, gate-weighted
 * combine with the shared output and the optional residual.
 * With shared_bits 8 or 4 the shared FFN is weight-only quantized (Section 4.3): its activations
 * (x, and h rounded to bf16) stay bf16, the integer codes enter the bf16 tensor-core MMAs exactly
 * (|q| <= 127 is representable), accumulation is fp32 and the row scale multiplies the finished sum.
 *
 *   x_bf16         in   [T, d] bf16 contiguous, 16-B aligned
 *   residual_bf16  in   [T, d] bf16 or NULL; may alias out_bf16
 *   out_bf16       out  [T, d] bf16; must not alias x_bf16
 *   taps           NULL or a struct of optional outputs
 *   ws, ws_bytes   scratch, >= mote_workspace_bytes(d,f,E,k,T), 256-B aligned
 * Pinned arithmetic: per sorted row, g = fl32(acc_g) * (alpha_g * (beta/127)), u likewise,
 * h = bf16_rn(u * silu(g)) with silu evaluated by a fixed fp32 sequence, so that the integer
 * stages that follow are reproducible bit for bit.
 * T = 0 is a no-op.  Errors: d%16, f%16 != 0, E/k out of range -> ERR_SHAPE; ERR_WORKSPACE;
 * ERR_ALIGN; a forced path whose conditions (see MOTE_PATH_*) do not hold -> ERR_SHAPE.
 */
mote_status_t mote_moe_forward(const mote_layer_t* L, const void* x_bf16,
                               const void* residual_bf16, int64_t T, void* out_bf16,
                               const mote_taps_t* taps, void* ws, size_t ws_bytes, void* stream);

/* Same layer with HOST input and output: copies x_host (and residual_host if non-NULL) to the
 * device, runs mote_moe_forward, copies the result to out_host and waits for the stream.  Host
 * buffers should be page-locked for the copies to be asynchronous.  Needs
 * mote_layer_workspace_bytes(...) + mote_host_staging_bytes(d, T) bytes of device scratch.
 * From 4096 tokens on the call runs the layer as two halves of the tokens (Eq. 2-4 treat every
 * token on its own, so the result is bit-identical to the one-piece call): the second half's input
 * copy runs beside the first half's layer and the first half's output copy beside the second
 * half's layer, on two copy streams that the library creates on the calling thread's first such
 * call on a device and keeps (like the library's other per-device state they do not survive a
 * cudaDeviceReset).  The copies start after the work already queued on `stream`; when the call
 * returns, `stream` and both copy streams are idle. */
size_t mote_host_staging_bytes(int d, int64_t T_max);
mote_status_t mote_moe_forward_host(const mote_layer_t* L, const void* x_host,
                                    const void* residual_host, int64_t T, void* out_host,
                                    void* ws, size_t ws_bytes, void* stream);

/* ------------------------------------------------------------------------------------------------
 * mote_rms_norm -- the LN of Eq. 2 for callers that chain layers: RMS normalisation (as in the
 * Qwen2.5 models the paper up-cycles), unit gain:
 *     y[t, :] = bf16( x[t, :] * rsqrt( mean_j x[t, j]^2 + eps ) )        fp32 arithmetic
 * x_bf16, y_bf16: [T, d] bf16 contiguous, 16-B aligned; y may alias x.  Errors: d % 8 != 0 -> ERR_SHAPE.
 */
mote_status_t mote_rms_norm(const void* x_bf16, int64_t T, int64_t d, float eps, void* y_bf16, void* stream);

/* ------------------------------------------------------------------------------------------------
 * mote_stack_forward -- n_layers MoTE FFN layers back to back as Eq. 1-2 chain them (the attention
 * sub-block of a transformer layer is not part of this):
 *
 *     x_l = bf16( x_{l-1} + FFN_l(n_l) + MoE_l(n_l) ),  n_l = LN(x_{l-1}),   l = 1 .. n_layers,  x_0 = x
 *
 * LN is mote_rms_norm with rms_eps when rms_eps > 0, and the identity when rms_eps == 0.  Each step
 * is mote_moe_forward(layer l, n_l, residual = x_{l-1}); everything is chained on one stream and
 * nothing synchronises in between.
 *
 *   layers_host        in   HOST array of n_layers layer descriptions; all layers share d, f may differ
 *   x_bf16             in   [T, d] bf16 device
 *   out_bf16           out  [T, d] bf16 device = x_{n_layers}; must not alias x_bf16
 *   layer_inputs_bf16  out  NULL, or [n_layers, T, d] bf16 device: the residual stream x_{l-1} entering
 *                           every layer l (parity tap; n_l follows from it with mote_rms_norm)
 *   ws, ws_bytes            >= mote_stack_workspace_bytes(...), 256-B aligned
 * Errors: as mote_moe_forward; n_layers < 1, layers of different d or rms_eps < 0 -> ERR_SHAPE.
 */
size_t mote_stack_workspace_bytes(const mote_layer_t* layers_host, int n_layers, int64_t T_max);
mote_status_t mote_stack_forward(const mote_layer_t* layers_host, int n_layers, float rms_eps, const void* x_bf16,
                                 int64_t T, void* out_bf16, void* layer_inputs_bf16, void* ws, size_t ws_bytes,
                                 void* stream);

/* mote_moe_forward with a CUDA event recorded on `stream` between the stages; waits for the stream
 * and writes the device time of each stage, in milliseconds, to stage_ms_host[MOTE_N_STAGES]:
 *   0 route (Eq. 3)   1 dispatch   2 Q_a(x) (Eq. 8)   3 gate/up ternary GEMM (Eq. 6)   4 Q_a(h)
 *   5 down ternary GEMM (Eq. 5)   6 shared gate/up   7 shared down (Eq. 2)   8 combine (Eq. 2, 4)
 * A stage that a path folds into its neighbour reports 0: the tensor path does the combine in the
 * shared-down epilogue (stage 7); the decode path reports its prologue (Q_a(x), router, dispatch)
 * as stage 0 and its two streaming kernels, which cover the routed AND the shared expert (and, in
 * the second one, the combine), as stages 3 and 5.  An RTN prefill's code expansion counts
 * into stage 6.  Stages run back to back on one
 * stream here even if mote_moe_forward overlaps some of them. */
enum { MOTE_N_STAGES = 9 };
mote_status_t mote_moe_forward_profile(const mote_layer_t* L, const void* x_bf16,
                                       const void* residual_bf16, int64_t T, void* out_bf16,
                                       void* ws, size_t ws_bytes, void* stream, float* stage_ms_host);

/* Reads (and clears) the device status word kept in the first 4 bytes of a workspace: MOTE_OK, or
 * MOTE_ERR_DEVICE_TIMEOUT if a kernel gave up a bounded wait (every device-side wait of the GEMM
 * kernels has a time limit; a CTA whose wait runs out stops working, lets copies in flight land,
 * releases its tensor memory, raises this word and returns normally, so the context stays usable
 * and the output of that call is invalid).  Synchronises the stream itself.
 * The word is cleared at the start of every mote_moe_forward / mote_moe_forward_host call and once
 * at the start of mote_stack_forward (not between its layers), so it reports the last such call. */
mote_status_t mote_device_status(void* ws, void* stream);

/* Diagnostic for the mechanism above (no counterpart in the paper): enqueues one thread block that
 * waits, with the GEMM kernels' own bounded wait, on a barrier nothing ever arrives at.  After about
 * limit_ns nanoseconds the wait gives up and the block raises the status word in ws[0..3] exactly
 * as a GEMM would; nothing faults and nothing hangs.  mote_device_status(ws) then returns
 * MOTE_ERR_DEVICE_TIMEOUT once, and MOTE_OK afterwards.
 *   ws        device memory, at least 4 bytes, 256-B aligned (any workspace will do)
 *   limit_ns  1 000 .. 100 000 000 (1 us .. 100 ms); outside -> ERR_SHAPE */
mote_status_t mote_selftest_bounded_wait(void* ws, uint64_t limit_ns, void* stream);

/* Measurement aid (no counterpart in the paper): the int8 tensor-core speed of light of the device,
 * as a kernel to be timed by the caller.  One thread block per SM issues n_batches * 64
 * tcgen05.mma.kind::i8 instructions of the routed expert GEMMs' shape (M128 x N256 x K32,
 * s8 x u8 -> s32) on operands resident in shared memory: no loads, no unpacking, no epilogue.
 * Enqueues one kernel on `stream` and writes the number of integer operations it performs
 * (2 per multiply-accumulate, all SMs) to *ops_host; time the kernel with events on `stream` and
 * divide.  ws: 256-B aligned device memory of at least 4 bytes whose first word receives the device
 * status (see mote_device_status).  n_batches: 1 .. 100000 (about 6 us each). */
mote_status_t mote_int8_mma_peak(void* ws, int n_batches, double* ops_host, void* stream);

/* Number of kernels the last mote_moe_forward call on this thread enqueued. */
int mote_last_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* MOTE_H_ */
