"""CPU oracle for the forward pass of one Mixture-of-Ternary-Experts (MoTE) FFN layer.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the layer
computes, written from the paper's equations (Eq. 2-10 of Section 3.1).  Only the test-suite,
the smoke check and the benchmark's `cpu_baseline` / `--impl reference` legs may import it.  It
shares no code, table or constant with the CUDA library and imports nothing from it.

Conventions
-----------
* bf16 tensors travel as ``uint16`` arrays holding the raw bit patterns.
* A weight matrix is ``W[m, n]`` with ``n`` the reduction ("in") dimension: ``y = W x``
  (Section 3.1: ``W in R^{m x n}``, ``Y = Q_w(W) Q_a(x)``).
* Integer stages are exact.  Floating-point stages are fp64, EXCEPT the few places where a
  float feeds a rounding that decides an integer (the codes, the int8 activations, the bf16
  hidden state h): those are written as explicit sequences of single correctly-rounded fp32
  operations (multiply, add, subtract, divide, round-to-nearest-even) so that an independent
  implementation can reproduce them bit for bit.

Parity pins: every function here is pinned by tests/test_oracle_pins.py (closed forms,
invariants, integer special cases, brute-force loops, the paper's Table 1 / Table 3 memory
figures).  The accuracy tables of the paper need trained weights and public evaluation sets and
are out of scope: "parity unpinned" applies to trained-model behaviour only.
"""
from __future__ import annotations

import math

import numpy as np

F32 = np.float32
EPS_SCALE = F32(1e-5)      # guard for alpha and beta (zero matrix / zero token)

# --------------------------------------------------------------------------------------------
# bf16 <-> fp32 (format definition: bf16 is the upper 16 bits of an IEEE binary32)
# --------------------------------------------------------------------------------------------


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float32."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def f32_to_bf16_rn(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round-to-nearest, ties-to-even); returns uint16 bit patterns.
    Finite inputs only."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


# --------------------------------------------------------------------------------------------
# Eq. 10  RoundClip
# --------------------------------------------------------------------------------------------


def round_clip(x: np.ndarray, a: float, b: float) -> np.ndarray:
    """Eq. 10: max(a, min(b, round(x))), round = nearest integer, ties to even."""
    return np.maximum(a, np.minimum(b, np.rint(x)))


# --------------------------------------------------------------------------------------------
# Eq. 7, 9  absmean ternary weight quantizer, and the INT2 storage of Section 3.1
# --------------------------------------------------------------------------------------------


def absmean_alpha(W: np.ndarray) -> np.float32:
    """Eq. 9: alpha = ||W||_1 / (n m).

    The sum of |w| is taken exactly (math.fsum returns the correctly rounded fp64 value of the
    exact sum), divided by n*m in fp64 and rounded once to fp32.  The result is clamped below
    by 1e-5 so that an all-zero matrix does not divide by zero in Eq. 7."""
    W = np.asarray(W, dtype=np.float32)
    total = math.fsum(np.abs(W).astype(np.float64).ravel().tolist())
    alpha = F32(total / float(W.size))
    return max(alpha, EPS_SCALE)


def ternarize(W: np.ndarray):
    """Eq. 7: Q_w(W) = alpha * RoundClip(W / alpha, -1, 1).

    Returns (codes int8 in {-1,0,1}, alpha fp32).  W / alpha is a true fp32 division."""
    W = np.asarray(W, dtype=np.float32)
    alpha = absmean_alpha(W)
    codes = round_clip(W / alpha, -1.0, 1.0).astype(np.int8)
    return codes, alpha


def pack_codes(codes: np.ndarray) -> np.ndarray:
    """INT2 storage (Section 3.1, last paragraph).  Stored value u = code + 1 in {0,1,2};
    four consecutive elements of the reduction dimension share a byte, element j occupying
    bits [2*(j%4), 2*(j%4)+1].  codes[m, n] -> uint8[m, n/4]."""
    m, n = codes.shape
    assert n % 4 == 0
    u = (codes.astype(np.int16) + 1).astype(np.uint8).reshape(m, n // 4, 4)
    return (u[:, :, 0] | (u[:, :, 1] << 2) | (u[:, :, 2] << 4) | (u[:, :, 3] << 6)).astype(np.uint8)


def unpack_codes(packed: np.ndarray) -> np.ndarray:
    """Inverse of pack_codes: uint8[m, n/4] -> int8[m, n]."""
    m, n4 = packed.shape
    out = np.empty((m, n4, 4), dtype=np.int8)
    for j in range(4):
        out[:, :, j] = ((packed >> (2 * j)) & 3).astype(np.int8) - 1
    return out.reshape(m, n4 * 4)


# --------------------------------------------------------------------------------------------
# Eq. 8  per-token absmax int8 activation quantizer
# --------------------------------------------------------------------------------------------


def quant_act(x_bf16: np.ndarray):
    """Eq. 8-9: beta = ||x||_inf per token, q = RoundClip(127 x / beta, -128, 127).

    x_bf16: uint16[T, d] bf16 bit patterns.  Returns (q int8[T,d], beta fp32[T], rowsum
    int32[T]).  127*x is exact in fp32 for a bf16 x; the division is a true fp32 division;
    beta is clamped below by 1e-5 (an all-zero token gives q = 0)."""
    x = bf16_to_f32(x_bf16)
    beta = np.maximum(np.max(np.abs(x), axis=1), EPS_SCALE).astype(np.float32)
    t = F32(127.0) * x
    q = round_clip(t / beta[:, None], -128.0, 127.0).astype(np.int8)
    rowsum = q.astype(np.int32).sum(axis=1, dtype=np.int32)
    return q, beta, rowsum


def dequant_act(q: np.ndarray, beta: np.ndarray) -> np.ndarray:
    """Q_a(x) of Eq. 8 as real numbers (fp64): beta/127 * q."""
    return q.astype(np.float64) * (beta.astype(np.float64)[:, None] / 127.0)


# --------------------------------------------------------------------------------------------
# Eq. 3  router, top-k selection (GShard-style, no capacity limit, no token dropping)
# --------------------------------------------------------------------------------------------


def router(x_bf16, Wr, bias, k: int, norm_topk: int):
    """Eq. 3: logits f(x) = Wr x (+ bias) in fp64; P = softmax over all E experts.

    Selection: the k largest logits, a tie going to the lower expert index; selected experts
    are listed in descending logit order.  Gate weights: norm_topk=1 -> softmax over the k
    selected logits (sums to 1); norm_topk=0 -> P(x)_i of Eq. 3 itself.
    Returns dict(logits f64[T,E], idx int32[T,k], w f64[T,k], near_tie bool[T]) where near_tie
    marks tokens whose k-th and (k+1)-th logits differ by less than 1e-5."""
    x = bf16_to_f32(x_bf16).astype(np.float64)
    Wr = np.asarray(Wr, dtype=np.float64)
    T = x.shape[0]
    E = Wr.shape[0]
    assert 1 <= k <= E
    logits = x @ Wr.T
    if bias is not None:
        logits = logits + np.asarray(bias, dtype=np.float64)[None, :]
    # stable sort of -logit keeps the lower index first among equals
    order = np.argsort(-logits, axis=1, kind="stable")
    idx = order[:, :k].astype(np.int32)
    sel = np.take_along_axis(logits, idx, axis=1)
    lmax = logits.max(axis=1, keepdims=True)
    if norm_topk:
        ex = np.exp(sel - lmax)
        w = ex / ex.sum(axis=1, keepdims=True)
    else:
        ex_all = np.exp(logits - lmax)
        w = np.exp(sel - lmax) / ex_all.sum(axis=1, keepdims=True)
    if k < E:
        nxt = np.take_along_axis(logits, order[:, k:k + 1], axis=1)[:, 0]
        near_tie = (sel[:, k - 1] - nxt) < 1e-5
    else:
        near_tie = np.zeros(T, dtype=bool)
    return dict(logits=logits, idx=idx, w=w, near_tie=near_tie)


def load_balance_stats(logits: np.ndarray, idx: np.ndarray, E: int):
    """The two per-expert factors of the load-balancing loss (Eq. 12) for a batch of tokens:
    t_i = number of (token, slot) pairs routed to expert i, and sum_x P(x)_i, the routing
    probabilities of Eq. 3 (softmax over all E experts) summed over the batch.  fp64."""
    logits = np.asarray(logits, dtype=np.float64)
    ex = np.exp(logits - logits.max(axis=1, keepdims=True))
    P = ex / ex.sum(axis=1, keepdims=True)
    t = np.bincount(np.asarray(idx).ravel(), minlength=E).astype(np.int64)
    return t, P.sum(axis=0)


def balance_loss(t: np.ndarray, prob_sum: np.ndarray, n_tokens: int) -> float:
    """Eq. 12 as printed: L_balance = E / |X| * sum_i t_i * sum_x P(x)_i."""
    E = len(t)
    return float(E) / float(n_tokens) * float(np.sum(np.asarray(t, np.float64) * np.asarray(prob_sum, np.float64)))


def dispatch(idx: np.ndarray, E: int):
    """Group the T*k (token, slot) pairs by expert, keeping (token, slot) order inside each
    expert (a stable counting sort).  pair p = t*k + j.
    Returns offsets int32[E+1], perm int32[P] (pair -> sorted row), inv int32[P] (row -> pair)."""
    flat = np.asarray(idx, dtype=np.int64).ravel()
    P = flat.size
    counts = np.bincount(flat, minlength=E)
    offsets = np.zeros(E + 1, dtype=np.int32)
    offsets[1:] = np.cumsum(counts)
    inv = np.argsort(flat, kind="stable").astype(np.int32)
    perm = np.empty(P, dtype=np.int32)
    perm[inv] = np.arange(P, dtype=np.int32)
    return offsets, perm, inv


# --------------------------------------------------------------------------------------------
# Eq. 6  SiLU of the gate, evaluated in fp32 by a fixed sequence of correctly-rounded operations
# --------------------------------------------------------------------------------------------

_LOG2E = F32(1.4426950408889634)
# Taylor coefficients of 2^r = sum_i (r ln2)^i / i!, i = 0..6, each rounded to fp32
_EXP2_C = [F32((math.log(2.0) ** i) / math.factorial(i)) for i in range(7)]


def exp_neg_pinned(g: np.ndarray) -> np.ndarray:
    """exp(-g) for fp32 g, as a fixed sequence of single fp32 operations:

        t  = clamp((-g) * log2(e), -125, 125)         one multiply
        n  = rint(t);  r = t - n                      r in [-1/2, 1/2], subtraction exact
        p  = c6; p = p*r + c_i  (i = 5 .. 0)          multiply and add rounded separately
        E  = p * 2^n                                  exact scaling (n in [-125, 125])

    The degree-6 polynomial has truncation error 1.2e-7 relative; together with the rounding
    of t the result is within ~|g| * 1e-7 + 4e-7 relative of exp(-g) on |g| <= 86."""
    g = np.asarray(g, dtype=np.float32)
    t = (-g) * _LOG2E
    t = np.minimum(np.maximum(t, F32(-125.0)), F32(125.0))
    n = np.rint(t)
    r = t - n
    p = np.full_like(r, _EXP2_C[6])
    for i in range(5, -1, -1):
        p = p * r
        p = p + _EXP2_C[i]
    scale = ((n.astype(np.int32) + np.int32(127)) << np.int32(23)).view(np.float32)
    return p * scale


def silu_pinned(g: np.ndarray) -> np.ndarray:
    """sigma of Eq. 6: SiLU(g) = g / (1 + exp(-g)); one fp32 add and one true fp32 division
    on top of exp_neg_pinned."""
    g = np.asarray(g, dtype=np.float32)
    den = F32(1.0) + exp_neg_pinned(g)
    return g / den


# --------------------------------------------------------------------------------------------
# Eq. 5-6  one ternary GLU expert on the rows routed to it
# --------------------------------------------------------------------------------------------


def int_matmul_exact(q: np.ndarray, codes: np.ndarray) -> np.ndarray:
    """acc[r, c] = sum_j q[r, j] * codes[c, j] as exact integers (int32).

    Evaluated with a float64 matrix product: every partial sum is an integer of magnitude at
    most 128 * n < 2^53, so each fp64 addition is exact whatever the summation order."""
    acc = q.astype(np.float64) @ codes.astype(np.float64).T
    return acc.astype(np.int32)


def dequant_scale(alpha: np.float32, beta: np.ndarray) -> np.ndarray:
    """Scale of one ternary linear output row: alpha * (beta / 127), two fp32 operations
    (Section 3.1: Y = Q_w(W) Q_a(x) = alpha * beta/127 * (codes . q))."""
    return F32(alpha) * (np.asarray(beta, dtype=np.float32) / F32(127.0))


def ternary_expert(qx, beta_x, codes_gate, alpha_gate, codes_up, alpha_up, codes_down, alpha_down):
    """Eq. 5-6 for the rows qx[r, d] (already Q_a-quantized, scales beta_x[r]).

        acc_g = codes_gate . qx,  acc_u = codes_up . qx                    exact int32
        g = fl32(acc_g) * c_g,  u = fl32(acc_u) * c_u                      fp32, c = alpha*(beta/127)
        h = bf16( u * silu(g) )                                            fp32 multiply, one rounding
        qh, beta_h = Q_a(h)                                                Eq. 8 on the bf16 h
        acc_d = codes_down . qh                                            exact int32
        y = acc_d * alpha_down * (beta_h / 127)                            fp64

    h is rounded to bf16 before Q_a because the model around the quantized linears runs in
    BF16; Q_a therefore always sees a bf16 tensor, for x and for h alike."""
    acc_g = int_matmul_exact(qx, codes_gate)
    acc_u = int_matmul_exact(qx, codes_up)
    c_g = dequant_scale(alpha_gate, beta_x)[:, None]
    c_u = dequant_scale(alpha_up, beta_x)[:, None]
    g = acc_g.astype(np.float32) * c_g
    u = acc_u.astype(np.float32) * c_u
    h_bf16 = f32_to_bf16_rn(u * silu_pinned(g))
    qh, beta_h, _ = quant_act(h_bf16)
    acc_d = int_matmul_exact(qh, codes_down)
    y = acc_d.astype(np.float64) * float(alpha_down) * (beta_h.astype(np.float64)[:, None] / 127.0)
    return dict(acc_gate=acc_g, acc_up=acc_u, h_bf16=h_bf16, qh=qh, beta_h=beta_h,
                acc_down=acc_d, y=y)


# --------------------------------------------------------------------------------------------
# Eq. 2  shared full-precision expert (the dense checkpoint's SwiGLU FFN, bf16 weights)
# --------------------------------------------------------------------------------------------


def shared_ffn(x_bf16, Wg_bf16, Wu_bf16, Wd_bf16) -> np.ndarray:
    """FFN(x) = W_down ( SiLU(W_gate x) * (W_up x) ), fp64 throughout on the bf16 values,
    no intermediate rounding.  Wg, Wu: [f, d]; Wd: [d, f]."""
    x = bf16_to_f32(x_bf16).astype(np.float64)
    Wg = bf16_to_f32(Wg_bf16).astype(np.float64)
    Wu = bf16_to_f32(Wu_bf16).astype(np.float64)
    Wd = bf16_to_f32(Wd_bf16).astype(np.float64)
    g = x @ Wg.T
    u = x @ Wu.T
    h = u * (g / (1.0 + np.exp(-g)))
    return h @ Wd.T


# --------------------------------------------------------------------------------------------
# Section 4.3  post-training quantization of the shared expert: round-to-nearest (RTN), weight-only
# --------------------------------------------------------------------------------------------


def rtn_quantize(W: np.ndarray, bits: int):
    """RTN absmax quantizer of a weight matrix W[m, n] to `bits`-bit signed integers (8 or 4), one
    scale per output row (the absmax form of Eq. 8-10 applied to the rows of W):

        qmax   = 2^(bits-1) - 1                        127 or 7
        beta_r = max(max_j |W[r, j]|, 1e-5)
        q[r,j] = RoundClip(qmax * W[r, j] / beta_r, -qmax, qmax)
        scale_r = beta_r / qmax                        dequantized weight = scale_r * q[r, j]

    Written as single fp32 operations (one multiply, one true division, round half to even) so
    that the integer codes are reproducible bit for bit.  Returns (q int8 [m, n], scale f32 [m])."""
    if bits not in (8, 4):
        raise ValueError("bits must be 8 or 4")
    W = np.asarray(W, dtype=np.float32)
    qmax = F32(2 ** (bits - 1) - 1)
    beta = np.maximum(np.max(np.abs(W), axis=1), EPS_SCALE).astype(np.float32)
    t = qmax * W
    q = round_clip(t / beta[:, None], -float(qmax), float(qmax)).astype(np.int8)
    scale = (beta / qmax).astype(np.float32)
    return q, scale


def pack_int4(q: np.ndarray) -> np.ndarray:
    """Storage of 4-bit codes: stored nibble u = q + 8 (1..15); every 8 consecutive elements of a
    row form one little-endian 32-bit word whose nibble p (bits 4p..4p+3) holds element 2p and
    whose nibble 4+p holds element 2p+1, p = 0..3.  q: int8 [m, n], n % 8 == 0.  Returns uint8
    [m, n/2] (the words' bytes in memory order)."""
    q = np.asarray(q, dtype=np.int8)
    m, n = q.shape
    if n % 8:
        raise ValueError("n must be a multiple of 8")
    u = (q.astype(np.int32) + 8).astype(np.uint32).reshape(m, n // 8, 8)
    words = np.zeros((m, n // 8), dtype=np.uint32)
    for p in range(4):
        words |= u[:, :, 2 * p] << np.uint32(4 * p)
        words |= u[:, :, 2 * p + 1] << np.uint32(16 + 4 * p)
    return words.astype("<u4").view(np.uint8).reshape(m, n // 2)


def unpack_int4(packed: np.ndarray) -> np.ndarray:
    """Inverse of pack_int4: uint8 [m, n/2] -> int8 [m, n]."""
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    m, nb = packed.shape
    words = packed.view("<u4").astype(np.uint32)
    q = np.zeros((m, nb // 4, 8), dtype=np.int32)
    for p in range(4):
        q[:, :, 2 * p] = ((words >> np.uint32(4 * p)) & np.uint32(15)).astype(np.int32) - 8
        q[:, :, 2 * p + 1] = ((words >> np.uint32(16 + 4 * p)) & np.uint32(15)).astype(np.int32) - 8
    return q.reshape(m, nb * 2).astype(np.int8)


def rtn_dequant(q: np.ndarray, scale: np.ndarray) -> np.ndarray:
    """The weights a weight-only quantized linear multiplies by: scale_r * q[r, j], in fp64."""
    return np.asarray(scale, dtype=np.float64)[:, None] * np.asarray(q, dtype=np.float64)


def shared_ffn_rtn(x_bf16, gate, up, down) -> np.ndarray:
    """FFN(x) of Eq. 2 with RTN weight-only quantized matrices: each of gate, up, down is a pair
    (q int8, scale f32[rows]); activations stay bf16 values; fp64 throughout, no intermediate
    rounding."""
    x = bf16_to_f32(x_bf16).astype(np.float64)
    g = x @ rtn_dequant(*gate).T
    u = x @ rtn_dequant(*up).T
    h = u * (g / (1.0 + np.exp(-g)))
    return h @ rtn_dequant(*down).T


def quantize_shared(layer: dict, bits: int) -> dict:
    """Copy of `layer` whose shared expert is RTN-quantized to `bits` bits (Section 4.3): adds
    layer["sh_rtn"] = {"bits", "gate": (q, scale), "up": ..., "down": ...}."""
    out = dict(layer)
    out["sh_rtn"] = {"bits": bits}
    for name in ("gate", "up", "down"):
        out["sh_rtn"][name] = rtn_quantize(bf16_to_f32(layer["sh_" + name]), bits)
    return out


# --------------------------------------------------------------------------------------------
# Eq. 1-2  LN in front of the layer: RMS normalisation with unit gain (Qwen2.5's norm)
# --------------------------------------------------------------------------------------------


def rms_norm(x_bf16: np.ndarray, eps: float) -> np.ndarray:
    """LN(x) of Eq. 2 as the Qwen2.5 backbone applies it: x / sqrt(mean(x^2) + eps) per token,
    no mean subtraction, unit gain; fp64 on the bf16 values, not rounded."""
    x = bf16_to_f32(x_bf16).astype(np.float64)
    return x / np.sqrt(np.mean(x * x, axis=1, keepdims=True) + eps)


# --------------------------------------------------------------------------------------------
# Eq. 2, 4  the whole layer
# --------------------------------------------------------------------------------------------


def moe_forward(layer: dict, x_bf16: np.ndarray, residual_bf16=None, token_subset=None,
                near_tie_choice=None):
    """out = [residual +] FFN(x) + sum_j w_j * FFN^T_{e_j}(x)   (Eq. 2 and Eq. 4).

    layer: dict with d, f, E, k, norm_topk, Wr[E,d] f32, router_bias[E] f32 or None,
      codes_gate/up [E][f,d] int8, codes_down [E][d,f] int8, alpha_gate/up/down f32[E],
      sh_gate/sh_up [f,d] uint16, sh_down [d,f] uint16; optional sh_rtn (see quantize_shared):
      the shared expert then runs on its RTN-quantized weights (Section 4.3).
    token_subset: optional sorted int array; if given, the expert and shared stages are
      evaluated for those tokens only (tokens are independent of each other), while routing and
      dispatch are still computed for every token.  Row-indexed results are then in the order
      of the subset's pairs sorted by (expert, token, slot); `rows` gives their rows in the
      full dispatch.
    near_tie_choice: optional int32[T, k].  For the tokens the router flags as near ties (k-th
      and (k+1)-th logit closer than 1e-5, where an fp32 router may legitimately pick the other
      expert) the selection is taken from this array instead, and the gate weights are
      recomputed from the oracle's own logits; every other token keeps the oracle's selection.
    Returns a dict of every intermediate named after the stages above."""
    E, k = layer["E"], layer["k"]
    T, d = x_bf16.shape
    r = router(x_bf16, layer["Wr"], layer.get("router_bias"), k, layer["norm_topk"])
    if near_tie_choice is not None and r["near_tie"].any():
        for t in np.nonzero(r["near_tie"])[0]:
            sel_idx = np.asarray(near_tie_choice[t], dtype=np.int32)
            lg = r["logits"][t]
            ex = np.exp(lg[sel_idx] - lg.max())
            denom = ex.sum() if layer["norm_topk"] else np.exp(lg - lg.max()).sum()
            r["idx"][t] = sel_idx
            r["w"][t] = ex / denom
    offsets, perm, inv = dispatch(r["idx"], E)
    qx, beta_x, rowsum_x = quant_act(x_bf16)

    toks = np.arange(T) if token_subset is None else np.asarray(token_subset, dtype=np.int64)
    pair_ids = (toks[:, None] * k + np.arange(k)[None, :]).ravel()
    rows = np.sort(perm[pair_ids]) if pair_ids.size else np.zeros(0, dtype=np.int32)
    row_pairs = inv[rows]
    row_tok = row_pairs // k
    row_exp = r["idx"].ravel()[row_pairs] if rows.size else np.zeros(0, dtype=np.int32)
    R = rows.size
    f = layer["f"]
    acc_gate = np.zeros((R, f), np.int32)
    acc_up = np.zeros((R, f), np.int32)
    h_bf16 = np.zeros((R, f), np.uint16)
    qh = np.zeros((R, f), np.int8)
    beta_h = np.zeros(R, np.float32)
    acc_down = np.zeros((R, d), np.int32)
    y = np.zeros((R, d), np.float64)
    for e in range(E):
        m = np.nonzero(row_exp == e)[0]
        if m.size == 0:
            continue
        t = row_tok[m]
        res = ternary_expert(qx[t], beta_x[t],
                             layer["codes_gate"][e], layer["alpha_gate"][e],
                             layer["codes_up"][e], layer["alpha_up"][e],
                             layer["codes_down"][e], layer["alpha_down"][e])
        acc_gate[m] = res["acc_gate"]; acc_up[m] = res["acc_up"]; h_bf16[m] = res["h_bf16"]
        qh[m] = res["qh"]; beta_h[m] = res["beta_h"]; acc_down[m] = res["acc_down"]; y[m] = res["y"]

    if layer.get("sh_rtn"):
        rtn = layer["sh_rtn"]
        shared = shared_ffn_rtn(x_bf16[toks], rtn["gate"], rtn["up"], rtn["down"])
    else:
        shared = shared_ffn(x_bf16[toks], layer["sh_gate"], layer["sh_up"], layer["sh_down"])
    out = shared.copy()
    if residual_bf16 is not None:
        out += bf16_to_f32(residual_bf16[toks]).astype(np.float64)
    # local row of each (subset token, slot) pair
    row_of_pair = {int(p): i for i, p in enumerate(row_pairs)}
    for i, t in enumerate(toks):
        for j in range(k):
            out[i] += r["w"][t, j] * y[row_of_pair[int(t) * k + j]]
    return dict(logits=r["logits"], topk_idx=r["idx"], topk_w=r["w"], near_tie=r["near_tie"],
                offsets=offsets, perm=perm, inv=inv, qx=qx, beta_x=beta_x, rowsum_x=rowsum_x,
                tokens=toks, rows=rows, row_tok=row_tok, row_exp=row_exp,
                acc_gate=acc_gate, acc_up=acc_up, h_bf16=h_bf16, qh=qh, beta_h=beta_h,
                acc_down=acc_down, y=y, shared_out=shared, out=out)


def build_layer(master: dict) -> dict:
    """Offline step of the path: ternarize every routed matrix (Eq. 7, 9) of a layer given as
    fp32 master weights (dict with W_gate/W_up [E,f,d], W_down [E,d,f] and the other fields
    passed through)."""
    E = master["E"]
    layer = {key: master[key] for key in ("d", "f", "E", "k", "norm_topk", "Wr", "router_bias",
                                           "sh_gate", "sh_up", "sh_down")}
    for name in ("gate", "up", "down"):
        codes, alphas = [], []
        for e in range(E):
            c, a = ternarize(master["W_" + name][e])
            codes.append(c); alphas.append(a)
        layer["codes_" + name] = codes
        layer["alpha_" + name] = np.array(alphas, dtype=np.float32)
    return layer


# --------------------------------------------------------------------------------------------
# Storage accounting (Table 1, Table 3, Section 1): expert memory in bytes
# --------------------------------------------------------------------------------------------


def expert_memory_bytes(n_layers: int, d: int, f: int, n_routed: int,
                        shared_bits: float = 16.0, routed_bits: float = 2.0,
                        n_shared: int = 1) -> float:
    """Bytes of the FFN experts of a model: per layer, each expert holds 3*d*f weights
    (gate, up, down); scales and metadata are not counted (as in the paper's tables)."""
    per_expert = 3.0 * d * f
    return n_layers * per_expert * (n_shared * shared_bits + n_routed * routed_bits) / 8.0
