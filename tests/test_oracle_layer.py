"""Layer-level pins for the CPU oracle: integer special cases, the real-number definition of
Eq. 4-8 evaluated by an independent route, brute-force loops on a tiny layer, and the
structural properties of dispatch and combine."""
import math

import numpy as np
import pytest

from oracle import mote_oracle as O
from workloads import synth


def _bf16(x):
    return O.f32_to_bf16_rn(np.asarray(x, np.float32))


def _tiny_layer(seed=11, d=16, f=32, E=3, k=2, T=5, **kw):
    wl = synth.custom("tiny", d, f, E, k, T, seed, **kw)
    master = synth.master_layer(wl)
    return wl, master, O.build_layer(master), synth.tokens(wl)


# ------------------------------------------------------------------ P5: integer special case
def test_ternary_linear_reduces_to_integer_matmul():
    rng = np.random.default_rng(21)
    a = np.float32(0.375)
    S = rng.integers(-1, 2, size=(24, 40))
    W = (S * a).astype(np.float32)
    codes, alpha = O.ternarize(W)
    # alpha = a * nnz/(nm) <= a, so |W/alpha| >= 1 on the support: codes = sign(W)
    assert np.array_equal(codes, S)
    xi = rng.integers(-127, 128, size=(6, 40))
    xi[:, 3] = -127
    q, beta, _ = O.quant_act(_bf16(xi))
    acc = O.int_matmul_exact(q, codes)
    assert np.array_equal(acc, xi.astype(np.int64) @ S.T.astype(np.int64))
    # Y = Q_w(W) Q_a(x) = alpha * (sign(W) . x) because beta/127 = 1
    c = O.dequant_scale(alpha, beta)
    assert np.all(c == alpha)


def test_int_matmul_exact_against_python_ints():
    rng = np.random.default_rng(22)
    q = rng.integers(-127, 128, size=(3, 2048)).astype(np.int8)
    q[0, :] = 127
    c = rng.integers(-1, 2, size=(4, 2048)).astype(np.int8)
    c[0, :] = 1                                        # extreme accumulator 127 * 2048
    acc = O.int_matmul_exact(q, c)
    for r in range(3):
        for m in range(4):
            assert int(acc[r, m]) == sum(int(a) * int(b) for a, b in zip(q[r], c[m]))


# ------------------------------------------------------------------ Eq. 5-8 by the definition
def test_expert_matches_real_number_definition():
    """Evaluate Eq. 5-6 with Q_w(W) and Q_a(x) as real matrices (fp64) and libm exp; the
    oracle's staged integer/fp32 route must agree up to its stated roundings."""
    wl, master, layer, x = _tiny_layer(seed=12, d=64, f=96, E=2, k=1, T=7)
    qx, beta_x, _ = O.quant_act(x)
    e = 1
    res = O.ternary_expert(qx, beta_x, layer["codes_gate"][e], layer["alpha_gate"][e],
                           layer["codes_up"][e], layer["alpha_up"][e],
                           layer["codes_down"][e], layer["alpha_down"][e])
    Qa_x = O.dequant_act(qx, beta_x)                                    # [T, d]
    Qw_g = float(layer["alpha_gate"][e]) * layer["codes_gate"][e].astype(np.float64)
    Qw_u = float(layer["alpha_up"][e]) * layer["codes_up"][e].astype(np.float64)
    Qw_d = float(layer["alpha_down"][e]) * layer["codes_down"][e].astype(np.float64)
    g = Qa_x @ Qw_g.T
    u = Qa_x @ Qw_u.T
    h_real = u * (g / (1.0 + np.exp(-g)))
    h = O.bf16_to_f32(res["h_bf16"]).astype(np.float64)
    # one bf16 rounding (half an ulp: at most 2^-8 relative) plus ~1e-6 of fp32 evaluation
    assert np.all(np.abs(h - h_real) <= np.abs(h_real) * (2 ** -8 + 2e-5) + 1e-15)  # fp64 noise where acc = 0
    assert np.mean(np.abs(h - h_real)) <= np.mean(np.abs(h_real)) * 2 ** -9
    # down projection from the oracle's own (bf16) h, by the real-number definition
    y_real = O.dequant_act(res["qh"], res["beta_h"]) @ Qw_d.T
    assert np.allclose(res["y"], y_real, rtol=1e-12, atol=1e-18)
    # and Q_a(h) is the quantizer of test_oracle_pins applied to h
    qh2, bh2, _ = O.quant_act(res["h_bf16"])
    assert np.array_equal(qh2, res["qh"]) and np.array_equal(bh2, res["beta_h"])


# ------------------------------------------------------------------ P8: brute force, tiny layer
def test_tiny_layer_brute_force():
    wl, master, layer, x = _tiny_layer()
    d, f, E, k, T = wl.d, wl.f, wl.E, wl.k, wl.T
    out = O.moe_forward(layer, x)
    xf = [[float(v) for v in row] for row in O.bf16_to_f32(x)]
    Wr = master["Wr"].astype(np.float64)
    sh = {n: O.bf16_to_f32(master[n]).astype(np.float64) for n in ("sh_gate", "sh_up", "sh_down")}
    for t in range(T):
        # router by loops
        logits = [sum(xf[t][j] * Wr[e, j] for j in range(d)) for e in range(E)]
        order = sorted(range(E), key=lambda e: (-logits[e], e))[:k]
        assert order == out["topk_idx"][t].tolist()
        ex = [math.exp(logits[e] - max(logits)) for e in order]
        gate_w = [v / sum(ex) for v in ex]
        # Q_a(x) by scalar arithmetic on Python floats (fp64 is exact enough away from ties)
        beta = max(abs(v) for v in xf[t])
        q = [max(-128, min(127, round(127 * v / beta))) for v in xf[t]]
        assert q == out["qx"][t].tolist()
        total = [0.0] * d
        for j, e in enumerate(order):
            cg, cu, cd = (layer["codes_" + n][e] for n in ("gate", "up", "down"))
            ag, au, ad = (float(layer["alpha_" + n][e]) for n in ("gate", "up", "down"))
            row = int(out["perm"][t * k + j])
            acc_g = [sum(int(cg[c, i]) * q[i] for i in range(d)) for c in range(f)]
            acc_u = [sum(int(cu[c, i]) * q[i] for i in range(d)) for c in range(f)]
            assert acc_g == out["acc_gate"][row].tolist()
            assert acc_u == out["acc_up"][row].tolist()
            # h in real arithmetic, compared through the bf16 grid
            h = []
            for c in range(f):
                g = acc_g[c] * ag * beta / 127
                u = acc_u[c] * au * beta / 127
                h.append(u * g / (1 + math.exp(-g)))
            h_or = O.bf16_to_f32(out["h_bf16"][row]).astype(np.float64)
            assert np.all(np.abs(h_or - np.array(h)) <= np.abs(h) * 2 ** -8 + 1e-30)
            # down projection from the oracle's h
            bh = max(float(np.max(np.abs(h_or))), 1e-5)
            qh = [max(-128, min(127, round(127 * v / bh))) for v in h_or.tolist()]
            diff = np.abs(np.array(qh) - out["qh"][row].astype(int))
            assert diff.max() <= 1 and (diff > 0).mean() < 0.05       # fp64 vs fp32 near ties
            qh = out["qh"][row].astype(int).tolist()
            acc_d = [sum(int(cd[c, i]) * qh[i] for i in range(f)) for c in range(d)]
            assert acc_d == out["acc_down"][row].tolist()
            for c in range(d):
                total[c] += gate_w[j] * acc_d[c] * ad * bh / 127
        # shared expert by loops
        g = [sum(sh["sh_gate"][c, i] * xf[t][i] for i in range(d)) for c in range(f)]
        u = [sum(sh["sh_up"][c, i] * xf[t][i] for i in range(d)) for c in range(f)]
        hs = [u[c] * g[c] / (1 + math.exp(-g[c])) for c in range(f)]
        for c in range(d):
            total[c] += sum(sh["sh_down"][c, i] * hs[i] for i in range(f))
        assert np.allclose(out["out"][t], total, rtol=1e-9, atol=1e-12)


# ------------------------------------------------------------------ P7: structure
def test_token_permutation_equivariance_and_subsets():
    wl, master, layer, x = _tiny_layer(seed=13, d=32, f=64, E=4, k=2, T=12)
    base = O.moe_forward(layer, x)
    pm = np.random.default_rng(0).permutation(wl.T)
    shuf = O.moe_forward(layer, x[pm])
    assert np.array_equal(shuf["out"], base["out"][pm])
    # evaluating a subset of tokens gives the same rows
    sub = np.array([1, 4, 9])
    part = O.moe_forward(layer, x, token_subset=sub)
    assert np.array_equal(part["out"], base["out"][sub])
    assert np.array_equal(part["acc_down"], base["acc_down"][part["rows"]])
    assert np.array_equal(part["h_bf16"], base["h_bf16"][part["rows"]])


def test_residual_is_added_and_single_expert_needs_no_dispatch():
    wl, master, layer, x = _tiny_layer(seed=14, d=32, f=64, E=1, k=1, T=6)
    res = _bf16(np.random.default_rng(1).standard_normal((wl.T, wl.d)))
    a = O.moe_forward(layer, x)
    b = O.moe_forward(layer, x, residual_bf16=res)
    assert np.allclose(b["out"] - a["out"], O.bf16_to_f32(res).astype(np.float64), atol=1e-12)
    # E = 1, k = 1: gate weight is 1, the layer is one ternary FFN plus the shared FFN
    assert np.all(a["topk_w"] == 1.0) and np.array_equal(a["perm"], np.arange(wl.T))
    qx, bx, _ = O.quant_act(x)
    direct = O.ternary_expert(qx, bx, layer["codes_gate"][0], layer["alpha_gate"][0],
                              layer["codes_up"][0], layer["alpha_up"][0],
                              layer["codes_down"][0], layer["alpha_down"][0])
    sh = O.shared_ffn(x, layer["sh_gate"], layer["sh_up"], layer["sh_down"])
    assert np.allclose(a["out"], direct["y"] + sh, rtol=1e-12, atol=1e-15)


def test_idle_expert_contributes_nothing():
    wl, master, layer, x = _tiny_layer(seed=15, d=32, f=64, E=4, k=1, T=8)
    bias = np.array([0, 0, -1e4, 0], np.float32)        # expert 2 can never win
    layer["router_bias"] = bias
    a = O.moe_forward(layer, x)
    assert a["offsets"][3] == a["offsets"][2]
    layer["codes_down"][2] = layer["codes_down"][2] * 0 + 1     # tamper with the idle expert
    b = O.moe_forward(layer, x)
    assert np.array_equal(a["out"], b["out"])


def test_workload_generators_are_seeded():
    wl = synth.WORKLOADS["c1"]
    a, b = synth.tokens(wl), synth.tokens(wl)
    assert np.array_equal(a, b) and a.shape == (64, 256) and a.dtype == np.uint16
    Wr, bias = synth.router_weights(synth.WORKLOADS["c3"], 0)
    p = np.exp(bias.astype(np.float64))
    assert abs(p.sum() - 1) < 1e-6 and abs(p[0] - 0.398) < 1e-3    # Zipf(1.1) over 8 experts
    x2 = O.bf16_to_f32(synth.tokens(synth.WORKLOADS["c2"], T=512)).astype(np.float64)
    big = (x2.std(axis=0) > 10).sum()
    assert big == 9                                                  # round(0.01 * 896)


# ------------------------------------------------------------------ Section 4.3: RTN shared expert
@pytest.mark.parametrize("bits", [8, 4])
def test_rtn_layer_equals_plain_layer_when_rtn_is_lossless(bits):
    # shared weights that already sit on the RTN grid (integers up to qmax times a power of two per
    # row, qmax attained): quantization changes nothing, so the layer must equal the bf16 layer
    wl, master, _, x = _tiny_layer(seed=31, d=32, f=64, E=3, k=2, T=6)
    rng = np.random.default_rng(70 + bits)
    qmax = 2 ** (bits - 1) - 1
    for name, shape in (("sh_gate", (64, 32)), ("sh_up", (64, 32)), ("sh_down", (32, 64))):
        Wi = rng.integers(-qmax, qmax + 1, size=shape)
        Wi[:, 0] = qmax
        row_scale = 2.0 ** rng.integers(-9, -5, size=(shape[0], 1))
        master[name] = _bf16(Wi * row_scale)
        assert np.array_equal(O.bf16_to_f32(master[name]).astype(np.float64), Wi * row_scale)
    layer = O.build_layer(master)
    plain = O.moe_forward(layer, x)
    rtn = O.moe_forward(O.quantize_shared(layer, bits), x)
    assert np.allclose(rtn["shared_out"], plain["shared_out"], rtol=1e-12, atol=0)
    assert np.allclose(rtn["out"], plain["out"], rtol=1e-12, atol=0)


@pytest.mark.parametrize("bits", [8, 4])
def test_rtn_shared_ffn_brute_force_and_error_scale(bits):
    wl, master, layer, x = _tiny_layer(seed=32, d=16, f=32, E=2, k=1, T=3)
    ql = O.quantize_shared(layer, bits)
    (qg, sg), (qu, su), (qd, sd) = (ql["sh_rtn"][n] for n in ("gate", "up", "down"))
    xf = O.bf16_to_f32(x).astype(np.float64)
    got = O.shared_ffn_rtn(x, (qg, sg), (qu, su), (qd, sd))
    for t in range(3):
        h = []
        for r in range(32):
            g = sum(float(sg[r]) * int(qg[r, j]) * xf[t, j] for j in range(16))
            u = sum(float(su[r]) * int(qu[r, j]) * xf[t, j] for j in range(16))
            h.append(u * g / (1.0 + math.exp(-g)))
        for c in range(16):
            ref = sum(float(sd[c]) * int(qd[c, r]) * h[r] for r in range(32))
            assert math.isclose(got[t, c], ref, rel_tol=1e-10, abs_tol=1e-15)
    # the quantized FFN approaches the bf16 FFN as the grid refines: INT8 error far below INT4 error
    plain = O.shared_ffn(x, layer["sh_gate"], layer["sh_up"], layer["sh_down"])
    rel = np.linalg.norm(got - plain) / np.linalg.norm(plain)
    assert rel < (0.05 if bits == 8 else 0.6)


# ------------------------------------------------------------------ Eq. 3-4 with an imposed selection
@pytest.mark.parametrize("norm_topk", [1, 0])
def test_near_tie_choice_takes_the_other_valid_pick_and_recomputes_the_gate(norm_topk):
    """A token whose k-th and (k+1)-th logits tie exactly may be routed either way by an fp32
    router.  moe_forward(near_tie_choice=...) must take the imposed selection for that token only,
    give it the gate weights of Eq. 3 (softmax over the selected k, or over all E experts) from
    the oracle's own logits, and leave every other token alone."""
    d, f, E, k, T = 16, 32, 4, 2, 3
    wl = synth.custom("tie", d, f, E, k, T, 31, norm_topk=norm_topk)
    master = synth.master_layer(wl)
    # hand-made router: token 0 has logits (2, 1, 1, -1): experts 1 and 2 tie for the second slot
    Wr = np.zeros((E, d), np.float32)
    Wr[0, 0], Wr[1, 0], Wr[2, 0], Wr[3, 0] = 2.0, 1.0, 1.0, -1.0
    Wr[:, 1] = [0.5, -0.25, 3.0, 0.125]                 # tokens 1, 2 use channel 1: no tie
    master["Wr"], master["router_bias"] = Wr, None
    layer = O.build_layer(master)
    xf = np.zeros((T, d), np.float32)
    xf[0, 0] = 1.0
    xf[1, 1] = 1.0
    xf[2, 1] = -2.0
    xf[:, 2:] = np.random.default_rng(5).standard_normal((T, d - 2)).astype(np.float32)
    x = _bf16(xf)
    base = O.moe_forward(layer, x)
    assert base["near_tie"].tolist() == [True, False, False]
    assert base["topk_idx"][0].tolist() == [0, 1]        # ties go to the lower index
    # the other valid pick for token 0; nonsense for the unflagged tokens, which must be ignored
    choice = np.array([[0, 2], [3, 3], [1, 1]], np.int32)
    got = O.moe_forward(layer, x, near_tie_choice=choice)
    assert got["topk_idx"][0].tolist() == [0, 2]
    assert np.array_equal(got["topk_idx"][1:], base["topk_idx"][1:])
    assert np.array_equal(got["topk_w"][1:], base["topk_w"][1:])
    assert np.array_equal(got["out"][1:], base["out"][1:])
    # gate weights of token 0 by scalar arithmetic on the exact logits (2, 1, 1, -1)
    lg = [2.0, 1.0, 1.0, -1.0]
    sel = [0, 2]
    den = sum(math.exp(lg[e]) for e in (sel if norm_topk else range(E)))
    want = [math.exp(lg[e]) / den for e in sel]
    assert np.allclose(got["topk_w"][0], want, rtol=1e-12)
    assert np.allclose(got["topk_w"][0], base["topk_w"][0], rtol=1e-12)   # equal logits, equal weights
    if norm_topk:
        assert abs(got["topk_w"][0].sum() - 1.0) < 1e-12
    else:
        assert got["topk_w"][0].sum() < 0.9              # the mass of the unselected experts is missing
    # dispatch follows the imposed selection, and the output is the sum over the imposed experts:
    # recompute token 0 from the per-expert stages
    assert np.array_equal(np.diff(got["offsets"]), np.bincount(got["topk_idx"].ravel(), minlength=E))
    qx, bx, _ = O.quant_act(x[:1])
    total = O.shared_ffn(x[:1], layer["sh_gate"], layer["sh_up"], layer["sh_down"])[0]
    for j, e in enumerate(sel):
        r = O.ternary_expert(qx, bx, layer["codes_gate"][e], layer["alpha_gate"][e], layer["codes_up"][e],
                             layer["alpha_up"][e], layer["codes_down"][e], layer["alpha_down"][e])
        total = total + want[j] * r["y"][0]
    assert np.allclose(got["out"][0], total, rtol=1e-12, atol=1e-15)
    # experts 1 and 2 hold different weights, so the imposed pick really changes the result
    assert not np.allclose(got["out"][0], base["out"][0], rtol=1e-6)
