"""Pins for the CPU oracle: everything here checks oracle/mote_oracle.py against something
other than itself -- figures the paper prints, closed forms, invariants, integer special
cases, library routines, and brute-force loops on tiny inputs."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import mote_oracle as O
from workloads import synth

HERE = os.path.dirname(os.path.abspath(__file__))


# ------------------------------------------------------------------ P1: storage accounting
def _memory_rows():
    rows = []
    with open(os.path.join(HERE, "golden", "paper_memory_figures.txt")) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            p = [s.strip() for s in line.split("|")]
            rows.append((p[0], int(p[1]), int(p[2]), int(p[3]), int(p[4]), float(p[5]),
                         int(p[6]), float(p[7]), p[8]))
    return rows


@pytest.mark.parametrize("row", _memory_rows(), ids=lambda r: r[0])
def test_expert_memory_matches_paper_tables(row):
    _, L, d, f, n_sh, sh_bits, n_r, r_bits, printed = row
    gib = O.expert_memory_bytes(L, d, f, n_r, shared_bits=sh_bits, routed_bits=r_bits,
                                n_shared=n_sh) / 2 ** 30
    assert f"{gib:.1f}" == printed, (gib, printed)


def test_intro_memory_example_16_experts():
    # Section 1: Qwen2.5-3B, every FFN replaced by 16 bf16 experts: 5.2 GB -> 73.2 GB of
    # non-embedding weights.  Attention/norm parameters per layer (16 heads, 2 KV heads of
    # 128, hidden 2048, q/k/v biases, two RMSNorm weights) are the public architecture.
    L, d, f = 36, 2048, 11008
    attn = (d * d + d) + 2 * (d * 256 + 256) + d * d + 2 * d
    other = (L * attn + d) * 2
    dense = other + O.expert_memory_bytes(L, d, f, 0, n_shared=1)
    moe16 = other + O.expert_memory_bytes(L, d, f, 16, routed_bits=16, n_shared=0)
    assert f"{dense / 2**30:.1f}" == "5.2"
    assert f"{moe16 / 2**30:.1f}" == "73.2"


def test_ratio_38_percent():
    # Section 4.2: MoTE 3B needs 38 % of MoE-LLaVA's expert memory
    a = O.expert_memory_bytes(36, 2048, 11008, 4)
    b = O.expert_memory_bytes(36, 2048, 11008, 4, routed_bits=16, n_shared=0)
    assert round(100 * a / b) == 38


# ------------------------------------------------------------------ bf16 helpers vs library
def test_bf16_conversions_match_torch():
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.standard_normal(20000).astype(np.float32) * 3,
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40],
                                 dtype=np.float32)])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = O.f32_to_bf16_rn(x)
    assert np.array_equal(got, want)
    back = torch.from_numpy(want.view(np.int16)).view(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(O.bf16_to_f32(got), back)


def test_bf16_ties_to_even_by_hand():
    # 1 + 2^-8 is exactly half-way between bf16 1.0 (even) and 1.0078125 (odd): goes to 1.0;
    # 1.0078125 + 2^-8 is half-way between odd 0x3F81 and even 0x3F82: goes to 0x3F82.
    x = np.array([1.0 + 2.0 ** -8, 1.0078125 + 2.0 ** -8], dtype=np.float32)
    assert O.f32_to_bf16_rn(x).tolist() == [0x3F80, 0x3F82]


# ------------------------------------------------------------------ Eq. 10
def test_round_clip_by_hand():
    x = np.array([-7.2, -1.5, -0.5, -0.4, 0.5, 0.51, 1.5, 2.5, 9.0], dtype=np.float32)
    assert O.round_clip(x, -1, 1).tolist() == [-1, -1, -0.0, -0.0, 0, 1, 1, 1, 1]
    assert O.round_clip(np.array([126.5, 127.5, -128.5, -300.0]), -128, 127).tolist() == \
        [126, 127, -128, -128]


# ------------------------------------------------------------------ P2: Q_w definition
def test_qw_invariants():
    rng = np.random.default_rng(2)
    W = (rng.standard_normal((96, 200)) * 0.02).astype(np.float32)
    codes, alpha = O.ternarize(W)
    assert set(np.unique(codes).tolist()) <= {-1, 0, 1}
    # alpha equals the mean of |W| (exact rational arithmetic), rounded once
    exact = sum(Fraction(float(abs(v))) for v in W.ravel()) / W.size
    assert abs(Fraction(float(alpha)) - exact) <= Fraction(float(np.spacing(alpha))) / 2 + \
        Fraction(1, 2 ** 80)
    # sign symmetry and power-of-two scaling
    c2, a2 = O.ternarize(-W)
    assert np.array_equal(c2, -codes) and a2 == alpha
    c3, a3 = O.ternarize(W * np.float32(8.0))
    assert np.array_equal(c3, codes) and a3 == alpha * np.float32(8.0)
    # codes are the nearest of {-1,0,1} to W/alpha in exact arithmetic
    ratio = W.astype(np.float64) / float(alpha)
    nearest = np.clip(np.round(ratio), -1, 1)
    off = np.abs(np.abs(ratio) - 0.5) > 1e-6       # away from the rounding boundary
    assert np.array_equal(codes[off], nearest[off].astype(np.int8))


def test_qw_zero_matrix_and_threshold():
    codes, alpha = O.ternarize(np.zeros((4, 8), np.float32))
    assert alpha == np.float32(1e-5) and not codes.any()
    # |W| = alpha/2 exactly is a tie: ties-to-even sends +-0.5 to 0, +-1.5 to +-1 (clipped 2 -> 1)
    W = np.array([[0.5, -0.5, 1.5, -1.5, 1.0, -1.0, 1.0, 1.0]], np.float32)   # mean |W| = 1
    codes, alpha = O.ternarize(W)
    assert alpha == 1.0 and codes.tolist() == [[0, 0, 1, -1, 1, -1, 1, 1]]


def test_qw_gaussian_closed_form():
    # P3: W ~ N(0, s^2): alpha/s -> sqrt(2/pi); P(code = 0) = erf(sqrt(2/pi) / (2 sqrt 2))
    s = 0.02
    W = (torch.randn((1500, 2000), generator=torch.Generator().manual_seed(5)) * s).numpy()
    codes, alpha = O.ternarize(W)
    assert abs(alpha / s - math.sqrt(2 / math.pi)) < 2e-3
    p0 = math.erf(math.sqrt(2 / math.pi) / (2 * math.sqrt(2)))
    assert abs((codes == 0).mean() - p0) < 2e-3
    assert abs((codes == 1).mean() - (1 - p0) / 2) < 2e-3


def test_pack_layout_by_hand():
    codes = np.array([[-1, 0, 1, 1, 0, 0, 0, -1]], np.int8)
    packed = O.pack_codes(codes)
    # u = code+1 = [0,1,2,2 | 1,1,1,0]; element j sits in bits 2j..2j+1 of its byte
    assert packed.tolist() == [[0 | (1 << 2) | (2 << 4) | (2 << 6), 1 | (1 << 2) | (1 << 4)]]
    rng = np.random.default_rng(3)
    c = rng.integers(-1, 2, size=(17, 64)).astype(np.int8)
    p = O.pack_codes(c)
    assert p.shape == (17, 16) and np.array_equal(O.unpack_codes(p), c)
    # the bit pair 0b11 never occurs
    assert not np.any([((p >> s) & 3) == 3 for s in (0, 2, 4, 6)])


# ------------------------------------------------------------------ P4: Q_a definition
def _bf16(x):
    return O.f32_to_bf16_rn(np.asarray(x, np.float32))


def test_qa_invariants():
    rng = np.random.default_rng(4)
    x = _bf16(rng.standard_normal((50, 96)) * 3)
    x[7] = 0                                           # an all-zero token
    q, beta, rowsum = O.quant_act(x)
    xf = O.bf16_to_f32(x).astype(np.float64)
    assert np.abs(q.astype(int)).max() <= 127
    nz = np.abs(xf).max(axis=1) > 0
    assert np.all(np.abs(q[nz].astype(int)).max(axis=1) == 127)
    assert not q[7].any() and beta[7] == np.float32(1e-5)
    assert np.array_equal(beta[nz].astype(np.float64), np.abs(xf[nz]).max(axis=1))
    assert np.array_equal(rowsum, q.astype(np.int64).sum(axis=1))
    # dequantisation error bound |x - beta q / 127| <= beta / 254
    err = np.abs(xf - O.dequant_act(q, beta))
    assert np.all(err <= beta.astype(np.float64)[:, None] / 254 * (1 + 1e-6))
    # power-of-two scale invariance
    x4 = _bf16(O.bf16_to_f32(x) * np.float32(4))
    q4, beta4, _ = O.quant_act(x4)
    assert np.array_equal(q4, q) and np.array_equal(beta4[nz], beta[nz] * 4)


def test_qa_integer_tokens_are_lossless():
    # P5: integer entries in [-127,127] with max |x| = 127 -> beta = 127 and q = x
    rng = np.random.default_rng(5)
    xi = rng.integers(-127, 128, size=(9, 64))
    xi[:, 0] = 127
    q, beta, _ = O.quant_act(_bf16(xi))
    assert np.all(beta == 127) and np.array_equal(q, xi)


# ------------------------------------------------------------------ P9: pinned SiLU
def test_exp_and_silu_accuracy():
    g = np.linspace(-30, 30, 240001).astype(np.float32)
    got = O.exp_neg_pinned(g).astype(np.float64)
    want = np.exp(-g.astype(np.float64))
    rel = np.abs(got - want) / want
    assert rel.max() < 5e-6, rel.max()
    assert np.all(rel[np.abs(g) <= 1] < 6e-7)
    s = O.silu_pinned(g).astype(np.float64)
    sw = g.astype(np.float64) / (1 + want)
    assert np.max(np.abs(s - sw) / np.maximum(np.abs(sw), 1e-30)) < 5e-6
    assert O.silu_pinned(np.float32(0.0)) == 0
    big = np.array([25.0, 60.0, 200.0, 1e4], np.float32)
    assert np.array_equal(O.silu_pinned(big), big)
    neg = O.silu_pinned(np.array([-100.0, -1e4], np.float32))
    assert np.all(neg <= 0) and np.all(np.abs(neg) < 1e-30)
    # monotone increasing to the right of its minimum (x ~ -1.278)
    gm = np.linspace(-1.2, 20, 50001).astype(np.float32)
    assert np.all(np.diff(O.silu_pinned(gm).astype(np.float64)) >= 0)


# ------------------------------------------------------------------ P6: router
def test_router_properties():
    rng = np.random.default_rng(6)
    T, d, E = 40, 32, 6
    x = _bf16(rng.standard_normal((T, d)))
    Wr = O.bf16_to_f32(_bf16(rng.standard_normal((E, d)) * 0.3))
    bias = rng.standard_normal(E).astype(np.float32)
    for k in (1, 2, 6):
        r = O.router(x, Wr, bias, k, 1)
        assert np.allclose(r["w"].sum(axis=1), 1.0, atol=1e-12)
        if k == 1:
            assert np.all(r["w"] == 1.0)
        # descending order and really the k largest
        sel = np.take_along_axis(r["logits"], r["idx"], axis=1)
        assert np.all(np.diff(sel, axis=1) <= 0)
        assert np.all(np.sort(r["logits"], axis=1)[:, ::-1][:, :k] == sel)
    # k = E without renormalisation is the plain softmax of Eq. 3 (library routine)
    r = O.router(x, Wr, bias, E, 0)
    sm = torch.softmax(torch.from_numpy(r["logits"]), dim=1).numpy()
    assert np.allclose(r["w"], np.take_along_axis(sm, r["idx"], axis=1), rtol=1e-12, atol=0)
    # logits by an explicit loop
    xf = O.bf16_to_f32(x).astype(np.float64)
    for t in (0, 17):
        for e in range(E):
            acc = sum(xf[t, j] * float(Wr[e, j]) for j in range(d)) + float(bias[e])
            assert abs(acc - r["logits"][t, e]) < 1e-12
    # permuting the experts permutes the indices
    pm = rng.permutation(E)
    r2 = O.router(x, Wr[pm], bias[pm], 2, 1)
    r1 = O.router(x, Wr, bias, 2, 1)
    assert np.array_equal(pm[r2["idx"]], r1["idx"])
    # norm_topk=0 with k<E: the selected probabilities of the full softmax
    r0 = O.router(x, Wr, bias, 2, 0)
    sm0 = torch.softmax(torch.from_numpy(r0["logits"]), dim=1).numpy()
    assert np.allclose(r0["w"], np.take_along_axis(sm0, r0["idx"], axis=1), rtol=1e-12)


def test_router_ties_go_to_lower_index_and_are_flagged():
    x = _bf16(np.ones((1, 4)))
    Wr = np.zeros((5, 4), np.float32)
    Wr[1] = Wr[3] = Wr[4] = 0.25                       # three equal logits of 1.0
    r = O.router(x, Wr, None, 2, 1)
    assert r["idx"].tolist() == [[1, 3]] and bool(r["near_tie"][0])
    r = O.router(x, Wr, np.array([0, 0.5, 0, 0.25, 0], np.float32), 2, 1)
    assert r["idx"].tolist() == [[1, 3]] and not bool(r["near_tie"][0])


# ------------------------------------------------------------------ dispatch
def test_dispatch_is_a_stable_counting_sort():
    rng = np.random.default_rng(7)
    E, T, k = 5, 23, 2
    idx = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    idx[idx == 3] = 0                                  # expert 3 gets nothing
    offsets, perm, inv = O.dispatch(idx, E)
    want = sorted(range(T * k), key=lambda p: (idx.ravel()[p], p))
    assert inv.tolist() == want
    assert np.array_equal(perm[inv], np.arange(T * k))
    for e in range(E):
        assert offsets[e + 1] - offsets[e] == int((idx == e).sum())
    assert offsets[4] == offsets[3]


# ------------------------------------------------------------------ LN of Eq. 2 (RMS norm)
def test_rms_norm_against_library_and_invariants():
    rng = np.random.default_rng(21)
    x = O.f32_to_bf16_rn((rng.standard_normal((7, 96)) * np.array([[0.01], [1], [30], [1], [2], [5], [0.5]])).astype(np.float32))
    got = O.rms_norm(x, 1e-6)
    xt = torch.from_numpy(O.bf16_to_f32(x).astype(np.float64))
    want = torch.nn.functional.rms_norm(xt, (96,), eps=1e-6).numpy()          # library routine, fp64
    assert np.allclose(got, want, rtol=1e-12, atol=0)
    assert np.allclose(np.sqrt(np.mean(got * got, axis=1))[1:], 1.0, atol=1e-5)   # unit rms (eps negligible)
    # scale invariance for power-of-two scalings (exact in bf16), eps -> 0
    x4 = O.f32_to_bf16_rn(O.bf16_to_f32(x) * np.float32(4.0))
    assert np.allclose(O.rms_norm(x4, 0.0), O.rms_norm(x, 0.0), rtol=1e-12)
    # a one-hot row of height a normalises to sqrt(d) at that position
    one = np.zeros((1, 64), np.float32); one[0, 5] = -3.0
    r = O.rms_norm(O.f32_to_bf16_rn(one), 0.0)
    assert abs(r[0, 5] + 8.0) < 1e-12 and np.count_nonzero(r) == 1
    # all-zero row stays zero when eps > 0
    assert np.all(O.rms_norm(np.zeros((1, 16), np.uint16), 1e-6) == 0)


# ------------------------------------------------------------------ Section 4.3: RTN of the shared expert
@pytest.mark.parametrize("bits", [8, 4])
def test_rtn_invariants(bits):
    rng = np.random.default_rng(40 + bits)
    qmax = 2 ** (bits - 1) - 1
    W = O.bf16_to_f32(_bf16(rng.standard_normal((37, 96)) * 0.02))
    W[5] = 0                                           # an all-zero output row
    q, scale = O.rtn_quantize(W, bits)
    Wd = W.astype(np.float64)
    assert q.dtype == np.int8 and np.abs(q.astype(int)).max() == qmax
    nz = np.abs(Wd).max(axis=1) > 0
    assert np.all(np.abs(q[nz].astype(int)).max(axis=1) == qmax)       # the absmax element maps to +-qmax
    assert not q[5].any()
    # scale = absmax / qmax, to one fp32 rounding
    assert np.allclose(scale[nz].astype(np.float64), np.abs(Wd[nz]).max(axis=1) / qmax, rtol=2 ** -23)
    # round-to-nearest: |w - scale*q| <= scale/2 (+ the fp32 roundings of the pinned sequence)
    err = np.abs(Wd - O.rtn_dequant(q, scale))
    assert np.all(err <= scale.astype(np.float64)[:, None] * (0.5 + 1e-5))
    # odd symmetry and power-of-two scale invariance
    qn, sn = O.rtn_quantize(-W, bits)
    assert np.array_equal(qn, -q) and np.array_equal(sn, scale)
    q8, s8 = O.rtn_quantize(W * np.float32(8), bits)
    assert np.array_equal(q8, q) and np.array_equal(s8[nz], scale[nz] * 8)
    # nearest grid point by brute force in exact rational arithmetic, away from ties
    for r in (0, 11, 36):
        beta = Fraction(float(np.abs(W[r]).max()))
        for j in range(0, 96, 7):
            t = Fraction(float(W[r, j])) * qmax / beta
            lo = math.floor(t)
            if abs(t - lo - Fraction(1, 2)) > Fraction(1, 1000):
                assert int(q[r, j]) == (lo if t - lo < Fraction(1, 2) else lo + 1)


@pytest.mark.parametrize("bits", [8, 4])
def test_rtn_integer_rows_are_lossless(bits):
    # rows of integers in [-qmax, qmax] (times a power of two) that attain qmax: q = the integers, scale = 2^j
    rng = np.random.default_rng(50 + bits)
    qmax = 2 ** (bits - 1) - 1
    Wi = rng.integers(-qmax, qmax + 1, size=(12, 64))
    Wi[:, 3] = qmax
    q, scale = O.rtn_quantize((Wi * 0.25).astype(np.float32), bits)
    assert np.array_equal(q, Wi) and np.all(scale == np.float32(0.25))
    assert np.array_equal(O.rtn_dequant(q, scale), Wi * 0.25)


def test_rtn_int8_is_eq8_applied_to_weight_rows():
    # with 8 bits the quantizer is Eq. 8 with a weight row in the place of a token
    rng = np.random.default_rng(60)
    Wb = _bf16(rng.standard_normal((21, 80)) * 0.02)
    q, scale = O.rtn_quantize(O.bf16_to_f32(Wb), 8)
    qa, beta, _ = O.quant_act(Wb)
    assert np.array_equal(q, qa) and np.array_equal(scale, beta / np.float32(127))


def test_int4_storage_by_hand_and_size():
    # one word by hand: elements 0..7 = -8+u with u = 1..8 -> nibbles (e0,e2,e4,e6 | e1,e3,e5,e7)
    q = np.array([[-7, -6, -5, -4, -3, -2, -1, 0]], dtype=np.int8)
    packed = O.pack_int4(q)
    word = int.from_bytes(bytes(packed[0]), "little")
    assert word == 0x8642_7531
    # independent decoder: python integers
    rng = np.random.default_rng(61)
    q = rng.integers(-7, 8, size=(5, 48)).astype(np.int8)
    packed = O.pack_int4(q)
    assert packed.shape == (5, 24) and packed.dtype == np.uint8          # 4 bits per weight
    for r in range(5):
        for w in range(6):
            word = int.from_bytes(bytes(packed[r, 4 * w:4 * w + 4]), "little")
            for p in range(4):
                assert ((word >> (4 * p)) & 15) - 8 == q[r, 8 * w + 2 * p]
                assert ((word >> (16 + 4 * p)) & 15) - 8 == q[r, 8 * w + 2 * p + 1]
    assert np.array_equal(O.unpack_int4(packed), q)
    # bytes per weight behind the Table 3 footprints: 1 (INT8) and 1/2 (INT4), scales not counted
    q8, _ = O.rtn_quantize(rng.standard_normal((16, 64)).astype(np.float32), 8)
    assert q8.nbytes == 16 * 64 and packed.nbytes * 2 == q.size


# ------------------------------------------------------------------ Eq. 12: load-balance factors
def test_load_balance_stats_and_loss():
    rng = np.random.default_rng(80)
    T, E, k = 57, 6, 2
    logits = rng.standard_normal((T, E)) * 2
    idx = np.argsort(-logits, axis=1, kind="stable")[:, :k]
    t, S = O.load_balance_stats(logits, idx, E)
    assert t.sum() == T * k and math.isclose(S.sum(), T, rel_tol=1e-12)     # probabilities sum to 1 per token
    # brute force
    for i in range(E):
        assert t[i] == sum(1 for tt in range(T) for j in range(k) if idx[tt, j] == i)
        ref = sum(math.exp(logits[tt, i]) / sum(math.exp(v) for v in logits[tt]) for tt in range(T))
        assert math.isclose(S[i], ref, rel_tol=1e-12)
    assert np.allclose(S, torch.softmax(torch.from_numpy(logits), dim=1).sum(0).numpy(), rtol=1e-12)
    # uniform router, top-1, perfectly balanced batch: t_i = T/E and sum_x P_i = T/E, so Eq. 12 gives T
    T = 24
    t, S = O.load_balance_stats(np.zeros((T, E)), (np.arange(T) % E)[:, None], E)
    assert np.all(t == T // E) and np.allclose(S, T / E)
    assert math.isclose(O.balance_loss(t, S, T), T, rel_tol=1e-12)
    # everything routed to one expert that also holds all the probability: E times larger
    lg = np.full((T, E), -1e3); lg[:, 2] = 0.0
    t, S = O.load_balance_stats(lg, np.full((T, 1), 2), E)
    assert math.isclose(O.balance_loss(t, S, T), E * T, rel_tol=1e-12)
