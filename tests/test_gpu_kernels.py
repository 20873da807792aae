"""GPU parity of the three stand-alone entry points against the CPU oracle (bit-exact integer
stages, gate weights within 1e-6)."""
import numpy as np
import pytest
import torch

from oracle import mote_oracle as O
from workloads import synth
from parity_utils import bf16_bits, bf16_tensor

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mote():
    import paper_2506_14435_b200 as m
    return m


def _randn(shape, seed, scale=1.0):
    return (torch.randn(shape, generator=torch.Generator().manual_seed(seed)) * scale).numpy()


@pytest.mark.parametrize("m,n,scale", [(1, 16, 0.02), (7, 48, 0.02), (256, 512, 0.02), (300, 1008, 1.0),
                                       (4864, 896, 0.02), (129, 11008, 0.02), (64, 64, 1e-30), (64, 64, 1e30)])
def test_ternarize_pack_fp32(mote, m, n, scale):
    W = _randn((m, n), 100 + m + n, scale).astype(np.float32)
    codes, alpha = O.ternarize(W)
    packed, a = mote.mote_ternarize_pack(torch.from_numpy(W).cuda())
    assert a.item() == alpha
    assert np.array_equal(packed.cpu().numpy(), O.pack_codes(codes))


def test_ternarize_pack_special_values(mote):
    W = np.zeros((8, 32), np.float32)
    packed, a = mote.mote_ternarize_pack(torch.from_numpy(W).cuda())
    assert a.item() == np.float32(1e-5) and np.all(packed.cpu().numpy() == 0x55)
    # exact ties at +-0.5 and +-1.5 of alpha, subnormals, wide exponent spread
    W = np.tile(np.array([0.5, -0.5, 1.5, -1.5, 1.0, -1.0, 1.0, 1.0], np.float32), (4, 4))
    codes, alpha = O.ternarize(W)
    packed, a = mote.mote_ternarize_pack(torch.from_numpy(W).cuda())
    assert a.item() == alpha == 1.0 and np.array_equal(packed.cpu().numpy(), O.pack_codes(codes))
    rng = np.random.default_rng(3)
    W = (rng.standard_normal((64, 256)) * np.exp2(rng.integers(-140, 60, size=(64, 256)))).astype(np.float32)
    codes, alpha = O.ternarize(W)
    packed, a = mote.mote_ternarize_pack(torch.from_numpy(W).cuda())
    assert a.item() == alpha and np.array_equal(packed.cpu().numpy(), O.pack_codes(codes))


def test_ternarize_pack_bf16_input(mote):
    Wb = O.f32_to_bf16_rn(_randn((96, 320), 5, 0.02).astype(np.float32))
    codes, alpha = O.ternarize(O.bf16_to_f32(Wb))
    packed, a = mote.mote_ternarize_pack(bf16_tensor(Wb))
    assert a.item() == alpha and np.array_equal(packed.cpu().numpy(), O.pack_codes(codes))


@pytest.mark.parametrize("T,d", [(1, 16), (5, 48), (64, 256), (300, 896), (33, 1536), (17, 2048), (9, 4864),
                                 (6, 8960), (5, 11008), (3, 32768)])
def test_quant_act(mote, T, d):
    x = O.f32_to_bf16_rn(_randn((T, d), 7 * T + d, 3.0).astype(np.float32))
    if T > 2:
        x[1] = 0
        x[2, : d // 2] = 0
    q, beta, rowsum = O.quant_act(x)
    gq, gb, gs = mote.mote_quant_act(bf16_tensor(x))
    assert np.array_equal(gq.cpu().numpy(), q)
    assert np.array_equal(gb.cpu().numpy(), beta)
    assert np.array_equal(gs.cpu().numpy(), rowsum)


def test_quant_act_strided_rows_and_outliers(mote):
    wl = synth.WORKLOADS["c2"]
    x = synth.tokens(wl, T=200)
    wide = np.zeros((200, wl.d + 64), np.uint16)
    wide[:, : wl.d] = x
    xt = bf16_tensor(wide)[:, : wl.d]
    q, beta, rowsum = O.quant_act(x)
    gq, gb, gs = mote.mote_quant_act(xt)
    assert np.array_equal(gq.cpu().numpy(), q) and np.array_equal(gb.cpu().numpy(), beta)
    assert np.array_equal(gs.cpu().numpy(), rowsum)
    assert gq.abs().max().item() == 127


@pytest.mark.parametrize("name,T,k,norm", [("c1", 64, 2, 1), ("c1", 64, 1, 0), ("c1", 64, 4, 0), ("c3", 64, 2, 1),
                                           ("c3", 1, 2, 1), ("c4", 1000, 2, 1), ("c4", 257, 8, 0)])
def test_route_topk(mote, name, T, k, norm):
    wl = synth.WORKLOADS[name]
    x = synth.tokens(wl, T=T)
    Wr, bias = synth.router_weights(wl, 0)
    ref = O.router(x, Wr, bias, k, norm)
    idx, w, logits = mote.mote_route_topk(bf16_tensor(x), torch.from_numpy(Wr).cuda(),
                                          None if bias is None else torch.from_numpy(bias).cuda(), k, norm,
                                          want_logits=True)
    idx, w, logits = idx.cpu().numpy(), w.cpu().numpy(), logits.cpu().numpy()
    assert np.max(np.abs(logits - ref["logits"])) < 2e-5
    ok = ~ref["near_tie"]
    assert np.array_equal(idx[ok], ref["idx"][ok])
    assert np.max(np.abs(w[ok].astype(np.float64) - ref["w"][ok])) <= 1e-6
    if norm:
        assert np.allclose(w.sum(axis=1), 1.0, atol=1e-6)


def test_route_topk_many_experts_and_ties(mote):
    rng = np.random.default_rng(11)
    T, d, E = 50, 64, 64
    x = O.f32_to_bf16_rn(rng.standard_normal((T, d)).astype(np.float32))
    Wr = O.bf16_to_f32(O.f32_to_bf16_rn((rng.standard_normal((E, d)) * 0.1).astype(np.float32)))
    Wr[40] = Wr[3]                                   # an exact tie: the lower index must win
    ref = O.router(x, Wr, None, 8, 1)
    idx, w, _ = mote.mote_route_topk(bf16_tensor(x), torch.from_numpy(Wr).cuda(), None, 8, 1)
    idx = idx.cpu().numpy()
    for t in range(T):
        if 3 in idx[t] and 40 in idx[t]:
            assert list(idx[t]).index(3) < list(idx[t]).index(40)
    ok = ~ref["near_tie"]
    assert np.array_equal(idx[ok], ref["idx"][ok])


def test_quant_act_every_bf16_value_under_many_scales(mote):
    """The kernels evaluate 127*x/beta as x * fl(127 * fl(1/beta)) and divide only near a rounding
    tie; this must give the oracle's integer for EVERY bf16 x with |x| <= beta.  Each row holds beta
    and all non-negative (or all non-positive) bf16 values below it."""
    rng = np.random.default_rng(77)
    betas = [0x3F80, 0x4040, 0x42FE, 0x3F81, 0x3FFF, 0x3400, 0x4B00, 0x0080, 0x1234, 0x7000]   # bf16 bit patterns
    betas += [int(b) for b in rng.integers(0x2000, 0x6000, size=50)]
    rows = []
    for b in betas:
        vals = np.arange(0, b + 1, dtype=np.uint32)            # all magnitudes up to beta (bit patterns are ordered)
        if len(vals) > 32768:
            vals = np.concatenate([vals[-16384:], rng.choice(vals[:-16384], 16384, replace=False)])
        for sign in (0, 0x8000):
            row = np.zeros(32768, np.uint16)
            row[: len(vals)] = (vals | sign).astype(np.uint16)
            row[len(vals) - 1 if len(vals) <= 32768 else 0] = b   # beta itself, positive
            rows.append(row)
    x = np.stack(rows)
    q, beta, rowsum = O.quant_act(x)
    gq, gb, gs = mote.mote_quant_act(bf16_tensor(x))
    assert np.array_equal(gb.cpu().numpy(), beta)
    assert np.array_equal(gq.cpu().numpy(), q)
    assert np.array_equal(gs.cpu().numpy(), rowsum)


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("m,n,scale,dtype", [(1, 16, 0.02, "bf16"), (7, 48, 0.02, "f32"), (300, 1008, 1.0, "bf16"),
                                             (129, 11008, 0.02, "bf16"), (64, 896, 0.02, "f32"),
                                             (33, 65536, 0.02, "bf16"), (16, 64, 1e-30, "f32")])
def test_rtn_quant(mote, m, n, scale, dtype, bits):
    W = _randn((m, n), 900 + m + n + bits, scale).astype(np.float32)
    if m > 4:
        W[3] = 0.0                                  # an all-zero row
    if dtype == "bf16":
        Wb = O.f32_to_bf16_rn(W)
        q_ref, s_ref = O.rtn_quantize(O.bf16_to_f32(Wb), bits)
        q, sc = mote.mote_rtn_quant(bf16_tensor(Wb), bits)
    else:
        q_ref, s_ref = O.rtn_quantize(W, bits)
        q, sc = mote.mote_rtn_quant(torch.from_numpy(W).cuda(), bits)
    want = q_ref if bits == 8 else O.pack_int4(q_ref)
    assert np.array_equal(q.cpu().numpy(), want)
    assert np.array_equal(sc.cpu().numpy(), s_ref)


@pytest.mark.parametrize("bits", [8, 4])
def test_rtn_quant_ties_and_errors(mote, bits):
    # exact half-integer quotients: rows of k + 1/2 multiples of beta/qmax
    qmax = 2 ** (bits - 1) - 1
    base = np.arange(-qmax, qmax + 1, dtype=np.float32)
    row = np.concatenate([base, base[:-1] + 0.5])
    row = np.resize(row, 64).astype(np.float32)
    row[0] = qmax
    W = np.tile(row, (5, 1)) * np.float32(0.125)
    q_ref, s_ref = O.rtn_quantize(W, bits)
    q, sc = mote.mote_rtn_quant(torch.from_numpy(W).cuda(), bits)
    assert np.array_equal(q.cpu().numpy(), q_ref if bits == 8 else O.pack_int4(q_ref))
    assert np.array_equal(sc.cpu().numpy(), s_ref)
    with pytest.raises(mote.MoteError) as ei:
        mote.mote_rtn_quant(torch.zeros((4, 24), device="cuda"), bits)       # n % 16 != 0
    assert ei.value.status == 2
    with pytest.raises(mote.MoteError) as ei:
        mote.mote_rtn_quant(torch.zeros((4, 32), device="cuda"), 3)
    assert ei.value.status == 2


@pytest.mark.parametrize("T,d,E,k,bias", [(1, 64, 4, 1, False), (300, 256, 8, 2, True), (4096, 896, 4, 2, False),
                                          (777, 128, 64, 8, True)])
def test_route_stats(mote, T, d, E, k, bias):
    # Eq. 12: tokens per expert exactly, summed routing probabilities to fp32 accuracy
    x = O.f32_to_bf16_rn(_randn((T, d), 60 + T, 1.0).astype(np.float32))
    Wr = O.bf16_to_f32(O.f32_to_bf16_rn(_randn((E, d), 61 + T, 0.05).astype(np.float32)))
    b = _randn((E,), 62 + T, 0.5).astype(np.float32) if bias else None
    idx, w, logits = mote.mote_route_topk(bf16_tensor(x), torch.from_numpy(Wr).cuda(),
                                          None if b is None else torch.from_numpy(b).cuda(), k, want_logits=True)
    cnt, ps = mote.mote_route_stats(logits, idx)
    t_ref, s_ref = O.load_balance_stats(logits.cpu().numpy(), idx.cpu().numpy(), E)
    assert np.array_equal(cnt.cpu().numpy(), t_ref)
    assert np.allclose(ps.cpu().numpy(), s_ref, rtol=2e-5, atol=1e-6)
    assert cnt.sum().item() == T * k and abs(ps.sum().item() - T) <= 1e-4 * T
    # against the oracle's own router (fp64 logits): same counts away from near ties
    r = O.router(x, Wr, b, k, 1)
    if not r["near_tie"].any():
        t2, s2 = O.load_balance_stats(r["logits"], r["idx"], E)
        assert np.array_equal(cnt.cpu().numpy(), t2)
        assert np.allclose(ps.cpu().numpy(), s2, rtol=1e-4, atol=1e-5)


def test_bounded_wait_runs_out_and_is_reported_once(mote):
    # The GEMM kernels bound every device-side wait; here the wait itself is exercised in the only
    # safe form: one thread block waits on a barrier nothing arrives at, gives up after 1 ms,
    # takes the GEMM's teardown and returns.  Nothing faults; the context keeps working.
    import time
    lib = mote.lib
    ws = torch.empty(4096, dtype=torch.uint8, device="cuda")
    ws.zero_()
    assert lib.mote_device_status(ws.data_ptr(), None) == 0
    t0 = time.perf_counter()
    assert lib.mote_selftest_bounded_wait(ws.data_ptr(), 1_000_000, None) == 0
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 1.0               # ~1 ms wait + 0.2 ms drain, not the 2 s default
    assert lib.mote_device_status(ws.data_ptr(), None) == 7     # MOTE_ERR_DEVICE_TIMEOUT
    assert lib.mote_device_status(ws.data_ptr(), None) == 0     # reading clears it
    # the context is intact: an ordinary kernel runs and gives the right answer afterwards
    x = torch.arange(64 * 256, device="cuda", dtype=torch.float32).reshape(64, 256).to(torch.bfloat16)
    q, beta, _ = mote.mote_quant_act(x)
    torch.cuda.synchronize()
    want_q, want_beta, _ = O.quant_act(x.cpu().view(torch.int16).numpy().view(np.uint16))
    assert np.array_equal(q.cpu().numpy(), want_q) and np.array_equal(beta.cpu().numpy(), want_beta)
    # argument checks happen on the host
    assert lib.mote_selftest_bounded_wait(None, 1_000_000, None) == 1
    assert lib.mote_selftest_bounded_wait(ws.data_ptr(), 10, None) == 2
    assert lib.mote_selftest_bounded_wait(ws.data_ptr(), 10**10, None) == 2


def test_status_word_survives_the_layers_of_a_stack_and_is_cleared_by_the_next_call(mote):
    # a stack clears the status word once at its start and not between its layers; a fresh top-level
    # call clears what an earlier one left
    wl = synth.custom("st", 128, 256, 4, 2, 8, 4300, n_layers=2, w_std=0.08)
    layers = [mote.MoteLayer.from_master(synth.master_layer(wl, layer=l)) for l in range(2)]
    stack = mote.MoteStack(layers)
    x = torch.from_numpy(synth.tokens(wl).view(np.int16).copy()).view(torch.bfloat16).cuda()
    mote.mote_stack_forward(stack, x)
    ws = stack._ws
    assert mote.lib.mote_device_status(ws.data_ptr(), None) == 0
    assert mote.lib.mote_selftest_bounded_wait(ws.data_ptr(), 1_000_000, None) == 0
    # a single layer call inside a stack must not clear: emulate by checking the stack's own clear
    mote.mote_stack_forward(stack, x)
    assert mote.lib.mote_device_status(ws.data_ptr(), None) == 0    # cleared at the start of the stack
    assert mote.lib.mote_selftest_bounded_wait(ws.data_ptr(), 1_000_000, None) == 0
    assert mote.lib.mote_device_status(ws.data_ptr(), None) == 7


def test_int8_mma_peak_kernel_runs_and_its_time_follows_the_work(mote):
    from paper_2506_14435_b200.binding import mote_int8_mma_peak
    a = mote_int8_mma_peak(400)
    b = mote_int8_mma_peak(800)
    # twice the MMAs take about twice as long (the kernel really issues them), and the rate is that
    # of a tensor pipe (far above what CUDA cores can do: 148 SMs x 128 lanes x 2 GHz x 8 = 0.3 POP/s)
    assert 1.7 < b["ms"][0] / a["ms"][0] < 2.3
    assert 1000.0 < b["tops_best"] < 6000.0
