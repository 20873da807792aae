"""The stand-alone streaming kernels on inputs larger than the 126 MB L2 (what their HBM figures in
profiles/ are captured on): the same bit-exact comparisons with the oracle as at small sizes, at a
size where the grid-stride loops wrap many times and every byte comes from DRAM."""
import numpy as np
import pytest
import torch

from oracle import mote_oracle as O
from parity_utils import bf16_bits, bf16_tensor

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mote():
    import paper_2506_14435_b200 as m
    return m


def _gauss(shape, seed, scale):
    return (torch.randn(shape, generator=torch.Generator().manual_seed(seed)) * scale).numpy()


def test_ternarize_pack_larger_than_l2(mote):
    W = _gauss((6144, 8192), 11, 0.02).astype(np.float32)          # 201 MB of fp32
    codes, alpha = O.ternarize(W)
    packed, a = mote.mote_ternarize_pack(torch.from_numpy(W).cuda())
    assert a.item() == alpha
    assert np.array_equal(packed.cpu().numpy(), O.pack_codes(codes))


@pytest.mark.parametrize("bits", [8, 4])
def test_rtn_quant_larger_than_l2(mote, bits):
    Wb = O.f32_to_bf16_rn(_gauss((8192, 10240), 12 + bits, 0.02).astype(np.float32))     # 168 MB of bf16
    q_ref, s_ref = O.rtn_quantize(O.bf16_to_f32(Wb), bits)
    q, sc = mote.mote_rtn_quant(bf16_tensor(Wb), bits)
    assert np.array_equal(q.cpu().numpy(), q_ref if bits == 8 else O.pack_int4(q_ref))
    assert np.array_equal(sc.cpu().numpy(), s_ref)


def test_quant_act_and_rms_norm_larger_than_l2(mote):
    T, d = 40960, 2048                                                                  # 168 MB of bf16
    x_bits = O.f32_to_bf16_rn(_gauss((T, d), 13, 3.0).astype(np.float32))
    x = bf16_tensor(x_bits)
    q, beta, rowsum = mote.mote_quant_act(x)
    q_ref, beta_ref, rs_ref = O.quant_act(x_bits)
    assert np.array_equal(q.cpu().numpy(), q_ref)
    assert np.array_equal(beta.cpu().numpy(), beta_ref) and np.array_equal(rowsum.cpu().numpy(), rs_ref)
    del q, q_ref
    y = O.bf16_to_f32(bf16_bits(mote.mote_rms_norm(x, 1e-6))).astype(np.float64)
    rows = np.arange(0, T, 97)                                     # the fp64 reference on a stride of rows
    want = O.rms_norm(x_bits[rows], 1e-6)
    assert np.all(np.abs(y[rows] - want) <= np.abs(want) * 2.0 ** -8 + 1e-30)


def test_route_topk_larger_than_l2(mote):
    T, d, E, k = 40960, 2048, 16, 2
    x_bits = O.f32_to_bf16_rn(_gauss((T, d), 14, 1.0).astype(np.float32))
    Wr = O.bf16_to_f32(O.f32_to_bf16_rn(_gauss((E, d), 15, 0.02).astype(np.float32)))
    bias = _gauss((E,), 16, 0.5).astype(np.float32)
    ref = O.router(x_bits, Wr, bias, k, 1)
    idx, w, logits = mote.mote_route_topk(bf16_tensor(x_bits), torch.from_numpy(Wr).cuda(), torch.from_numpy(bias).cuda(),
                                          k, 1, want_logits=True)
    assert np.max(np.abs(logits.cpu().numpy().astype(np.float64) - ref["logits"])) < 2e-5
    ok = ~ref["near_tie"]
    assert np.array_equal(idx.cpu().numpy()[ok], ref["idx"][ok]) and ok.mean() > 0.99
    assert np.max(np.abs(w.cpu().numpy().astype(np.float64)[ok] - ref["w"][ok])) <= 1e-6
