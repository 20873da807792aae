"""The helpers the GPU parity tests lean on must themselves reject what they are there to reject
(checked here on the CPU, on hand-made cases)."""
import numpy as np
import pytest

from oracle import mote_oracle as O
from workloads import synth
from parity_utils import assert_elementwise_close, assert_valid_near_tie_pick, shared_rounding_sigma


def test_near_tie_validity_accepts_either_side_of_the_tie_only():
    logits = [5.0, 3.0, 3.0 - 5e-6, 0.0]                # experts 1 and 2 within 1e-5 of each other
    assert_valid_near_tie_pick([0, 1], logits, 2)
    assert_valid_near_tie_pick([0, 2], logits, 2)
    # drops the clear winner; repeats an expert; takes a clear loser; wrong order
    for bad in ([1, 2], [1, 1], [0, 0], [0, 3], [1, 0], [2, 0]):
        with pytest.raises(AssertionError):
            assert_valid_near_tie_pick(bad, logits, 2)
    # a three-way tie for the last two of three slots
    logits = [1.0, 1.0 + 2e-6, 7.0, 1.0 - 3e-6, -2.0]
    for ok in ([2, 1, 0], [2, 0, 3], [2, 3, 1]):
        assert_valid_near_tie_pick(ok, logits, 3)
    with pytest.raises(AssertionError):
        assert_valid_near_tie_pick([2, 1, 4], logits, 3)


def test_elementwise_bound_catches_one_wrong_element_that_the_norm_would_miss():
    # a tiny shared expert: the GPU's only liberty is the bf16 rounding of h, emulated here
    wl = synth.custom("helper", 32, 64, 2, 1, 40, 77, w_std=0.3)
    layer = O.build_layer(synth.master_layer(wl))
    x = synth.tokens(wl)
    ref = O.shared_ffn(x, layer["sh_gate"], layer["sh_up"], layer["sh_down"])
    sigma = shared_rounding_sigma(layer, x)
    xf = O.bf16_to_f32(x).astype(np.float64)
    Wg, Wu, Wd = (O.bf16_to_f32(layer["sh_" + n]).astype(np.float64) for n in ("gate", "up", "down"))
    g = xf @ Wg.T
    h = (xf @ Wu.T) * (g / (1.0 + np.exp(-g)))
    h_bf16 = O.bf16_to_f32(O.f32_to_bf16_rn(h.astype(np.float32))).astype(np.float64)
    got = h_bf16 @ Wd.T
    assert np.abs(got - ref).max() > 0                                    # the rounding is visible ...
    assert_elementwise_close(got, ref, sigma, "bf16 h")                   # ... and inside the bound
    assert np.abs(got - ref).max() < 6 * sigma.max()
    got[17, 10] += 20 * sigma[17, 10] + 0.02 * abs(ref[17, 10])           # one element off
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) < 5e-3         # the Frobenius test passes it
    with pytest.raises(AssertionError):
        assert_elementwise_close(got, ref, sigma, "planted")
