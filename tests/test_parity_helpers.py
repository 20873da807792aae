"""The helpers the GPU parity tests lean on must themselves reject what they are there to reject
(checked here on the CPU, on hand-made cases)."""
import numpy as np
import pytest

from parity_utils import assert_elementwise_close, assert_valid_near_tie_pick


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
    rng = np.random.default_rng(3)
    ref = rng.standard_normal((64, 256))
    got = ref * (1.0 + 2.0 ** -10 * rng.uniform(-1, 1, ref.shape))       # bf16-rounding-sized noise
    assert_elementwise_close(got, ref, "noise")
    got[17, 100] += 0.25                                                  # one element off by a quarter
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) < 5e-3         # the Frobenius test passes it
    with pytest.raises(AssertionError):
        assert_elementwise_close(got, ref, "planted")
