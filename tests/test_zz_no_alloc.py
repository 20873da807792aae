"""mote_ternarize_pack_static, the entry point for callers that cannot allocate device memory
(a fully committed memory pool, a plug-in inside a host that owns all allocations, a loop that
cannot take an allocation's device-wide synchronisation).  It keeps its scratch in a device array
built into the library instead of taking a workspace, and must give the very bytes that
mote_ternarize_pack gives.  The scratch survives between calls, so the check is made on two calls
in a row with different matrices: stale sums left by the first would change the second's alpha.

This file sorts last on purpose: a run that stops at the first failure has then already run every
other test."""
import numpy as np
import pytest
import torch

from oracle import mote_oracle as O


@pytest.fixture(scope="module")
def mote():
    import paper_2506_14435_b200 as m
    return m


def _w(shape, seed, scale, dtype=torch.float32):
    return (torch.randn(shape, generator=torch.Generator().manual_seed(seed)) * scale).to(dtype).cuda()


@pytest.mark.gpu
def test_static_scratch_matches_workspace_entry_point_twice_in_a_row(mote):
    cases = [_w((512, 1024), 41, 0.02), _w((96, 320), 42, 3.0), _w((256, 512), 43, 0.02, torch.bfloat16)]
    for i, W in enumerate(cases):
        m, n = W.shape
        want_packed, want_alpha = mote.mote_ternarize_pack(W)
        packed = torch.full((m, n // 4), 0xFF, dtype=torch.uint8, device="cuda")
        alpha = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated()
        free_before = torch.cuda.mem_get_info()[0]
        mote.mote_ternarize_pack_static(W, packed, alpha)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        # the driver's view too, which would also see an allocation made inside the library (from the
        # second call on: the first use of a library on a device may load its code there)
        if i > 0:
            assert torch.cuda.mem_get_info()[0] >= free_before
        # integer and byte work: bit-exact, as everywhere else in the suite
        assert alpha.item() == want_alpha.item()
        assert torch.equal(packed, want_packed)
        # and against the oracle directly (Eq. 7, 9), not only through the other entry point
        codes, a = O.ternarize(W.float().cpu().numpy())
        assert alpha.item() == float(a)
        assert np.array_equal(packed.cpu().numpy(), O.pack_codes(codes))


def test_static_scratch_rejects_oversize_and_bad_arguments(mote):
    import ctypes as C
    lib = mote.lib
    fake, odd = C.c_void_p(0x1000), C.c_void_p(0x1004)
    assert lib.mote_ternarize_pack_static(fake, 0, 1 << 16, (1 << 15) + 16, fake, fake, None) == 8   # > 2^31 elements
    assert lib.mote_ternarize_pack_static(None, 0, 4, 16, fake, fake, None) == 1
    assert lib.mote_ternarize_pack_static(fake, 0, 4, 12, fake, fake, None) == 2
    assert lib.mote_ternarize_pack_static(odd, 0, 4, 16, fake, fake, None) == 3
    assert lib.mote_ternarize_pack_static(fake, 9, 4, 16, fake, fake, None) == 5
