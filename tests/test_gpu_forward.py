"""GPU parity of the whole layer (mote_moe_forward through the C ABI) against the CPU oracle:
every integer stage bit-exact, the bf16 output within 5e-3 relative Frobenius error."""
import numpy as np
import pytest
import torch

from oracle import mote_oracle as O
from workloads import synth
from parity_utils import bf16_bits, bf16_tensor, check_forward, check_packed_layer, check_shared_codes

pytestmark = pytest.mark.gpu

SIMT, TENSOR, STREAM = 1, 2, 3
BOTH = [pytest.param(SIMT, id="simt"), pytest.param(TENSOR, id="tensor")]
ALL = BOTH + [pytest.param(STREAM, id="stream")]


@pytest.fixture(scope="module")
def mote():
    import paper_2506_14435_b200 as m
    return m


def _setup(mote, wl, path=1):
    master = synth.master_layer(wl)
    layer_or = O.build_layer(master)
    layer_gpu = mote.MoteLayer.from_master(master, path=path)
    return master, layer_or, layer_gpu


@pytest.mark.parametrize("path", ALL)
def test_c1_full_parity(mote, path):
    wl = synth.WORKLOADS["c1"]
    master, layer_or, layer_gpu = _setup(mote, wl, path)
    check_packed_layer(layer_gpu, layer_or)
    rep = check_forward(mote, layer_gpu, layer_or, synth.tokens(wl))
    assert rep["rel_fro"] < 5e-3


@pytest.mark.parametrize("d,f,E,k,T,kw,path", [
    (16, 32, 3, 2, 5, {}, SIMT),
    (48, 80, 2, 1, 1, {}, SIMT),
    (64, 112, 5, 5, 33, {}, SIMT),                       # k = E
    (256, 512, 4, 2, 300, dict(outlier_frac=0.02), SIMT),
    (128, 256, 8, 2, 77, dict(bias="zipf"), SIMT),
    (128, 384, 4, 1, 130, dict(norm_topk=0), SIMT),
    (128, 128, 2, 1, 1, {}, TENSOR),                      # one row, one k-step
    (256, 512, 4, 2, 300, dict(outlier_frac=0.02), TENSOR),   # ragged tails in every expert
    (128, 256, 8, 2, 77, dict(bias="zipf"), TENSOR),
    (128, 384, 4, 1, 130, dict(norm_topk=0), TENSOR),     # down projection with 128-wide tiles
    (384, 640, 3, 3, 515, {}, TENSOR),                    # k = E, several row tiles per expert
    (128, 256, 64, 8, 200, {}, TENSOR),                   # many experts, k = 8: 128 pairs per router block
    (256, 128, 16, 4, 1000, dict(bias="normal"), TENSOR), # more row tiles than experts, uneven loads
    (128, 256, 64, 8, 70, {}, SIMT),
    (64, 128, 3, 3, 5, {}, STREAM),                       # k = E, one short reduction step
    (128, 192, 2, 1, 1, {}, STREAM),                      # one token
    (896, 4864, 4, 2, 17, dict(outlier_frac=0.01), STREAM),   # d/4 = 224 bytes: a ragged last step
    (256, 512, 4, 2, 64, dict(bias="zipf"), STREAM),      # the largest batch, uneven expert loads
    (192, 320, 8, 1, 33, dict(norm_topk=0), STREAM),
    (128, 256, 64, 8, 37, {}, STREAM),                    # many experts, k = 8
    # a handful of pairs
    (256, 512, 4, 2, 2, {}, STREAM),                      # two tokens, top-2
    (128, 256, 2, 1, 3, dict(norm_topk=0), STREAM),       # three pairs on two experts
    (128, 320, 8, 4, 1, {}, STREAM),                      # one token, k = 4
    (896, 4864, 4, 2, 2, dict(outlier_frac=0.01), STREAM),
    (192, 320, 1, 1, 4, {}, STREAM),                      # one expert takes all four rows
    (512, 1024, 8, 2, 13, dict(bias="zipf"), STREAM),    # 9..16 tokens: the two-column-tile kernels
])
def test_small_shapes(mote, d, f, E, k, T, kw, path):
    wl = synth.custom("small", d, f, E, k, T, 2000 + d + f + T, **kw)
    master, layer_or, layer_gpu = _setup(mote, wl, path)
    check_packed_layer(layer_gpu, layer_or)
    check_forward(mote, layer_gpu, layer_or, synth.tokens(wl))


@pytest.mark.parametrize("path", BOTH)
def test_idle_and_overloaded_experts_residual_and_aliasing(mote, path):
    wl = synth.custom("skew", 128, 256, 4, 2, 97, 3001)
    master = synth.master_layer(wl)
    master["router_bias"] = np.array([50.0, -50.0, 40.0, -60.0], np.float32)   # experts 1 and 3 idle
    layer_or = O.build_layer(master)
    layer_gpu = mote.MoteLayer.from_master(master, path=path)
    x = synth.tokens(wl)
    res = synth.tokens(wl, stream=1)
    rep = check_forward(mote, layer_gpu, layer_or, x, residual_bits=res)
    assert rep["counts"].tolist() == [97, 0, 97, 0]
    rep2 = check_forward(mote, layer_gpu, layer_or, x, residual_bits=res, out_alias_residual=True)
    assert torch.equal(rep["out"], rep2["out"])


@pytest.mark.parametrize("path", BOTH)
def test_run_to_run_determinism_and_token_permutation(mote, path):
    wl = synth.custom("det", 256, 512, 4, 2, 200, 3002)
    master, layer_or, layer_gpu = _setup(mote, wl, path)
    x = bf16_tensor(synth.tokens(wl))
    a = mote.mote_moe_forward(layer_gpu, x).clone()
    b = mote.mote_moe_forward(layer_gpu, x).clone()
    assert torch.equal(a, b)
    pm = torch.randperm(wl.T, generator=torch.Generator().manual_seed(1)).cuda()
    c = mote.mote_moe_forward(layer_gpu, x[pm].contiguous())
    assert torch.equal(c, a[pm])


def test_stream_path_idle_experts_residual_determinism(mote):
    wl = synth.custom("skew", 128, 256, 4, 2, 40, 3003)
    master = synth.master_layer(wl)
    master["router_bias"] = np.array([50.0, -50.0, 40.0, -60.0], np.float32)   # experts 1 and 3 idle
    layer_or = O.build_layer(master)
    layer_gpu = mote.MoteLayer.from_master(master, path=STREAM)
    x = synth.tokens(wl)
    res = synth.tokens(wl, stream=1)
    rep = check_forward(mote, layer_gpu, layer_or, x, residual_bits=res)
    assert rep["counts"].tolist() == [40, 0, 40, 0]
    rep2 = check_forward(mote, layer_gpu, layer_or, x, residual_bits=res, out_alias_residual=True)
    assert torch.equal(rep["out"], rep2["out"])
    xt = bf16_tensor(x)
    pm = torch.randperm(wl.T, generator=torch.Generator().manual_seed(2)).cuda()
    a = mote.mote_moe_forward(layer_gpu, xt).clone()
    c = mote.mote_moe_forward(layer_gpu, xt[pm].contiguous())
    assert torch.equal(c, a[pm])


def test_stream_path_rejects_large_batches(mote):
    wl = synth.custom("big", 128, 256, 4, 2, 65, 3004)
    master = synth.master_layer(wl)
    layer_gpu = mote.MoteLayer.from_master(master, path=STREAM)
    with pytest.raises(mote.MoteError) as ei:
        mote.mote_moe_forward(layer_gpu, bf16_tensor(synth.tokens(wl)))
    assert ei.value.status == 2


def test_zero_tokens_is_a_noop(mote):
    wl = synth.WORKLOADS["c1"]
    master, layer_or, layer_gpu = _setup(mote, wl)
    x = torch.empty((0, wl.d), dtype=torch.bfloat16, device="cuda")
    out = mote.mote_moe_forward(layer_gpu, x)
    assert out.shape == (0, wl.d)


@pytest.mark.parametrize("path", ALL)
@pytest.mark.parametrize("T", synth.C3_BATCHES)
def test_c3_decode_batches(mote, T, path, c3_layers):
    wl, layer_or, layer_gpu = c3_layers
    layer_gpu.path = path
    rep = check_forward(mote, layer_gpu, layer_or, synth.tokens(wl, T=T))
    assert rep["rel_fro"] < 5e-3


@pytest.fixture(scope="module")
def c3_layers(mote):
    wl = synth.WORKLOADS["c3"]
    master, layer_or, layer_gpu = _setup(mote, wl)
    check_packed_layer(layer_gpu, layer_or)
    return wl, layer_or, layer_gpu


def test_host_buffer_entry_point(mote):
    from paper_2506_14435_b200.binding import mote_moe_forward_host
    wl = synth.WORKLOADS["c1"]
    master, layer_or, layer_gpu = _setup(mote, wl)
    xb = synth.tokens(wl)
    x_host = torch.from_numpy(xb.view(np.int16).copy()).view(torch.bfloat16).pin_memory()
    out_host = torch.empty_like(x_host).pin_memory()
    mote_moe_forward_host(layer_gpu, x_host, out_host)
    want = mote.mote_moe_forward(layer_gpu, x_host.cuda())
    assert torch.equal(out_host, want.cpu())


@pytest.mark.parametrize("T,with_residual", [(4096, False), (4133, True), (9000, True)])
def test_host_buffer_entry_point_long_prefill(mote, T, with_residual):
    """From 4096 tokens on the host call runs the layer as two halves with the copies of one half
    beside the layer of the other: the result must equal the one-piece device call bit for bit
    (tokens are independent, Eq. 2-4), for an even and for a ragged split.  (The device call is
    what the other tests compare with the oracle.)"""
    from paper_2506_14435_b200.binding import mote_moe_forward_host
    wl = synth.Workload("host_pipe", 128, 256, 8, 2, T, seed=77, bias="zipf")
    master, layer_or, layer_gpu = _setup(mote, wl)
    pin = lambda bits: torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).pin_memory()
    x_host = pin(synth.tokens(wl))
    res_host = pin(synth.tokens(wl, stream=1)) if with_residual else None
    out_host = torch.empty_like(x_host).pin_memory()
    for _ in range(2):                                   # the second call reuses the copy streams
        out_host.zero_()
        mote_moe_forward_host(layer_gpu, x_host, out_host, res_host)
        want = mote.mote_moe_forward(layer_gpu, x_host.cuda(), residual=None if res_host is None else res_host.cuda())
        assert torch.equal(out_host, want.cpu())


# ------------------------------------------------------------------ Section 4.3: RTN-coded shared expert
@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("d,f,E,k,T,kw,path", [
    (16, 32, 3, 2, 5, {}, SIMT),
    (64, 112, 5, 5, 33, {}, SIMT),
    (128, 128, 2, 1, 1, {}, TENSOR),                      # one row, two k-steps
    (256, 512, 4, 2, 300, dict(outlier_frac=0.02), TENSOR),
    (128, 384, 4, 1, 130, dict(norm_topk=0), TENSOR),     # down projection with 128-wide tiles
    (384, 640, 3, 3, 515, {}, TENSOR),                    # several row tiles, 160-wide down tiles (128 + 32 rows)
    (896, 4864, 4, 2, 160, dict(outlier_frac=0.01), TENSOR),  # 224-wide down tiles
    (256, 512, 4, 2, 900, {}, TENSOR),                    # long enough for the codes to be expanded once per call
    (64, 128, 3, 3, 5, {}, STREAM),                       # one short reduction step (32 bytes of 4-bit codes)
    (128, 192, 2, 1, 1, {}, STREAM),
    (896, 4864, 4, 2, 17, dict(outlier_frac=0.01), STREAM),
    (256, 512, 4, 2, 64, dict(bias="zipf"), STREAM),
])
def test_rtn_shared_expert(mote, d, f, E, k, T, kw, path, bits):
    wl = synth.custom("rtn", d, f, E, k, T, 4000 + d + f + T, **kw)
    master, layer_or, layer_gpu = _setup(mote, wl, path)
    layer_or = O.quantize_shared(layer_or, bits)
    layer_gpu = layer_gpu.quantize_shared(bits)
    check_shared_codes(layer_gpu, layer_or)
    check_forward(mote, layer_gpu, layer_or, synth.tokens(wl))


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("path", ALL)
def test_rtn_shared_expert_c3_decode(mote, path, bits, c3_layers):
    wl, layer_or, layer_gpu = c3_layers
    layer_or = O.quantize_shared(layer_or, bits)
    layer_q = layer_gpu.quantize_shared(bits, path=path)
    check_shared_codes(layer_q, layer_or)
    for T in (1, 33):
        rep = check_forward(mote, layer_q, layer_or, synth.tokens(wl, T=T))
        assert rep["rel_fro"] < 5e-3


def test_rtn_shared_expert_rejects_missing_scales(mote):
    wl = synth.WORKLOADS["c1"]
    master, layer_or, layer_gpu = _setup(mote, wl)
    layer_q = layer_gpu.quantize_shared(8)
    layer_q.tensors["sh_up_scale"] = None
    with pytest.raises(mote.MoteError) as ei:
        mote.mote_moe_forward(layer_q, bf16_tensor(synth.tokens(wl)))
    assert ei.value.status == 1
    layer_gpu.shared_bits = 5
    with pytest.raises(mote.MoteError) as ei:
        mote.mote_moe_forward(layer_gpu, bf16_tensor(synth.tokens(wl)))
    assert ei.value.status == 2


@pytest.mark.parametrize("bits", [8, 4])
def test_rtn_prefill_expanding_once_or_inside_the_gemm_agree(mote, bits):
    # with only mote_workspace_bytes() of scratch a long prefill expands the codes inside the GEMM;
    # with mote_layer_workspace_bytes() it expands them once: same integers, same sums
    import ctypes as C
    wl = synth.custom("rtn", 256, 512, 4, 2, 900, 4321)
    master, layer_or, layer_gpu = _setup(mote, wl, TENSOR)
    layer_q = layer_gpu.quantize_shared(bits)
    x = bf16_tensor(synth.tokens(wl))
    small = mote.lib.mote_workspace_bytes(wl.d, wl.f, wl.E, wl.k, wl.T)
    s = layer_q.struct()
    assert mote.lib.mote_layer_workspace_bytes(C.byref(s), wl.T) == small + 6 * wl.d * wl.f
    assert mote.lib.mote_layer_workspace_bytes(C.byref(layer_gpu.struct()), wl.T) == small
    ws = torch.empty(small, dtype=torch.uint8, device="cuda")
    out1 = torch.empty_like(x)
    st = mote.lib.mote_moe_forward(C.byref(s), x.data_ptr(), None, wl.T, out1.data_ptr(), None, ws.data_ptr(), small,
                                   C.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert st == 0
    out2 = mote.mote_moe_forward(layer_q, x)
    torch.cuda.synchronize()
    assert torch.equal(out1, out2)


@pytest.mark.parametrize("T", [5, 200])
def test_output_and_residual_aligned_to_16_bytes_only(mote, T):
    # the C ABI promises kernels nothing beyond 16-byte alignment of out and residual: a view that
    # starts 16 bytes into an allocation must give the bits of the aligned call (the tensor path's
    # fused combine uses 32-byte accesses only where the pointers allow them)
    wl = synth.custom("align", 128, 256, 4, 2, T, 4400, w_std=0.08)
    layer = mote.MoteLayer.from_master(synth.master_layer(wl))
    x = bf16_tensor(synth.tokens(wl))
    res = bf16_tensor(synth.tokens(wl, stream=1))
    want = mote.mote_moe_forward(layer, x, residual=res)
    n = T * wl.d
    res_buf = torch.empty(n + 8, dtype=torch.bfloat16, device="cuda")
    out_buf = torch.empty(n + 8, dtype=torch.bfloat16, device="cuda")
    res16 = res_buf[8:].view(T, wl.d)
    out16 = out_buf[8:].view(T, wl.d)
    res16.copy_(res)
    assert res16.data_ptr() % 32 == 16 and out16.data_ptr() % 32 == 16
    got = mote.mote_moe_forward(layer, x, residual=res16, out=out16)
    torch.cuda.synchronize()
    assert torch.equal(got, want)
