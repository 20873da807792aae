"""mote_stack_forward: layers chained with the residual between them (the c5 workload's shape of
use).  Each layer is checked against the oracle ON THE GPU'S OWN LAYER INPUT (a bf16 rounding
difference upstream may legitimately flip a routing decision downstream, so parity is per layer),
and the chain must equal the same layers called one by one, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import mote_oracle as O
from workloads import synth
from parity_utils import REL_FRO_TOL, assert_elementwise_close, assert_valid_near_tie_pick, bf16_bits, bf16_tensor, shared_rounding_sigma

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mote():
    import paper_2506_14435_b200 as m
    return m


@pytest.mark.parametrize("T,d", [(1, 64), (5, 896), (33, 2048), (300, 256), (3, 8192)])
def test_rms_norm(mote, T, d):
    rng = np.random.default_rng(T * 31 + d)
    x = O.f32_to_bf16_rn((rng.standard_normal((T, d)) * rng.uniform(0.01, 40.0, size=(T, 1))).astype(np.float32))
    if T > 2:
        x[1] = 0
    want = O.rms_norm(x, 1e-6)
    got = O.bf16_to_f32(bf16_bits(mote.mote_rms_norm(bf16_tensor(x), 1e-6))).astype(np.float64)
    # fp32 arithmetic and one bf16 rounding: within one bf16 ulp (2^-8 relative) of the fp64 value
    assert np.all(np.abs(got - want) <= np.abs(want) * 2.0 ** -8 + 1e-30)
    err = np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30)
    assert err <= REL_FRO_TOL


@pytest.mark.parametrize("rms_eps,shared_bits", [(1e-6, 16), (0.0, 16), (1e-6, 8), (1e-6, 4)])
@pytest.mark.parametrize("T", [1, 24, 40, 150])      # decode path (1, 24) and tensor-core path (40: K-split shared down; 150)
def test_small_stack_per_layer_parity(mote, T, rms_eps, shared_bits):
    n_layers = 5
    wl = synth.custom("stack", 128, 256, 4, 2, T, 4100, n_layers=n_layers, w_std=0.08)
    masters = [synth.master_layer(wl, layer=l) for l in range(n_layers)]
    layers = [mote.MoteLayer.from_master(m) for m in masters]
    if shared_bits != 16:                             # Section 4.3: RTN-coded shared experts
        layers = [l.quantize_shared(shared_bits) for l in layers]
    stack = mote.MoteStack(layers)
    x_bits = synth.tokens(wl)
    x = bf16_tensor(x_bits)
    taps = torch.zeros((n_layers, T, wl.d), dtype=torch.bfloat16, device="cuda")
    out = mote.mote_stack_forward(stack, x, layer_inputs=taps, rms_eps=rms_eps)
    torch.cuda.synchronize()
    assert torch.equal(taps[0], x)
    norm = (lambda t: mote.mote_rms_norm(t.contiguous(), rms_eps)) if rms_eps > 0 else (lambda t: t.contiguous())
    # the chain equals layer-by-layer calls
    cur = x
    for l, layer in enumerate(layers):
        assert torch.equal(taps[l], cur)
        cur = mote.mote_moe_forward(layer, norm(cur), residual=cur)
    assert torch.equal(cur, out)
    # every layer against the oracle, on the GPU's own input and residual of that layer
    for l in range(n_layers):
        layer_or = O.build_layer(masters[l])
        if shared_bits != 16:
            layer_or = O.quantize_shared(layer_or, shared_bits)
        res = taps[l].contiguous()
        xin_t = norm(res)
        got_t = taps[l + 1] if l + 1 < n_layers else out
        idx_taps = layers[l].alloc_taps(T, names=["topk_idx"])
        mote.mote_moe_forward(layers[l], xin_t, residual=res, taps=idx_taps)
        ref = O.moe_forward(layer_or, bf16_bits(xin_t), residual_bf16=bf16_bits(res),
                            near_tie_choice=idx_taps["topk_idx"].cpu().numpy())
        got = O.bf16_to_f32(bf16_bits(got_t)).astype(np.float64)
        err = np.linalg.norm(got - ref["out"]) / np.linalg.norm(ref["out"])
        assert err <= REL_FRO_TOL, (l, err)


def test_c5_shape_stack_matches_layer_by_layer(mote):
    wl = synth.WORKLOADS["c5"]
    layers = [mote.MoteLayer.from_device_draws(wl.d, wl.f, wl.E, wl.k, wl.norm_topk, synth.device_draw(wl, l, "cuda"))
              for l in range(2)]
    stack = mote.MoteStack(layers)
    for T in (1, 32, 300):
        x = synth.device_tokens(wl, "cuda", T=T)
        out = mote.mote_stack_forward(stack, x)
        cur = x
        for layer in layers:
            cur = mote.mote_moe_forward(layer, mote.mote_rms_norm(cur, 1e-6), residual=cur)
        assert torch.equal(cur, out)
        assert torch.isfinite(out.float()).all()


def test_stack_argument_errors(mote):
    import ctypes as C
    from paper_2506_14435_b200.binding import mote_layer_t
    lib = mote.lib
    arr = (mote_layer_t * 2)(mote_layer_t(128, 256, 4, 2, 1, 0), mote_layer_t(256, 256, 4, 2, 1, 0))
    assert lib.mote_stack_workspace_bytes(arr, 2, 8) == 0            # layers of different d
    fake = C.c_void_p(0x1000)
    eps = C.c_float(1e-6)
    assert lib.mote_stack_forward(arr, 0, eps, fake, 4, C.c_void_p(0x2000), None, fake, 1 << 20, None) == 2
    assert lib.mote_stack_forward(None, 1, eps, fake, 4, C.c_void_p(0x2000), None, fake, 1 << 20, None) == 1
    assert lib.mote_stack_forward(arr, 1, eps, fake, 4, fake, None, fake, 1 << 20, None) == 2    # out aliases x
    assert lib.mote_stack_forward(arr, 1, C.c_float(-1.0), fake, 4, C.c_void_p(0x2000), None, fake, 1 << 20, None) == 2
    assert lib.mote_rms_norm(fake, 4, 12, eps, fake, None) == 2 and lib.mote_rms_norm(None, 4, 16, eps, fake, None) == 1


@pytest.mark.parametrize("T", [1, 200])
def test_stack_forward_can_be_captured_in_a_cuda_graph(mote, T):
    # the library only enqueues on the caller's stream: a captured step replays to the same bits
    n_layers = 3
    wl = synth.custom("graph", 128, 256, 4, 2, T, 4200, n_layers=n_layers, w_std=0.08)
    layers = [mote.MoteLayer.from_master(synth.master_layer(wl, layer=l)) for l in range(n_layers)]
    stack = mote.MoteStack(layers)
    x = bf16_tensor(synth.tokens(wl))
    out = torch.empty_like(x)
    want = mote.mote_stack_forward(stack, x).clone()          # also the warm-up (first-call set-up, workspace)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        mote.mote_stack_forward(stack, x, out=out)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        mote.mote_stack_forward(stack, x, out=out)
    for _ in range(3):
        out.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, want)
    # new input in the same buffer, same graph
    x2 = bf16_tensor(synth.tokens(wl, stream=1))
    want2 = mote.mote_stack_forward(stack, x2).clone()
    x.copy_(x2)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, want2)


def test_c5_shape_stack_per_layer_parity_on_the_gpus_own_inputs(mote):
    """Three layers of the c5 stack at its own shape (d2048 f11008 E16 k2, bf16 shared expert),
    host-drawn weights, a decode batch of 32: every layer is compared with the oracle on the
    residual stream the GPU itself produced for it (stands for layers sampled from the 36-layer
    stack: every layer has the same shape and its own seeded weights)."""
    n_layers, T = 3, 32
    wl = synth.WORKLOADS["c5"].with_T(T)
    layers, oracles = [], []
    for l in range(n_layers):
        master = synth.master_layer(wl, layer=l)
        layers.append(mote.MoteLayer.from_master(master))
        oracles.append(O.build_layer(master))
        del master
    stack = mote.MoteStack(layers)
    x = bf16_tensor(synth.tokens(wl))
    taps = torch.zeros((n_layers, T, wl.d), dtype=torch.bfloat16, device="cuda")
    out = mote.mote_stack_forward(stack, x, layer_inputs=taps)
    torch.cuda.synchronize()
    assert mote.lib.mote_device_status(stack._ws.data_ptr(), None) == 0
    assert torch.equal(taps[0], x)
    for l in range(n_layers):
        res = taps[l].contiguous()
        xin = mote.mote_rms_norm(res, 1e-6)
        got_t = taps[l + 1] if l + 1 < n_layers else out
        # the stack's layer equals a stand-alone call on the same input, bit for bit
        idx_taps = layers[l].alloc_taps(T, names=["topk_idx"])
        alone = mote.mote_moe_forward(layers[l], xin, residual=res, taps=idx_taps)
        assert torch.equal(alone, got_t), l
        ref = O.moe_forward(oracles[l], bf16_bits(xin), residual_bf16=bf16_bits(res),
                            near_tie_choice=idx_taps["topk_idx"].cpu().numpy())
        for t in np.nonzero(ref["near_tie"])[0]:
            assert_valid_near_tie_pick(idx_taps["topk_idx"][t].cpu().numpy(), ref["logits"][t], wl.k)
        assert np.array_equal(idx_taps["topk_idx"].cpu().numpy(), ref["topk_idx"])
        got = O.bf16_to_f32(bf16_bits(got_t)).astype(np.float64)
        err = np.linalg.norm(got - ref["out"]) / np.linalg.norm(ref["out"])
        assert err <= REL_FRO_TOL, (l, err)
        assert_elementwise_close(got, ref["out"], shared_rounding_sigma(oracles[l], bf16_bits(xin)), f"layer {l}")
