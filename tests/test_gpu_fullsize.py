"""Parity at the full sizes of the prefill workloads, in the launch configuration bench.py times
(automatic path selection).  Routing, dispatch and Q_a(x) are compared for every token; the expert
stages and the output for a token sample the oracle can afford: the tokens owning the first and
last row of every expert segment, the rows on both sides of every 128- and 256-row tile boundary,
and a seeded random remainder (tokens are independent of each other, so a sample is a valid check).
Packed weights and alpha are compared for every matrix."""
import numpy as np
import pytest
import torch

from oracle import mote_oracle as O
from workloads import synth
from parity_utils import bf16_tensor, check_forward, check_packed_layer, check_shared_codes

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mote():
    import paper_2506_14435_b200 as m
    return m


def _sampled_parity(mote, wl, n_random, max_boundary_tokens, shared_bits=16):
    master = synth.master_layer(wl)
    layer_or = O.build_layer(master)
    layer_gpu = mote.MoteLayer.from_master(master)
    check_packed_layer(layer_gpu, layer_or)
    if shared_bits != 16:
        layer_or = O.quantize_shared(layer_or, shared_bits)
        layer_gpu = layer_gpu.quantize_shared(shared_bits)
        check_shared_codes(layer_gpu, layer_or)
    x_bits = synth.tokens(wl)
    r = O.router(x_bits, layer_or["Wr"], layer_or.get("router_bias"), wl.k, wl.norm_topk)
    offsets, perm, inv = O.dispatch(r["idx"], wl.E)
    toks = synth.sample_tokens(offsets, inv, wl.k, wl.T, n_random=n_random, seed=wl.seed)
    if len(toks) > max_boundary_tokens + n_random:
        rng = np.random.default_rng(wl.seed)
        toks = np.sort(rng.choice(toks, size=max_boundary_tokens + n_random, replace=False))
    toks = toks[~r["near_tie"][toks]]          # a near tie may legitimately move a token to another expert
    rep = check_forward(mote, layer_gpu, layer_or, x_bits, token_subset=toks)
    assert rep["tokens"] >= min(64, wl.T)
    return rep


def test_c2_full_size_sampled(mote):
    rep = _sampled_parity(mote, synth.WORKLOADS["c2"], n_random=96, max_boundary_tokens=400)
    assert rep["rel_fro"] < 5e-3


@pytest.mark.parametrize("bits", [8, 4])
def test_c2_full_size_sampled_rtn_shared_expert(mote, bits):
    rep = _sampled_parity(mote, synth.WORKLOADS["c2"], n_random=64, max_boundary_tokens=100, shared_bits=bits)
    assert rep["rel_fro"] < 5e-3


def test_c4_full_size_sampled(mote):
    rep = _sampled_parity(mote, synth.WORKLOADS["c4"], n_random=64, max_boundary_tokens=200)
    assert rep["rel_fro"] < 5e-3
    assert rep["counts"].min() >= 0 and rep["counts"].sum() == 2 * 8192


@pytest.mark.parametrize("T", [1, 48, 333])
def test_paper_configuration_top1_full_softmax_gate(mote, T):
    # the paper's 0.5B model layer: 1 shared + 4 routed experts, top-1, gate weight = P(x)_i of Eq. 3
    wl = synth.WORKLOADS["p05"].with_T(T)
    master = synth.master_layer(wl)
    layer_or = O.build_layer(master)
    layer_gpu = mote.MoteLayer.from_master(master)
    rep = check_forward(mote, layer_gpu, layer_or, synth.tokens(wl))
    assert rep["rel_fro"] < 5e-3
    assert rep["counts"].sum() == T


@pytest.mark.parametrize("bits", [8, 4])
def test_paper_3b_layer_rtn_shared_expert_decode_and_prefill(mote, bits):
    # the operating points of the paper's Table 3: the 3B model's layer with the shared expert in INT8 / INT4
    wl = synth.WORKLOADS["p3"]
    master = synth.master_layer(wl)
    layer_or = O.quantize_shared(O.build_layer(master), bits)
    layer_gpu = mote.MoteLayer.from_master(master).quantize_shared(bits)
    check_shared_codes(layer_gpu, layer_or)
    for T in (1, 160):
        rep = check_forward(mote, layer_gpu, layer_or, synth.tokens(wl.with_T(T)))
        assert rep["rel_fro"] < 5e-3


@pytest.mark.parametrize("T", [1, 32])
def test_c5_shape_decode_layer(mote, T):
    # one layer of the c5 stack at its own shape (d2048 f11008, 16 routed experts, top-2, bf16 shared
    # expert), host-drawn weights, automatic path (the weight stream at these batch sizes), every tap
    wl = synth.WORKLOADS["c5"].with_T(T)
    master = synth.master_layer(wl, layer=0)
    layer_or = O.build_layer(master)
    layer_gpu = mote.MoteLayer.from_master(master)
    check_packed_layer(layer_gpu, layer_or)
    del master
    rep = check_forward(mote, layer_gpu, layer_or, synth.tokens(wl))
    assert rep["tokens"] == T and rep["counts"].sum() == 2 * T
    assert rep["rel_fro"] < 5e-3
