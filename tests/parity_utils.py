"""Helpers for the GPU parity tests: run the library through its C ABI on seeded inputs and
compare every intermediate with the CPU oracle."""
import numpy as np
import torch

from oracle import mote_oracle as O

REL_FRO_TOL = 5e-3      # bf16 layer output against the fp64 oracle
GATE_W_TOL = 1e-6
NEAR_TIE_GAP = 1e-5     # k-th and (k+1)-th logit closer than this: either pick is valid


def assert_valid_near_tie_pick(pick, logits, k: int):
    """A flagged token's selection must still be A correct top-k up to the tie: k distinct experts,
    every expert clearly above the oracle's k-th logit among them, none clearly below it, listed in
    descending logit order (up to the same gap)."""
    pick = [int(e) for e in pick]
    logits = np.asarray(logits, dtype=np.float64)
    kth = np.sort(logits)[::-1][k - 1]
    assert len(set(pick)) == k, pick
    must = set(np.nonzero(logits > kth + NEAR_TIE_GAP)[0].tolist())
    may = set(np.nonzero(logits >= kth - NEAR_TIE_GAP - 1e-12)[0].tolist())
    assert must <= set(pick) <= may, (pick, logits.tolist())
    sel = logits[pick]
    assert np.all(sel[:-1] >= sel[1:] - NEAR_TIE_GAP - 1e-12), (pick, sel.tolist())


def shared_rounding_sigma(layer_or: dict, x_bits: np.ndarray) -> np.ndarray:
    """Standard deviation, per output element, of what the one unavoidable intermediate rounding does
    to the shared expert's output: the kernels hold h = up * SiLU(gate) as bf16, i.e. every h_i is
    off by a relative error of at most 2^-9 (spread like a uniform variable: deviation 2^-9/sqrt 3),
    independent between i, so  s_c = sum_i Wd[c,i] h_i  is off by a variable of deviation
        sigma_c = 2^-9 / sqrt(3) * sqrt( sum_i (Wd[c,i] h_i)^2 ).
    Evaluated in fp64 from the same inputs the oracle gets (this is test arithmetic, not the oracle)."""
    x = O.bf16_to_f32(x_bits).astype(np.float64)
    if layer_or.get("sh_rtn"):
        Wg, Wu, Wd = (O.rtn_dequant(*layer_or["sh_rtn"][n]) for n in ("gate", "up", "down"))
    else:
        Wg, Wu, Wd = (O.bf16_to_f32(layer_or["sh_" + n]).astype(np.float64) for n in ("gate", "up", "down"))
    g = x @ Wg.T
    h = (x @ Wu.T) * (g / (1.0 + np.exp(-g)))
    return 2.0 ** -9 / np.sqrt(3.0) * np.sqrt((h * h) @ (Wd * Wd).T)


def assert_elementwise_close(got: np.ndarray, ref: np.ndarray, sigma: np.ndarray, what: str):
    """Per-element bound beside the Frobenius norm (which one wrong element cannot fail).  The GPU
    result differs from the fp64 oracle by the rounding of the shared expert's h to bf16 (deviation
    sigma per element, see shared_rounding_sigma; never more than 8 sigma in practice: the error is a
    sum of bounded independent terms) and by the final rounding of the value itself (2^-9 relative for
    a bf16 output; taken as 2^-8 to leave room for the fp32 accumulation order)."""
    bound = 8.0 * sigma + 2.0 ** -8 * np.abs(ref) + 1e-30
    bad = np.abs(got - ref) > bound
    assert not bad.any(), (what, int(bad.sum()), float(np.max(np.abs(got - ref) / bound)))


def bf16_tensor(bits: np.ndarray, device="cuda") -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(device)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def oracle_layer_from_master(master: dict) -> dict:
    return O.build_layer(master)


def check_packed_layer(layer_gpu, layer_or: dict):
    """Packed bytes and alpha of every routed matrix: bit-exact."""
    for name in ("gate", "up", "down"):
        packed = layer_gpu.tensors[name + "_packed"].cpu().numpy()
        alpha = layer_gpu.tensors["alpha_" + name].cpu().numpy()
        for e in range(layer_or["E"]):
            want = O.pack_codes(layer_or["codes_" + name][e])
            assert np.array_equal(packed[e], want), (name, e)
            assert alpha[e] == layer_or["alpha_" + name][e], (name, e, alpha[e], layer_or["alpha_" + name][e])


def check_forward(mote, layer_gpu, layer_or: dict, x_bits: np.ndarray, residual_bits=None, token_subset=None,
                  out_alias_residual=False):
    """Runs mote_moe_forward with every tap and compares with the oracle.  Returns a report."""
    T, d = x_bits.shape
    k, E, f = layer_or["k"], layer_or["E"], layer_or["f"]
    x = bf16_tensor(x_bits)
    res = None if residual_bits is None else bf16_tensor(residual_bits)
    taps = layer_gpu.alloc_taps(T)
    out_buf = res if out_alias_residual else None
    out = mote.mote_moe_forward(layer_gpu, x, residual=res, out=out_buf, taps=taps)
    torch.cuda.synchronize()
    assert mote.lib.mote_device_status(layer_gpu._ws.data_ptr(), None) == 0, "a device-side wait timed out"
    row_taps = ("acc_gate", "acc_up", "h_bf16", "qh", "beta_h", "acc_down", "y")
    g = {n: t.cpu() for n, t in taps.items() if n not in row_taps and n != "shared_out"}
    g_idx = g["topk_idx"].numpy()

    ref = O.moe_forward(layer_or, x_bits, residual_bits, token_subset=token_subset, near_tie_choice=g_idx)
    near = ref["near_tie"]
    # routing: indices equal everywhere (near-tie tokens were aligned to the GPU's valid choice)
    for t in np.nonzero(near)[0]:
        assert_valid_near_tie_pick(g_idx[t], ref["logits"][t], k)
    assert np.array_equal(g_idx, ref["topk_idx"])
    assert np.max(np.abs(g["topk_w"].numpy().astype(np.float64) - ref["topk_w"])) <= GATE_W_TOL
    assert np.array_equal(g["offsets"].numpy(), ref["offsets"])
    assert np.array_equal(g["perm"].numpy(), ref["perm"])
    assert np.array_equal(g["qx"].numpy(), ref["qx"])
    assert np.array_equal(g["beta_x"].numpy(), ref["beta_x"])
    # row- and token-indexed taps: only the oracle's rows travel to the host
    rows_dev = torch.from_numpy(ref["rows"].astype(np.int64)).cuda()
    toks = ref["tokens"]
    toks_dev = torch.from_numpy(np.asarray(toks, dtype=np.int64)).cuda()
    for n in row_taps:
        g[n] = taps[n][rows_dev].cpu()
    assert np.array_equal(g["acc_gate"].numpy(), ref["acc_gate"])
    assert np.array_equal(g["acc_up"].numpy(), ref["acc_up"])
    assert np.array_equal(bf16_bits(g["h_bf16"]), ref["h_bf16"])
    assert np.array_equal(g["qh"].numpy(), ref["qh"])
    assert np.array_equal(g["beta_h"].numpy(), ref["beta_h"])
    assert np.array_equal(g["acc_down"].numpy(), ref["acc_down"])
    y = g["y"].numpy().astype(np.float64)
    assert np.allclose(y, ref["y"], rtol=2e-6, atol=1e-12)
    sh = taps["shared_out"][toks_dev].cpu().numpy().astype(np.float64)
    sh_err = np.linalg.norm(sh - ref["shared_out"]) / max(np.linalg.norm(ref["shared_out"]), 1e-30)
    assert sh_err <= REL_FRO_TOL, sh_err
    sigma = shared_rounding_sigma(layer_or, x_bits[toks])
    assert_elementwise_close(sh, ref["shared_out"], sigma, "shared_out")
    out_f = O.bf16_to_f32(bf16_bits(out[toks_dev])).astype(np.float64)
    err = np.linalg.norm(out_f - ref["out"]) / max(np.linalg.norm(ref["out"]), 1e-30)
    assert err <= REL_FRO_TOL, err
    assert_elementwise_close(out_f, ref["out"], sigma, "out")
    # the launch configuration that is timed passes no taps (other epilogue branches, no fp32 copy
    # of the shared output): it must give the very same bits
    if not out_alias_residual:
        plain = mote.mote_moe_forward(layer_gpu, x, residual=res)
        torch.cuda.synchronize()
        assert torch.equal(plain, out), "tap-less call differs from the tapped one"
    return dict(rel_fro=err, shared_rel_fro=sh_err, near_ties=int(near.sum()), tokens=len(toks),
                out=out, counts=np.diff(ref["offsets"]))


def check_shared_codes(layer_gpu, layer_or: dict):
    """RTN codes and row scales of the shared expert (Section 4.3): bit-exact."""
    rtn = layer_or["sh_rtn"]
    assert layer_gpu.shared_bits == rtn["bits"]
    for name in ("gate", "up", "down"):
        q, scale = rtn[name]
        got = layer_gpu.tensors["sh_" + name].cpu().numpy()
        want = q if rtn["bits"] == 8 else O.pack_int4(q)
        assert got.dtype == want.dtype and np.array_equal(got, want), name
        assert np.array_equal(layer_gpu.tensors["sh_" + name + "_scale"].cpu().numpy(), scale), name
