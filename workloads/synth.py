"""Seeded synthetic inputs for the MoTE FFN-layer workloads.

This module only draws random numbers and shapes them; it contains none of the method's
arithmetic (no quantizer, no router, no GEMM).  Both the CUDA path's tests and the CPU oracle
receive the very same arrays produced here.

All arrays are numpy.  bf16 tensors are uint16 bit patterns (the rounding of a random draw to
bf16 is data preparation, done with torch's converter).

Workloads (shapes from the Qwen2.5 0.5B / 1.5B / 3B FFN dimensions the paper's models use,
Section 4.1; 1 shared + E routed experts; the synthetic tensors stand in for the activations
of the public instruction / evaluation sets, which an FFN layer only sees as [T, d] rows):

  c1  d=256  f=512   E=4  k=2  T=64                      plain N(0,1) tokens
  c2  d=896  f=4864  E=4  k=2  T=4096                    1 % of channels scaled x20
  c3  d=1536 f=8960  E=8  k=2  T in {1,8,32,64}          router bias ln p_e, p_e ~ (e+1)^-1.1
  c4  d=2048 f=11008 E=16 k=2  T=8192                    outlier channels, router bias N(0,0.5^2)
  c5  36 layers of c4's shape, T in {1,32,2048}          plain tokens, no bias
  p05 / p15 / p3  the paper's own MoTE models: E=4, top-1, gate = softmax over all experts,
      24 / 28 / 36 layers of the Qwen2.5-0.5B / 1.5B / 3B FFN shape, 2048-token sequences
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch

MAT_GATE, MAT_UP, MAT_DOWN, MAT_SH_GATE, MAT_SH_UP, MAT_SH_DOWN, MAT_ROUTER, MAT_BIAS, MAT_X = range(9)


@dataclass(frozen=True)
class Workload:
    name: str
    d: int
    f: int
    E: int
    k: int
    T: int
    seed: int
    n_layers: int = 1
    norm_topk: int = 1
    outlier_frac: float = 0.0      # fraction of channels multiplied by outlier_gain
    outlier_gain: float = 20.0
    bias: str = "none"             # "none" | "zipf" | "normal"
    w_std: float = 0.02

    def with_T(self, T: int) -> "Workload":
        return replace(self, T=T)


WORKLOADS = {
    "c1": Workload("c1", 256, 512, 4, 2, 64, 1001),
    "c2": Workload("c2", 896, 4864, 4, 2, 4096, 1002, outlier_frac=0.01),
    "c3": Workload("c3", 1536, 8960, 8, 2, 64, 1003, bias="zipf"),
    "c4": Workload("c4", 2048, 11008, 16, 2, 8192, 1004, outlier_frac=0.01, bias="normal"),
    "c5": Workload("c5", 2048, 11008, 16, 2, 2048, 1005, n_layers=36),
    # the configuration the paper trains and evaluates (Section 4.1, App. B): 1 shared + 4 routed
    # experts, top-1, the gate weight is P(x)_i of Eq. 3 over all experts; 2048-token sequences
    "p05": Workload("p05", 896, 4864, 4, 1, 2048, 1011, n_layers=24, norm_topk=0),
    "p15": Workload("p15", 1536, 8960, 4, 1, 2048, 1012, n_layers=28, norm_topk=0),
    "p3": Workload("p3", 2048, 11008, 4, 1, 2048, 1013, n_layers=36, norm_topk=0),
}
C3_BATCHES = (1, 8, 32, 64)
C5_BATCHES = (1, 32, 2048)


def _gen(wl: Workload, layer: int, expert: int, mat: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(((wl.seed * 1009 + layer) * 1009 + expert) * 1009 + mat)
    return g


def _to_bf16_bits(t: torch.Tensor) -> np.ndarray:
    return t.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16).copy()


def routed_matrix(wl: Workload, layer: int, expert: int, mat: int) -> np.ndarray:
    """fp32 master weights of one routed matrix: gate/up are [f, d], down is [d, f]."""
    shape = (wl.d, wl.f) if mat == MAT_DOWN else (wl.f, wl.d)
    return (torch.randn(shape, generator=_gen(wl, layer, expert, mat), dtype=torch.float32)
            * wl.w_std).numpy()


def shared_matrix(wl: Workload, layer: int, mat: int) -> np.ndarray:
    """bf16 bit patterns of one shared-expert matrix (sh_gate/sh_up [f,d], sh_down [d,f])."""
    shape = (wl.d, wl.f) if mat == MAT_SH_DOWN else (wl.f, wl.d)
    w = torch.randn(shape, generator=_gen(wl, layer, 0, mat), dtype=torch.float32) * wl.w_std
    return _to_bf16_bits(w)


def router_weights(wl: Workload, layer: int):
    """(Wr fp32[E,d] with bf16-representable values, bias fp32[E] or None)."""
    w = torch.randn((wl.E, wl.d), generator=_gen(wl, layer, 0, MAT_ROUTER), dtype=torch.float32)
    Wr = (w * wl.w_std).to(torch.bfloat16).to(torch.float32).numpy().copy()
    if wl.bias == "zipf":
        p = np.arange(1, wl.E + 1, dtype=np.float64) ** -1.1
        bias = np.log(p / p.sum()).astype(np.float32)
    elif wl.bias == "normal":
        b = torch.randn((wl.E,), generator=_gen(wl, layer, 0, MAT_BIAS), dtype=torch.float32) * 0.5
        bias = b.numpy().copy()
    else:
        bias = None
    return Wr, bias


def tokens(wl: Workload, T: int | None = None, stream: int = 0) -> np.ndarray:
    """bf16 bit patterns of x[T, d]: N(0,1), optionally with outlier channels."""
    T = wl.T if T is None else T
    g = _gen(wl, 0, stream, MAT_X)
    x = torch.randn((T, wl.d), generator=g, dtype=torch.float32)
    n_out = int(round(wl.outlier_frac * wl.d))
    if n_out > 0:
        chans = torch.randperm(wl.d, generator=g)[:n_out]
        x[:, chans] *= wl.outlier_gain
    return _to_bf16_bits(x)


def master_layer(wl: Workload, layer: int = 0) -> dict:
    """All fp32 master weights of one layer in memory (use for shapes up to c4)."""
    Wr, bias = router_weights(wl, layer)
    m = dict(d=wl.d, f=wl.f, E=wl.E, k=wl.k, norm_topk=wl.norm_topk, Wr=Wr, router_bias=bias)
    for name, mat in (("gate", MAT_GATE), ("up", MAT_UP), ("down", MAT_DOWN)):
        m["W_" + name] = np.stack([routed_matrix(wl, layer, e, mat) for e in range(wl.E)])
    for name, mat in (("sh_gate", MAT_SH_GATE), ("sh_up", MAT_SH_UP), ("sh_down", MAT_SH_DOWN)):
        m[name] = shared_matrix(wl, layer, mat)
    return m


def custom(name: str, d: int, f: int, E: int, k: int, T: int, seed: int, **kw) -> Workload:
    return Workload(name, d, f, E, k, T, seed, **kw)


def sample_tokens(offsets: np.ndarray, inv: np.ndarray, k: int, T: int, n_random: int,
                  tile_rows=(128, 256), seed: int = 0) -> np.ndarray:
    """Pick tokens for sampled parity at full size: the tokens owning the first and last row of
    every expert segment, the rows on both sides of every tile boundary inside a segment, and a
    seeded random remainder.  offsets/inv describe the expert-sorted order (row -> pair)."""
    rows = set()
    P = int(offsets[-1])
    for e in range(len(offsets) - 1):
        a, b = int(offsets[e]), int(offsets[e + 1])
        if b <= a:
            continue
        rows.update((a, b - 1))
        for tr in tile_rows:
            for r in range(a + tr, b, tr):
                rows.update((r - 1, r))
    toks = {int(inv[r]) // k for r in rows if 0 <= r < P}
    rng = np.random.default_rng(seed)
    if n_random > 0:
        toks.update(int(t) for t in rng.choice(T, size=min(n_random, T), replace=False))
    return np.array(sorted(toks), dtype=np.int64)


def device_draw(wl: Workload, layer: int, device):
    """Returns draw(name, expert) producing the tensors of one layer directly on `device`, for
    layer stacks that would take minutes to draw on the host (c5: 36 layers of 0.8 G weights).
    Same distributions and seeding scheme as the host generators but a different random stream,
    so these tensors are for timing and for GPU-against-GPU consistency checks, never for the oracle.
    name: "gate" | "up" | "down" (fp32 [f,d] / [d,f]), "sh_gate" | "sh_up" | "sh_down" (bf16),
    "Wr" (fp32 [E,d], bf16-representable), "bias" (fp32 [E] or None)."""
    ids = dict(gate=MAT_GATE, up=MAT_UP, down=MAT_DOWN, sh_gate=MAT_SH_GATE, sh_up=MAT_SH_UP, sh_down=MAT_SH_DOWN,
               Wr=MAT_ROUTER, bias=MAT_BIAS)

    def gen(expert, mat):
        g = torch.Generator(device=device)
        g.manual_seed(((wl.seed * 1009 + layer) * 1009 + expert) * 1009 + mat)
        return g

    def draw(name: str, expert: int = 0):
        mat = ids[name]
        if name == "Wr":
            w = torch.randn((wl.E, wl.d), generator=gen(0, mat), device=device, dtype=torch.float32) * wl.w_std
            return w.to(torch.bfloat16).to(torch.float32)
        if name == "bias":
            if wl.bias == "zipf":
                p = torch.arange(1, wl.E + 1, dtype=torch.float64) ** -1.1
                return torch.log(p / p.sum()).to(torch.float32).to(device)
            if wl.bias == "normal":
                return torch.randn((wl.E,), generator=gen(0, mat), device=device, dtype=torch.float32) * 0.5
            return None
        shape = (wl.d, wl.f) if name in ("down", "sh_down") else (wl.f, wl.d)
        w = torch.randn(shape, generator=gen(expert, mat), device=device, dtype=torch.float32) * wl.w_std
        return w.to(torch.bfloat16) if name.startswith("sh_") else w

    return draw


def device_tokens(wl: Workload, device, T: int | None = None, stream: int = 0) -> torch.Tensor:
    """x[T, d] bf16 drawn on the device (N(0,1), optional outlier channels); see device_draw."""
    T = wl.T if T is None else T
    g = torch.Generator(device=device)
    g.manual_seed(((wl.seed * 1009) * 1009 + stream) * 1009 + MAT_X)
    x = torch.randn((T, wl.d), generator=g, device=device, dtype=torch.float32)
    n_out = int(round(wl.outlier_frac * wl.d))
    if n_out > 0:
        chans = torch.randperm(wl.d, generator=g, device=device)[:n_out]
        x[:, chans] *= wl.outlier_gain
    return x.to(torch.bfloat16)
