"""ctypes binding of libmote.so.  Argument marshalling only: every step of the layer runs in the
library's kernels.  torch is used for device memory and streams."""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libmote.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2506_14435_b200.build`; "
                      "there is no fallback path")
lib = C.CDLL(_LIB_PATH)

PATH_AUTO, PATH_SIMT, PATH_TENSOR, PATH_STREAM = 0, 1, 2, 3
DTYPE_F32, DTYPE_BF16 = 0, 1


class mote_layer_t(C.Structure):
    _fields_ = [("d", C.c_int32), ("f", C.c_int32), ("E", C.c_int32), ("k", C.c_int32),
                ("norm_topk", C.c_int32), ("path", C.c_int32),
                ("Wr", C.c_void_p), ("router_bias", C.c_void_p),
                ("gate_packed", C.c_void_p), ("up_packed", C.c_void_p), ("down_packed", C.c_void_p),
                ("alpha_gate", C.c_void_p), ("alpha_up", C.c_void_p), ("alpha_down", C.c_void_p),
                ("sh_gate", C.c_void_p), ("sh_up", C.c_void_p), ("sh_down", C.c_void_p),
                ("shared_bits", C.c_int32),
                ("sh_gate_scale", C.c_void_p), ("sh_up_scale", C.c_void_p), ("sh_down_scale", C.c_void_p)]


TAP_FIELDS = ["topk_idx", "topk_w", "offsets", "perm", "qx", "beta_x", "acc_gate", "acc_up", "h_bf16",
              "qh", "beta_h", "acc_down", "y", "shared_out"]


class mote_taps_t(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in TAP_FIELDS]


lib.mote_status_string.restype = C.c_char_p
lib.mote_status_string.argtypes = [C.c_int]
lib.mote_ternarize_workspace_bytes.restype = C.c_size_t
lib.mote_ternarize_workspace_bytes.argtypes = []
lib.mote_ternarize_pack.restype = C.c_int
lib.mote_ternarize_pack.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p,
                                    C.c_void_p, C.c_size_t, C.c_void_p]
lib.mote_ternarize_pack_static.restype = C.c_int
lib.mote_ternarize_pack_static.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p,
                                           C.c_void_p]
lib.mote_rtn_quant.restype = C.c_int
lib.mote_rtn_quant.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
lib.mote_quant_act.restype = C.c_int
lib.mote_quant_act.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p,
                               C.c_void_p, C.c_void_p]
lib.mote_route_topk.restype = C.c_int
lib.mote_route_topk.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                                C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
lib.mote_route_stats.restype = C.c_int
lib.mote_route_stats.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
lib.mote_workspace_bytes.restype = C.c_size_t
lib.mote_workspace_bytes.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_int64]
lib.mote_layer_workspace_bytes.restype = C.c_size_t
lib.mote_layer_workspace_bytes.argtypes = [C.POINTER(mote_layer_t), C.c_int64]
lib.mote_host_staging_bytes.restype = C.c_size_t
lib.mote_host_staging_bytes.argtypes = [C.c_int, C.c_int64]
lib.mote_moe_forward.restype = C.c_int
lib.mote_moe_forward.argtypes = [C.POINTER(mote_layer_t), C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p,
                                 C.POINTER(mote_taps_t), C.c_void_p, C.c_size_t, C.c_void_p]
lib.mote_stack_workspace_bytes.restype = C.c_size_t
lib.mote_stack_workspace_bytes.argtypes = [C.POINTER(mote_layer_t), C.c_int, C.c_int64]
lib.mote_stack_forward.restype = C.c_int
lib.mote_stack_forward.argtypes = [C.POINTER(mote_layer_t), C.c_int, C.c_float, C.c_void_p, C.c_int64, C.c_void_p,
                                   C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
lib.mote_rms_norm.restype = C.c_int
lib.mote_rms_norm.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_float, C.c_void_p, C.c_void_p]
lib.mote_moe_forward_host.restype = C.c_int
lib.mote_moe_forward_host.argtypes = [C.POINTER(mote_layer_t), C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p,
                                      C.c_void_p, C.c_size_t, C.c_void_p]
lib.mote_moe_forward_profile.restype = C.c_int
lib.mote_moe_forward_profile.argtypes = [C.POINTER(mote_layer_t), C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p,
                                         C.c_void_p, C.c_size_t, C.c_void_p, C.POINTER(C.c_float)]
lib.mote_device_status.restype = C.c_int
lib.mote_device_status.argtypes = [C.c_void_p, C.c_void_p]
lib.mote_selftest_bounded_wait.restype = C.c_int
lib.mote_selftest_bounded_wait.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p]
lib.mote_int8_mma_peak.restype = C.c_int
lib.mote_int8_mma_peak.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_double), C.c_void_p]
lib.mote_last_launch_count.restype = C.c_int
lib.mote_last_launch_count.argtypes = []


class MoteError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib.mote_status_string(status).decode()} (status {status})")


def _check(status: int, where: str):
    if status != 0:
        raise MoteError(status, where)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _need_cuda(*ts):
    for t in ts:
        if t is not None and (not t.is_cuda or not t.is_contiguous()):
            raise ValueError("expected contiguous CUDA tensors")


def mote_ternarize_pack(W: torch.Tensor):
    """Eq. 7, 9: W[m, n] (fp32 or bf16, CUDA) -> (packed uint8[m, n/4], alpha float32[1])."""
    _need_cuda(W)
    m, n = W.shape
    dt = {torch.float32: DTYPE_F32, torch.bfloat16: DTYPE_BF16}[W.dtype]
    packed = torch.empty((m, max(n // 4, 1)), dtype=torch.uint8, device=W.device)
    alpha = torch.empty(1, dtype=torch.float32, device=W.device)
    ws_bytes = lib.mote_ternarize_workspace_bytes()
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=W.device)
    _check(lib.mote_ternarize_pack(_ptr(W), dt, m, n, _ptr(packed), _ptr(alpha), _ptr(ws), ws_bytes, _stream()),
           "mote_ternarize_pack")
    return packed, alpha


def mote_ternarize_pack_static(W: torch.Tensor, packed: torch.Tensor, alpha: torch.Tensor):
    """mote_ternarize_pack for callers that may not allocate: the caller passes the outputs
    (packed uint8[m, n/4], alpha float32[1]) and the library uses its built-in 2 KiB of device
    scratch, so neither this wrapper nor the call behind it allocates device memory.  At most 2^31
    elements; calls on one device must not overlap (they share the scratch)."""
    _need_cuda(W, packed, alpha)
    m, n = W.shape
    dt = {torch.float32: DTYPE_F32, torch.bfloat16: DTYPE_BF16}[W.dtype]
    if packed.dtype != torch.uint8 or packed.numel() != m * n // 4 or alpha.dtype != torch.float32:
        raise ValueError("packed must be uint8[m, n/4] and alpha float32[1]")
    _check(lib.mote_ternarize_pack_static(_ptr(W), dt, m, n, _ptr(packed), _ptr(alpha), _stream()),
           "mote_ternarize_pack_static")
    return packed, alpha


def mote_rtn_quant(W: torch.Tensor, bits: int):
    """Section 4.3: RTN absmax codes of W[m, n] (fp32 or bf16, CUDA), one scale per row.
    Returns (q, scale float32[m]); q is int8[m, n] for bits = 8 and uint8[m, n/2] for bits = 4."""
    _need_cuda(W)
    m, n = W.shape
    dt = {torch.float32: DTYPE_F32, torch.bfloat16: DTYPE_BF16}[W.dtype]
    if bits == 8:
        q = torch.empty((m, n), dtype=torch.int8, device=W.device)
    else:
        q = torch.empty((m, max(n // 2, 1)), dtype=torch.uint8, device=W.device)
    scale = torch.empty(m, dtype=torch.float32, device=W.device)
    _check(lib.mote_rtn_quant(_ptr(W), dt, m, n, bits, _ptr(q), _ptr(scale), _stream()), "mote_rtn_quant")
    return q, scale


def mote_quant_act(x: torch.Tensor, want_rowsum: bool = True):
    """Eq. 8: x[T, d] bf16 (CUDA; rows may be strided) -> (q int8[T,d], beta f32[T], rowsum i32[T])."""
    if not x.is_cuda or x.dtype != torch.bfloat16 or x.stride(1) != 1:
        raise ValueError("expected a CUDA bf16 matrix with unit inner stride")
    T, d = x.shape
    q = torch.empty((T, d), dtype=torch.int8, device=x.device)
    beta = torch.empty(T, dtype=torch.float32, device=x.device)
    rowsum = torch.empty(T, dtype=torch.int32, device=x.device) if want_rowsum else None
    _check(lib.mote_quant_act(_ptr(x), T, d, x.stride(0) if T > 1 else d, _ptr(q), _ptr(beta), _ptr(rowsum),
                              _stream()), "mote_quant_act")
    return q, beta, rowsum


def mote_route_topk(x, Wr, bias, k: int, norm_topk: int = 1, want_logits: bool = False):
    """Eq. 3: returns (topk_idx int32[T,k], topk_w f32[T,k], logits f32[T,E] or None)."""
    _need_cuda(x, Wr, bias)
    T, d = x.shape
    E = Wr.shape[0]
    idx = torch.empty((T, k), dtype=torch.int32, device=x.device)
    w = torch.empty((T, k), dtype=torch.float32, device=x.device)
    logits = torch.empty((T, E), dtype=torch.float32, device=x.device) if want_logits else None
    _check(lib.mote_route_topk(_ptr(x), T, d, _ptr(Wr), _ptr(bias), E, k, norm_topk, _ptr(idx), _ptr(w),
                               _ptr(logits), _stream()), "mote_route_topk")
    return idx, w, logits


def mote_route_stats(logits: torch.Tensor, topk_idx: torch.Tensor):
    """Eq. 12: (tokens_per_expert int32[E], prob_sum f32[E]) of a routed batch."""
    _need_cuda(logits, topk_idx)
    T, E = logits.shape
    k = topk_idx.shape[1]
    cnt = torch.empty(E, dtype=torch.int32, device=logits.device)
    ps = torch.empty(E, dtype=torch.float32, device=logits.device)
    _check(lib.mote_route_stats(_ptr(logits), _ptr(topk_idx), T, E, k, _ptr(cnt), _ptr(ps), _stream()),
           "mote_route_stats")
    return cnt, ps


class MoteLayer:
    """Device-resident weights of one MoTE layer plus its mote_layer_t."""

    def __init__(self, d, f, E, k, norm_topk, Wr, router_bias, gate_packed, up_packed, down_packed,
                 alpha_gate, alpha_up, alpha_down, sh_gate, sh_up, sh_down, path=PATH_AUTO,
                 shared_bits=16, sh_gate_scale=None, sh_up_scale=None, sh_down_scale=None):
        self.d, self.f, self.E, self.k, self.norm_topk, self.path = d, f, E, k, norm_topk, path
        self.shared_bits = shared_bits
        self.tensors = dict(Wr=Wr, router_bias=router_bias, gate_packed=gate_packed, up_packed=up_packed,
                            down_packed=down_packed, alpha_gate=alpha_gate, alpha_up=alpha_up,
                            alpha_down=alpha_down, sh_gate=sh_gate, sh_up=sh_up, sh_down=sh_down,
                            sh_gate_scale=sh_gate_scale, sh_up_scale=sh_up_scale, sh_down_scale=sh_down_scale)
        _need_cuda(*self.tensors.values())
        self._ws = None

    @classmethod
    def from_master(cls, master: dict, device="cuda", path=PATH_AUTO):
        """Offline step: upload fp32 master weights (numpy, see workloads.synth.master_layer) and
        ternarize every routed matrix on the device with mote_ternarize_pack."""
        d, f, E = master["d"], master["f"], master["E"]
        dev = torch.device(device)
        packed = {}
        alphas = {}
        for name, shape in (("gate", (f, d)), ("up", (f, d)), ("down", (d, f))):
            buf = torch.empty((E, shape[0], shape[1] // 4), dtype=torch.uint8, device=dev)
            al = torch.empty(E, dtype=torch.float32, device=dev)
            for e in range(E):
                W = torch.from_numpy(master["W_" + name][e]).to(dev)
                p, a = mote_ternarize_pack(W)
                buf[e].copy_(p)
                al[e:e + 1].copy_(a)
            packed[name], alphas[name] = buf, al

        def bf16(bits):
            return torch.from_numpy(bits.view("int16")).view(torch.bfloat16).to(dev)

        bias = master.get("router_bias")
        return cls(d, f, E, master["k"], master["norm_topk"], torch.from_numpy(master["Wr"]).to(dev),
                   None if bias is None else torch.from_numpy(bias).to(dev),
                   packed["gate"], packed["up"], packed["down"], alphas["gate"], alphas["up"], alphas["down"],
                   bf16(master["sh_gate"]), bf16(master["sh_up"]), bf16(master["sh_down"]), path=path)

    @classmethod
    def from_device_draws(cls, d, f, E, k, norm_topk, draw, device="cuda", path=PATH_AUTO):
        """Offline step with weights that are already on the device: draw(name, expert) returns
        fp32 CUDA matrices for "gate"/"up"/"down", bf16 ones for "sh_gate"/"sh_up"/"sh_down",
        fp32 "Wr" and "bias" (or None); every routed matrix goes through mote_ternarize_pack."""
        dev = torch.device(device)
        packed, alphas = {}, {}
        for name, shape in (("gate", (f, d)), ("up", (f, d)), ("down", (d, f))):
            buf = torch.empty((E, shape[0], shape[1] // 4), dtype=torch.uint8, device=dev)
            al = torch.empty(E, dtype=torch.float32, device=dev)
            for e in range(E):
                p, a = mote_ternarize_pack(draw(name, e).contiguous())
                buf[e].copy_(p)
                al[e:e + 1].copy_(a)
            packed[name], alphas[name] = buf, al
        return cls(d, f, E, k, norm_topk, draw("Wr").contiguous(), draw("bias"),
                   packed["gate"], packed["up"], packed["down"], alphas["gate"], alphas["up"], alphas["down"],
                   draw("sh_gate").contiguous(), draw("sh_up").contiguous(), draw("sh_down").contiguous(), path=path)

    def quantize_shared(self, bits: int, path=None) -> "MoteLayer":
        """Section 4.3: a layer with the same routed experts whose (bf16) shared expert is replaced
        by its RTN INT8 / INT4 codes (mote_rtn_quant on the device)."""
        if self.shared_bits != 16:
            raise ValueError("the shared expert is quantized already")
        t = dict(self.tensors)
        for name in ("sh_gate", "sh_up", "sh_down"):
            t[name], t[name + "_scale"] = mote_rtn_quant(self.tensors[name], bits)
        return MoteLayer(self.d, self.f, self.E, self.k, self.norm_topk, path=self.path if path is None else path,
                         shared_bits=bits, **t)

    def struct(self) -> mote_layer_t:
        t = self.tensors
        s = mote_layer_t(self.d, self.f, self.E, self.k, self.norm_topk, self.path)
        for name in ("Wr", "router_bias", "gate_packed", "up_packed", "down_packed", "alpha_gate", "alpha_up",
                     "alpha_down", "sh_gate", "sh_up", "sh_down", "sh_gate_scale", "sh_up_scale", "sh_down_scale"):
            setattr(s, name, None if t[name] is None else t[name].data_ptr())
        s.shared_bits = self.shared_bits
        return s

    def workspace(self, T: int, host_staging: bool = False) -> torch.Tensor:
        need = lib.mote_layer_workspace_bytes(C.byref(self.struct()), T)
        if need == 0:
            raise MoteError(2, "mote_layer_workspace_bytes")
        if host_staging:
            need += lib.mote_host_staging_bytes(self.d, T)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=self.tensors["Wr"].device)
        return self._ws

    def alloc_taps(self, T: int, names=TAP_FIELDS):
        dev = self.tensors["Wr"].device
        P, d, f, E, k = T * self.k, self.d, self.f, self.E, self.k
        spec = dict(topk_idx=((T, k), torch.int32), topk_w=((T, k), torch.float32),
                    offsets=((E + 1,), torch.int32), perm=((P,), torch.int32), qx=((T, d), torch.int8),
                    beta_x=((T,), torch.float32), acc_gate=((P, f), torch.int32), acc_up=((P, f), torch.int32),
                    h_bf16=((P, f), torch.bfloat16), qh=((P, f), torch.int8), beta_h=((P,), torch.float32),
                    acc_down=((P, d), torch.int32), y=((P, d), torch.float32),
                    shared_out=((T, d), torch.float32))
        return {n: torch.zeros(spec[n][0], dtype=spec[n][1], device=dev) for n in names}


def mote_moe_forward(layer: MoteLayer, x: torch.Tensor, residual=None, out=None, taps: dict | None = None):
    """Eq. 2-8 for x[T, d] bf16 (CUDA).  Returns out[T, d] bf16; fills the tensors in `taps`."""
    _need_cuda(x, residual, out)
    T = x.shape[0]
    if out is None:
        out = torch.empty_like(x)
    ws = layer.workspace(T)
    s = layer.struct()
    tp = None
    if taps is not None:
        tp = mote_taps_t()
        for n, t in taps.items():
            setattr(tp, n, t.data_ptr())
        tp = C.byref(tp)
    _check(lib.mote_moe_forward(C.byref(s), _ptr(x), _ptr(residual), T, _ptr(out), tp, _ptr(ws), ws.numel(),
                                _stream()), "mote_moe_forward")
    return out


def mote_moe_forward_host(layer: MoteLayer, x_host: torch.Tensor, out_host: torch.Tensor, residual_host=None):
    """Same layer with (pinned) host tensors in and out; synchronises the stream."""
    T = x_host.shape[0]
    ws = layer.workspace(T, host_staging=True)
    s = layer.struct()
    _check(lib.mote_moe_forward_host(C.byref(s), _ptr(x_host), _ptr(residual_host), T, _ptr(out_host), _ptr(ws),
                                     ws.numel(), _stream()), "mote_moe_forward_host")
    return out_host


class MoteStack:
    """A list of MoteLayer run back to back with the residual between layers (mote_stack_forward)."""

    def __init__(self, layers):
        self.layers = list(layers)
        self._structs = (mote_layer_t * len(self.layers))(*[l.struct() for l in self.layers])
        self._ws = None

    def workspace(self, T: int) -> torch.Tensor:
        need = lib.mote_stack_workspace_bytes(self._structs, len(self.layers), T)
        if need == 0:
            raise MoteError(2, "mote_stack_workspace_bytes")
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=self.layers[0].tensors["Wr"].device)
        return self._ws


def mote_rms_norm(x: torch.Tensor, eps: float = 1e-6, out=None):
    """The LN of Eq. 2 (RMS normalisation, unit gain) of x[T, d] bf16."""
    _need_cuda(x, out)
    if out is None:
        out = torch.empty_like(x)
    _check(lib.mote_rms_norm(_ptr(x), x.shape[0], x.shape[1], eps, _ptr(out), _stream()), "mote_rms_norm")
    return out


def mote_stack_forward(stack: MoteStack, x: torch.Tensor, out=None, layer_inputs=None, rms_eps: float = 1e-6):
    """x[T, d] bf16 -> x_L[T, d] bf16 after all layers (Eq. 1-2 chained, LN = RMS norm; rms_eps = 0
    chains the layers without normalisation); layer_inputs ([L, T, d] bf16) receives the residual
    stream entering every layer."""
    _need_cuda(x, out, layer_inputs)
    T = x.shape[0]
    if out is None:
        out = torch.empty_like(x)
    ws = stack.workspace(T)
    _check(lib.mote_stack_forward(stack._structs, len(stack.layers), rms_eps, _ptr(x), T, _ptr(out), _ptr(layer_inputs),
                                  _ptr(ws), ws.numel(), _stream()), "mote_stack_forward")
    return out


STAGE_NAMES = ["route", "dispatch", "quant_x", "gateup_ternary", "quant_h", "down_ternary", "shared_gateup",
               "shared_down", "combine"]


def mote_moe_forward_profile(layer: MoteLayer, x: torch.Tensor, out=None, residual=None) -> dict:
    """One forward with CUDA events between the stages; returns {stage: milliseconds}."""
    _need_cuda(x, residual, out)
    T = x.shape[0]
    if out is None:
        out = torch.empty_like(x)
    ws = layer.workspace(T)
    s = layer.struct()
    ms = (C.c_float * len(STAGE_NAMES))()
    _check(lib.mote_moe_forward_profile(C.byref(s), _ptr(x), _ptr(residual), T, _ptr(out), _ptr(ws), ws.numel(),
                                        _stream(), ms), "mote_moe_forward_profile")
    return dict(zip(STAGE_NAMES, [float(v) for v in ms]))


def mote_int8_mma_peak(n_batches: int, repeats: int = 5) -> dict:
    """Times the library's MMA-only kernel (mote_int8_mma_peak) with CUDA events on the current
    stream, `repeats` launches back to back after one warm-up: returns {"tops_best", "tops_median",
    "ms" (sorted), "ms_in_order", "ops" (per launch)}."""
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    ops = C.c_double(0.0)
    stream = torch.cuda.current_stream()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(repeats + 2)]
    evs[0].record(stream)
    for i in range(repeats + 1):
        _check(lib.mote_int8_mma_peak(_ptr(ws), n_batches, C.byref(ops), _stream()), "mote_int8_mma_peak")
        evs[i + 1].record(stream)
    torch.cuda.synchronize()
    times = [evs[i].elapsed_time(evs[i + 1]) for i in range(1, repeats + 1)]
    _check(lib.mote_device_status(_ptr(ws), _stream()), "mote_int8_mma_peak (device)")
    in_order = list(times)
    times.sort()
    return {"tops_best": ops.value / (times[0] * 1e-3) / 1e12,
            "tops_median": ops.value / (times[len(times) // 2] * 1e-3) / 1e12, "ms": times,
            "ms_in_order": in_order, "ops": ops.value}
