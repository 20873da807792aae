"""The C-ABI library loads without a GPU, exports every symbol include/mote.h declares, and
rejects bad arguments on the host before anything is launched."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def mote():
    from paper_2506_14435_b200 import build
    build.build()
    import paper_2506_14435_b200 as m
    return m


def test_every_declared_symbol_is_exported(mote):
    text = open(os.path.join(ROOT, "include", "mote.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = set(re.findall(r"\b(mote_[a-z_0-9]+)\s*\(", text))
    assert {"mote_ternarize_pack", "mote_quant_act", "mote_route_topk", "mote_moe_forward"} <= names
    for n in names:
        assert hasattr(mote.lib, n), n


def test_status_strings(mote):
    for st in range(8):
        assert mote.lib.mote_status_string(st)
    assert mote.lib.mote_status_string(0) == b"ok"


def test_workspace_query(mote):
    wb = mote.lib.mote_workspace_bytes
    assert wb(256, 512, 4, 2, 64) > 0
    assert wb(256, 512, 4, 2, 128) > wb(256, 512, 4, 2, 64)
    assert wb(250, 512, 4, 2, 64) == 0          # d % 16
    assert wb(256, 512, 4, 5, 64) == 0          # k > E
    assert wb(256, 512, 65, 2, 64) == 0         # E > MOTE_MAX_EXPERTS
    assert wb(256, 512, 4, 2, -1) == 0
    assert mote.lib.mote_host_staging_bytes(256, 64) >= 3 * 64 * 256 * 2


def test_host_side_argument_errors(mote):
    lib = mote.lib
    NULL = None
    fake = C.c_void_p(0x1000)                    # aligned, never dereferenced: checks run first
    odd = C.c_void_p(0x1004)
    # ternarize_pack
    assert lib.mote_ternarize_pack(NULL, 0, 4, 16, fake, fake, fake, 4096, NULL) == 1
    assert lib.mote_ternarize_pack(fake, 7, 4, 16, fake, fake, fake, 4096, NULL) == 5
    assert lib.mote_ternarize_pack(fake, 0, 4, 12, fake, fake, fake, 4096, NULL) == 2
    assert lib.mote_ternarize_pack(fake, 0, 0, 16, fake, fake, fake, 4096, NULL) == 2
    assert lib.mote_ternarize_pack(odd, 0, 4, 16, fake, fake, fake, 4096, NULL) == 3
    assert lib.mote_ternarize_pack(fake, 0, 4, 16, fake, fake, fake, 8, NULL) == 4
    # quant_act
    assert lib.mote_quant_act(fake, 4, 20, 20, fake, fake, NULL, NULL) == 2
    assert lib.mote_quant_act(fake, -1, 16, 16, fake, fake, NULL, NULL) == 2
    assert lib.mote_quant_act(fake, 4, 32, 16, fake, fake, NULL, NULL) == 2      # ldx < d
    assert lib.mote_quant_act(NULL, 4, 16, 16, fake, fake, NULL, NULL) == 1
    assert lib.mote_quant_act(odd, 4, 16, 16, fake, fake, NULL, NULL) == 3
    assert lib.mote_quant_act(NULL, 0, 16, 16, NULL, NULL, NULL, NULL) == 0      # T = 0 is a no-op
    # route_topk
    assert lib.mote_route_topk(fake, 4, 16, fake, NULL, 4, 5, 1, fake, fake, NULL, NULL) == 2
    assert lib.mote_route_topk(fake, 4, 16, fake, NULL, 65, 2, 1, fake, fake, NULL, NULL) == 2
    assert lib.mote_route_topk(fake, 4, 16, fake, NULL, 16, 9, 1, fake, fake, NULL, NULL) == 2
    assert lib.mote_route_topk(fake, 4, 16, NULL, NULL, 4, 2, 1, fake, fake, NULL, NULL) == 1
    # moe_forward
    from paper_2506_14435_b200.binding import mote_layer_t
    L = mote_layer_t(256, 512, 4, 2, 1, 0)
    ws = C.c_void_p(0x10000)
    assert lib.mote_moe_forward(None, fake, NULL, 4, fake, None, ws, 1 << 30, NULL) == 1
    assert lib.mote_moe_forward(C.byref(L), fake, NULL, 4, fake, None, ws, 1 << 30, NULL) == 1   # null weights
    assert lib.mote_moe_forward(C.byref(L), NULL, NULL, 0, NULL, None, NULL, 0, NULL) == 0       # T = 0
    Lbad = mote_layer_t(250, 512, 4, 2, 1, 0)
    assert lib.mote_moe_forward(C.byref(Lbad), fake, NULL, 4, fake, None, ws, 1 << 30, NULL) == 2
    for name, ctype in mote_layer_t._fields_[6:]:
        if ctype is C.c_void_p:
            setattr(L, name, 0x2000)
    L.router_bias = None
    assert lib.mote_moe_forward(C.byref(L), fake, NULL, 4, fake, None, ws, 1 << 30, NULL) == 2   # out aliases x
    other = C.c_void_p(0x3000)
    assert lib.mote_moe_forward(C.byref(L), fake, NULL, 4, other, None, ws, 16, NULL) == 4       # workspace
    assert lib.mote_moe_forward(C.byref(L), fake, NULL, 4, other, None, C.c_void_p(0x10010), 1 << 30, NULL) == 3
    # shared-expert storage: unknown width, RTN codes without their scales
    L.shared_bits = 5
    assert lib.mote_moe_forward(C.byref(L), fake, NULL, 4, other, None, ws, 1 << 30, NULL) == 2
    L.shared_bits = 4
    L.sh_down_scale = None
    assert lib.mote_moe_forward(C.byref(L), fake, NULL, 4, other, None, ws, 1 << 30, NULL) == 1
    # rtn_quant
    assert lib.mote_rtn_quant(NULL, 1, 4, 16, 8, fake, fake, NULL) == 1
    assert lib.mote_rtn_quant(fake, 9, 4, 16, 8, fake, fake, NULL) == 5
    assert lib.mote_rtn_quant(fake, 1, 4, 24, 8, fake, fake, NULL) == 2
    assert lib.mote_rtn_quant(fake, 1, 4, 16, 2, fake, fake, NULL) == 2
    assert lib.mote_rtn_quant(odd, 1, 4, 16, 4, fake, fake, NULL) == 3
    # route_stats
    assert lib.mote_route_stats(fake, fake, 4, 65, 2, fake, fake, NULL) == 2
    assert lib.mote_route_stats(fake, fake, 4, 4, 2, NULL, fake, NULL) == 1
    assert lib.mote_route_stats(NULL, fake, 4, 4, 2, fake, fake, NULL) == 1
