"""B200 (sm_100a) forward pass of a Mixture-of-Ternary-Experts FFN layer: Python binding over the
C-ABI library libmote.so.  Importing this package loads the library and fails loudly if it has
not been built (python -m paper_2506_14435_b200.build)."""
from .binding import (MoteError, MoteLayer, PATH_AUTO, PATH_SIMT, PATH_STREAM, PATH_TENSOR, lib,
                      mote_moe_forward, mote_quant_act, mote_route_topk, mote_ternarize_pack)

__all__ = ["MoteError", "MoteLayer", "lib", "mote_ternarize_pack", "mote_quant_act", "mote_route_topk",
           "mote_moe_forward", "PATH_AUTO", "PATH_SIMT", "PATH_TENSOR", "PATH_STREAM"]
