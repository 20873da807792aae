"""B200 (sm_100a) forward pass of a Mixture-of-Ternary-Experts FFN layer: Python binding over the
C-ABI library libmote.so.  The binding (and with it the library) is loaded on first use of any
name below and fails loudly if the library has not been built
(python -m paper_2506_14435_b200.build); there is no fallback path."""

_EXPORTS = ["MoteError", "MoteLayer", "lib", "mote_ternarize_pack", "mote_ternarize_pack_static", "mote_rtn_quant", "mote_quant_act", "mote_route_topk", "mote_route_stats",
            "mote_moe_forward", "mote_moe_forward_host", "MoteStack", "mote_stack_forward", "mote_rms_norm", "mote_moe_forward_profile", "PATH_AUTO", "PATH_SIMT",
            "PATH_TENSOR", "PATH_STREAM", "STAGE_NAMES"]
__all__ = list(_EXPORTS)


def __getattr__(name):
    if name in _EXPORTS:
        from . import binding
        return getattr(binding, name)
    raise AttributeError(name)
