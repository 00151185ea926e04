"""B200-native token-centric MoE layer (gate, dispatch, expert FFN, combine).

`binding` exposes the C-ABI entry points of libtcmoe.so; `synth` draws the
seeded synthetic workloads; `build` compiles the library in-tree.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding", "build"]
