"""Double quantization (AsyLPG / Sparse-AsyLPG / Acc-AsyLPG) hot path for NVIDIA B200.

``binding`` exposes the C ABI of ``libdq.so`` (see include/dq.h) with the same names; ``synth`` holds the
seeded synthetic input generators; ``build`` compiles the library in-tree.
"""
from .binding import *  # noqa: F401,F403
from .binding import EXPORTS, LIB_PATH, lib  # noqa: F401
