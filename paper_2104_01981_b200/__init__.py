"""B200-native sparse gradient compression (top-k with error feedback, W-worker decode-sum).

``api`` binds the C-ABI library ``libgc.so`` (CUDA, sm_100a); ``synth`` holds the seeded
synthetic workloads; ``build`` compiles the library in-tree.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "api", "build"]
