"""LongGen efficient-layer attention for B200: C-ABI CUDA library plus a thin binding.

`binding` loads the in-tree shared library lazily (and raises if it is missing);
`synth` draws the seeded synthetic workloads; `build` compiles the library with nvcc.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding", "build"]
