"""EliteKV decode attention for NVIDIA B200 (sm_100a): thin Python binding over libelitekv.so.

`binding` loads the CUDA library on first use and raises if it is missing; `inputs` holds the
seeded synthetic workloads; `build` compiles the library in-tree.
"""
from . import inputs  # noqa: F401  (pure data generation, no CUDA needed)

__all__ = ["inputs", "binding", "build"]
