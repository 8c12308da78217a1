"""Per-layer approximate cache look-up of Freeze Inference (arXiv 2002.02645) for NVIDIA B200 (sm_100a).

`binding` wraps the C ABI of include/fi.h; `datagen` draws the seeded synthetic workloads; `build` compiles the
CUDA library in-tree.
"""
from . import build, datagen  # noqa: F401

__all__ = ["build", "datagen", "binding"]
