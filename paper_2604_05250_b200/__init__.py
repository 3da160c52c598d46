"""B200 (sm_100a) library for the data-parallel core of one DualDiffusion
verification step: bidirectional attention and the fused verification kernel.

The compute lives in ``csrc/`` behind the C ABI declared in
``include/dualdiff.h``; ``binding`` marshals arguments to it and nothing more.
Importing the package does not load the CUDA library; the first call does, and
fails loudly if the library has not been built.
"""
from . import synth  # noqa: F401  (seeded input generators; no CUDA needed)

__all__ = ["synth", "binding", "build"]
