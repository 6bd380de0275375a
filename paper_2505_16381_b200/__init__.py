"""PaTH attention (blockwise training hot path) for NVIDIA B200 (sm_100a).

The compute lives in a C-ABI shared library built from ``csrc/``; ``binding``
marshals arguments to it and nothing else.  Importing this package does not load
the library; the first call does, and fails loudly if it has not been built.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding", "build", "autograd"]
