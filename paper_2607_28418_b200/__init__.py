"""WIDE hot path for NVIDIA B200: token-wise dynamic-width execution of a transformer layer.

``binding`` wraps the C-ABI library (libwide.so, built from csrc/ by ``build``); ``synth`` holds
the seeded synthetic workloads.  Importing the package does not load the library.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding", "build"]
