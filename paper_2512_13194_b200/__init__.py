"""EARS speculative-decoding verification step, CUDA (sm_100a) implementation.

``verify`` and friends call the C-ABI library built from ``csrc/``; there is no
CPU fallback.  ``synth`` holds the seeded synthetic workloads.
"""
from . import synth  # noqa: F401
