"""CPU oracle for the EARS verification step (TEST INFRASTRUCTURE).

Loads ``ears_oracle.c`` (plain fp64 C, built with gcc) through ctypes.  Nothing in
the CUDA package imports this; only tests, the smoke check and the benchmark's
CPU-baseline leg do.
"""
from .ears_oracle import (  # noqa: F401
    OracleResult,
    build,
    entropy,
    entropy_uncertainty,
    inverse_cdf,
    half_to_double,
    max_threads,
    philox4x32_10,
    row_softmax,
    softmax,
    uniform_accept,
    uniform_final,
    verify,
    verify_greedy,
)
