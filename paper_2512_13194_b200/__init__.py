"""EARS speculative-decoding verification step, CUDA (sm_100a) implementation.

``verify`` and friends call the C-ABI library built from ``csrc/`` (declared in
``include/ears.h``); there is no CPU fallback.  ``synth`` holds the seeded
synthetic workloads, ``shard`` the batch partition used across GPUs and
the driver of the vocabulary-sharded step.
"""
from . import shard, synth  # noqa: F401
from .sampler import EarsSampler, StepResult  # noqa: F401
from .binding import (  # noqa: F401
    DEV_INVALID_INPUT,
    DEV_TIMEOUT,
    EarsError,
    ShardStep,
    class_counts,
    decision_counts,
    describe_plan,
    last_device_status,
    load_library,
    philox_device,
    profile_begin,
    profile_end,
    selftest_bounded_wait,
    set_path,
    set_plan,
    shutdown,
    verify,
    verify_abi,
    verify_greedy,
    verify_host,
    verify_noalloc,
    version,
    workspace_bytes,
    workspace_device_status,
)
