"""Host-side checks that need no GPU: the library builds, loads, exports every symbol the
header declares, and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import pytest

import paper_2512_13194_b200 as ears
from paper_2512_13194_b200 import build as ears_build
from paper_2512_13194_b200.shard import shard_range

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ears.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ears_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = ears_build.build()
    lib = ctypes.CDLL(path)
    names = declared_symbols()
    assert "ears_verify" in names and "ears_verify_ex" in names and len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n
    assert ears.version() == 100


def test_status_strings():
    lib = ears.load_library()
    seen = {lib.ears_status_string(s).decode() for s in range(0, -8, -1)}
    assert len(seen) == 8 and "ok" in seen
    assert lib.ears_status_string(-99).decode() == "unknown status"


def test_bad_arguments_are_rejected_on_the_host():
    lib = ears.load_library()
    buf = (ctypes.c_float * 64)()
    p = ctypes.addressof(buf)
    ok = dict(t=p, d=p, x=p, B=1, K=1, V=4, T=1.0, beta=0.1, out_len=p, out_tok=p)

    def call(**kw):
        a = dict(ok, **kw)
        return lib.ears_verify_f32(a["t"], a["d"], a["x"], a["B"], a["K"], a["V"], a["T"], a["beta"], 0, 0,
                                   a["out_len"], a["out_tok"], None)

    assert call(t=None) == -1 and call(d=None) == -1 and call(x=None) == -1
    assert call(out_len=None) == -1 and call(out_tok=None) == -1
    assert call(B=0) == -2 and call(K=0) == -2 and call(V=0) == -2 and call(K=65) == -2
    assert call(V=2**30 + 1) == -2
    assert call(B=2**31 - 1, K=64, V=2**30) == -2
    assert call(T=0.0) == -3 and call(T=-1.0) == -3 and call(T=float("nan")) == -3 and call(T=float("inf")) == -3
    assert call(beta=-0.1) == -3 and call(beta=float("nan")) == -3
    assert call(t=p + 2) == -4 and call(d=p + 1) == -4
    assert lib.ears_verify_ex(7, p, p, p, 1, 1, 4, 1.0, 0.1, 0, 0, 0, p, p, None, None, None, None, None,
                              None, 0, None) == -3
    assert lib.ears_verify_ex(0, p, p, p, 1, 1, 4, 1.0, 0.1, 0, 0, -1, p, p, None, None, None, None, None,
                              None, 0, None) == -3
    assert lib.ears_verify_ex(0, p, p, p, 1, 1, 4, 1.0, 0.1, 0, 0, 0, p, p, None, None, None, None, None,
                              p + 4, 1 << 20, None) == -4
    assert lib.ears_verify_host(0, None, p, p, 1, 1, 4, 1.0, 0.1, 0, 0, 0, p, p, None) == -1
    # the allocation-free entry point judges its arguments before it looks for a device
    lib.ears_verify_noalloc.argtypes = ([ctypes.c_int] + [ctypes.c_void_p] * 3 + [ctypes.c_int] * 3 + [ctypes.c_float] * 2
                                        + [ctypes.c_uint64] * 2 + [ctypes.c_int64] + [ctypes.c_void_p] * 4)

    def noalloc(dtype=0, t=p, B=1, K=1, V=4, T=1.0, beta=0.1, b_first=0):
        return lib.ears_verify_noalloc(dtype, t, p, p, B, K, V, T, beta, 0, 0, b_first, p, p, None, None)

    assert noalloc(t=None) == -1
    assert noalloc(dtype=9) == -3 and noalloc(T=0.0) == -3 and noalloc(T=float("nan")) == -3 and noalloc(beta=-1.0) == -3
    assert noalloc(b_first=-1) == -3
    assert noalloc(B=0) == -2 and noalloc(K=65) == -2
    assert noalloc(t=p + 2) == -4
    assert noalloc(B=40000, K=8, V=16) == -5          # beyond the fixed scratch array
    assert lib.ears_set_plan(3, 0) == -3 and lib.ears_set_plan(0, 0) == 0
    assert lib.ears_philox_device(None, None, -1, None) == -2
    assert lib.ears_philox_device(None, None, 0, None) == 0


def test_workspace_bound_is_monotone_enough():
    assert ears.workspace_bytes(0, 1, 1) == 0
    small = ears.workspace_bytes(1, 4, 32000)
    big = ears.workspace_bytes(512, 3, 256000)
    assert 0 < small < big < 64 << 20


def test_shard_ranges_tile_the_batch():
    for B in (0, 1, 7, 512):
        for world in (1, 2, 3, 8):
            spans = [shard_range(B, r, world) for r in range(world)]
            assert spans[0][0] == 0 and sum(n for _, n in spans) == B
            for (a, n), (b, _) in zip(spans, spans[1:]):
                assert a + n == b
            assert max(n for _, n in spans) - min(n for _, n in spans) <= 1
    with pytest.raises(ValueError):
        shard_range(4, 2, 2)
