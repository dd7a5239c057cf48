"""ctypes binding of the fp64 C oracle (TEST INFRASTRUCTURE, see ears_oracle.c).

Argument marshalling only; every number is computed in ``ears_oracle.c``.
Logits may be numpy float32 or float16 arrays, numpy uint16 arrays holding bf16 bit
patterns, or CPU torch tensors of dtype float32 / bfloat16.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ears_oracle.c")
_LIB = os.path.join(_HERE, "libears_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile ears_oracle.c with gcc (no fast-math: IEEE double semantics kept)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    c = ctypes
    lib.ears_oracle_philox4x32_10.argtypes = [c.POINTER(c.c_uint32)] * 3
    lib.ears_oracle_philox4x32_10.restype = None
    lib.ears_oracle_uniform_accept.argtypes = [c.c_uint64, c.c_uint64, c.c_int64, c.c_int]
    lib.ears_oracle_uniform_accept.restype = c.c_double
    lib.ears_oracle_uniform_final.argtypes = [c.c_uint64, c.c_uint64, c.c_int64, c.c_int]
    lib.ears_oracle_uniform_final.restype = c.c_double
    lib.ears_oracle_softmax.argtypes = [c.c_void_p, c.c_int, c.c_double, c.c_void_p,
                                        c.POINTER(c.c_double), c.POINTER(c.c_double)]
    lib.ears_oracle_softmax.restype = c.c_int
    lib.ears_oracle_inverse_cdf.argtypes = [c.c_void_p, c.c_int, c.c_double, c.c_double,
                                            c.POINTER(c.c_double), c.POINTER(c.c_double),
                                            c.POINTER(c.c_double), c.POINTER(c.c_int),
                                            c.POINTER(c.c_int)]
    lib.ears_oracle_inverse_cdf.restype = c.c_int
    lib.ears_oracle_verify.argtypes = (
        [c.c_void_p, c.c_void_p, c.c_int, c.c_void_p, c.c_int, c.c_int, c.c_int,
         c.c_float, c.c_float, c.c_uint64, c.c_uint64, c.c_int64, c.c_double]
        + [c.c_void_p] * 11 + [c.c_int])
    lib.ears_oracle_verify.restype = c.c_int
    lib.ears_oracle_verify_var.argtypes = (
        [c.c_void_p, c.c_void_p, c.c_int, c.c_void_p, c.c_int, c.c_int, c.c_int,
         c.c_float, c.c_float, c.c_void_p, c.c_void_p, c.c_int, c.c_uint64, c.c_uint64, c.c_int64, c.c_double]
        + [c.c_void_p] * 11 + [c.c_int])
    lib.ears_oracle_verify_var.restype = c.c_int
    lib.ears_oracle_verify_unc.argtypes = (
        [c.c_void_p, c.c_void_p, c.c_int, c.c_void_p, c.c_int, c.c_int, c.c_int,
         c.c_float, c.c_float, c.c_void_p, c.c_void_p, c.c_int, c.c_int, c.c_uint64, c.c_uint64, c.c_int64, c.c_double]
        + [c.c_void_p] * 12 + [c.c_int])
    lib.ears_oracle_verify_unc.restype = c.c_int
    lib.ears_oracle_entropy.argtypes = [c.c_void_p, c.c_int]
    lib.ears_oracle_entropy.restype = c.c_double
    lib.ears_oracle_entropy_uncertainty.argtypes = [c.c_double, c.c_int]
    lib.ears_oracle_entropy_uncertainty.restype = c.c_double
    lib.ears_oracle_verify_greedy.argtypes = [c.c_void_p, c.c_int, c.c_void_p, c.c_int, c.c_int, c.c_int,
                                              c.c_void_p, c.c_void_p, c.c_void_p]
    lib.ears_oracle_verify_greedy.restype = c.c_int
    lib.ears_oracle_row_softmax.argtypes = [c.c_void_p, c.c_int, c.c_int64, c.c_int, c.c_float, c.c_void_p]
    lib.ears_oracle_row_softmax.restype = c.c_int
    lib.ears_oracle_half_to_double.argtypes = [c.c_uint16]
    lib.ears_oracle_half_to_double.restype = c.c_double
    lib.ears_oracle_max_threads.argtypes = []
    lib.ears_oracle_max_threads.restype = c.c_int
    _lib = lib
    return lib


def _as_logits(a):
    """-> (contiguous numpy array, dtype code 0=fp32 / 1=bf16 bits / 2=fp16 bits)."""
    if not isinstance(a, np.ndarray):  # torch tensor on the CPU
        import torch
        a = a.detach().contiguous()
        if a.dtype == torch.bfloat16:
            return a.view(torch.int16).numpy().view(np.uint16), 1
        if a.dtype == torch.float32:
            return a.numpy(), 0
        if a.dtype == torch.float16:
            return a.view(torch.int16).numpy().view(np.uint16), 2
        raise TypeError(f"unsupported logits dtype {a.dtype}")
    a = np.ascontiguousarray(a)
    if a.dtype == np.float32:
        return a, 0
    if a.dtype == np.uint16:
        return a, 1
    if a.dtype == np.float16:
        return a.view(np.uint16), 2
    raise TypeError(f"unsupported logits dtype {a.dtype}")


def _as_tokens(x):
    if not isinstance(x, np.ndarray):
        x = x.detach().cpu().numpy()
    return np.ascontiguousarray(x, dtype=np.int32)


def philox4x32_10(ctr, key):
    lib = _load()
    c = (ctypes.c_uint32 * 4)(*[int(v) & 0xFFFFFFFF for v in ctr])
    k = (ctypes.c_uint32 * 2)(*[int(v) & 0xFFFFFFFF for v in key])
    o = (ctypes.c_uint32 * 4)()
    lib.ears_oracle_philox4x32_10(c, k, o)
    return tuple(int(v) for v in o)


def uniform_accept(seed: int, offset: int, b: int, k: int) -> float:
    return float(_load().ears_oracle_uniform_accept(seed, offset, b, k))


def uniform_final(seed: int, offset: int, b: int, K: int) -> float:
    return float(_load().ears_oracle_uniform_final(seed, offset, b, K))


def softmax(logits, T: float):
    """-> (p, m, Z) of one row; raises ValueError for a row without a softmax."""
    lib = _load()
    l = np.ascontiguousarray(logits, dtype=np.float64)
    p = np.empty_like(l)
    m, Z = ctypes.c_double(), ctypes.c_double()
    rc = lib.ears_oracle_softmax(l.ctypes.data, l.size, float(T), p.ctypes.data,
                                 ctypes.byref(m), ctypes.byref(Z))
    if rc:
        raise ValueError("row has NaN, +inf or no finite entry")
    return p, m.value, Z.value


def inverse_cdf(r, u: float, band: float = 1e-6):
    """-> dict(token, S, lo, hi, band_lo, band_hi); token -1 when S <= 0."""
    lib = _load()
    r = np.ascontiguousarray(r, dtype=np.float64)
    S, lo, hi = ctypes.c_double(), ctypes.c_double(), ctypes.c_double()
    blo, bhi = ctypes.c_int(), ctypes.c_int()
    tok = lib.ears_oracle_inverse_cdf(r.ctypes.data, r.size, float(u), float(band),
                                      ctypes.byref(S), ctypes.byref(lo), ctypes.byref(hi),
                                      ctypes.byref(blo), ctypes.byref(bhi))
    return dict(token=int(tok), S=S.value, lo=lo.value, hi=hi.value,
                band_lo=blo.value, band_hi=bhi.value)


def entropy(p) -> float:
    """Shannon entropy (nats) of a distribution."""
    p = np.ascontiguousarray(p, dtype=np.float64)
    return float(_load().ears_oracle_entropy(p.ctypes.data, p.size))


def entropy_uncertainty(H: float, V: int) -> float:
    return float(_load().ears_oracle_entropy_uncertainty(float(H), int(V)))


def row_softmax(logits, row_index: int, V: int, temperature: float):
    lib = _load()
    a, code = _as_logits(logits)
    p = np.empty(V, dtype=np.float64)
    rc = lib.ears_oracle_row_softmax(a.ctypes.data, code, int(row_index), int(V),
                                     float(temperature), p.ctypes.data)
    if rc:
        raise ValueError("row has no softmax")
    return p


def half_to_double(bits: int) -> float:
    return float(_load().ears_oracle_half_to_double(int(bits) & 0xFFFF))


def max_threads() -> int:
    return int(_load().ears_oracle_max_threads())


@dataclass
class OracleResult:
    accept_len: np.ndarray   # [B] int32
    tokens: np.ndarray       # [B,K+1] int32
    pt_tok: np.ndarray       # [B,K] float64
    pd_tok: np.ndarray       # [B,K]
    max_pt: np.ndarray       # [B,K]
    margin: np.ndarray       # [B,K]  R - max(U - Tol, 0)
    cls: np.ndarray          # [B,K] uint8: 0 reject, 1 direct, 2 pardon
    resid_mass: np.ndarray   # [B]
    cdf_margin: np.ndarray   # [B]
    band_lo: np.ndarray      # [B] int32
    band_hi: np.ndarray      # [B] int32
    entropy: np.ndarray = None   # [B,K] H(P_t) in nats, when asked for


def verify(target_logits, draft_logits, draft_tokens, temperature: float, beta: float,
           seed: int = 0, offset: int = 0, b_first: int = 0, band: float = 1e-6,
           nthreads: int = 1, seq_temperature=None, seq_beta=None,
           stop_at_first_reject: bool = False, uncertainty: str = "maxprob", want_entropy: bool = False) -> OracleResult:
    """seq_temperature / seq_beta: optional [B] float32 arrays replacing the scalars per sequence.
    stop_at_first_reject: rows after a sequence's first rejection are not read (nor validated).
    uncertainty: "maxprob" (1 - max P_t, Sec. 3.2) or "entropy" (H(P_t) / ln V, Sec. 5 item 1).
    want_entropy: also report H(P_t) per position (always reported with uncertainty="entropy")."""
    lib = _load()
    t, ct = _as_logits(target_logits)
    d, cd = _as_logits(draft_logits)
    if ct != cd:
        raise TypeError("target and draft logits must share a dtype")
    x = _as_tokens(draft_tokens)
    B, K1, V = t.shape
    K = K1 - 1
    if d.shape != (B, K, V) or x.shape != (B, K):
        raise ValueError("shape mismatch")
    acc = np.empty(B, np.int32)
    tok = np.empty((B, K + 1), np.int32)
    f = lambda *s: np.zeros(s, np.float64)
    res = OracleResult(acc, tok, f(B, K), f(B, K), f(B, K), f(B, K), np.zeros((B, K), np.uint8),
                       f(B), f(B), np.full(B, -1, np.int32), np.full(B, -1, np.int32))
    st = None if seq_temperature is None else np.ascontiguousarray(np.asarray(seq_temperature, dtype=np.float32))
    sb = None if seq_beta is None else np.ascontiguousarray(np.asarray(seq_beta, dtype=np.float32))
    if (st is not None and st.shape != (B,)) or (sb is not None and sb.shape != (B,)):
        raise ValueError("per-sequence arrays must have shape [B]")
    mode = {"maxprob": 0, "entropy": 1}[uncertainty]
    if mode == 1 or want_entropy:
        res.entropy = f(B, K)
    rc = lib.ears_oracle_verify_unc(
        t.ctypes.data, d.ctypes.data, ct, x.ctypes.data, B, K, V,
        float(temperature), float(beta), None if st is None else st.ctypes.data,
        None if sb is None else sb.ctypes.data, int(bool(stop_at_first_reject)), mode,
        int(seed), int(offset), int(b_first), float(band),
        acc.ctypes.data, tok.ctypes.data, res.pt_tok.ctypes.data, res.pd_tok.ctypes.data,
        res.max_pt.ctypes.data, res.margin.ctypes.data, res.cls.ctypes.data,
        res.resid_mass.ctypes.data, res.cdf_margin.ctypes.data,
        res.band_lo.ctypes.data, res.band_hi.ctypes.data,
        None if res.entropy is None else res.entropy.ctypes.data, int(nthreads))
    if rc:
        raise ValueError(f"ears_oracle_verify rejected its arguments (rc={rc})")
    return res


def verify_greedy(target_logits, draft_tokens):
    """The temperature -> 0 limit of the step: -> (accept_len [B], tokens [B,K+1], argmax [B,K+1])."""
    lib = _load()
    t, ct = _as_logits(target_logits)
    x = _as_tokens(draft_tokens)
    B, K1, V = t.shape
    K = K1 - 1
    if x.shape != (B, K):
        raise ValueError("shape mismatch")
    acc = np.empty(B, np.int32)
    tok = np.empty((B, K + 1), np.int32)
    am = np.empty((B, K + 1), np.int32)
    rc = lib.ears_oracle_verify_greedy(t.ctypes.data, ct, x.ctypes.data, B, K, V, acc.ctypes.data, tok.ctypes.data,
                                       am.ctypes.data)
    if rc:
        raise ValueError(f"ears_oracle_verify_greedy rejected its arguments (rc={rc})")
    return acc, tok, am
