"""ctypes binding of libears.so (include/ears.h).  Argument marshalling only:
torch supplies device memory and streams, every step runs in the CUDA library.
There is no fallback: a missing library or a failing call raises."""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import build as _build

EARS_DTYPE_F32, EARS_DTYPE_BF16, EARS_DTYPE_F16 = 0, 1, 2
DEV_INVALID_INPUT, DEV_TIMEOUT = 1, 2

_lib = None


class EarsError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"ears status {status}: {message}")
        self.status = status


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """Loads (and, when sources are newer, rebuilds) the in-tree CUDA library."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    if path is None:
        path = os.environ.get("EARS_LIBRARY")      # another build of the same library (a variant under test)
    if path is None:
        path = _build.LIB
        if not os.path.exists(path):
            path = _build.build()
    lib = ctypes.CDLL(path)
    c = ctypes
    common = [c.c_void_p, c.c_void_p, c.c_void_p, c.c_int, c.c_int, c.c_int, c.c_float, c.c_float,
              c.c_uint64, c.c_uint64]
    for name in ("ears_verify_f32", "ears_verify_bf16", "ears_verify_f16", "ears_verify"):
        fn = getattr(lib, name)
        fn.argtypes = common + [c.c_void_p, c.c_void_p, c.c_void_p]
        fn.restype = c.c_int
    lib.ears_verify_ex.argtypes = ([c.c_int] + common + [c.c_int64] + [c.c_void_p] * 7
                                   + [c.c_void_p, c.c_size_t, c.c_void_p])
    lib.ears_verify_ex.restype = c.c_int
    lib.ears_verify_var.argtypes = ([c.c_int] + common[:8] + [c.c_void_p, c.c_void_p, c.c_uint] + common[8:] + [c.c_int64]
                                    + [c.c_void_p] * 7 + [c.c_void_p, c.c_size_t, c.c_void_p])
    lib.ears_verify_var.restype = c.c_int
    lib.ears_verify_entropy.argtypes = ([c.c_int] + common[:8] + [c.c_void_p, c.c_void_p, c.c_uint] + common[8:] + [c.c_int64]
                                        + [c.c_void_p] * 8 + [c.c_void_p, c.c_size_t, c.c_void_p])
    lib.ears_verify_entropy.restype = c.c_int
    lib.ears_verify_greedy.argtypes = [c.c_int, c.c_void_p, c.c_void_p, c.c_int, c.c_int, c.c_int, c.c_void_p, c.c_void_p,
                                       c.c_void_p, c.c_size_t, c.c_void_p]
    lib.ears_verify_greedy.restype = c.c_int
    lib.ears_verify_host.argtypes = [c.c_int] + common + [c.c_int64, c.c_void_p, c.c_void_p, c.c_void_p]
    lib.ears_verify_host.restype = c.c_int
    lib.ears_verify_noalloc.argtypes = [c.c_int] + common + [c.c_int64, c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p]
    lib.ears_verify_noalloc.restype = c.c_int
    shard_head = [c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_int, c.c_int, c.c_int, c.c_int, c.c_int]
    lib.ears_shard_workspace_bytes.argtypes = [c.c_int, c.c_int, c.c_int, c.c_int]
    lib.ears_shard_workspace_bytes.restype = c.c_size_t
    lib.ears_shard_stats.argtypes = shard_head + [c.c_float, c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p]
    lib.ears_shard_stats.restype = c.c_int
    lib.ears_shard_decide.argtypes = shard_head + [c.c_int, c.c_void_p, c.c_float, c.c_float, c.c_uint64, c.c_uint64,
                                                   c.c_int64, c.c_void_p, c.c_void_p, c.c_void_p,
                                                   c.c_void_p, c.c_size_t, c.c_void_p]
    lib.ears_shard_decide.restype = c.c_int
    lib.ears_shard_pick.argtypes = shard_head + [c.c_int, c.c_int, c.c_void_p, c.c_void_p, c.c_float, c.c_uint64,
                                                 c.c_uint64, c.c_int64, c.c_void_p, c.c_void_p, c.c_size_t, c.c_void_p]
    lib.ears_shard_pick.restype = c.c_int
    lib.ears_workspace_bytes.argtypes = [c.c_int, c.c_int, c.c_int]
    lib.ears_workspace_bytes.restype = c.c_size_t
    lib.ears_last_device_status.argtypes = [c.c_void_p]
    lib.ears_last_device_status.restype = c.c_int
    lib.ears_workspace_device_status.argtypes = [c.c_void_p, c.c_void_p]
    lib.ears_workspace_device_status.restype = c.c_int
    lib.ears_last_decision_counts.argtypes = [c.c_void_p, c.POINTER(c.c_uint32)]
    lib.ears_last_decision_counts.restype = c.c_int
    lib.ears_workspace_decision_counts.argtypes = [c.c_void_p, c.c_void_p, c.POINTER(c.c_uint32)]
    lib.ears_workspace_decision_counts.restype = c.c_int
    lib.ears_selftest_bounded_wait.argtypes = [c.c_int, c.c_void_p]
    lib.ears_selftest_bounded_wait.restype = c.c_int
    lib.ears_philox_device.argtypes = [c.c_void_p, c.c_void_p, c.c_int, c.c_void_p]
    lib.ears_philox_device.restype = c.c_int
    lib.ears_set_plan.argtypes = [c.c_int, c.c_int]
    lib.ears_set_plan.restype = c.c_int
    lib.ears_set_path.argtypes = [c.c_int, c.c_int]
    lib.ears_set_path.restype = c.c_int
    lib.ears_describe_plan.argtypes = [c.c_int, c.c_int, c.c_int, c.c_int, c.c_char_p, c.c_size_t]
    lib.ears_describe_plan.restype = c.c_int
    lib.ears_profile_begin.argtypes = [c.c_int]
    lib.ears_profile_begin.restype = c.c_int
    lib.ears_profile_end.argtypes = [c.c_void_p, c.c_int, c.POINTER(c.c_int)]
    lib.ears_profile_end.restype = c.c_int
    lib.ears_status_string.argtypes = [c.c_int]
    lib.ears_status_string.restype = c.c_char_p
    lib.ears_last_cuda_error.argtypes = []
    lib.ears_last_cuda_error.restype = c.c_char_p
    lib.ears_version.argtypes = []
    lib.ears_version.restype = c.c_int
    lib.ears_shutdown.argtypes = []
    lib.ears_shutdown.restype = None
    _lib = lib
    return lib


def _check(rc: int):
    if rc != 0:
        lib = load_library()
        msg = lib.ears_status_string(rc).decode()
        extra = lib.ears_last_cuda_error().decode()
        raise EarsError(rc, msg + (f" ({extra})" if extra and rc == -6 else ""))


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return EARS_DTYPE_F32
    if t.dtype == torch.bfloat16:
        return EARS_DTYPE_BF16
    if t.dtype == torch.float16:
        return EARS_DTYPE_F16
    raise TypeError(f"logits must be float32, bfloat16 or float16, got {t.dtype}")


def _shapes(target_logits, draft_logits, draft_tokens):
    if target_logits.dim() != 3 or draft_logits.dim() != 3 or draft_tokens.dim() != 2:
        raise ValueError("expected target [B,K+1,V], draft [B,K,V], tokens [B,K]")
    B, K1, V = target_logits.shape
    K = K1 - 1
    if tuple(draft_logits.shape) != (B, K, V) or tuple(draft_tokens.shape) != (B, K):
        raise ValueError("shape mismatch between target, draft and tokens")
    if draft_logits.dtype != target_logits.dtype:
        raise TypeError("target and draft logits must share a dtype")
    return B, K, V


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def verify(target_logits: torch.Tensor, draft_logits: torch.Tensor, draft_tokens: torch.Tensor,
           temperature: float, beta: float, seed: int = 0, offset: int = 0, *, b_first: int = 0,
           stats: bool = False, workspace: Optional[torch.Tensor] = None, stream=None,
           seq_temperature: Optional[torch.Tensor] = None, seq_beta: Optional[torch.Tensor] = None,
           stop_at_first_reject: bool = False, uncertainty: str = "maxprob", entropy: bool = False):
    """One EARS verification step on the current CUDA device.

    Returns (accept_len [B] int32, tokens [B,K+1] int32) and, with ``stats=True``, a dict with
    pt_tok, pd_tok, max_pt [B,K] float64, cls [B,K] uint8 and resid_mass [B] float64.
    ``uncertainty="entropy"`` scales the tolerance by H(P_t) / ln V instead of 1 - max P_t
    (EARS_FLAG_ENTROPY_UNCERTAINTY); ``entropy=True`` adds H(P_t) [B,K] float64 to the returned dict
    (which is then returned even without ``stats``).
    ``seq_temperature`` / ``seq_beta``: optional float32 CUDA tensors [B] that replace the scalar
    for each sequence (ears_verify_var).  ``stop_at_first_reject``: rows after a sequence's first
    rejection are not part of the step (EARS_FLAG_STOP_AT_FIRST_REJECT).
    The call is asynchronous on ``stream`` (default: torch's current stream).
    """
    lib = load_library()
    B, K, V = _shapes(target_logits, draft_logits, draft_tokens)
    dev = target_logits.device
    if dev.type != "cuda" or draft_logits.device != dev or draft_tokens.device != dev:
        raise ValueError("all inputs must live on the same CUDA device")
    t = target_logits.contiguous()
    d = draft_logits.contiguous()
    x = draft_tokens.to(torch.int32).contiguous()
    with torch.cuda.device(dev):
        acc = torch.empty(B, dtype=torch.int32, device=dev)
        tok = torch.empty((B, K + 1), dtype=torch.int32, device=dev)
        st = None
        ptrs = [None] * 5
        if stats:
            st = dict(pt_tok=torch.empty((B, K), dtype=torch.float64, device=dev),
                      pd_tok=torch.empty((B, K), dtype=torch.float64, device=dev),
                      max_pt=torch.empty((B, K), dtype=torch.float64, device=dev),
                      cls=torch.empty((B, K), dtype=torch.uint8, device=dev),
                      resid_mass=torch.zeros(B, dtype=torch.float64, device=dev))
            ptrs = [st[k].data_ptr() for k in ("pt_tok", "pd_tok", "max_pt", "cls", "resid_mass")]
        ws_ptr, ws_bytes = (None, 0) if workspace is None else (workspace.data_ptr(), workspace.numel() * workspace.element_size())
        if uncertainty not in ("maxprob", "entropy"):
            raise ValueError("uncertainty must be 'maxprob' or 'entropy'")
        ent = None
        if entropy:
            ent = torch.empty((B, K), dtype=torch.float64, device=dev)
            st = {} if st is None else st
            st["entropy"] = ent
        if seq_temperature is None and seq_beta is None and not stop_at_first_reject and uncertainty == "maxprob" and ent is None:
            rc = lib.ears_verify_ex(_dtype_code(t), t.data_ptr(), d.data_ptr(), x.data_ptr(), B, K, V,
                                    float(temperature), float(beta), int(seed), int(offset), int(b_first),
                                    acc.data_ptr(), tok.data_ptr(), *ptrs, ws_ptr, ws_bytes, _stream_ptr(stream))
        else:
            arrs = []
            for a in (seq_temperature, seq_beta):
                if a is not None:
                    if a.device != dev or a.dtype != torch.float32 or a.shape != (B,):
                        raise ValueError("per-sequence arrays must be float32 CUDA tensors of shape [B]")
                    a = a.contiguous()
                arrs.append(a)
            flags = (1 if stop_at_first_reject else 0) | (2 if uncertainty == "entropy" else 0)
            head = (_dtype_code(t), t.data_ptr(), d.data_ptr(), x.data_ptr(), B, K, V, float(temperature), float(beta),
                    None if arrs[0] is None else arrs[0].data_ptr(), None if arrs[1] is None else arrs[1].data_ptr(),
                    flags, int(seed), int(offset), int(b_first), acc.data_ptr(), tok.data_ptr())
            if uncertainty == "entropy" or ent is not None:
                rc = lib.ears_verify_entropy(*head, *ptrs, None if ent is None else ent.data_ptr(), ws_ptr, ws_bytes,
                                             _stream_ptr(stream))
            else:
                rc = lib.ears_verify_var(*head, *ptrs, ws_ptr, ws_bytes, _stream_ptr(stream))
    _check(rc)
    return (acc, tok, st) if st is not None else (acc, tok)


def verify_greedy(target_logits: torch.Tensor, draft_tokens: torch.Tensor, *, workspace: Optional[torch.Tensor] = None,
                  stream=None):
    """The temperature -> 0 limit of the step (ears_verify_greedy): a draft token is accepted iff it is
    the top token of its target row.  Returns (accept_len [B] int32, tokens [B,K+1] int32)."""
    lib = load_library()
    if target_logits.dim() != 3 or draft_tokens.dim() != 2:
        raise ValueError("expected target_logits [B,K+1,V] and draft_tokens [B,K]")
    B, K1, V = target_logits.shape
    K = K1 - 1
    if draft_tokens.shape != (B, K) or K < 1:
        raise ValueError("shape mismatch")
    dev = target_logits.device
    if dev.type != "cuda" or draft_tokens.device != dev:
        raise ValueError("all inputs must live on the same CUDA device")
    t = target_logits.contiguous()
    x = draft_tokens.to(torch.int32).contiguous()
    with torch.cuda.device(dev):
        acc = torch.empty(B, dtype=torch.int32, device=dev)
        tok = torch.empty((B, K + 1), dtype=torch.int32, device=dev)
        ws_ptr, ws_bytes = (None, 0) if workspace is None else (workspace.data_ptr(), workspace.numel() * workspace.element_size())
        rc = lib.ears_verify_greedy(_dtype_code(t), t.data_ptr(), x.data_ptr(), B, K, V, acc.data_ptr(), tok.data_ptr(),
                                    ws_ptr, ws_bytes, _stream_ptr(stream))
    _check(rc)
    return acc, tok


def verify_abi(name: str, target_logits, draft_logits, draft_tokens, temperature, beta, seed, offset,
               stream=None):
    """Calls one of the 13-argument entry points (ears_verify, ears_verify_f32, ears_verify_bf16, ears_verify_f16) as is."""
    lib = load_library()
    B, K, V = _shapes(target_logits, draft_logits, draft_tokens)
    dev = target_logits.device
    acc = torch.empty(B, dtype=torch.int32, device=dev)
    tok = torch.empty((B, K + 1), dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        rc = getattr(lib, name)(target_logits.data_ptr(), draft_logits.data_ptr(), draft_tokens.data_ptr(),
                                B, K, V, float(temperature), float(beta), int(seed), int(offset),
                                acc.data_ptr(), tok.data_ptr(), _stream_ptr(stream))
    _check(rc)
    return acc, tok


def verify_host(target_logits: torch.Tensor, draft_logits: torch.Tensor, draft_tokens: torch.Tensor,
                temperature: float, beta: float, seed: int = 0, offset: int = 0, *, b_first: int = 0,
                out_accept_len: Optional[torch.Tensor] = None, out_tokens: Optional[torch.Tensor] = None,
                stream=None):
    """Same step with CPU tensors (pinned memory recommended): the library copies the inputs
    to the device, runs the kernels, copies the results back and waits.  Returns CPU tensors."""
    lib = load_library()
    B, K, V = _shapes(target_logits, draft_logits, draft_tokens)
    for a in (target_logits, draft_logits, draft_tokens):
        if a.device.type != "cpu" or not a.is_contiguous():
            raise ValueError("verify_host takes contiguous CPU tensors")
    if draft_tokens.dtype != torch.int32:
        raise TypeError("draft_tokens must be int32")
    acc = out_accept_len if out_accept_len is not None else torch.empty(B, dtype=torch.int32)
    tok = out_tokens if out_tokens is not None else torch.empty((B, K + 1), dtype=torch.int32)
    rc = lib.ears_verify_host(_dtype_code(target_logits), target_logits.data_ptr(), draft_logits.data_ptr(),
                              draft_tokens.data_ptr(), B, K, V, float(temperature), float(beta), int(seed),
                              int(offset), int(b_first), acc.data_ptr(), tok.data_ptr(), _stream_ptr(stream))
    _check(rc)
    return acc, tok


NOALLOC_SCRATCH_BYTES = 8 << 20


def verify_noalloc(target_logits, draft_logits, draft_tokens, temperature, beta, seed, offset, *,
                   out_accept_len: torch.Tensor, out_tokens: torch.Tensor, b_first: int = 0,
                   out_device_status: Optional[torch.Tensor] = None, stream=None) -> None:
    """ears_verify_noalloc: the step for callers that cannot allocate device memory.

    Every buffer, outputs included, is the caller's (this wrapper creates no tensor); the
    library's scratch is a fixed array inside the library.  Shapes needing more scratch than
    NOALLOC_SCRATCH_BYTES raise EarsError(-5).  Calls that may overlap on the GPU share that
    one array and race: keep them on one stream or otherwise ordered.
    """
    lib = load_library()
    B, K, V = _shapes(target_logits, draft_logits, draft_tokens)
    for a in (target_logits, draft_logits, draft_tokens, out_accept_len, out_tokens):
        if not a.is_cuda or not a.is_contiguous():
            raise ValueError("verify_noalloc takes contiguous CUDA tensors and converts nothing")
    if draft_tokens.dtype != torch.int32 or out_accept_len.dtype != torch.int32 or out_tokens.dtype != torch.int32:
        raise TypeError("token and output tensors must be int32")
    if out_accept_len.numel() != B or tuple(out_tokens.shape) != (B, K + 1):
        raise ValueError("outputs must be [B] and [B,K+1]")
    with torch.cuda.device(target_logits.device):
        rc = lib.ears_verify_noalloc(_dtype_code(target_logits), target_logits.data_ptr(), draft_logits.data_ptr(),
                                     draft_tokens.data_ptr(), B, K, V, float(temperature), float(beta), int(seed),
                                     int(offset), int(b_first), out_accept_len.data_ptr(), out_tokens.data_ptr(),
                                     None if out_device_status is None else out_device_status.data_ptr(),
                                     _stream_ptr(stream))
    _check(rc)


def class_counts(stats: dict, accept_len: torch.Tensor) -> dict:
    """Counts of the three-way decision of Sec. 3.2 step 5 over the positions that were decided,
    i.e. up to and including each sequence's first rejection: {"direct": .., "pardon": .., "reject": ..}
    from the ``cls`` output of ``verify(..., stats=True)``."""
    cls = stats["cls"]
    B, K = cls.shape
    n = accept_len.clamp(min=-1).to(torch.int64)
    upto = torch.where(n < 0, torch.zeros_like(n), torch.clamp(n + 1, max=K))
    live = torch.arange(K, device=cls.device)[None, :] < upto[:, None]
    return {"direct": int(((cls == 1) & live).sum()), "pardon": int(((cls == 2) & live).sum()),
            "reject": int(((cls == 0) & live).sum())}


def workspace_bytes(B: int, K: int, V: int) -> int:
    return int(load_library().ears_workspace_bytes(B, K, V))


def last_device_status(stream=None) -> int:
    rc = load_library().ears_last_device_status(_stream_ptr(stream))
    if rc < 0:
        _check(rc)
    return rc


def decision_counts(stream=None, workspace: Optional[torch.Tensor] = None) -> dict:
    """Device-side counts of the three-way decision (Sec. 3.2 step 5) of the most recent call on
    ``stream`` (or on ``workspace``): {"direct", "pardon", "reject", "invalid"}; waits for the stream."""
    out = (ctypes.c_uint32 * 4)()
    lib = load_library()
    if workspace is None:
        _check(lib.ears_last_decision_counts(_stream_ptr(stream), out))
    else:
        _check(lib.ears_workspace_decision_counts(workspace.data_ptr(), _stream_ptr(stream), out))
    return {"direct": int(out[0]), "pardon": int(out[1]), "reject": int(out[2]), "invalid": int(out[3])}


def workspace_device_status(workspace: torch.Tensor, stream=None) -> int:
    rc = load_library().ears_workspace_device_status(workspace.data_ptr(), _stream_ptr(stream))
    if rc < 0:
        _check(rc)
    return rc


def selftest_bounded_wait(limit_ms: int = 50, stream=None) -> int:
    """Runs the bounded-wait self-test; returns the raw status (-7 = the wait gave up as designed)."""
    return int(load_library().ears_selftest_bounded_wait(int(limit_ms), _stream_ptr(stream)))


def philox_device(ctr_key: torch.Tensor) -> torch.Tensor:
    """ctr_key [n,6] int32/uint32 bit patterns on the GPU -> [n,4] words (int32 bit patterns)."""
    lib = load_library()
    ck = ctr_key.contiguous()
    out = torch.empty((ck.shape[0], 4), dtype=torch.int32, device=ck.device)
    with torch.cuda.device(ck.device):
        _check(lib.ears_philox_device(ck.data_ptr(), out.data_ptr(), ck.shape[0], _stream_ptr(None)))
    return out


def set_plan(loader: int = 0, parts: int = 0) -> None:
    _check(load_library().ears_set_plan(loader, parts))


class ShardStep:
    """One device's part of a verification step whose vocabulary is split across devices: the
    three local phases of ``ears_shard_stats`` / ``_decide`` / ``_pick``.  The caller exchanges the
    small results between the phases (``shard.verify_vocab_sharded`` does it with a communicator).

    target_shard [B,K+1,Vs] and draft_shard [B,K,Vs] hold columns [v_first, v_first+Vs) of a
    vocabulary of V entries; draft_tokens [B,K] int32 are ids in [0, V)."""

    def __init__(self, target_shard: torch.Tensor, draft_shard: torch.Tensor, draft_tokens: torch.Tensor,
                 v_first: int, V: int, temperature: float, beta: float, seed: int = 0, offset: int = 0,
                 b_first: int = 0):
        if not target_shard.is_cuda:
            raise RuntimeError("ears: the step runs on CUDA devices only")
        self.t, self.d, self.x = target_shard.contiguous(), draft_shard.contiguous(), draft_tokens.contiguous()
        self.B, K1, self.Vs = self.t.shape
        self.K = K1 - 1
        if self.d.shape != (self.B, self.K, self.Vs) or self.x.shape != (self.B, self.K) or self.x.dtype != torch.int32:
            raise ValueError("shape or dtype mismatch")
        if self.d.dtype != self.t.dtype:
            raise TypeError("target and draft logits must share a dtype")
        self.dtype = _dtype_code(self.t)
        self.v_first, self.V = int(v_first), int(V)
        self.T, self.beta, self.seed, self.offset, self.b_first = float(temperature), float(beta), int(seed), int(offset), int(b_first)
        self.lib = load_library()
        dev = self.t.device
        nbytes = self.lib.ears_shard_workspace_bytes(self.dtype, self.B, self.K, self.Vs)
        if nbytes == 0:
            raise EarsError(-2, "bad shape")
        self.ws = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        self.acc = torch.empty(self.B, dtype=torch.int32, device=dev)
        self.tok = torch.empty((self.B, self.K + 1), dtype=torch.int32, device=dev)

    def _head(self):
        return (self.dtype, self.t.data_ptr(), self.d.data_ptr(), self.x.data_ptr(), self.B, self.K, self.Vs, self.V,
                self.v_first)

    def _stream(self):
        return torch.cuda.current_stream(self.t.device).cuda_stream

    def stats(self) -> torch.Tensor:
        """-> [B (2K+1), 4] float32: (m, s, token logit, token column here) per row of the local columns."""
        out = torch.empty((self.B * (2 * self.K + 1), 4), dtype=torch.float32, device=self.t.device)
        with torch.cuda.device(self.t.device):
            _check(self.lib.ears_shard_stats(*self._head(), self.T, out.data_ptr(), self.ws.data_ptr(), self.ws.numel(),
                                             self._stream()))
        return out

    def decide(self, all_stats: torch.Tensor) -> torch.Tensor:
        """all_stats [n_shards, B (2K+1), 4] -> [B] float64: local mass of the row each sequence draws from."""
        all_stats = all_stats.contiguous()
        self.n_shards = int(all_stats.shape[0])
        if all_stats.shape[1:] != (self.B * (2 * self.K + 1), 4) or all_stats.dtype != torch.float32:
            raise ValueError("all_stats must be [n_shards, B (2K+1), 4] float32")
        mass = torch.empty(self.B, dtype=torch.float64, device=self.t.device)
        with torch.cuda.device(self.t.device):
            _check(self.lib.ears_shard_decide(*self._head(), self.n_shards, all_stats.data_ptr(), self.T, self.beta,
                                              self.seed, self.offset, self.b_first, self.acc.data_ptr(), self.tok.data_ptr(),
                                              mass.data_ptr(), self.ws.data_ptr(), self.ws.numel(), self._stream()))
        return mass

    def pick(self, shard: int, all_stats: torch.Tensor, all_mass: torch.Tensor):
        """-> (accept_len [B], tokens [B,K+1]); tokens[b, n] holds the drawn token only on the device
        that owns it (-1 elsewhere): an element-wise MAX over devices completes it."""
        all_stats, all_mass = all_stats.contiguous(), all_mass.contiguous()
        if all_mass.shape != (self.n_shards, self.B) or all_mass.dtype != torch.float64:
            raise ValueError("all_mass must be [n_shards, B] float64")
        with torch.cuda.device(self.t.device):
            _check(self.lib.ears_shard_pick(*self._head(), self.n_shards, int(shard), all_stats.data_ptr(),
                                            all_mass.data_ptr(), self.T, self.seed, self.offset, self.b_first,
                                            self.tok.data_ptr(), self.ws.data_ptr(), self.ws.numel(), self._stream()))
        return self.acc, self.tok


def set_path(path: int = 0, cluster: int = 0) -> None:
    """0 = automatic; path 1 streaming kernel with the shared-memory ring, 2 resident (cluster) kernel,
    3 streaming kernel reading straight from global memory, 4 cluster-streamed kernel; cluster = CTAs
    per cluster (paths 2 and 4; 0 = chosen by the library).  A forced path that cannot take a call's
    shape makes that call fail with EARS_ERR_SHAPE."""
    _check(load_library().ears_set_path(path, cluster))


def describe_plan(dtype: str, B: int, K: int, V: int) -> str:
    """The launch plan a call with these sizes would use on the current device ("fp32", "bf16" or "fp16")."""
    buf = ctypes.create_string_buffer(256)
    _check(load_library().ears_describe_plan({"fp32": 0, "bf16": 1, "fp16": 2}[dtype], B, K, V, buf, len(buf)))
    return buf.value.decode()


def profile_begin(max_calls: int) -> None:
    _check(load_library().ears_profile_begin(int(max_calls)))


def profile_end(capacity: int):
    """-> per-call device durations (ms) of the verification kernel."""
    a = (ctypes.c_float * capacity)()
    n = ctypes.c_int(0)
    _check(load_library().ears_profile_end(a, capacity, ctypes.byref(n)))
    return list(a[:n.value])


def version() -> int:
    return int(load_library().ears_version())


def shutdown() -> None:
    load_library().ears_shutdown()
