"""The allocation-free entry point (ears_verify_noalloc) against the ordinary one.

Some callers cannot allocate device memory when they verify (a thread capturing a CUDA
graph, a server that handed all memory to its own pool, a thread that must stay off the
allocator's lock).  For them the library carries a fixed scratch array; this file checks,
through the C ABI, that the step run on that array gives the same accept lengths and tokens
as the ordinary entry point, on two calls in a row (the array keeps the first call's
contents, so the second call proves that what must start at zero is cleared), and that
shapes too large for the array are refused.  It is collected last on purpose.
"""
import gc

import numpy as np
import pytest
import torch

import oracle
from oracle.parity import assert_parity, compare
from paper_2512_13194_b200 import synth

pytestmark = pytest.mark.gpu


def test_noalloc_matches_ordinary_entry_twice_in_a_row(ears):
    dev = "cuda:0"
    cases = [synth.tiny_inputs(9, 4, 24000, "fp32", seed=61), synth.tiny_inputs(5, 3, 40001, "bf16", seed=62)]
    for w, t, d, x in cases:
        tg, dg, xg = t.to(dev), d.to(dev), x.to(dev)
        acc = torch.empty(w.B, dtype=torch.int32, device=dev)
        tok = torch.empty((w.B, w.K + 1), dtype=torch.int32, device=dev)
        status = torch.full((1,), 77, dtype=torch.int32, device=dev)
        for call, (offset, beta) in enumerate([(3, 0.1), (4, 0.6)]):       # back to back, same scratch
            ref_len, ref_tok = ears.verify(tg, dg, xg, 0.9, beta, 5, offset, b_first=2)
            acc.fill_(-9)
            tok.fill_(-9)
            gc.collect()                       # tensors that earlier tests left in reference cycles go now, not mid-call
            torch.cuda.synchronize()
            before = torch.cuda.memory_allocated()
            free_before = torch.cuda.mem_get_info()[0]
            ears.verify_noalloc(tg, dg, xg, 0.9, beta, 5, offset, b_first=2, out_accept_len=acc, out_tokens=tok,
                                out_device_status=status)
            torch.cuda.synchronize()
            assert torch.cuda.memory_allocated() == before
            assert torch.cuda.mem_get_info()[0] >= free_before      # no driver-level allocation either
            assert status.item() == 0
            # same kernels, same launch plan, same inputs: bit-exact, the bar of the parity tests
            assert torch.equal(acc, ref_len), (call, acc, ref_len)
            assert torch.equal(tok, ref_tok), (call, tok, ref_tok)
            # and against the oracle, with the near-tie rules of the parity tests
            ora = oracle.verify(t, d, x, 0.9, beta, seed=5, offset=offset, b_first=2)
            assert_parity(compare(acc.cpu().numpy(), tok.cpu().numpy(), ora, w.K, inputs=(t, d, 0.9)), max_explained=1)


def test_noalloc_allocates_nothing_once_its_kernels_are_loaded(ears):
    """The first use of an element type and kernel on a device loads code (the driver allocates for
    that once); the call after it must not allocate at all.  Here the allocation-free entry point
    itself makes the first use: fp16 logits under each kernel, a warm-up call, then a measured one."""
    dev = "cuda:0"
    for path, (B, K, V) in ((2, (3, 2, 9000)), (3, (3, 2, 70000)), (1, (3, 2, 70000))):
        w, t, d, x = synth.tiny_inputs(B, K, V, "fp16", seed=64 + path)
        tg, dg, xg = t.to(dev), d.to(dev), x.to(dev)
        acc = torch.empty(B, dtype=torch.int32, device=dev)
        tok = torch.empty((B, K + 1), dtype=torch.int32, device=dev)
        ears.set_path(path, 0)
        try:
            ears.verify_noalloc(tg, dg, xg, 1.1, 0.2, 8, 1, out_accept_len=acc, out_tokens=tok)    # warm-up: loads the kernel
            gc.collect()
            torch.cuda.synchronize()
            before, free_before = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
            ears.verify_noalloc(tg, dg, xg, 1.1, 0.2, 8, 2, out_accept_len=acc, out_tokens=tok)
            torch.cuda.synchronize()
            assert torch.cuda.memory_allocated() == before
            assert torch.cuda.mem_get_info()[0] >= free_before
        finally:
            ears.set_path(0, 0)
        ora = oracle.verify(t, d, x, 1.1, 0.2, seed=8, offset=2)
        assert_parity(compare(acc.cpu().numpy(), tok.cpu().numpy(), ora, K, inputs=(t, d, 1.1)), max_explained=1)


def test_noalloc_marks_invalid_sequences_and_reports_status(ears):
    dev = "cuda:0"
    w, t, d, x = synth.tiny_inputs(4, 2, 3000, "fp32", seed=63)
    x = x.clone()
    x[1, 0] = 3000                                                      # out of range
    tg, dg, xg = t.to(dev), d.to(dev), x.to(dev)
    acc = torch.empty(4, dtype=torch.int32, device=dev)
    tok = torch.empty((4, 3), dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    ears.verify_noalloc(tg, dg, xg, 1.0, 0.1, 1, 1, out_accept_len=acc, out_tokens=tok, out_device_status=status)
    torch.cuda.synchronize()
    assert acc[1].item() == -1 and status.item() & ears.DEV_INVALID_INPUT
    ref_len, ref_tok = ears.verify(tg, dg, xg, 1.0, 0.1, 1, 1)
    assert torch.equal(acc, ref_len) and torch.equal(tok, ref_tok)


def test_noalloc_refuses_shapes_beyond_its_scratch(ears):
    dev = "cuda:0"
    B, K, V = 40000, 8, 16          # about 24 MB of per-row bookkeeping: more than the 8 MiB array
    assert ears.workspace_bytes(B, K, V) > 8 << 20
    t = torch.zeros((B, K + 1, V), device=dev)
    d = torch.zeros((B, K, V), device=dev)
    x = torch.zeros((B, K), dtype=torch.int32, device=dev)
    acc = torch.full((B,), -9, dtype=torch.int32, device=dev)
    tok = torch.full((B, K + 1), -9, dtype=torch.int32, device=dev)
    with pytest.raises(ears.EarsError) as e:
        ears.verify_noalloc(t, d, x, 1.0, 0.1, 0, 0, out_accept_len=acc, out_tokens=tok)
    assert e.value.status == -5 and "workspace" in str(e.value)
    torch.cuda.synchronize()
    assert torch.all(acc == -9)     # nothing was enqueued
