"""GPU parity: the CUDA library (through its C ABI) against the fp64 oracle, element
by element on the same seeded inputs."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2512_13194_b200 import synth
from oracle.parity import Tally, assert_parity, compare

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def run_both(ears, w, t, d, x, T, beta, seed=0, offset=0, b_first=0, nthreads=8):
    dev = torch.device("cuda:0")
    acc, tok, st = ears.verify(t.to(dev), d.to(dev), x.to(dev), T, beta, seed, offset, b_first=b_first, stats=True)
    # the same call without the optional outputs (the resident kernel then decides in fp32 unless
    # R is close to the threshold) must give the same lengths and tokens
    acc2, tok2 = ears.verify(t.to(dev), d.to(dev), x.to(dev), T, beta, seed, offset, b_first=b_first)
    torch.cuda.synchronize()
    assert ears.last_device_status() & ears.DEV_TIMEOUT == 0
    assert torch.equal(acc, acc2) and torch.equal(tok, tok2)
    ora = oracle.verify(t.cpu(), d.cpu(), x.cpu(), T, beta, seed=seed, offset=offset, b_first=b_first,
                        nthreads=nthreads)
    stats = {k: v.cpu().numpy() for k, v in st.items()}
    tally = compare(acc.cpu().numpy(), tok.cpu().numpy(), ora, w.K, stats, inputs=(t.cpu(), d.cpu(), T))
    # the mass the final token was drawn from
    ok = ora.accept_len >= 0
    np.testing.assert_allclose(stats["resid_mass"][ok], ora.resid_mass[ok], rtol=2e-5)
    assert np.array_equal(stats["cls"][ok] != 0, ora.cls[ok] != 0) or tally.flagged_decisions > 0
    return tally, acc, tok, ora


def test_device_philox_known_answers(ears):
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            if not line.startswith("#") and line.strip():
                rows.append([int(v, 16) for v in line.split()])
    ck = torch.from_numpy(np.array([r[:6] for r in rows], dtype=np.uint32).view(np.int32)).cuda()
    out = ears.philox_device(ck).cpu().numpy().view(np.uint32)
    assert out.tolist() == [r[6:] for r in rows]
    rng = np.random.default_rng(0)
    rnd = rng.integers(0, 2**32, (4096, 6), dtype=np.uint64).astype(np.uint32)
    got = ears.philox_device(torch.from_numpy(rnd.view(np.int32)).cuda()).cpu().numpy().view(np.uint32)
    for i in range(0, 4096, 97):
        assert tuple(got[i].tolist()) == oracle.philox4x32_10(rnd[i, :4].tolist(), rnd[i, 4:].tolist())


SHAPES = [
    # B, K, V, dtype
    (1, 1, 1, "fp32"), (2, 3, 7, "fp32"), (3, 2, 8, "bf16"), (2, 2, 9, "bf16"),
    (2, 3, 1023, "fp32"), (3, 1, 1025, "bf16"), (2, 2, 4096, "fp32"), (2, 2, 4097, "fp32"),
    (2, 2, 8192, "bf16"), (1, 4, 8200, "bf16"), (4, 5, 32000, "fp32"), (3, 4, 32001, "bf16"),
    (2, 3, 70001, "fp32"), (5, 7, 50000, "bf16"), (1, 64, 515, "fp32"), (700, 2, 130, "fp32"),
    (3, 2, 8, "fp16"), (3, 1, 1025, "fp16"), (1, 4, 8200, "fp16"), (3, 4, 32001, "fp16"), (5, 7, 50000, "fp16"),
    (300, 2, 700, "fp16"),
]


# (path, cluster): 1 = streaming kernel with the shared-memory ring; 3 = streaming kernel reading straight from
# global memory; 2 = resident kernel with 1..16 CTAs per cluster (0 = automatic); 4 = the cluster-streamed kernel
# (clusters stream their slices; the second pass of a first rejection is shared out among all CTAs)
PATHS = [(1, 0), (3, 0), (2, 0), (2, 1), (2, 2), (2, 4), (2, 8), (2, 16), (4, 0), (4, 1), (4, 2), (4, 4), (4, 8), (4, 16)]


@pytest.fixture
def forced_path(ears):
    """Forces one of the two kernels for the duration of a test."""
    def force(path, cluster=0):
        ears.set_path(path, cluster)
    yield force
    ears.set_path(0, 0)


@pytest.mark.parametrize("path,cluster", PATHS)
@pytest.mark.parametrize("B,K,V,dtype", SHAPES)
def test_parity_shapes(ears, forced_path, B, K, V, dtype, path, cluster):
    """Tiny to medium cases: several chunks, ragged tails, unaligned rows (element-wise loader),
    empty slices in large clusters; under every kernel and cluster size."""
    forced_path(path, cluster)
    tally = Tally()
    for seed, (T, beta) in enumerate([(1.0, 0.0), (0.8, 0.3), (1.3, 1.0)]):
        w, t, d, x = synth.tiny_inputs(B, K, V, dtype, seed=100 + seed, temperature=T)
        try:
            tl, *_ = run_both(ears, w, t, d, x, T, beta, seed=seed, offset=7 * seed)
        except ears.EarsError as e:
            if path == 2 and cluster and e.status == -2 and 2 * V * (4 if dtype == "fp32" else 2) > 60000 * cluster:
                pytest.skip("a pair of rows does not fit a cluster of this size")
            raise
        tally.merge(tl)
    assert_parity(tally, max_explained=1)
    assert tally.max_rel_prob_err < 1e-5


@pytest.mark.parametrize("path", [0, 1, 3, 4])
@pytest.mark.parametrize("idx", [1, 2, 3, 4])
def test_parity_workloads(ears, forced_path, idx, path):
    """Workloads 1-4 at full size, in the automatic launch configuration (the resident kernel for
    workloads 1-2, the cluster-streamed kernel for workloads 3-4) and with the other kernels forced."""
    forced_path(path)
    w = synth.workload(idx)
    temps = w.temperatures or (w.temperature,)
    betas = w.betas or (w.beta,)
    tally = Tally()
    lens = []
    for T in temps:
        t, d, x = synth.make_inputs(w, "cpu", temperature=T)
        for beta in betas:
            for offset in range(3):
                tl, acc, tok, ora = run_both(ears, w, t, d, x, T, beta, seed=w.verify_seed, offset=offset)
                tally.merge(tl)
                lens.append(float(ora.accept_len.mean()))
    assert_parity(tally)
    assert tally.max_rel_prob_err < 1e-5
    print(f"\n{w.name}: rows={tally.rows} explained={tally.explained} flagged_dec={tally.flagged_decisions} "
          f"flagged_tok={tally.flagged_tokens} max_rel={tally.max_rel_prob_err:.2e} mean_len={np.mean(lens):.2f}")


@pytest.mark.parametrize("cluster", [0, 1, 2, 4])
@pytest.mark.parametrize("B,K,V,dtype,beta", [(96, 7, 20000, "bf16", 0.0), (600, 3, 9000, "fp32", 0.0), (40, 31, 3000, "bf16", 0.05),
                                              (130, 2, 70001, "fp16", 0.0)])
def test_parity_shared_second_pass(ears, forced_path, B, K, V, dtype, beta, cluster):
    """The cluster-streamed kernel with most sequences rejected somewhere and more positions than CTA
    slots: many second-pass jobs in the queue at once, pieces served between items and by CTAs that have
    run out of them, for every cluster size; K = 31 takes the path without the per-sequence word; the
    device-side counters see every sequence exactly once."""
    forced_path(4, cluster)
    w, t, d, x = synth.tiny_inputs(B, K, V, dtype, seed=77, temperature=1.1)
    tally, _, _, ora = run_both(ears, w, t, d, x, 1.1, beta, seed=5, offset=11)
    assert_parity(tally, max_explained=2)
    if beta == 0.0:
        assert (ora.accept_len < K).sum() >= B // 4   # many second-pass jobs
    got = ears.decision_counts()        # of run_both's last call (the one without the optional outputs)
    want = oracle_class_counts(ora, K)
    assert got["invalid"] == 0
    # (a decision the oracle flags as a near-tie could be classed either way; a flipped decision also
    # changes which later positions count)
    if tally.flagged_decisions == 0:
        assert got == want, (got, want)
    else:
        assert abs(sum(got.values()) - sum(want.values())) <= K * tally.flagged_decisions


@pytest.mark.parametrize("path", [0, 1, 3, 4])
@pytest.mark.parametrize("idx,B", [(2, 8), (3, 32), (4, 128), (4, 24)])
def test_parity_fp16_workload_shapes(ears, forced_path, idx, B, path):
    """The 2-byte workloads with IEEE binary16 logits instead of bfloat16 (same values before
    rounding), in the automatic launch configuration and with each streaming kernel forced."""
    from dataclasses import replace
    forced_path(path)
    w = replace(synth.workload(idx), dtype="fp16", B=B)
    t, d, x = synth.make_inputs(w, "cpu")
    assert t.dtype == torch.float16
    tally = Tally()
    for offset, beta in enumerate([w.beta, 0.0]):
        tl, *_ = run_both(ears, w, t, d, x, w.temperature, beta, seed=w.verify_seed, offset=offset)
        tally.merge(tl)
    assert_parity(tally)
    assert tally.max_rel_prob_err < 1e-5


@pytest.mark.parametrize("path", [1, 2, 3, 4])
def test_probabilities_are_tight_on_rows_far_below_their_maximum(ears, forced_path, path):
    """Rows of workload 3 (one logit 8 above the rest: every other term of Z sits near 2^-17, where
    the fp32 product l c is coarse).  A correction of the wrong sign for the rounding of m c doubled
    that error to 1e-6 and moved final tokens beyond the 1e-6 band once per million rows; the bound
    here is well below that and above what the arithmetic gives (3e-7)."""
    forced_path(path)
    w = synth.workload(3)
    t, d, x = synth.make_inputs(w, "cpu")
    tl, *_ = run_both(ears, w, t, d, x, w.temperature, w.beta, seed=w.verify_seed, offset=0)
    assert_parity(tl)
    print(f"\npath {path}: max relative probability error {tl.max_rel_prob_err:.2e}")
    assert tl.max_rel_prob_err < 7e-7


@pytest.mark.parametrize("path,V", [(0, 256000), (3, 256000), (4, 256000), (0, 131072), (3, 131072), (1, 131072)])
@pytest.mark.parametrize("beta", [1.0, 0.0])
def test_parity_largest_workload(ears, forced_path, beta, path, V):
    """Full size of the largest configuration, in the launch configuration the benchmark times
    (path 0, V = 256000: the ring kernel) and with the kernel that reads straight from global memory
    forced; and the same batch with rows of 512 KB (V = 131072), which the automatic rule gives to
    that kernel.  beta = 0 is added because at beta = 1 nearly everything is accepted and the
    residual path idles."""
    from dataclasses import replace
    forced_path(path)
    w = replace(synth.workload(5), V=V)
    plan = ears.describe_plan(w.dtype, w.B, w.K, w.V).split(":")[0]
    assert plan == {(0, 256000): "streaming", (0, 131072): "direct"}.get((path, V)) \
        or plan == {1: "streaming", 3: "direct", 4: "cluster-streamed"}.get(path)
    t, d, x = synth.make_inputs(w, "cuda:0")
    acc, tok, st = ears.verify(t, d, x, w.temperature, beta, 0, 3, stats=True)
    torch.cuda.synchronize()
    assert ears.last_device_status() == 0
    ora = oracle.verify(t.cpu(), d.cpu(), x.cpu(), w.temperature, beta, seed=0, offset=3,
                        nthreads=oracle.max_threads())
    tally = compare(acc.cpu().numpy(), tok.cpu().numpy(), ora, w.K, {k: v.cpu().numpy() for k, v in st.items()},
                    inputs=(t.cpu(), d.cpu(), w.temperature))
    # One step of 3584 rows cannot resolve a rate of 1e-4 (the soak runs over 1e6 rows do: 3-5e-5 under every
    # kernel, i.e. 0.1-0.2 expected here); what this step checks is that nothing is unexplained.
    assert_parity(tally, max_explained=3)
    assert tally.max_rel_prob_err < 1e-5
    if beta == 0.0:
        assert (ora.accept_len < w.K).mean() > 0.3
    print(f"\ncfg5 beta={beta}: explained={tally.explained} flagged_tok={tally.flagged_tokens} "
          f"max_rel={tally.max_rel_prob_err:.2e} mean_len={ora.accept_len.mean():.2f}")


def test_launch_plans_agree(ears):
    """Loader (bulk copy vs element-wise) and row splitting only change summation order."""
    w, t, d, x = synth.tiny_inputs(6, 3, 40000, "bf16", seed=5)
    try:
        results = []
        for plan in [(0, 0), (1, 1), (2, 0), (1, 3), (2, 5), (1, 1000)]:
            ears.set_plan(*plan)
            tl, acc, tok, _ = run_both(ears, w, t, d, x, 1.0, 0.2, seed=3, offset=1)
            assert_parity(tl, max_explained=1)
            results.append((acc.cpu(), tok.cpu()))
    finally:
        ears.set_plan(0, 0)
    same = sum(torch.equal(r[1], results[0][1]) for r in results)
    assert same >= len(results) - 1


def test_kernels_agree(ears, forced_path):
    """The streaming and the resident kernel (any cluster size, either loader) give the same
    accept lengths and, up to summation order at a CDF boundary, the same tokens."""
    w, t, d, x = synth.tiny_inputs(7, 4, 24000, "bf16", seed=15, noise=1.5)
    dev = "cuda:0"
    tg, dg, xg = t.to(dev), d.to(dev), x.to(dev)
    results = []
    try:
        for path, cluster, loader in [(1, 0, 0), (3, 0, 0), (3, 0, 2), (2, 0, 0), (2, 1, 0), (2, 2, 2), (2, 4, 0), (2, 8, 2), (2, 16, 0),
                                      (4, 0, 0), (4, 1, 2), (4, 2, 0), (4, 8, 2), (4, 16, 0)]:
            forced_path(path, cluster)
            ears.set_plan(loader, 0)
            acc, tok = ears.verify(tg, dg, xg, 1.0, 0.1, 4, 9)
            torch.cuda.synchronize()
            assert ears.last_device_status() == 0
            results.append((acc.cpu(), tok.cpu()))
    finally:
        ears.set_plan(0, 0)
    assert (results[0][0] < 4).any() and (results[0][0] == 4).any()    # both kinds of final token occur
    for acc, tok in results[1:]:
        assert torch.equal(acc, results[0][0])
    same = sum(torch.equal(r[1], results[0][1]) for r in results)
    assert same >= len(results) - 1


def test_forced_resident_path_refuses_rows_that_do_not_fit(ears, forced_path):
    forced_path(2)
    w, t, d, x = synth.tiny_inputs(1, 1, 600000, "fp32", seed=3)
    with pytest.raises(ears.EarsError) as e:
        ears.verify(t.cuda(), d.cuda(), x.cuda(), 1.0, 0.1, 0, 0)
    assert e.value.status == -2


@pytest.mark.parametrize("dtype", ["fp32", "fp16", "bf16"])
@pytest.mark.parametrize("path", [1, 2, 3, 4])
def test_invalid_sequences_are_marked(ears, forced_path, path, dtype):
    """Unusable data marks its own sequence and nothing else.  For the 2-byte types the NaNs sit in
    an odd and in an even lane of a packed pair (the packed maximum drops NaNs, so they must reach
    the sum), alone in a row that is otherwise ordinary, and next to the row's maximum."""
    forced_path(path)
    B, V = 13, 5000
    w, t, d, x = synth.tiny_inputs(B, 3, V, dtype, seed=9)
    t = t.clone(); d = d.clone(); x = x.clone()
    x[1, 0] = V
    x[2, 2] = -3
    t[3, 1, 77] = float("nan")        # odd lane
    d[4, 0, 4999] = float("inf")
    t[5, 3, :] = float("-inf")        # a row with nothing finite
    t[6, 2, 78] = float("nan")        # even lane
    d[7, 1, 4096] = float("nan")      # first entry of a 16-byte vector, draft row
    top = int(t[8, 0].float().argmax())
    t[8, 0, top ^ 1] = float("nan")   # the partner of the row's maximum in its packed pair
    t[9, 3, 4999] = float("inf")      # +inf in the extra row, last entry
    t[0, 0, 10:500] = float("-inf")   # masked vocabulary entries are legal
    d[0, 0, 10:500] = float("-inf")
    x[0, 0] = 5
    bad = list(range(1, 10))
    dev = "cuda:0"
    acc, tok = ears.verify(t.to(dev), d.to(dev), x.to(dev), 1.0, 0.1, 1, 2)
    torch.cuda.synchronize()
    assert ears.last_device_status() & ears.DEV_INVALID_INPUT
    ora = oracle.verify(t, d, x, 1.0, 0.1, seed=1, offset=2)
    assert ora.accept_len[bad].tolist() == [-1] * len(bad)
    assert (ora.accept_len[[0, 10, 11, 12]] >= 0).all()
    tl = compare(acc.cpu().numpy(), tok.cpu().numpy(), ora, 3, inputs=(t, d, 1.0))
    assert_parity(tl, max_explained=0)
    # the next call starts from a clean status
    acc, tok = ears.verify(t[10:].to(dev), d[10:].to(dev), x[10:].to(dev), 1.0, 0.1, 1, 2, b_first=10)
    assert ears.last_device_status() == 0
    assert torch.equal(acc.cpu(), torch.from_numpy(ora.accept_len[10:]))


def test_batch_shards_match_full_batch(ears):
    from paper_2512_13194_b200.shard import shard_range
    w, t, d, x = synth.tiny_inputs(11, 4, 9000, "bf16", seed=21)
    dev = "cuda:0"
    full_len, full_tok = ears.verify(t.to(dev), d.to(dev), x.to(dev), 0.9, 0.1, 5, 17)
    for world in (2, 3):
        for rank in range(world):
            lo, n = shard_range(11, rank, world)
            a, k = ears.verify(t[lo:lo + n].to(dev), d[lo:lo + n].to(dev), x[lo:lo + n].to(dev), 0.9, 0.1, 5, 17,
                               b_first=lo)
            assert torch.equal(a, full_len[lo:lo + n]) and torch.equal(k, full_tok[lo:lo + n])


def test_entry_points_agree(ears):
    """13-argument symbols, caller-owned workspace, a side stream and the host-buffer entry."""
    dev = "cuda:0"
    for dtype, name in (("fp32", "ears_verify_f32"), ("bf16", "ears_verify_bf16"), ("fp16", "ears_verify_f16"),
                        ("fp32", "ears_verify")):
        w, t, d, x = synth.tiny_inputs(5, 3, 12000, dtype, seed=33)
        tg, dg, xg = t.to(dev), d.to(dev), x.to(dev)
        ref_len, ref_tok = ears.verify(tg, dg, xg, 1.1, 0.2, 9, 4)
        a, k = ears.verify_abi(name, tg, dg, xg, 1.1, 0.2, 9, 4)
        assert torch.equal(a, ref_len) and torch.equal(k, ref_tok)
        ws = torch.empty(ears.workspace_bytes(5, 3, 12000) + 256, dtype=torch.uint8, device=dev)
        ws = ws[(-ws.data_ptr()) % 256:]
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            a, k = ears.verify(tg, dg, xg, 1.1, 0.2, 9, 4, workspace=ws, stream=side)
        side.synchronize()
        assert torch.equal(a, ref_len) and torch.equal(k, ref_tok)
        assert ears.workspace_device_status(ws, side) == 0
        with pytest.raises(ears.EarsError):
            ears.verify(tg, dg, xg, 1.1, 0.2, 9, 4, workspace=ws[:256])
        ha, hk = ears.verify_host(t.pin_memory(), d.pin_memory(), x.pin_memory(), 1.1, 0.2, 9, 4)
        assert torch.equal(ha, ref_len.cpu()) and torch.equal(hk, ref_tok.cpu())
        ha, hk = ears.verify_host(t, d, x, 1.1, 0.2, 9, 4)   # pageable memory works too
        assert torch.equal(ha, ref_len.cpu()) and torch.equal(hk, ref_tok.cpu())


def test_repeated_calls_are_reproducible(ears):
    w, t, d, x = synth.tiny_inputs(9, 5, 20000, "fp32", seed=44)
    dev = "cuda:0"
    tg, dg, xg = t.to(dev), d.to(dev), x.to(dev)
    first = ears.verify(tg, dg, xg, 1.0, 0.1, 1, 1)
    for _ in range(5):
        again = ears.verify(tg, dg, xg, 1.0, 0.1, 1, 1)
        assert torch.equal(again[0], first[0]) and torch.equal(again[1], first[1])
    other = ears.verify(tg, dg, xg, 1.0, 0.1, 1, 2)
    assert not torch.equal(other[1], first[1])


@pytest.mark.parametrize("B,K,V,dtype,T,beta", [
    (3, 64, 2051, "bf16", 1.0, 0.3),        # longest draft, unaligned rows, many rows per sequence
    (5000, 1, 96, "fp32", 0.9, 0.1),        # many tiny sequences: tickets and the publish queue under load
    (9, 2, 70000, "bf16", 1.0, 0.0),        # beta = 0 with a poor draft: nearly every sequence is rejected
    (9, 2, 70000, "fp32", 1.4, 50.0),       # huge tolerance: everything accepted, bonus path only
    (40, 3, 16384, "fp32", 1.0, 0.2),       # V an exact multiple of the slot size (no ragged chunk)
    (40, 3, 16385, "bf16", 1.0, 0.2),       # one element past it, unaligned
    (2, 1, 1000003, "fp32", 1.0, 0.05),     # a vocabulary of a million, unaligned: hundreds of chunks per row
])
def test_parity_extremes(ears, B, K, V, dtype, T, beta):
    """In the automatic launch configuration: the resident kernel except for the million-entry rows."""
    w, t, d, x = synth.tiny_inputs(B, K, V, dtype, seed=300 + K, noise=2.5 if beta == 0.0 else 0.5, temperature=T)
    tally = Tally()
    for offset in range(2):
        tl, acc, tok, ora = run_both(ears, w, t, d, x, T, beta, seed=11, offset=offset)
        tally.merge(tl)
    assert_parity(tally, max_explained=max(1, int(np.ceil(1e-4 * tally.rows))))
    if beta == 0.0:
        assert (ora.accept_len < K).mean() > 0.5
    if beta == 50.0:
        assert (ora.accept_len == K).all()


def test_alternating_shapes_share_one_workspace(ears):
    """Back-to-back calls of different shapes on one stream reuse (and regrow) the library's
    workspace; counters of an earlier call must never leak into the next."""
    dev = "cuda:0"
    cases = [synth.tiny_inputs(4, 3, 30000, "fp32", seed=71), synth.tiny_inputs(64, 2, 900, "bf16", seed=72),
             synth.tiny_inputs(2, 5, 130000, "bf16", seed=73)]
    gpu = [(w, t.to(dev), d.to(dev), x.to(dev)) for w, t, d, x in cases]
    first = [ears.verify(t, d, x, 1.0, 0.1, 2, 0) for _, t, d, x in gpu]
    for rep in range(3):
        for i in (2, 0, 1, 1, 0, 2):
            _, t, d, x = gpu[i]
            a, k = ears.verify(t, d, x, 1.0, 0.1, 2, 0)
            assert torch.equal(a, first[i][0]) and torch.equal(k, first[i][1])
    assert ears.last_device_status() == 0


def test_bounded_wait_gives_up_and_context_survives(ears):
    """A device-side wait that can never complete returns after its limit with the timeout status
    (no trap, no hang), and the same context keeps working."""
    import time
    t0 = time.perf_counter()
    rc = ears.selftest_bounded_wait(50)
    dt = time.perf_counter() - t0
    assert rc == -7                      # EARS_ERR_TIMEOUT: the wait gave up as designed
    assert 0.04 < dt < 1.5
    w, t, d, x = synth.tiny_inputs(3, 2, 5000, "fp32", seed=5)
    tl, *_ = run_both(ears, w, t, d, x, 1.0, 0.1)
    assert_parity(tl, max_explained=0)
    assert ears.load_library().ears_selftest_bounded_wait(0, None) == -3


@pytest.mark.parametrize("path,cluster", [(1, 0), (3, 0), (2, 0), (2, 4), (4, 0), (4, 2)])
@pytest.mark.parametrize("B,K,V,dtype", [(12, 3, 9000, "fp32"), (9, 4, 20001, "bf16"), (300, 2, 700, "bf16")])
def test_parity_per_sequence_temperature_and_beta(ears, forced_path, B, K, V, dtype, path, cluster):
    """ears_verify_var: every sequence with its own temperature and beta, against the oracle run
    with the same arrays; plus: equal entries reproduce the scalar call bit for bit, and an
    unusable entry invalidates only its own sequence."""
    forced_path(path, cluster)
    dev = "cuda:0"
    w, t, d, x = synth.tiny_inputs(B, K, V, dtype, seed=500 + K, noise=1.0)
    rng = np.random.default_rng(B)
    Ts = rng.uniform(0.5, 1.6, B).astype(np.float32)
    betas = rng.choice(np.array([0.0, 0.1, 0.3, 1.0], np.float32), B)
    tg, dg, xg = t.to(dev), d.to(dev), x.to(dev)
    Tg, bg = torch.from_numpy(Ts).to(dev), torch.from_numpy(betas).to(dev)
    tally = Tally()
    for offset in range(2):
        acc, tok, st = ears.verify(tg, dg, xg, 123.0, 456.0, 7, offset, b_first=3, stats=True, seq_temperature=Tg,
                                   seq_beta=bg)
        acc2, tok2 = ears.verify(tg, dg, xg, 123.0, 456.0, 7, offset, b_first=3, seq_temperature=Tg, seq_beta=bg)
        torch.cuda.synchronize()
        assert ears.last_device_status() == 0
        assert torch.equal(acc, acc2) and torch.equal(tok, tok2)
        ora = oracle.verify(t, d, x, 1.0, 0.0, seed=7, offset=offset, b_first=3, nthreads=8, seq_temperature=Ts,
                            seq_beta=betas)
        tally.merge(compare(acc.cpu().numpy(), tok.cpu().numpy(), ora, K, {k: v.cpu().numpy() for k, v in st.items()},
                            inputs=(t, d, Ts)))
    assert_parity(tally, max_explained=1)
    assert tally.max_rel_prob_err < 1e-5
    # equal entries == the scalar call
    ref = ears.verify(tg, dg, xg, 0.9, 0.25, 7, 1)
    same = ears.verify(tg, dg, xg, 5.0, 5.0, 7, 1, seq_temperature=torch.full((B,), 0.9, device=dev),
                       seq_beta=torch.full((B,), 0.25, device=dev))
    assert torch.equal(ref[0], same[0]) and torch.equal(ref[1], same[1])
    only_T = ears.verify(tg, dg, xg, 5.0, 0.25, 7, 1, seq_temperature=torch.full((B,), 0.9, device=dev))
    assert torch.equal(ref[0], only_T[0]) and torch.equal(ref[1], only_T[1])
    # unusable entries
    badT, badb = Ts.copy(), betas.copy()
    badT[1] = 0.0
    badT[4] = np.nan
    badb[2] = -1.0
    acc, tok = ears.verify(tg, dg, xg, 1.0, 0.0, 7, 0, b_first=3, seq_temperature=torch.from_numpy(badT).to(dev),
                           seq_beta=torch.from_numpy(badb).to(dev))
    torch.cuda.synchronize()
    assert ears.last_device_status() & ears.DEV_INVALID_INPUT
    ora = oracle.verify(t, d, x, 1.0, 0.0, seed=7, offset=0, b_first=3, nthreads=8, seq_temperature=badT, seq_beta=badb)
    assert ora.accept_len[[1, 2, 4]].tolist() == [-1, -1, -1]
    assert_parity(compare(acc.cpu().numpy(), tok.cpu().numpy(), ora, K, inputs=(t, d, np.where(np.isfinite(badT) & (badT > 0), badT, 1.0))),
                  max_explained=1)


@pytest.mark.parametrize("path", [1, 2, 3, 4])
def test_status_and_counters_start_clean_on_every_call_of_one_shape(ears, forced_path, path):
    """Calls of one shape on the library's workspace alternate between two counter blocks without
    a memset in between: a call that saw invalid input must not leak its status or counters."""
    forced_path(path)
    dev = "cuda:0"
    w, t, d, x = synth.tiny_inputs(7, 3, 6000, "fp32", seed=91)
    bad = x.clone()
    bad[2, 1] = 6000
    tg, dg, xg, bg = t.to(dev), d.to(dev), x.to(dev), bad.to(dev)
    ref = ears.verify(tg, dg, xg, 1.0, 0.2, 3, 0)
    assert ears.last_device_status() == 0
    for rep in range(4):
        a, k = ears.verify(tg, dg, bg, 1.0, 0.2, 3, 0)
        assert ears.last_device_status() == ears.DEV_INVALID_INPUT and a[2].item() == -1
        for _ in range(1 + rep % 2):       # odd and even numbers of clean calls in between
            a, k = ears.verify(tg, dg, xg, 1.0, 0.2, 3, 0)
            assert ears.last_device_status() == 0
            assert torch.equal(a, ref[0]) and torch.equal(k, ref[1])


@pytest.mark.parametrize("path,cluster", [(1, 0), (3, 0), (2, 0), (2, 2), (2, 8), (4, 0), (4, 1), (4, 4)])
@pytest.mark.parametrize("B,K,V,dtype", [(24, 4, 9000, "fp32"), (200, 3, 1500, "bf16"), (5, 6, 20001, "bf16")])
def test_parity_stop_at_first_reject(ears, forced_path, B, K, V, dtype, path, cluster):
    """EARS_FLAG_STOP_AT_FIRST_REJECT against the oracle in the same mode: same lengths and tokens
    as the full evaluation on clean data, and data planted after the first rejection (NaN, token out
    of range, a broken extra row) is ignored, while planted at the rejected position it invalidates."""
    forced_path(path, cluster)
    dev = "cuda:0"
    w, t, d, x = synth.tiny_inputs(B, K, V, dtype, seed=640 + K, noise=1.8)
    T, beta = 1.0, 0.05
    full = oracle.verify(t, d, x, T, beta, seed=4, offset=2, nthreads=8)
    n = full.accept_len
    assert (n < K).sum() >= 3
    t2, d2, x2 = t.clone(), d.clone(), x.clone()
    rej = [b for b in range(B) if n[b] < K]
    for i, b in enumerate(rej):
        if n[b] + 1 < K:
            k = int(n[b]) + 1
            if i % 3 == 0:
                t2[b, k, 3] = float("nan")
            elif i % 3 == 1:
                x2[b, k] = V + 7
            else:
                d2[b, k, :] = float("-inf")
        if i % 2 == 0:
            t2[b, K, 0] = float("inf")
    if len(rej) > 4:
        b = rej[-1]
        t2[b, int(n[b]), 1] = float("nan")      # at the rejected position: invalid in either mode
    tally = Tally()
    for tt, dd, xx in ((t, d, x), (t2, d2, x2)):
        acc, tok, st = ears.verify(tt.to(dev), dd.to(dev), xx.to(dev), T, beta, 4, 2, stats=True, stop_at_first_reject=True)
        acc2, tok2 = ears.verify(tt.to(dev), dd.to(dev), xx.to(dev), T, beta, 4, 2, stop_at_first_reject=True)
        torch.cuda.synchronize()
        assert ears.last_device_status() & ears.DEV_TIMEOUT == 0
        assert torch.equal(acc, acc2) and torch.equal(tok, tok2)
        ora = oracle.verify(tt, dd, xx, T, beta, seed=4, offset=2, nthreads=8, stop_at_first_reject=True)
        tally.merge(compare(acc.cpu().numpy(), tok.cpu().numpy(), ora, K, inputs=(tt, dd, T)))
        # per-position outputs exist up to the first rejection
        pt = st["pt_tok"].cpu().numpy()
        for b in range(B):
            if ora.accept_len[b] >= 0:
                upto = min(int(ora.accept_len[b]) + 1, K)
                np.testing.assert_allclose(pt[b, :upto], ora.pt_tok[b, :upto], rtol=1e-5, atol=1e-30)
    assert_parity(tally, max_explained=1)
    clean = ears.verify(t.to(dev), d.to(dev), x.to(dev), T, beta, 4, 2)
    stop = ears.verify(t.to(dev), d.to(dev), x.to(dev), T, beta, 4, 2, stop_at_first_reject=True)
    assert torch.equal(clean[0], stop[0]) and torch.equal(clean[1], stop[1])


def test_graph_replays_and_eager_calls_share_the_library_workspace(ears):
    """A call recorded into a CUDA graph (after a warm-up call, so nothing allocates during the
    capture) replays correctly any number of times, also interleaved with eager calls on the same
    stream: the counters of every execution start at zero."""
    dev = "cuda:0"
    w, t, d, x = synth.tiny_inputs(6, 3, 7000, "fp32", seed=17)
    tg, dg, xg = t.to(dev), d.to(dev), x.to(dev)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        ref = ears.verify(tg, dg, xg, 1.0, 0.2, 5, 3, stream=side)
        ref = ears.verify(tg, dg, xg, 1.0, 0.2, 5, 3, stream=side)
        side.synchronize()
        acc = torch.empty_like(ref[0])
        tok = torch.empty_like(ref[1])
        lib = ears.load_library()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            rc = lib.ears_verify_f32(tg.data_ptr(), dg.data_ptr(), xg.data_ptr(), 6, 3, 7000, 1.0, 0.2, 5, 3,
                                     acc.data_ptr(), tok.data_ptr(), torch.cuda.current_stream().cuda_stream)
        assert rc == 0
        cap_stream = side
    for rep in range(5):
        acc.fill_(-7)
        tok.fill_(-7)
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(acc, ref[0]) and torch.equal(tok, ref[1]), rep
        if rep % 2:
            with torch.cuda.stream(cap_stream):
                a, k = ears.verify(tg, dg, xg, 1.0, 0.2, 5, 3, stream=cap_stream)
            cap_stream.synchronize()
            assert torch.equal(a, ref[0]) and torch.equal(k, ref[1])


def test_workspace_recorded_in_a_graph_outlives_a_larger_call(ears):
    """A call recorded into a CUDA graph keeps pointing at the library's workspace of that moment.
    A later, larger call on the same stream needs a bigger workspace: the recorded one must stay
    allocated (the library parks it until shutdown), so that further replays still work."""
    dev = "cuda:0"
    w, t, d, x = synth.tiny_inputs(4, 2, 6000, "fp32", seed=23)
    wl, tl_, dl, xl = synth.tiny_inputs(40, 6, 90000, "fp32", seed=24)     # needs a much larger workspace
    assert ears.workspace_bytes(40, 6, 90000) > 4 * ears.workspace_bytes(4, 2, 6000)
    tg, dg, xg = t.to(dev), d.to(dev), x.to(dev)
    side = torch.cuda.Stream()
    lib = ears.load_library()
    with torch.cuda.stream(side):
        ref = ears.verify(tg, dg, xg, 1.0, 0.2, 5, 3, stream=side)
        side.synchronize()
        acc, tok = torch.empty_like(ref[0]), torch.empty_like(ref[1])
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            rc = lib.ears_verify_f32(tg.data_ptr(), dg.data_ptr(), xg.data_ptr(), 4, 2, 6000, 1.0, 0.2, 5, 3,
                                     acc.data_ptr(), tok.data_ptr(), torch.cuda.current_stream().cuda_stream)
        assert rc == 0
        big_ref = oracle.verify(tl_, dl, xl, 1.0, 0.2, seed=5, offset=3, nthreads=8)
        a, k = ears.verify(tl_.to(dev), dl.to(dev), xl.to(dev), 1.0, 0.2, 5, 3, stream=side)   # grows the workspace
        side.synchronize()
        assert_parity(compare(a.cpu().numpy(), k.cpu().numpy(), big_ref, 6, inputs=(tl_, dl, 1.0)), max_explained=1)
    for rep in range(3):
        acc.fill_(-7)
        tok.fill_(-7)
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(acc, ref[0]) and torch.equal(tok, ref[1]), rep
    with torch.cuda.stream(side):
        again = ears.verify(tg, dg, xg, 1.0, 0.2, 5, 3, stream=side)
    side.synchronize()
    assert torch.equal(again[0], ref[0]) and torch.equal(again[1], ref[1])
    assert ears.last_device_status(side) == 0


def oracle_class_counts(ora, K):
    want = {"direct": 0, "pardon": 0, "reject": 0, "invalid": int((ora.accept_len < 0).sum())}
    for b in range(len(ora.accept_len)):
        if ora.accept_len[b] >= 0:
            for k in range(min(int(ora.accept_len[b]) + 1, K)):
                want[("reject", "direct", "pardon")[int(ora.cls[b, k])]] += 1
    return want


def test_decision_class_counts_match_the_oracle(ears):
    """direct / pardon / reject (Sec. 3.2 step 5) counted over the decided positions, from the class output."""
    w, t, d, x = synth.tiny_inputs(64, 4, 3000, "fp32", seed=77, noise=1.2)
    acc, tok, st = ears.verify(t.cuda(), d.cuda(), x.cuda(), 1.0, 0.3, 2, 0, stats=True)
    got = ears.class_counts(st, acc)
    ora = oracle.verify(t, d, x, 1.0, 0.3, seed=2, offset=0)
    want = oracle_class_counts(ora, 4)
    want.pop("invalid")
    assert got == want and got["pardon"] > 0 and got["reject"] > 0
    assert got["reject"] == int((ora.accept_len < 4).sum())


@pytest.mark.parametrize("stop_first", [False, True])
@pytest.mark.parametrize("path,cluster", [(1, 0), (3, 0), (2, 0), (2, 4), (4, 0), (4, 2)])
def test_device_side_decision_counters(ears, forced_path, path, cluster, stop_first):
    """The counters the kernels keep themselves (no optional output asked for): direct / pardon /
    reject over what each sequence decided, and invalid sequences; with a caller workspace too; and
    every call starts them from zero."""
    forced_path(path, cluster)
    dev = "cuda:0"
    for dtype, V in (("fp32", 3000), ("bf16", 20001)):
        w, t, d, x = synth.tiny_inputs(96, 4, V, dtype, seed=78, noise=1.2)
        x = x.clone()
        x[5, 1] = V + 3
        x[17, 0] = -1
        tg, dg, xg = t.to(dev), d.to(dev), x.to(dev)
        ora = oracle.verify(t, d, x, 1.0, 0.3, seed=2, offset=0, nthreads=8, stop_at_first_reject=stop_first)
        # (a decision within 1e-5 of its threshold, or a ratio that close to U, could be classed either way)
        near = (np.abs(ora.margin) < 1e-5).any() or (np.abs(ora.pt_tok / np.maximum(ora.pd_tok, 1e-10)
                                                               - np.vectorize(lambda b, k: oracle.uniform_accept(2, 0, b, k))(
                                                                   *np.indices(ora.margin.shape))) < 1e-5).any()
        want = oracle_class_counts(ora, 4)
        for rep in range(2):
            ears.verify(tg, dg, xg, 1.0, 0.3, 2, 0, stop_at_first_reject=stop_first)
            got = ears.decision_counts()
            assert got["invalid"] == want["invalid"] >= 1
            if not near:
                assert got == want, (got, want)
            assert got["pardon"] > 0 and got["reject"] > 0
        ws = torch.empty(ears.workspace_bytes(96, 4, V) + 256, dtype=torch.uint8, device=dev)
        ws = ws[(-ws.data_ptr()) % 256:]
        ears.verify(tg, dg, xg, 1.0, 0.3, 2, 0, workspace=ws, stop_at_first_reject=stop_first)
        got_ws = ears.decision_counts(workspace=ws)
        if not near:
            assert got_ws == want
        # a clean batch afterwards: nothing left over
        ears.verify(tg[20:40], dg[20:40], xg[20:40], 1.0, 50.0, 2, 0, b_first=20, stop_at_first_reject=stop_first)
        clean = ears.decision_counts()
        assert clean["invalid"] == 0 and clean["reject"] == 0 and clean["direct"] + clean["pardon"] == 20 * 4


@pytest.mark.parametrize("path,cluster", [(1, 0), (3, 0), (2, 0), (2, 4), (4, 0), (4, 2)])
@pytest.mark.parametrize("B,K,V,dtype", [(6, 3, 9000, "fp32"), (5, 4, 20001, "bf16"), (3, 2, 70000, "fp16"), (200, 2, 700, "bf16")])
def test_parity_entropy_measure(ears, forced_path, B, K, V, dtype, path, cluster):
    """H(P_t) out of the same sweep against the oracle's (1e-5 relative, or 5e-7 absolute: H = ln Z - ...
    with Z an fp32 sum good to a few 1e-7, so that much of ln Z is the floor), and the step with H / ln V
    as the uncertainty (Sec. 5 item 1) against the oracle in the same mode; masked entries (-inf) must
    not disturb either; asking for the entropy alone leaves the printed rule's results untouched."""
    forced_path(path, cluster)
    dev = "cuda:0"
    w, t, d, x = synth.tiny_inputs(B, K, V, dtype, seed=700 + K, noise=1.2)
    t, d = t.clone(), d.clone()
    t[0, 0, 5:V // 2] = float("-inf")
    d[0, 0, 5:V // 2] = float("-inf")
    t[1 % B, 1, :] = 0.0                      # a flat row: H = ln V
    t[2 % B, K - 1, 3] += 60.0                # a (nearly) one-hot row: H ~ 0
    x = x.clone()
    x[0, 0] = 2
    tg, dg, xg = t.to(dev), d.to(dev), x.to(dev)
    tally = Tally()
    for offset, (T, beta) in enumerate([(1.0, 0.3), (0.8, 1.0), (1.4, 0.05)]):
        acc, tok, st = ears.verify(tg, dg, xg, T, beta, 9, offset, stats=True, uncertainty="entropy", entropy=True)
        acc2, tok2, st2 = ears.verify(tg, dg, xg, T, beta, 9, offset, uncertainty="entropy", entropy=True)
        torch.cuda.synchronize()
        assert ears.last_device_status() == 0
        assert torch.equal(acc, acc2) and torch.equal(tok, tok2)
        ora = oracle.verify(t, d, x, T, beta, seed=9, offset=offset, nthreads=8, uncertainty="entropy")
        tally.merge(compare(acc.cpu().numpy(), tok.cpu().numpy(), ora, K, {k: v.cpu().numpy() for k, v in st.items() if k != "entropy"},
                            inputs=(t, d, T)))
        H = st["entropy"].cpu().numpy()
        np.testing.assert_allclose(H, ora.entropy, rtol=1e-5, atol=5e-7)
        np.testing.assert_allclose(st2["entropy"].cpu().numpy(), ora.entropy, rtol=1e-5, atol=5e-7)
        assert abs(H[1 % B, 1] - np.log(V)) < 1e-5 * np.log(V)
        # the printed rule with the entropy as a by-product only
        ref = ears.verify(tg, dg, xg, T, beta, 9, offset)
        a3, k3, st3 = ears.verify(tg, dg, xg, T, beta, 9, offset, entropy=True)
        assert torch.equal(ref[0], a3) and torch.equal(ref[1], k3)
        np.testing.assert_allclose(st3["entropy"].cpu().numpy(), ora.entropy, rtol=1e-5, atol=5e-7)
    assert_parity(tally, max_explained=1)
    assert tally.max_rel_prob_err < 1e-5


def test_parity_entropy_measure_workload_rows(ears):
    """Rows of workloads 3 and 4 (peaked, flat and Zipf-shaped distributions at full vocabulary), in the
    automatic launch configuration."""
    from dataclasses import replace
    for idx, B in ((3, 32), (4, 48)):
        w = replace(synth.workload(idx), B=B)
        t, d, x = synth.make_inputs(w, "cpu")
        acc, tok, st = ears.verify(t.cuda(), d.cuda(), x.cuda(), w.temperature, w.beta, 0, 2, uncertainty="entropy", entropy=True)
        ora = oracle.verify(t, d, x, w.temperature, w.beta, seed=0, offset=2, nthreads=oracle.max_threads(), uncertainty="entropy")
        assert_parity(compare(acc.cpu().numpy(), tok.cpu().numpy(), ora, w.K, inputs=(t, d, w.temperature)))
        np.testing.assert_allclose(st["entropy"].cpu().numpy(), ora.entropy, rtol=1e-5, atol=5e-7)
