"""Long parity run (not collected by pytest): accumulates GPU-vs-oracle comparisons over many
verification steps of one workload and prints the disagreement counts.

    python tests/soak_parity.py <workload 1..5> <rows to cover> [beta] [dtype] [shards]

dtype (fp32 / bf16 / fp16) replaces the workload's element type; shards > 0 runs the
vocabulary-sharded step instead (that many column ranges, one after another on this device, the
exchanges done here).

Near-tie disagreements (explained by the oracle's margins) must stay below 1e-4 of rows; anything
unexplained is a failure.
"""
import os
import sys
from dataclasses import replace

import numpy as np
import torch

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import oracle  # noqa: E402
import paper_2512_13194_b200 as ears  # noqa: E402
from paper_2512_13194_b200 import synth  # noqa: E402
from paper_2512_13194_b200.shard import vocab_range  # noqa: E402
from oracle.parity import Tally, compare  # noqa: E402


def main():
    idx, want_rows = int(sys.argv[1]), int(float(sys.argv[2]))
    w = synth.workload(idx)
    beta = float(sys.argv[3]) if len(sys.argv) > 3 else w.beta
    if len(sys.argv) > 4:
        w = replace(w, dtype=sys.argv[4])
    shards = int(sys.argv[5]) if len(sys.argv) > 5 else 0
    t, d, x = synth.make_inputs(w, "cuda:0")
    th, dh, xh = t.cpu(), d.cpu(), x.cpu()
    tally, offset = Tally(), 0
    threads = min(oracle.max_threads(), len(os.sched_getaffinity(0)))
    parts = [vocab_range(w.V, r, shards) for r in range(shards)]
    cols = [(t[:, :, a:a + n].contiguous(), d[:, :, a:a + n].contiguous(), a) for a, n in parts]
    while shards and tally.rows < want_rows:
        steps = [ears.ShardStep(tc, dc, x, a, w.V, w.temperature, beta, w.verify_seed, offset) for tc, dc, a in cols]
        all_stats = torch.stack([s.stats() for s in steps])
        all_mass = torch.stack([s.decide(all_stats) for s in steps])
        outs = [s.pick(r, all_stats, all_mass) for r, s in enumerate(steps)]
        torch.cuda.synchronize()
        acc = outs[0][0]
        tok = torch.stack([o[1] for o in outs]).max(0).values
        assert all(torch.equal(o[0], acc) for o in outs), f"step {offset}: ranks disagree on accept lengths"
        ora = oracle.verify(th, dh, xh, w.temperature, beta, seed=w.verify_seed, offset=offset, nthreads=threads)
        tally.merge(compare(acc.cpu().numpy(), tok.cpu().numpy(), ora, w.K, inputs=(th, dh, w.temperature)))
        offset += 1
    while tally.rows < want_rows:
        acc, tok, st = ears.verify(t, d, x, w.temperature, beta, w.verify_seed, offset, stats=True)
        # without the optional outputs the resident kernel decides in fp32 away from the threshold
        acc2, tok2 = ears.verify(t, d, x, w.temperature, beta, w.verify_seed, offset)
        torch.cuda.synchronize()
        assert torch.equal(acc, acc2) and torch.equal(tok, tok2), f"step {offset}: outputs depend on stats"
        ora = oracle.verify(th, dh, xh, w.temperature, beta, seed=w.verify_seed, offset=offset, nthreads=threads)
        tally.merge(compare(acc.cpu().numpy(), tok.cpu().numpy(), ora, w.K, {k: v.cpu().numpy() for k, v in st.items()},
                            inputs=(th, dh, w.temperature)))
        offset += 1
    how = f"{shards} vocabulary shards" if shards else ears.describe_plan(w.dtype, w.B, w.K, w.V).split(':')[0] + " kernel"
    print(f"{w.name} {w.dtype} beta={beta} [{how}]: steps={offset} rows={tally.rows} sequences={tally.sequences} "
          f"explained decisions={tally.explained_decisions} tokens={tally.explained_tokens} "
          f"({tally.explained / tally.rows:.2e} of rows) unexplained={len(tally.unexplained)} "
          f"flagged decisions={tally.flagged_decisions} tokens={tally.flagged_tokens} "
          f"max rel prob err={tally.max_rel_prob_err:.2e}")
    if tally.unexplained:
        print("UNEXPLAINED:", tally.unexplained[:5])
        sys.exit(1)


if __name__ == "__main__":
    main()
