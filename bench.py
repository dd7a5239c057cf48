#!/usr/bin/env python
"""Benchmark of the EARS verification step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload 1..5]

One step = one pass of the whole hot path (statistics + decisions + first-reject scan +
final token) over one batch of synthetic logits.  The default workload is the largest
configuration (B=512, K=3, V=256000, fp32: 3.67 GB of logits, far larger than L2, so every
step streams from HBM).  With N > 1 (launched by torch.distributed.run, one rank per GPU)
each rank verifies its own batch of the same size with its global sequence offset: batch
sharding, no data-path collective, weak scaling.

Rank 0 prints ONE JSON line.  `--impl reference` times the fp64 CPU oracle instead (a
deliberately plain program) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "verify rows/s"
UNIT = "rows/s"
DATASHEET_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per sequence from one ncu capture of the named kernel on a
# small batch of the default workload (see profiles/); the traffic grows in proportion to the number
# of sequences.  Reported only while the kernel the plan names is the captured one; an entry is taken
# out (None) whenever its kernel changes after the capture.
NCU_DRAM_BYTES_PER_SEQUENCE = {
    # kernel name: (bytes per sequence, what was captured)
    "ears_verify_kernel": ((691050496 + 5236992) / 96,
                           "ncu dram__bytes_read.sum + dram__bytes_write.sum of ears_verify_kernel<float,6,false,false> on a 96-sequence "
                           "batch of this workload (profiles/ears_verify_kernel_cfg5.md), scaled by sequences"),
}


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    REASONS = {
        0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
        0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting",
        0x100: "display_clock_setting", 0x10: "sync_boost",
    }

    def __init__(self, index: int, period_s: float = 0.01):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self.trace = []          # (host time, SM MHz, reason names, watts) per sample
        self._halt = threading.Event()
        self.error = None

    def run(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM)
            while not self._halt.is_set():
                now = time.perf_counter()
                mhz = pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)
                self.samples.append(mhz)
                mask = pynvml.nvmlDeviceGetCurrentClocksEventReasons(h) if hasattr(
                    pynvml, "nvmlDeviceGetCurrentClocksEventReasons") else pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                names = tuple(name for bit, name in self.REASONS.items() if mask & bit)
                self.reasons.update(names)
                try:
                    watts = pynvml.nvmlDeviceGetPowerUsage(h) / 1000.0
                except Exception:
                    watts = None
                self.trace.append((now, mhz, names, watts))
                time.sleep(self.period)
        except Exception as e:  # NVML missing: report it rather than guess
            self.error = repr(e)

    def stop(self):
        self._halt.set()
        self.join(timeout=2)
        out = {"sm_mhz": statistics.median(self.samples) if self.samples else None,
               "sm_min_mhz": min(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}
        if self.error:
            out["error"] = self.error
        return out


def physical_gpu_index(local_index: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


def back_to_back(step, ears, gpu_index: int, n: int):
    """n steps back to back with the library's per-launch events and NVML samples beside them.
    -> (kernel_ms per launch, estimated host time of each launch, clock trace, clocks summary)."""
    import torch
    sampler = ClockSampler(gpu_index, period_s=0.004)
    sampler.start()
    time.sleep(0.03)
    ears.profile_begin(n)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for i in range(n):
        step(5000 + i)
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    kernel_ms = ears.profile_end(n)
    clocks = sampler.stop()
    # launches fill [t0, t1] in order; place each by its share of the summed kernel time
    total = sum(kernel_ms) or 1.0
    at, run = [], 0.0
    for k in kernel_ms:
        at.append(t0 + (t1 - t0) * (run + 0.5 * k) / total)
        run += k
    return kernel_ms, at, sampler.trace, clocks


def clock_at(trace, when):
    """The NVML sample nearest in time to `when` -> (MHz, reasons, watts) or None."""
    if not trace:
        return None
    import bisect
    times = [s[0] for s in trace]
    i = bisect.bisect_left(times, when)
    cand = [j for j in (i - 1, i) if 0 <= j < len(trace)]
    j = min(cand, key=lambda j: abs(times[j] - when))
    return trace[j][1:]


def bins_by_clock(kernel_ms, at, trace, logits_bytes, peak, width_mhz=50):
    """Kernel time binned by the SM clock sampled beside each launch."""
    groups = {}
    for k, when in zip(kernel_ms, at):
        c = clock_at(trace, when)
        if c is None:
            continue
        lo = int(c[0] // width_mhz) * width_mhz
        g = groups.setdefault(lo, {"ms": [], "mhz": [], "reasons": set(), "watts": []})
        g["ms"].append(k)
        g["mhz"].append(c[0])
        g["reasons"].update(c[1])
        if c[2] is not None:
            g["watts"].append(c[2])
    out = []
    for lo in sorted(groups, reverse=True):
        g = groups[lo]
        med = statistics.median(g["ms"])
        q = sorted(g["ms"])
        out.append({"sm_mhz_bin": [lo, lo + width_mhz], "launches": len(q), "kernel_us_median": med * 1e3,
                    "kernel_us_p10_p90": [q[len(q) // 10] * 1e3, q[(9 * len(q)) // 10 - (1 if len(q) >= 10 else 0)] * 1e3],
                    "gbs": logits_bytes / (med * 1e-3) / 1e9, "frac": logits_bytes / (med * 1e-3) / 1e9 / peak,
                    "us_x_mhz": med * 1e3 * statistics.median(g["mhz"]), "reasons": sorted(g["reasons"]),
                    "watts_median": statistics.median(g["watts"]) if g["watts"] else None})
    return out


def sustained(step, ears, gpu_index: int, ms_step: float, logits_bytes: int, peak: float, seconds: float = 0.6):
    """The kernel under continuous load: >= `seconds` of back-to-back steps appended after the timed
    region; the figure is the mean over the last half, with the clocks sampled during that half."""
    n = int(min(60000, max(100, seconds * 1e3 / max(ms_step, 1e-3))))
    kernel_ms, at, trace, _ = back_to_back(step, ears, gpu_index, n)
    half = kernel_ms[len(kernel_ms) // 2:]
    t_half = at[len(at) // 2]
    late = [s for s in trace if s[0] >= t_half]
    k = statistics.fmean(half)
    gbs = logits_bytes / (k * 1e-3) / 1e9
    return {"kernel_ms": k, "achieved": gbs, "frac": gbs / peak, "launches": n,
            "seconds": sum(kernel_ms) * 1e-3, "over": "last half of the launches",
            "clocks": {"sm_mhz": statistics.median(s[1] for s in late) if late else None,
                       "sm_min_mhz": min((s[1] for s in late), default=None),
                       "reasons": sorted({r for s in late for r in s[2]}), "samples": len(late)}}


def config_of(w, world: int) -> dict:
    """The workload as both arms of the benchmark report it."""
    return {"workload": w.name, "B_per_gpu": w.B, "K": w.K, "V": w.V, "logits_dtype": w.dtype,
            "temperature": w.temperature, "beta": w.beta, "parallelism": f"batch-shard x{world}",
            "l2": "inputs exceed L2 several times over; no flush needed" if w.logit_bytes > 512e6
                  else "inputs fit L2: warm-cache number"}


def final_token_bytes(accept_len, K: int, V: int, esize: int):
    """-> (formula, read_again).  formula: the workload's byte count for the final token (two rows
    after a rejection, one row for a bonus token).  read_again: what the kernel really streams a
    second time (only the two rows of a rejected position; the bonus row's sums are kept from the
    first pass), mostly out of L2."""
    n = accept_len[accept_len >= 0]
    rej, acc = (n < K).sum().item(), (n >= K).sum().item()
    return int((rej * 2 + acc) * V * esize), int(rej * 2 * V * esize)


def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2512_13194_b200 as ears
    from paper_2512_13194_b200 import synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}: launch with torch.distributed.run")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the verification step has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    ears.load_library()

    w = synth.workload(args.workload)
    if args.batch:
        w = w.with_batch(args.batch)
    # every rank holds a batch of the configured size; rank r owns global sequences [r*B, (r+1)*B)
    wr = w if world == 1 else dataclasses.replace(w, data_seed=w.data_seed + 7919 * rank)
    t, d, x = synth.make_inputs(wr, dev)
    b_first = rank * w.B
    K, V, esize = w.K, w.V, w.elem_bytes
    stream = torch.cuda.current_stream()

    def step(i):
        return ears.verify(t, d, x, w.temperature, w.beta, w.verify_seed, i, b_first=b_first)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(args.warmup, 3)):
        acc, tok = step(i)
    barrier()
    if ears.last_device_status() != 0:
        raise SystemExit("device status not clean after warm-up")

    sampler = ClockSampler(physical_gpu_index(local)) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.05)
    ears.profile_begin(args.steps)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for i in range(args.steps):
        acc, tok = step(1000 + i)
    e1.record(stream)
    barrier()
    ms_total = e0.elapsed_time(e1)
    kernel_ms = ears.profile_end(args.steps)
    clocks = sampler.stop() if sampler else None
    if ears.last_device_status() != 0:
        raise SystemExit("device status not clean after the timed region")

    ms = torch.tensor([ms_total], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    ms_step = ms.item() / args.steps
    rows_total = w.rows * world
    value = rows_total / (ms_step * 1e-3)

    logits_bytes = w.logit_bytes
    rs_formula, rs_again = final_token_bytes(acc, K, V, esize)
    step_bytes = logits_bytes + rs_formula
    k_avg = statistics.fmean(kernel_ms)
    plan = ears.describe_plan(w.dtype, w.B, K, V)
    kernel_name = {"resident": "ears_resident_kernel", "direct": "ears_direct_kernel",
                   "cluster-streamed": "ears_cstream_kernel"}.get(plan.split(":")[0], "ears_verify_kernel")
    if kernel_name == "ears_resident_kernel":
        rs_again = 0     # the rows of a position stay in shared memory until its token is drawn
    peak, peak_kind = measured_peak()
    # algorithmic HBM bytes of the kernel: every logit once.  The rows of the final token are a second
    # pass over bytes already counted (normally served by L2), so they are left out of the roofline.
    achieved = logits_bytes / (k_avg * 1e-3) / 1e9
    # the same kernel under continuous load (the timed region above may be too short for the power
    # management of the device to settle)
    sus = None
    if rank == 0 and world == 1 and not args.no_sustained:
        sus = sustained(step, ears, physical_gpu_index(local), ms_step, logits_bytes, peak)
    captured = NCU_DRAM_BYTES_PER_SEQUENCE.get(kernel_name) if args.workload == 5 else None

    # end to end through the host-buffer entry point: H2D of the inputs and D2H of the results every step
    th, dh, xh = (a.cpu().pin_memory() for a in (t, d, x))
    out_len = torch.empty(w.B, dtype=torch.int32).pin_memory()
    out_tok = torch.empty((w.B, K + 1), dtype=torch.int32).pin_memory()
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    ears.verify_host(th, dh, xh, w.temperature, w.beta, w.verify_seed, 0, b_first=b_first,
                     out_accept_len=out_len, out_tokens=out_tok)
    barrier()
    t0 = time.perf_counter()
    for i in range(e2e_steps):
        ears.verify_host(th, dh, xh, w.temperature, w.beta, w.verify_seed, 1000 + i, b_first=b_first,
                         out_accept_len=out_len, out_tokens=out_tok)
    torch.cuda.synchronize()
    e2e_s = torch.tensor([time.perf_counter() - t0], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(e2e_s, op=dist.ReduceOp.MAX)
    e2e_value = rows_total / (e2e_s.item() / e2e_steps)
    h2d = th.numel() * th.element_size() + dh.numel() * dh.element_size() + xh.numel() * 4
    d2h = out_len.numel() * 4 + out_tok.numel() * 4
    chk_len, chk_tok = step(1000 + e2e_steps - 1)
    assert torch.equal(out_len, chk_len.cpu()) and torch.equal(out_tok, chk_tok.cpu()), \
        "host entry disagrees with device entry"

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(w, th, dh, xh, args.cpu_sample)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": config_of(w, world),
            "mean_accept_len": float(acc.float().mean().item()), "launch_plan": plan,
            "gbs_step_formula": step_bytes / (ms_step * 1e-3) / 1e9,
            "bytes_per_step": {"logits": logits_bytes, "final_token_rows_formula": rs_formula,
                               "final_token_rows_streamed_again": rs_again},
            "kernel_ms": {kernel_name: k_avg, "median": statistics.median(kernel_ms), "min": min(kernel_ms)},
            "roofline": {"bound": "hbm", "kernel": kernel_name, "achieved": achieved, "peak": peak,
                         "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                         "frac_of_datasheet_8000": achieved / DATASHEET_HBM_GBS,
                         "traffic": captured[0] * w.B if captured else None,
                         "traffic_note": (captured[1] if captured else
                                          "no ncu capture of this kernel since it last changed"),
                         "sustained": sus},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps},
            "gpu_launches": args.steps,
            "clocks": clocks,
        }
        if cpu:
            line["cpu_baseline"] = cpu
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def cpu_baseline(w, th, dh, xh, sample: int):
    """The oracle as it stands on the host cores, on the first `sample` sequences of the workload."""
    import oracle
    n = min(sample, w.B)
    cores = min(oracle.max_threads(), len(os.sched_getaffinity(0)))
    t0 = time.perf_counter()
    oracle.verify(th[:n], dh[:n], xh[:n], w.temperature, w.beta, seed=w.verify_seed, offset=1000, nthreads=cores)
    dt = time.perf_counter() - t0
    return {"value": n * (2 * w.K + 1) / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {n} of {w.B} sequences of {w.name}, one step, {dt:.2f} s wall"}


def run_reference(args):
    """The fp64 oracle on the host cores; each step verifies a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2512_13194_b200 import synth
    w = synth.workload(args.workload)
    if args.batch:
        w = w.with_batch(args.batch)
    cores = min(oracle.max_threads(), len(os.sched_getaffinity(0)))
    warm = max(args.warmup, 1)
    # size the per-step sample so that (steps + warm-up) oracle calls take about two minutes
    probe_w = w.with_batch(min(w.B, 16))
    t, d, x = synth.make_inputs(probe_w, "cpu")
    t0 = time.perf_counter()
    oracle.verify(t, d, x, w.temperature, w.beta, seed=w.verify_seed, offset=0, nthreads=cores)
    per_seq = (time.perf_counter() - t0) / probe_w.B
    budget = 120.0 / (args.steps + warm)
    n = int(max(1, min(w.B, budget / max(per_seq, 1e-9))))
    if n > probe_w.B:
        n = (n // 16) * 16 or n
        t, d, x = synth.make_inputs(w.with_batch(n), "cpu")
    else:
        t, d, x = t[:n], d[:n], x[:n]
    for i in range(warm):
        oracle.verify(t, d, x, w.temperature, w.beta, seed=w.verify_seed, offset=i, nthreads=cores)
    t0 = time.perf_counter()
    for i in range(args.steps):
        oracle.verify(t, d, x, w.temperature, w.beta, seed=w.verify_seed, offset=1000 + i, nthreads=cores)
    dt = (time.perf_counter() - t0) / args.steps
    value = n * (2 * w.K + 1) / dt
    sample = f"first {n} of {w.B} sequences of {w.name} per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": warm, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(w, args.gpus),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }), flush=True)


def run_table(args):
    """All five workloads (with the sweep of workload 2) on one GPU: a markdown table of device
    times (cold = L2 flushed before every step, warm = back to back), throughput against the HBM
    roofline, oracle times on the host and the GPU-vs-oracle comparison.  Not the benchmark line."""
    import numpy as np
    import torch

    import oracle
    import paper_2512_13194_b200 as ears
    from paper_2512_13194_b200 import synth
    from oracle.parity import compare

    torch.cuda.set_device(0)
    ears.load_library()
    peak, peak_kind = measured_peak()
    cores = min(oracle.max_threads(), len(os.sched_getaffinity(0)))
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")   # > 4 x L2
    stream = torch.cuda.current_stream()

    def timed(fn, n, cold):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        for a, b in ev:
            if cold:
                flush.zero_()
            a.record(stream)
            fn()
            b.record(stream)
        torch.cuda.synchronize()
        return statistics.median(a.elapsed_time(b) for a, b in ev) * 1e3   # us

    print(f"| cfg | B | K | V | dtype | T | beta | mean accept_len | GPU us/step (cold / warm L2) | rows/s (cold) | "
          f"GB/s logits (cold) | % of {peak:.0f} ({peak_kind}) | % of 8000 | oracle s (1 thread) | "
          f"oracle s ({cores} threads) | disagreements / rows (explained / unexplained) | max rel. prob. error |")
    print("|" + "---|" * 17)
    for idx in range(1, 6):
        w = synth.workload(idx)
        for T in (w.temperatures or (w.temperature,)):
            t, d, x = synth.make_inputs(w, "cuda:0", temperature=T)
            th, dh, xh = t.cpu(), d.cpu(), x.cpu()
            for beta in (w.betas or (w.beta,)):
                run = lambda off=0: ears.verify(t, d, x, T, beta, w.verify_seed, off)
                for i in range(5):
                    run(i)
                n = 30 if idx == 5 else 100
                cold, warm = timed(run, n, True), timed(run, n, False)
                acc, tok, st = ears.verify(t, d, x, T, beta, w.verify_seed, 7, stats=True)
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                ora = oracle.verify(th, dh, xh, T, beta, seed=w.verify_seed, offset=7, nthreads=cores)
                o_n = time.perf_counter() - t0
                if idx < 5 or args.table_full:
                    t0 = time.perf_counter()
                    oracle.verify(th, dh, xh, T, beta, seed=w.verify_seed, offset=7, nthreads=1)
                    o_1 = f"{time.perf_counter() - t0:.3f}"
                else:
                    o_1 = f"~{o_n * cores:.1f} (threads x wall)"
                tl = compare(acc.cpu().numpy(), tok.cpu().numpy(), ora, w.K, {k: v.cpu().numpy() for k, v in st.items()},
                             inputs=(th, dh, T))
                gbs = w.logit_bytes / (cold * 1e-6) / 1e9
                print(f"| {idx} | {w.B} | {w.K} | {w.V} | {w.dtype} | {T} | {beta} | {float(ora.accept_len.mean()):.2f} | "
                      f"{cold:.1f} / {warm:.1f} | {w.rows / (cold * 1e-6):.3g} | {gbs:.0f} | {100 * gbs / peak:.1f} | "
                      f"{100 * gbs / DATASHEET_HBM_GBS:.1f} | {o_1} | {o_n:.3f} | {tl.explained + len(tl.unexplained)} / {tl.rows} "
                      f"({tl.explained} / {len(tl.unexplained)}) | {tl.max_rel_prob_err:.1e} |", flush=True)
            del t, d, x


def run_series(args):
    """The kernel under continuous load: --series N steps back to back on one GPU (N >= 1000 for the
    default workload keeps the device busy for more than half a second), the library's events around
    every launch, NVML sampled beside them.  Prints kernel time by position in the series and by
    sampled SM clock, and one JSON line with the bins.  Not the benchmark line."""
    import torch

    import paper_2512_13194_b200 as ears
    from paper_2512_13194_b200 import synth

    torch.cuda.set_device(0)
    ears.load_library()
    w = synth.workload(args.workload)
    if args.batch:
        w = w.with_batch(args.batch)
    t, d, x = synth.make_inputs(w, "cuda:0")
    peak, peak_kind = measured_peak()
    step = lambda i: ears.verify(t, d, x, w.temperature, w.beta, w.verify_seed, i)
    for i in range(max(args.warmup, 3)):
        step(i)
    torch.cuda.synchronize()
    time.sleep(0.5)      # let the device idle first: the series then shows the change of state from its start
    n = min(args.series, 60000)
    kernel_ms, at, trace, clocks = back_to_back(step, ears, physical_gpu_index(0), n)
    plan = ears.describe_plan(w.dtype, w.B, w.K, w.V)
    print(f"# {w.name}: {n} launches back to back, {sum(kernel_ms) * 1e-3:.2f} s of kernel time; plan: {plan}")
    print(f"# peak for the fractions: {peak:.1f} GB/s ({peak_kind})")
    print("| launches | kernel us (median) | GB/s | of peak | SM MHz beside (median) | reasons | W |")
    print("|---|---|---|---|---|---|---|")
    edges = sorted({0, 20, 50, 100, 200, 400, 800, 1600, 3200, 6400, 12800, 25600, n} & set(range(n + 1)) | {n})
    for a, b in zip(edges[:-1], edges[1:]):
        seg = kernel_ms[a:b]
        if not seg:
            continue
        med = statistics.median(seg)
        cs = [c for c in (clock_at(trace, when) for when in at[a:b]) if c]
        mhz = statistics.median(c[0] for c in cs) if cs else float("nan")
        reasons = sorted({r for c in cs for r in c[1]})
        watts = [c[2] for c in cs if c[2] is not None]
        gbs = w.logit_bytes / (med * 1e-3) / 1e9
        print(f"| {a + 1}-{b} | {med * 1e3:.1f} | {gbs:.0f} | {gbs / peak:.3f} | {mhz:.0f} | {','.join(reasons) or '-'} | "
              f"{statistics.median(watts) if watts else float('nan'):.0f} |")
    bins = bins_by_clock(kernel_ms, at, trace, w.logit_bytes, peak)
    print()
    print("| SM MHz bin | launches | kernel us median (p10-p90) | GB/s | of peak | us x MHz | reasons | W |")
    print("|---|---|---|---|---|---|---|---|")
    for b in bins:
        print(f"| {b['sm_mhz_bin'][0]}-{b['sm_mhz_bin'][1]} | {b['launches']} | {b['kernel_us_median']:.1f} "
              f"({b['kernel_us_p10_p90'][0]:.1f}-{b['kernel_us_p10_p90'][1]:.1f}) | {b['gbs']:.0f} | {b['frac']:.3f} | "
              f"{b['us_x_mhz']:.3g} | {','.join(b['reasons']) or '-'} | {b['watts_median'] or float('nan'):.0f} |")
    half = kernel_ms[n // 2:]
    k = statistics.fmean(half)
    print(json.dumps({"series": n, "workload": w.name, "plan": plan, "kernel_ms_first_20": statistics.fmean(kernel_ms[:20]),
                      "kernel_ms_last_half": k, "frac_last_half": w.logit_bytes / (k * 1e-3) / 1e9 / peak,
                      "peak": peak, "peak_kind": peak_kind, "clocks": clocks, "bins": bins}), flush=True)


def run_timeline(args):
    """Where one launch spends its time: builds (if needed) and loads the timeline variant of the
    library (-DEARS_TRACE, paper_2512_13194_b200/build.py --trace), runs one step of the chosen
    workload after an L2 flush and prints what the first CTAs recorded at the ends of their phases.
    Only the cluster kernel (resident and streamed forms) carries marks.  Not the benchmark line."""
    import ctypes

    import torch

    from paper_2512_13194_b200 import binding, build as ears_build, synth

    lib = binding.load_library(ears_build.build(trace=True))
    import paper_2512_13194_b200 as ears
    torch.cuda.set_device(0)
    w = synth.workload(args.workload)
    if args.batch:
        w = w.with_batch(args.batch)
    t, d, x = synth.make_inputs(w, "cuda:0")
    beta = w.beta if args.beta is None else args.beta
    ears.set_path(args.path, args.cluster)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    for i in range(3):
        ears.verify(t, d, x, w.temperature, beta, w.verify_seed, i, stop_at_first_reject=args.stop_first)
    torch.cuda.synchronize()
    flush.zero_()
    torch.cuda.synchronize()
    assert lib.ears_trace_reset() == 0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    acc, _ = ears.verify(t, d, x, w.temperature, beta, w.verify_seed, 7, stop_at_first_reject=args.stop_first)
    e1.record()
    torch.cuda.synchronize()
    n_ctas, n_ev = ctypes.c_int(), ctypes.c_int()
    buf = (ctypes.c_uint64 * (96 * 192 * 2))()
    counts = (ctypes.c_int * 96)()
    assert lib.ears_trace_read(buf, counts, ctypes.byref(n_ctas), ctypes.byref(n_ev)) == 0
    names = {0: "start", 1: "item", 2: "stats", 3: "exchange", 4: "decision", 5: "masses+pick", 6: "exit", 7: "job",
             10: "unit-chosen", 11: "piece-chosen", 12: "idle-chosen", 13: "exit-chosen", 15: "streamed", 16: "epilogue"}
    print(f"# {w.name} beta={beta}: {ears.describe_plan(w.dtype, w.B, w.K, w.V)}; event-timed {e0.elapsed_time(e1) * 1e3:.1f} us; "
          f"rejected sequences {float((acc < w.K).float().mean()):.2f}")
    ev = {}
    for c in range(n_ctas.value):
        ev[c] = [(buf[(c * n_ev.value + i) * 2], buf[(c * n_ev.value + i) * 2 + 1] >> 32, buf[(c * n_ev.value + i) * 2 + 1] & 0xffffffff)
                 for i in range(min(counts[c], n_ev.value))]
    t0 = min(e[0][0] for e in ev.values() if e)
    t_end = max(e[-1][0] for e in ev.values() if e)
    print(f"# first mark to last mark over the traced CTAs: {(t_end - t0) * 1e-3:.1f} us")
    # durations of each phase (time since the previous mark of the same CTA), over all traced CTAs
    dur = {}
    for c, e in ev.items():
        for a, b in zip(e[:-1], e[1:]):
            key = names.get(b[1], str(b[1])) + (" (none)" if b[1] == 5 and a[1] == 4 and (b[0] - a[0]) < 400 else "")
            dur.setdefault(key, []).append((b[0] - a[0]) * 1e-3)
    print("| phase (ends with this mark) | count | median us | p10 | p90 | total us per CTA |")
    print("|---|---|---|---|---|---|")
    ctas = sum(1 for e in ev.values() if e)
    for k, v in dur.items():
        v = sorted(v)
        print(f"| {k} | {len(v)} | {statistics.median(v):.2f} | {v[len(v) // 10]:.2f} | {v[(9 * len(v)) // 10 - 1 if len(v) > 9 else -1]:.2f} | {sum(v) / ctas:.1f} |")
    for c in (0, 1, n_ctas.value - 1):
        if ev.get(c):
            print(f"CTA {c}: " + " ".join(f"{names.get(tag, tag)}@{(ts - t0) * 1e-3:.1f}" + (f"[{arg}]" if tag in (1, 10) else "") for ts, tag, arg in ev[c][:40]))


def run_shard_table(args):
    """One rank's share of the vocabulary-sharded step, phase by phase, on one GPU: this rank's
    columns of every row with the synthetic distributions of the workload, the other ranks'
    statistics and masses stood in for by copies of this rank's own (same sizes; the exchanges
    themselves are not timed here).  L2 flushed before every step.  Not the benchmark line."""
    import torch

    import paper_2512_13194_b200 as ears
    from dataclasses import replace
    from paper_2512_13194_b200 import synth
    from paper_2512_13194_b200.shard import vocab_range

    torch.cuda.set_device(0)
    ears.load_library()
    peak, peak_kind = measured_peak()
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    ev = lambda: torch.cuda.Event(enable_timing=True)
    print(f"| workload | B | ranks | columns per rank | dtype | statistics us (GB/s, of {peak:.0f} {peak_kind}) | decisions + mass us "
          f"| pick us | exchanged bytes per rank |")
    print("|---|---|---|---|---|---|---|---|---|")
    cases = ((5, 512, 8), (5, 512, 2), (4, 1024, 8), (4, 128, 4), (3, 32, 2), (2, 4096, 2))
    if args.batch:   # one case (small ones for profiler captures)
        cases = ((args.workload, args.batch, args.ranks),)
    for idx, B, n in cases:
        w = replace(synth.workload(idx), B=B)
        _, Vs = vocab_range(w.V, 0, n)
        t, d, x = synth.make_inputs(replace(w, V=Vs), "cuda:0")
        step = ears.ShardStep(t, d, x, 0, w.V, w.temperature, w.beta, 0, 1)
        res = []
        for it in range(args.warmup + 9):
            flush.zero_()
            e = [ev() for _ in range(6)]
            e[0].record(); st = step.stats(); e[1].record()
            all_stats = st[None].repeat(n, 1, 1)
            all_stats[1:, :, 3] = 0          # every token claimed once
            e[2].record(); m = step.decide(all_stats); e[3].record()
            all_mass = m[None].repeat(n, 1)
            e[4].record(); step.pick(0, all_stats, all_mass); e[5].record()
            torch.cuda.synchronize()
            if it >= args.warmup:
                res.append(tuple(e[2 * i].elapsed_time(e[2 * i + 1]) * 1e3 for i in range(3)))
        res = sorted(res, key=sum)[len(res) // 2]
        nbytes = (t.numel() + d.numel()) * t.element_size()
        gbs = nbytes / res[0] / 1e3
        xbytes = B * (2 * w.K + 1) * 16 + B * 8 + B * (w.K + 1) * 4
        print(f"| {idx} | {B} | {n} | {Vs} | {w.dtype} | {res[0]:.1f} ({gbs:.0f}, {gbs / peak:.2f}) | {res[1]:.1f} | {res[2]:.1f} | {xbytes} |",
              flush=True)
        del t, d, x, step


def run_greedy_table(args):
    """The temperature -> 0 form (ears_verify_greedy: target rows only) on the five workloads' target
    rows and two larger batches, L2 flushed before every step.  Not the benchmark line."""
    import torch

    import paper_2512_13194_b200 as ears
    from dataclasses import replace
    from paper_2512_13194_b200 import synth

    torch.cuda.set_device(0)
    ears.load_library()
    peak, peak_kind = measured_peak()
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    print(f"| workload | B | dtype | target-row bytes | us per step | GB/s | of {peak:.0f} ({peak_kind}) |")
    print("|---|---|---|---|---|---|---|")
    cases = ((1, 0), (2, 0), (3, 0), (4, 0), (5, 0), (4, 1024), (2, 4096))
    if args.batch:   # one case (small ones for profiler captures)
        cases = ((args.workload, args.batch),)
    for idx, B in cases:
        w = synth.workload(idx)
        if B:
            w = replace(w, B=B)
        t, d, x = synth.make_inputs(w, "cuda:0")
        del d
        ts = []
        for it in range(args.warmup + 21):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); ears.verify_greedy(t, x); b.record()
            torch.cuda.synchronize()
            if it >= args.warmup:
                ts.append(a.elapsed_time(b) * 1e3)
        us = statistics.median(ts)
        nbytes = t.numel() * t.element_size()
        print(f"| {idx} | {w.B} | {w.dtype} | {nbytes} | {us:.1f} | {nbytes / us / 1e3:.0f} | {nbytes / us / 1e3 / peak:.2f} |", flush=True)
        del t, x


def run_early_table(args):
    """Leaving out what follows a sequence's first rejection (EARS_FLAG_STOP_AT_FIRST_REJECT) at large
    batches: the rows a step needs, and the time with the flag off and on (identical results
    required), L2 flushed before every step.  Not the benchmark line."""
    import torch

    import paper_2512_13194_b200 as ears
    from dataclasses import replace
    from paper_2512_13194_b200 import synth

    torch.cuda.set_device(0)
    ears.load_library()
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")

    def timed(fn, n=21):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        for a, b in ev:
            flush.zero_(); a.record(); fn(); b.record()
        torch.cuda.synchronize()
        return statistics.median(a.elapsed_time(b) * 1e3 for a, b in ev)

    print("| workload | B | beta | rows needed / rows | flag off: kernel, us | flag on: us |")
    print("|---|---|---|---|---|---|")
    for idx, B in ((4, 1024), (4, 256), (2, 4096), (3, 512), (5, 512)):
        w = replace(synth.workload(idx), B=B)
        t, d, x = synth.make_inputs(w, "cuda:0")
        for beta in (w.beta, 0.0):
            off = lambda: ears.verify(t, d, x, w.temperature, beta, 0, 1)
            on = lambda: ears.verify(t, d, x, w.temperature, beta, 0, 1, stop_at_first_reject=True)
            a0, t0 = off()
            p_off = ears.describe_plan(w.dtype, w.B, w.K, w.V).split(":")[0]
            a1, t1 = on()
            torch.cuda.synchronize()
            # the two calls may run different kernels: equal up to near-ties (a sanity check, not the parity test)
            assert (a0 != a1).sum() <= 2 and (t0 != t1).any(-1).sum() <= 8
            n = a0.clamp(min=0)
            need = int((2 * torch.clamp(n + 1, max=w.K) + (n == w.K)).sum())
            print(f"| {idx} | {B} | {beta} | {need} / {w.rows} ({need / w.rows:.2f}) | {p_off}, {timed(off):.1f} | {timed(on):.1f} |", flush=True)
        del t, d, x


def run_read_ceiling(args):
    """What library reductions reach on this GPU over a tensor of the benchmark workload's size
    (read-only traffic, unlike the read + write copy behind the measured peak): context for the
    roofline fraction.  Not the benchmark line."""
    import torch

    torch.cuda.set_device(0)
    peak, peak_kind = measured_peak()
    print(f"| dtype | GB | op | median ms | GB/s | of {peak:.0f} ({peak_kind}) |")
    print("|---|---|---|---|---|---|")
    for dt, n in ((torch.float32, 917504000), (torch.bfloat16, 1835008000)):
        x = torch.empty(n, dtype=dt, device="cuda").normal_()
        y = torch.empty_like(x)
        gb = x.numel() * x.element_size() / 1e9
        for name, fn, mult in (("sum (read only)", lambda: x.sum(), 1), ("max (read only)", lambda: x.max(), 1),
                               ("copy_ (read + write)", lambda: y.copy_(x), 2)):
            for _ in range(3):
                fn()
            ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(20)]
            for a, b in ev:
                a.record(); fn(); b.record()
            torch.cuda.synchronize()
            med = statistics.median(a.elapsed_time(b) for a, b in ev)
            print(f"| {str(dt).split('.')[-1]} | {gb:.2f} | {name} | {med:.3f} | {mult * gb / med * 1e3:.0f} | {mult * gb / med * 1e3 / peak:.2f} |", flush=True)
        del x, y


def run_path_table(args):
    """Every kernel forced in turn (ears_set_path) on the workloads and on larger batches of their
    shapes, L2 flushed before every step, median of 21 event-timed steps.  '-': that kernel cannot
    take the shape.  Not the benchmark line."""
    import torch

    import paper_2512_13194_b200 as ears
    from dataclasses import replace
    from paper_2512_13194_b200 import synth

    torch.cuda.set_device(0)
    ears.load_library()
    peak, peak_kind = measured_peak()
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    names = {0: "automatic", 1: "ring", 2: "resident", 3: "direct", 4: "cluster-streamed"}
    print(f"| shape | logits GB | beta | rejected sequences | automatic choice | " + " | ".join(f"{names[q]} us" for q in range(5))
          + f" | best GB/s (of {peak:.0f} {peak_kind}) |")
    print("|---|---|---|---|---|" + "---|" * 6)
    cases = ((1, 0, None), (2, 0, None), (3, 0, None), (4, 0, None), (5, 0, None), (4, 1024, 50.0), (4, 1024, None), (4, 1024, 0.0),
             (3, 512, None), (2, 4096, None), (1, 2048, None), (5, 512, 0.0),
             # between the workloads' sizes: where the automatic choice changes hands
             (1, 64, None), (2, 64, None), (2, 512, None), (3, 64, None), (3, 128, None), (3, 256, None),
             (4, 32, None), (4, 64, None), (4, 256, None), (4, 512, None), (5, 32, None), (5, 128, None))
    if args.batch:
        cases = ((args.workload, args.batch, args.beta),)
    for idx, B, beta in cases:
        w = synth.workload(idx)
        if B:
            w = replace(w, B=B)
        beta = w.beta if beta is None else beta
        t, d, x = synth.make_inputs(w, "cuda:0")
        nbytes = t.numel() * t.element_size() + d.numel() * d.element_size()
        cells, ref, best = [], None, None
        for q in range(5):
            ears.set_path(q, 0)
            try:
                acc, tok = ears.verify(t, d, x, w.temperature, beta, w.verify_seed, 1)
            except ears.EarsError:
                cells.append("-")
                continue
            torch.cuda.synchronize()
            if ref is None:
                ref = (acc, tok, ears.describe_plan(w.dtype, w.B, w.K, w.V).split(":")[0])
            else:   # every kernel must give the automatic choice's result (a sanity check, not the parity test: near-ties may differ)
                assert (acc != ref[0]).sum() <= 2 and (tok != ref[1]).any(-1).sum() <= 8
            ts = []
            for it in range(3 + 21):
                flush.zero_()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); ears.verify(t, d, x, w.temperature, beta, w.verify_seed, 1); b.record()
                torch.cuda.synchronize()
                if it >= 3:
                    ts.append(a.elapsed_time(b) * 1e3)
            us = statistics.median(ts)
            best = us if best is None else min(best, us)
            cells.append(f"{us:.1f}")
        ears.set_path(0, 0)
        rej = int((ref[0] < w.K).sum())
        print(f"| workload {idx} at B={w.B} | {nbytes / 1e9:.3f} | {beta} | {rej} | {ref[2]} | " + " | ".join(cells)
              + f" | {nbytes / best / 1e3:.0f} ({nbytes / best / 1e3 / peak:.2f}) |", flush=True)
        del t, d, x


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", type=int, default=5, help="1..5; the default is the largest configuration")
    ap.add_argument("--batch", type=int, default=0, help="override B (smaller cases for profiler captures)")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--cpu-sample", type=int, default=512, help="sequences given to the CPU baseline")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sustained", action="store_true", help="skip the appended run under continuous load")
    ap.add_argument("--timeline", action="store_true", help="print where one launch spends its time (timeline build) instead")
    ap.add_argument("--path", type=int, default=0, help="with --timeline: force a kernel (ears_set_path)")
    ap.add_argument("--cluster", type=int, default=0, help="with --timeline: CTAs per cluster")
    ap.add_argument("--beta", type=float, default=None, help="with --timeline: override the workload's beta")
    ap.add_argument("--stop-first", action="store_true", help="with --timeline: leave out what follows a first rejection")
    ap.add_argument("--series", type=int, default=0,
                    help="instead of the benchmark line: this many steps back to back, kernel time per launch "
                         "binned by the SM clock sampled beside it")
    ap.add_argument("--table", action="store_true", help="print the five-workload results table instead")
    ap.add_argument("--table-full", action="store_true", help="also time the 1-thread oracle on workload 5")
    ap.add_argument("--ranks", type=int, default=2, help="with --shard-table --batch: ranks the vocabulary is split over")
    ap.add_argument("--shard-table", action="store_true",
                    help="print per-phase times of one rank of the vocabulary-sharded step instead")
    ap.add_argument("--greedy-table", action="store_true", help="print times of the temperature -> 0 form instead")
    ap.add_argument("--path-table", action="store_true", help="print the time of every kernel, forced in turn, on a list of shapes instead")
    ap.add_argument("--early-table", action="store_true", help="print times with / without stopping at the first rejection instead")
    ap.add_argument("--read-ceiling", action="store_true", help="print what library reductions reach on this GPU instead")
    args = ap.parse_args()
    if args.timeline:
        run_timeline(args)
    elif args.series:
        run_series(args)
    elif args.greedy_table:
        run_greedy_table(args)
    elif args.path_table:
        run_path_table(args)
    elif args.early_table:
        run_early_table(args)
    elif args.read_ceiling:
        run_read_ceiling(args)
    elif args.shard_table:
        run_shard_table(args)
    elif args.table:
        run_table(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
