#!/usr/bin/env python
"""Benchmark of the CoS verification step.

A step is one cos_verify_run call over one synthetic batch: every (row, position) of the
workload is verified (combine, accept test, first-rejection scan, residual / bonus sample).
Prints ONE JSON line.  `value` is verified positions per second with the inputs resident in
device memory; `e2e` is the same through the host-pointer entry point (copies included);
`roofline` compares the kernel's algorithmic bytes per second with the measured copy bandwidth;
`cpu_baseline` times the float64 oracle on a bounded sample of the same workload.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg3] [--impl reference]
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2502_01662_b200 import synth  # noqa: E402
from paper_2502_01662_b200.binding import COS_RUN_EARLY_EXIT  # noqa: E402

HEADLINE = "cfg3"
# dram read + write bytes of one stage-0 launch from the ncu capture summarised under profiles/
TRAFFIC_BYTES = {"cfg3": 355332096}
FALLBACK_HBM_GBS = 6650.0
L2_BYTES = 126 * 1024 * 1024


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.samples = []

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            time.sleep(0.3)          # let the first sample land before the load starts
        except Exception:
            self.proc = None
        return self

    def __exit__(self, *exc):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=10)
        except Exception:
            self.proc.kill()
            out = ""
        for ln in out.strip().splitlines()[1:]:      # the first sample predates the load
            f = [x.strip() for x in ln.split(",")]
            try:
                self.samples.append((float(f[0]), float(f[1]), f[2:]))
            except Exception:
                pass

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({names[k] for s in self.samples for k, v in enumerate(s[2]) if v.lower().startswith("active")})
        return {"sm_mhz": float(np.median([s[0] for s in self.samples])), "sm_max_mhz": self.samples[0][1],
                "reasons": reasons, "samples": len(self.samples)}


def make_verifier(w, host_staging=False, device=0, cluster_size=0):
    from paper_2502_01662_b200 import CosVerifier
    return CosVerifier(w.n, w.combine, w.weights, w.temperature, w.gamma, w.vocab, w.batch, w.torch_dtype,
                       mask_model=w.mask_model, mask_alpha=w.mask_alpha, device=device, host_staging=host_staging,
                       cluster_size=cluster_size)


def rotating_inputs(w, device, rank):
    """Inputs whose total size exceeds L2; small workloads are replicated into distinct buffers."""
    base = synth.make_inputs(w, device)
    total = w.positions * w.bytes_per_position
    copies = 1 if total > 2 * L2_BYTES else min(256, int(np.ceil(3 * L2_BYTES / total)))
    sets = [base]
    for _ in range(copies - 1):
        sets.append(dict(base, logits=base["logits"].clone()))
    return sets


def time_device(w, verifier, sets, steps, warmup, row_base, sampler=None, flags=0):
    """K back-to-back launches between two CUDA events on the launching stream."""
    B, P, V = w.batch, w.gamma + 1, w.vocab
    dev = sets[0]["logits"].device
    outs = verifier._alloc_outs(B, P, V, dev, False, False)
    def step(k):
        s = sets[k % len(sets)]
        verifier.run(s["logits"], s["drafts"], s["proposer"], s["seed"], s["offset"] + k, row_base=row_base, outs=outs,
                     flags=flags)
    for k in range(warmup):
        step(k)
    torch.cuda.synchronize(dev)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if sampler:
        sampler.__enter__()
    # a long enough region for the clock sampler to see the load
    start.record()
    for k in range(steps):
        step(warmup + k)
    stop.record()
    torch.cuda.synchronize(dev)
    if sampler:
        sampler.__exit__()
    return start.elapsed_time(stop) / 1e3, outs


def time_e2e(w, device, steps, warmup, row_base):
    """The host-pointer call: pinned host inputs, copies in and out inside the timed region."""
    host = synth.make_inputs(w, "cpu")
    logits = host["logits"].pin_memory()
    drafts, prop = host["drafts"].pin_memory(), host["proposer"].pin_memory()
    v = make_verifier(w, host_staging=True, device=device)
    try:
        outs = v._alloc_outs(w.batch, w.gamma + 1, w.vocab, "cpu", False, False, pin=True)
        for k in range(warmup):
            v.run_host(logits, drafts, prop, host["seed"], k, row_base=row_base, outs=outs)
        torch.cuda.synchronize(device)
        t0 = time.perf_counter()
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        for k in range(steps):
            v.run_host(logits, drafts, prop, host["seed"], warmup + k, row_base=row_base, outs=outs)
        stop.record()
        torch.cuda.synchronize(device)
        wall = time.perf_counter() - t0
        dev_t = start.elapsed_time(stop) / 1e3
    finally:
        v.close()
    h2d = logits.numel() * logits.element_size() + drafts.numel() * 4 + prop.numel() * 4
    d2h = sum(t.numel() * t.element_size() for t in outs.values())
    return max(wall, dev_t), h2d, d2h


def oracle_sample(w, target_seconds=15.0, max_rows=None):
    """Times the oracle, as it stands, on the first rows of the workload (single thread):
    one row first, then as many more as fit the time budget."""
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import helpers
    made = {}
    def timed(rows, first_row):
        small = w.scaled(batch=first_row + rows, name=w.name)
        if small.batch not in made:
            made.clear()
            made[small.batch] = synth.make_inputs(small, "cpu")
        inputs = made[small.batch]
        t0 = time.perf_counter()
        helpers.run_oracle(small, inputs, rows=range(first_row, first_row + rows))
        return time.perf_counter() - t0
    t1 = timed(1, 0)
    more = int(target_seconds / t1) - 1
    more = max(0, min(more, (max_rows or w.batch) - 1, w.batch - 1))
    total_t, rows = t1, 1
    if more > 0:
        total_t += timed(more, 1)
        rows += more
    # a batch the oracle finishes in a second or two is verified again (whole) until about ten seconds are spent
    passes = 1
    if rows == w.batch:
        while total_t < 10.0 and passes < 64:
            total_t += timed(w.batch, 0)
            passes += 1
    return passes * rows * (w.gamma + 1) / total_t, rows, total_t, passes


def run_reference(args, w):
    """The oracle, as it stands, on host cores: each step verifies a bounded sample of the workload
    (whole rows, or the first positions of one row when the step budget is small), sized so that
    the run ends within a few minutes whatever --steps says."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import helpers
    P = w.gamma + 1
    max_rows = min(4, w.batch)
    base = synth.make_inputs(w.scaled(batch=max_rows, name=w.name), "cpu")
    def run_units(units):
        if units >= P:
            rows = min(max_rows, units // P)
            small = w.scaled(batch=max_rows, name=w.name)
            t0 = time.perf_counter()
            helpers.run_oracle(small, base, rows=range(rows))
            return rows * P, time.perf_counter() - t0
        small = w.scaled(batch=1, gamma=units - 1, name=w.name)
        part = dict(base, logits=base["logits"][:, :1, :units].contiguous(), drafts=base["drafts"][:1, :units - 1].contiguous(),
                    proposer=base["proposer"][:1])
        t0 = time.perf_counter()
        helpers.run_oracle(small, part)
        return units, time.perf_counter() - t0
    _, t_unit = run_units(1)
    budget = 150.0 / max(1, args.steps + args.warmup)
    units = int(max(1, min(max_rows * P, budget / max(t_unit, 1e-6))))
    total_pos, total_t = 0, 0.0
    for k in range(args.warmup + args.steps):
        done, dt = run_units(units)
        if k >= args.warmup:
            total_pos += done
            total_t += dt
    value = total_pos / total_t
    sample = (f"{units // P} rows x {P} positions" if units >= P else f"first {units} positions of one row") + f" of {w.name} per step"
    line = {
        "impl": "reference", "metric": "verified draft positions/sec", "value": value, "unit": "positions/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "n": w.n, "B": w.batch, "gamma": w.gamma, "V": w.vocab, "logits": w.dtype},
        "cpu_baseline": {"value": value, "unit": "positions/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "positions/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", default=HEADLINE, choices=sorted(synth.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cluster", type=int, default=0, help="thread blocks per position (0 = library default)")
    ap.add_argument("--all-configs", action="store_true", help="also time the other workloads (short loops)")
    ap.add_argument("--skip-cpu", action="store_true")
    ap.add_argument("--skip-e2e", action="store_true")
    args = ap.parse_args()
    w = synth.CONFIGS[args.config]
    if args.impl == "reference":
        run_reference(args, w)
        return
    if args.warmup < 3:
        args.warmup = 3
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    # each rank verifies its own shard of rows (the whole workload per rank: weak scaling);
    # rows are independent, so there is no collective on the data path
    row_base = rank * w.batch
    sets = rotating_inputs(w, dev, rank)
    verifier = make_verifier(w, device=local, cluster_size=args.cluster)
    info = verifier.info()
    sampler = ClockSampler(local) if rank == 0 else None
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize(dev)
    elapsed, outs = time_device(w, verifier, sets, args.steps, args.warmup, row_base, sampler)
    if dist is not None:
        t = torch.tensor([elapsed], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        elapsed = float(t.item())
        dist.barrier()
    # the dominant kernel (stage 0: every position once) timed by itself: CUDA events recorded by the
    # library on the launching stream around each of its launches
    stage_ms = None
    verifier.set_stage_timing(True)
    acc = None
    B, P, V = w.batch, w.gamma + 1, w.vocab
    touts = verifier._alloc_outs(B, P, V, dev, False, False)
    for k in range(60):
        s_ = sets[k % len(sets)]
        verifier.run(s_["logits"], s_["drafts"], s_["proposer"], s_["seed"], s_["offset"] + k, row_base=row_base, outs=touts)
        ms = verifier.stage_ms()
        if k >= 10:
            acc = ms if acc is None else [a_ + b_ for a_, b_ in zip(acc, ms)]
    stage_ms = [a_ / 50.0 for a_ in acc]
    verifier.set_stage_timing(False)
    verifier.close()
    mean_accept = float(outs["accept_count"].float().mean().item())

    e2e = None
    if not args.skip_e2e:
        e_steps = max(2, min(args.steps, 5))
        et, h2d, d2h = time_e2e(w, local, e_steps, 3, row_base)
        if dist is not None:
            t = torch.tensor([et], device=dev, dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            et = float(t.item())
        e2e = {"value": world * w.positions * e_steps / et, "unit": "positions/s", "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": e_steps}

    extra = None
    if args.all_configs and world == 1:
        extra = {}
        for name, ww in synth.CONFIGS.items():
            torch.cuda.empty_cache()
            s2 = rotating_inputs(ww, dev, 0)
            v2 = make_verifier(ww, device=local)
            k2 = max(20, args.steps // 4)
            t2, _ = time_device(ww, v2, s2, k2, 5, 0)
            # a variant, not the metric: with the early-exit hint positions behind a reported rejection go unread
            t3, _ = time_device(ww, v2, s2, k2, 5, 0, flags=COS_RUN_EARLY_EXIT)
            # the same calls captured once in a CUDA graph and replayed (one call per input copy, 64 at most)
            outs2 = v2._alloc_outs(ww.batch, ww.gamma + 1, ww.vocab, dev, False, False)
            ncap = min(len(s2), 64)
            graph = torch.cuda.CUDAGraph()
            torch.cuda.synchronize(dev)
            with torch.cuda.graph(graph):
                for q in range(ncap):
                    v2.run(s2[q]["logits"], s2[q]["drafts"], s2[q]["proposer"], s2[q]["seed"], s2[q]["offset"], outs=outs2)
            reps = max(3, k2 // ncap)
            for _ in range(2):
                graph.replay()
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record()
            for _ in range(reps):
                graph.replay()
            ev1.record()
            torch.cuda.synchronize(dev)
            t4 = ev0.elapsed_time(ev1) / 1e3
            del graph
            extra[name] = {"us_per_call": 1e6 * t2 / k2, "positions_per_s": ww.positions * k2 / t2,
                           "us_per_call_graph": 1e6 * t4 / (reps * ncap),
                           "GBps": ww.positions * ww.bytes_per_position * k2 / t2 / 1e9,
                           "cluster": v2.info()["cluster_size"], "buffers": len(s2),
                           "us_per_call_early_exit": 1e6 * t3 / k2}
            v2.close()
            del s2

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    peak, peak_kind = measured_peak()
    per_call = elapsed / args.steps
    bytes_per_launch = w.positions * w.bytes_per_position
    stage0 = stage_ms[0] / 1e3                      # seconds per launch of the dominant kernel
    achieved = bytes_per_launch / stage0 / 1e9
    per_launch = per_call
    line = {
        "metric": "verified draft positions/sec", "value": world * w.positions * args.steps / elapsed,
        "unit": "positions/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * per_launch, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "n": w.n, "combine": "prob_ensemble" if w.combine == 0 else "logit_linear",
                   "T": w.temperature, "B": w.batch, "gamma": w.gamma, "V": w.vocab, "logits": w.dtype,
                   "l2": "inputs larger than L2" if len(sets) == 1 else f"rotating over {len(sets)} input copies",
                   "cluster_size": info["cluster_size"], "resident_clusters": info["max_clusters"],
                   "mean_accept_count": mean_accept},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": TRAFFIC_BYTES.get(w.name), "peak_kind": peak_kind, "bytes_per_launch": bytes_per_launch,
                     "kernel": "cos_verify_kernel, stage 0 (every position: sweep, accept tests, row scan)",
                     "launch_us": [1e3 * m for m in stage_ms],
                     "whole_call": {"achieved": bytes_per_launch / per_call / 1e9,
                                    "frac": bytes_per_launch / per_call / 1e9 / peak}},
        "gpu_launches": args.steps * info["launches_per_run"],
        "clocks": sampler.summary() if sampler else None,
    }
    if e2e:
        line["e2e"] = e2e
    if extra:
        line["all_configs"] = extra
    if not args.skip_cpu:
        v, rows, dt, passes = oracle_sample(w)
        line["cpu_baseline"] = {"value": v, "unit": "positions/s", "cores": 1, "kind": "oracle",
                                "sample": f"first {rows} rows x {w.gamma + 1} positions of {w.name}, {passes} pass(es), {dt:.1f} s"}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
