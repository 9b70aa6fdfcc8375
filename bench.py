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
from paper_2502_01662_b200.binding import COS_RUN_EARLY_EXIT, COS_RUN_INPUTS_SETTLED  # noqa: E402,F401

HEADLINE = "cfg3"
# dram read + write bytes of one launch of the dominant kernel, as RECORDED in the ncu capture summarised under
# profiles/ (kernel name -> bytes); reported only while the kernel that runs carries the same name
TRAFFIC_BYTES = {"cos_verify_kernel": 355468544}   # profiles/cos_verify_kernel_cfg3.md, stage 0 on workload 3
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
REPORTED = ("cfg1", "cfg2", "cfg3", "cfg4", "cfg5", "cfg5_greedy")
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
    if sampler:
        # nvidia-smi takes a third of a second to start; the device is kept busy afterwards for 50 ms before the
        # warm-up steps, so that the timed region does not begin on a device that has just sat idle
        sampler.__enter__()
        t_busy = time.perf_counter()
        k = 0
        while time.perf_counter() - t_busy < 0.05:
            step(k)
            k += 1
            if k % 64 == 0:
                torch.cuda.synchronize(dev)
    for k in range(warmup):
        step(k)
    torch.cuda.synchronize(dev)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
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
    """The oracle, as it stands, on host cores (its C++ twin, OpenMP over rows, all threads): each step verifies a
    bounded sample of the workload (whole rows), sized so that the run ends within a few minutes whatever --steps
    says.  Rank 0 alone runs it."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import helpers
    from oracle import cos_oracle_native as nat
    P = w.gamma + 1
    threads = nat.max_threads()
    max_rows = min(w.batch, max(1, threads))
    small = w.scaled(batch=max_rows, name=w.name)
    base = synth.make_inputs(small, "cpu")
    def run_rows(rows):
        t0 = time.perf_counter()
        helpers.run_oracle(small, base, rows=range(rows), native=True)
        return time.perf_counter() - t0
    t_all = run_rows(max_rows)
    budget = 150.0 / max(1, args.steps + args.warmup)
    rows = max_rows if t_all <= budget else max(1, int(max_rows * budget / t_all))
    total_pos, total_t = 0, 0.0
    for k in range(args.warmup + args.steps):
        dt = run_rows(rows)
        if k >= args.warmup:
            total_pos += rows * P
            total_t += dt
    value = total_pos / total_t
    sample = f"{rows} rows x {P} positions of {w.name} per step (C++ twin of the oracle, {threads} threads)"
    line = {
        "impl": "reference", "metric": "verified draft positions/sec", "value": value, "unit": "positions/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "n": w.n, "B": w.batch, "gamma": w.gamma, "V": w.vocab, "logits": w.dtype},
        "cpu_baseline": {"value": value, "unit": "positions/s", "cores": min(threads, rows), "box_cores": os.cpu_count(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "positions/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def kernel_names(w, info):
    """What the launches of one call are (for the roofline's stage list)."""
    if info["one_launch"]:
        return ["cos_fused_kernel (every position: sweep, accept tests, row scan, token draw)"]
    names = ["cos_verify_kernel stage 0 (every position: sweep, accept tests, row scan)"]
    if info["launches_per_run"] == 2 and info.get("draw_items"):
        names.append("cos_fused_kernel, drawing items only (token draw, one sweep)")
    elif info["launches_per_run"] == 2 and w.combine == synth.COMBINE_PROB_ENSEMBLE and w.n > 2:
        names.append("cos_verify_kernel stage 4 (token draw, one sweep, a channel per model)")
    elif info["launches_per_run"] == 2:
        names.append("cos_verify_kernel stage 3 (token draw, one sweep)")
    elif info["launches_per_run"] == 3:
        names += ["cos_verify_kernel stage 1 (normalisers of the drawing positions)",
                  "cos_verify_kernel stage 2 (token masses and draw)"]
    return names


def measure_workload(w, dev, local, steps, warmup, row_base=0, sampler=None, cluster=0, stage_runs=30,
                     try_one_launch=False, one_launch=False):
    """One workload on one GPU: K back-to-back calls between two events, then the launches of a call one by one."""
    peak, _ = measured_peak()
    sets = rotating_inputs(w, dev, 0)
    verifier = make_verifier(w, device=local, cluster_size=cluster)
    if one_launch:
        verifier.set_one_launch(True)
    info = verifier.info()
    elapsed, outs = time_device(w, verifier, sets, steps, warmup, row_base, sampler)
    # the same calls with the promise that the inputs were complete before the timed region (they were): the
    # streaming launch of a call then overlaps the end of the previous call's drawing launch
    settled_steps = max(20, steps // 4)
    t_settled, _ = time_device(w, verifier, sets, settled_steps, 5, row_base, flags=COS_RUN_INPUTS_SETTLED)
    def one_call(flags):
        o = verifier._alloc_outs(w.batch, w.gamma + 1, w.vocab, dev, False, False)
        s0 = sets[0]
        for _ in range(2):          # the second of two calls in a row is the one that overlaps
            verifier.run(s0["logits"], s0["drafts"], s0["proposer"], s0["seed"], s0["offset"] + 4242, row_base=row_base,
                         outs=o, flags=flags)
        torch.cuda.synchronize(dev)
        return o
    o_plain, o_settled = one_call(0), one_call(COS_RUN_INPUTS_SETTLED)
    same = all(torch.equal(o_plain[k], o_settled[k]) for k in ("accept_count", "out_tokens", "row_status"))
    verifier.set_stage_timing(True)
    acc = None
    touts = verifier._alloc_outs(w.batch, w.gamma + 1, w.vocab, dev, False, False)
    for k in range(stage_runs + 5):
        s_ = sets[k % len(sets)]
        verifier.run(s_["logits"], s_["drafts"], s_["proposer"], s_["seed"], s_["offset"] + k, row_base=row_base, outs=touts)
        ms = verifier.stage_ms()
        if k >= 5:
            acc = ms if acc is None else [a_ + b_ for a_, b_ in zip(acc, ms)]
    stage_us = [1e3 * a_ / stage_runs for a_ in acc]
    verifier.set_stage_timing(False)
    verifier.close()
    nbytes = w.positions * w.bytes_per_position
    per_call = elapsed / steps
    stages = []
    for name, us in zip(kernel_names(w, info), stage_us):
        # every launch is charged the whole call's algorithmic bytes only if it reads them: the first one does
        gbps = nbytes / (us * 1e-6) / 1e9 if not stages else None
        stages.append({"kernel": name, "us": us, "GBps": gbps, "frac": (gbps / peak) if gbps else None})
    one_launch_us = drawing_launch_us = None
    if try_one_launch:
        v2 = make_verifier(w, device=local)
        try:
            v2.set_one_launch(1)
            t2, _ = time_device(w, v2, sets, max(20, steps // 4), 5, row_base)
            one_launch_us = 1e6 * t2 / max(20, steps // 4)
            v2.set_one_launch(2)
            t3, _ = time_device(w, v2, sets, max(20, steps // 4), 5, row_base)
            drawing_launch_us = 1e6 * t3 / max(20, steps // 4)
        except Exception:
            one_launch_us = None          # the one-launch form does not cover this configuration
        finally:
            v2.close()
    res = {"us_per_call": 1e6 * per_call, "positions_per_s": w.positions / per_call, "GBps": nbytes / per_call / 1e9,
           "frac": nbytes / per_call / 1e9 / peak, "frac_of_nominal_8TBps": nbytes / per_call / 1e9 / NOMINAL_HBM_GBS,
           "bytes_per_call": nbytes, "launches_per_call": info["launches_per_run"], "stages": stages,
           "buffers": len(sets), "one_launch": info["one_launch"],
           "inputs_settled": {"us_per_call": 1e6 * t_settled / settled_steps,
                              "frac": nbytes / (t_settled / settled_steps) / 1e9 / peak,
                              "what": "the same calls with COS_RUN_INPUTS_SETTLED: a call's streaming launch may read "
                                      "its inputs while the previous call's drawing launch drains"}}
    res["inputs_settled"]["same_rows_as_ordinary_calls"] = bool(same)
    if one_launch_us is not None:
        res["us_per_call_one_launch_form"] = one_launch_us   # the opt-in single-kernel form of the same run
        res["us_per_call_persistent_drawing_launch"] = drawing_launch_us   # staged streaming + the persistent kernel's drawing items
    return res, elapsed, outs, info, sets


def sustained_small_calls(w, dev, local, calls=256, contexts=8):
    """Many independent calls of a small workload on distinct buffers, spread over several contexts and streams,
    so that calls overlap on the device: the time per call once launch latency is hidden."""
    sets = rotating_inputs(w, dev, 0)
    vs = [make_verifier(w, device=local) for _ in range(contexts)]
    streams = [torch.cuda.Stream(device=dev) for _ in range(contexts)]
    outs = [v._alloc_outs(w.batch, w.gamma + 1, w.vocab, dev, False, False) for v in vs]
    def go(n, base):
        for k in range(n):
            c = k % contexts
            s_ = sets[(base + k) % len(sets)]
            vs[c].run(s_["logits"], s_["drafts"], s_["proposer"], s_["seed"], s_["offset"] + base + k, outs=outs[c],
                      stream=streams[c])
    torch.cuda.synchronize(dev)
    go(2 * contexts, 0)
    torch.cuda.synchronize(dev)
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record(torch.cuda.current_stream(dev))
    for st in streams:
        st.wait_stream(torch.cuda.current_stream(dev))
    go(calls, 1000)
    for st in streams:
        torch.cuda.current_stream(dev).wait_stream(st)
    t1.record(torch.cuda.current_stream(dev))
    torch.cuda.synchronize(dev)
    for v in vs:
        v.close()
    sec = t0.elapsed_time(t1) / 1e3 / calls
    nbytes = w.positions * w.bytes_per_position
    return {"us_per_call_sustained": 1e6 * sec, "positions_per_s_sustained": w.positions / sec,
            "GBps_sustained": nbytes / sec / 1e9, "contexts": contexts, "calls": calls, "buffers": len(sets)}


def three_streams(w, dev, local):
    """Independent calls of a workload dealt out over three contexts and streams: while one call's drawing launch
    finishes with one block per row, another call's streaming launch has the rest of the device."""
    peak, _ = measured_peak()
    r = sustained_small_calls(w, dev, local, calls=120 if w.positions * w.bytes_per_position < (1 << 30) else 45, contexts=3)
    return {"us_per_call": r["us_per_call_sustained"], "positions_per_s": r["positions_per_s_sustained"],
            "GBps": r["GBps_sustained"], "frac": r["GBps_sustained"] / peak, "contexts": 3, "calls": r["calls"],
            "what": "independent calls on three contexts and streams, between two events on the stream they fork from"}


def ceilings(dev):
    """Read-only and read-plus-exponential streaming ceilings of this device (library micro-kernels)."""
    from paper_2502_01662_b200.binding import measure_ceiling
    buf = (torch.randn(512 * 1024 * 1024, device=dev, dtype=torch.float32) * 3.0).to(torch.bfloat16)   # 1 GiB
    out = {"read_ceiling_GBps": measure_ceiling(0, buf), "ex2_ceiling_GBps": measure_ceiling(1, buf),
           "bytes": buf.numel() * 2, "what": "128-bit streaming loads over 1 GiB of bf16; ex2: one ex2.approx per entry"}
    del buf
    return out


def self_launch(args):
    """`--gpus N` without a launcher around us: start the N ranks here (one process per GPU)."""
    import socket
    with socket.socket() as s_:
        s_.bind(("127.0.0.1", 0))
        port = s_.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", default=HEADLINE, choices=sorted(synth.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cluster", type=int, default=0, help="thread blocks per position (0 = library default)")
    ap.add_argument("--one-launch", action="store_true", help="time the opt-in single-kernel form of a run instead")
    ap.add_argument("--headline-only", action="store_true", help="skip the per-workload table and the ceilings")
    ap.add_argument("--skip-cpu", action="store_true")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--backend", default="nccl", choices=["nccl", "gloo"],
                    help="gloo: launcher self-test on CPU (no verification is timed; see tests/test_bench_launcher.py)")
    args = ap.parse_args()
    w = synth.CONFIGS[args.config]
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        self_launch(args)
    if args.impl == "reference":
        run_reference(args, w)
        return
    if args.warmup < 3:
        args.warmup = 3
    if args.backend == "gloo":
        launcher_self_test(args, world, rank)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but the launcher started {world} rank(s)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    # each rank verifies its own shard of rows (the whole workload per rank: weak scaling);
    # rows are independent, so there is no collective on the data path
    row_base = rank * w.batch
    sampler = ClockSampler(local) if rank == 0 else None
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize(dev)
    head, elapsed, outs, info, sets = measure_workload(w, dev, local, args.steps, args.warmup, row_base, sampler,
                                                       cluster=args.cluster, one_launch=args.one_launch)
    if dist is not None:
        t = torch.tensor([elapsed], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        elapsed = float(t.item())
        dist.barrier()
    mean_accept = float(outs["accept_count"].float().mean().item())
    n_sets = len(sets)
    del sets

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

    table, ceil = None, None
    extra_launches = 0
    if not args.headline_only and world == 1:
        table = {}
        for name in REPORTED:
            ww = synth.CONFIGS[name]
            torch.cuda.empty_cache()
            if name == w.name:
                table[name] = {k: v for k, v in head.items()}
                table[name]["three_streams"] = three_streams(ww, dev, local)
                continue
            k2 = 400 if ww.positions * ww.bytes_per_position < (1 << 30) else 100
            res, _, _, inf2, s2 = measure_workload(ww, dev, local, k2, 5, stage_runs=20, try_one_launch=True)
            del s2
            extra_launches += (k2 + 5 + 25) * inf2["launches_per_run"]
            if name == "cfg2":
                res.update(sustained_small_calls(ww, dev, local))
            res["three_streams"] = three_streams(ww, dev, local)
            table[name] = res
        torch.cuda.empty_cache()
        ceil = ceilings(dev)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    peak, peak_kind = measured_peak()
    per_call = elapsed / args.steps
    bytes_per_call = w.positions * w.bytes_per_position
    achieved = bytes_per_call / per_call / 1e9
    dominant = head["stages"][0]["kernel"].split(" ")[0]
    line = {
        "metric": "verified draft positions/sec", "value": world * w.positions * args.steps / elapsed,
        "unit": "positions/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * per_call, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "input_dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "n": w.n, "combine": "prob_ensemble" if w.combine == 0 else "logit_linear",
                   "T": w.temperature, "B": w.batch, "gamma": w.gamma, "V": w.vocab, "logits": w.dtype,
                   "l2": "inputs larger than L2" if n_sets == 1 else f"rotating over {n_sets} input copies",
                   "before_warmup": "clock sampler started, then 50 ms of untimed calls, then the W warm-up steps",
                   "cluster_size": info["cluster_size"], "resident_clusters": info["max_clusters"],
                   "one_launch": info["one_launch"], "items_per_position": info["items_per_position"],
                   "mean_accept_count": mean_accept},
        # the WHOLE call: algorithmic bytes of the batch over the time of all launches of a call
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": TRAFFIC_BYTES.get(dominant), "peak_kind": peak_kind, "bytes_per_launch": bytes_per_call,
                     "frac_of_nominal_8TBps": achieved / NOMINAL_HBM_GBS, "kernel": head["stages"][0]["kernel"],
                     "launches_per_call": head["launches_per_call"], "stages": head["stages"],
                     # not the headline: the same calls under the caller's promise that their inputs were complete
                     # earlier (true of this loop), which lets consecutive calls overlap
                     "inputs_settled": head.get("inputs_settled"),
                     # not the headline either: independent calls on three contexts and streams overlap one call's
                     # drawing launch with another's streaming launch
                     "three_streams": (table or {}).get(w.name, {}).get("three_streams")},
        "gpu_launches": args.steps * info["launches_per_run"],
        "clocks": sampler.summary() if sampler else None,
    }
    if e2e:
        line["e2e"] = e2e
    if table:
        line["configs"] = table
    if ceil:
        line["ceilings"] = ceil
    if not args.skip_cpu:
        line["cpu_baseline"] = cpu_baseline(w)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def native_sample(w, threads, target_seconds=6.0):
    """The oracle's C++ twin on the first rows of the workload with `threads` host threads (0 = all)."""
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import helpers
    from oracle import cos_oracle_native as nat
    used = threads if threads > 0 else nat.max_threads()
    rows = min(w.batch, max(1, used))
    small = w.scaled(batch=rows, name=w.name)
    inputs = synth.make_inputs(small, "cpu")
    t0 = time.perf_counter()
    helpers.run_oracle(small, inputs, native=True, threads=threads)
    t1 = time.perf_counter() - t0
    reps = int(max(0, min(2000, target_seconds / max(t1, 1e-3) - 1)))
    for _ in range(reps):
        helpers.run_oracle(small, inputs, native=True, threads=threads)
    total = time.perf_counter() - t0
    return (reps + 1) * rows * (w.gamma + 1) / total, rows, total, used


def cpu_baseline(w):
    """The oracle, as it stands, on this machine's host cores, on a bounded sample of the workload: its C++ twin on all
    cores (the headline value) and on one, and the Python oracle on one core."""
    v_all, rows_all, dt_all, used = native_sample(w, 0)
    v_one, rows_one, dt_one, _ = native_sample(w, 1, target_seconds=4.0)
    v_py, rows_py, dt_py, passes = oracle_sample(w, target_seconds=6.0)
    return {"value": v_all, "unit": "positions/s", "cores": used, "box_cores": os.cpu_count(), "kind": "oracle",
            "sample": f"first {rows_all} rows x {w.gamma + 1} positions of {w.name}, {dt_all:.1f} s (C++ twin of the oracle, OpenMP over rows)",
            "one_thread": {"value": v_one, "sample": f"{rows_one} row(s), {dt_one:.1f} s"},
            "python_oracle_one_thread": {"value": v_py, "sample": f"{rows_py} row(s), {passes} pass(es), {dt_py:.1f} s"}}


def launcher_self_test(args, world, rank):
    """CPU check of the multi-rank plumbing (no GPU, no verification): ranks meet, each times a stand-in step,
    the maximum over ranks is taken, rank 0 prints the line with n_gpus = world size."""
    import torch.distributed as dist
    dist.init_process_group("gloo")
    dist.barrier()
    t0 = time.perf_counter()
    time.sleep(0.01 * (rank + 1))            # rank r "works" for (r + 1) * 10 ms
    elapsed = time.perf_counter() - t0
    t = torch.tensor([elapsed], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.barrier()
    if rank == 0:
        print(json.dumps({"metric": "launcher self-test", "n_gpus": world, "max_elapsed_s": float(t.item()),
                          "own_elapsed_s": elapsed, "backend": "gloo", "gpu_launches": 0}))
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
