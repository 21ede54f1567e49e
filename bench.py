#!/usr/bin/env python
"""Benchmark of the Kimad+ compression pass on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..5] [--impl kimad|reference]

One "step" is one kimad_step(): the whole hot path (EF21 difference, error curves, knapsack DP,
Top-K select, pack, EF21 update) for all simulated workers of one GPU on one batch of synthetic
gradients.  Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank runs its own set of
workers on its own GPU (the path shards by worker: no collective on the data path) and the time is
the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2312_08053_b200 import workloads  # noqa: E402
from paper_2312_08053_b200.dist import max_over_ranks, barrier, init_distributed  # noqa: E402

METRIC = "compressed_gradient_elements_per_second"
UNIT = "elements/s"

# DRAM traffic of the dominant kernel per input element: dram__bytes_read.sum + dram__bytes_write.sum of one
# launch of the sweep kernel in an ncu capture on workload 3 (inputs larger than L2), divided by the elements of
# that launch.  Every element is read once from each input and one code byte written for it, so the figure
# carries over to the other workloads; it has to be re-captured when the sweep's data movement changes.
NCU_TRAFFIC_BYTES_PER_ELEM = {"sweep": 9.27}

# algorithmic bytes per input element of each stage (what the stage must move at least once)
STAGE_ALGO_BYTES = {"sweep": 9.0,  # read grad + g, write one code byte per element
                    "select_count": 1.0, "select_write": 8.0}


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return float(json.load(open(p))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id):
        self.rows, self.proc, self.gpu_id = [], None, gpu_id

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu_id), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()

    def summary(self, t0, t1):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = [r for (t, r) in self.rows if t0 <= t <= t1] or [r for (_, r) in self.rows]
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except Exception:
                continue
            for name, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def run_reference(args, rank):
    """The oracle, as it stands, on the host cores: each step is one oracle pass over a bounded sample
    (shrunk tensors, same layer list / distributions / budget trace) of the configured workload."""
    if rank != 0:
        return
    from oracle import kimad_oracle as ko

    wl_full = workloads.workload(args.config)
    target = 3_000_000
    div = max(1, int(np.ceil(wl_full.N * wl_full.n_workers / target)))
    wl = workloads.workload(args.config, div)
    bw = workloads.bandwidth_trace(wl, 64)
    grads = [workloads.gradients(wl, s).numpy() for s in range(2)]
    state = np.zeros((wl.n_workers, wl.N), np.float32)
    times = []
    for s in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        r = ko.step(wl.layer_sizes, wl.n_workers, wl.ratio_grid, wl.D, wl.value_dtype, grads[s % 2], state,
                    bw[s % len(bw)], wl.t_target, cap=wl.N)
        dt = time.perf_counter() - t0
        state = r.state
        if s >= args.warmup:
            times.append(dt)
    ms = 1e3 * float(np.mean(times))
    elems = wl.N * wl.n_workers
    val = elems / (ms * 1e-3)
    sample = f"{wl.name}: {wl.n_workers} workers x {wl.N} elements per step (tensors shrunk {div}x)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": _dtype_label(wl_full), "data": "synthetic",
        "config": {"workload": wl_full.name, "cfg": args.config, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": ko.get_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def cpu_baseline(cfg):
    """Oracle timed on a bounded sample (about 10-30 s of CPU work) of the same workload."""
    from oracle import kimad_oracle as ko

    wl_full = workloads.workload(cfg)
    total = wl_full.N * wl_full.n_workers

    def one(target):
        div = max(1, int(np.ceil(total / target)))
        wl = workloads.workload(cfg, div)
        bw = workloads.bandwidth_trace(wl, 8)
        grads = workloads.gradients(wl, 0).numpy()
        state = np.zeros_like(grads)
        t0 = time.perf_counter()
        ko.step(wl.layer_sizes, wl.n_workers, wl.ratio_grid, wl.D, wl.value_dtype, grads, state, bw[3], wl.t_target,
                cap=wl.N)
        return wl, div, time.perf_counter() - t0

    wl, div, dt = one(8_000_000)              # calibration run, not reported
    rate = wl.N * wl.n_workers / dt
    wl, div, dt = one(min(total, max(8_000_000, rate * 15.0)))  # about 15 s of oracle work
    return {"value": wl.N * wl.n_workers / dt, "unit": UNIT, "cores": ko.get_threads(), "kind": "oracle",
            "sample": f"1 oracle step on {wl.name}: {wl.n_workers} workers x {wl.N} elements "
                      f"(tensors shrunk {div}x), {dt:.1f} s"}


TARGET_FRAC = 0.60  # of the HBM roofline on compulsory bytes, for the workloads of 100 M parameters and more


def _dtype_label(wl):
    # the path computes in binary32 (difference, keys, sums of squares as exact integers); workload 5 packs bf16 values
    return "f32" if wl.value_dtype == 0 else "f32 (bf16 packed values)"


SCHEDULE = 0  # kimad_debug_set_schedule of every context the bench creates (--schedule)
ZERO_ROWS = 0.0  # fraction of exactly-zero rows in the token embedding's gradient (--zero-rows; workloads 4 and 5)


def _time_steps(kb, torch, wl, dev, rank, steps, warmup, max_buf_bytes=70e9):
    """Device-timed steps of one workload: returns (ctx, out, grads, state, bw, cap, per-step ms list, launches)."""
    W, N, L = wl.n_workers, wl.N, wl.L
    bw = workloads.bandwidth_trace(wl)
    bpe = 8 if wl.value_dtype == 0 else 6
    cap = int(min(N, np.max(bw) * wl.t_target / bpe + L + 1))
    ctx = kb.new_context(wl.layer_sizes, W, wl.ratio_grid, device=dev, D=wl.D, value_dtype=wl.value_dtype,
                         max_packed_elems=cap)
    kb.kimad_debug_set_schedule(ctx, SCHEDULE)
    out = kb.Packed(ctx, device=dev)
    # fresh gradients for every step (as in training), as far as the device memory allowed for them goes; beyond
    # that the buffers are cycled.  Every rank draws its own streams (seed offset by rank).
    n_bufs = int(max(2, min(warmup + steps, max_buf_bytes // (W * N * 4))))
    grads = [workloads.gradients(wl, 1000 * rank + s, device=dev, zero_rows=ZERO_ROWS) for s in range(n_bufs)]
    state = torch.zeros((W, N), dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()

    def step(s):
        kb.kimad_step(ctx, grads[s % n_bufs], state, bw[s % len(bw)], wl.t_target, out, stream)

    for s in range(warmup):
        step(s)
    torch.cuda.synchronize()
    return ctx, out, grads, state, bw, cap, step, n_bufs


def _stage_times(kb, ctx, step, first, n_prof):
    kb.kimad_debug_enable_stage_timing(ctx, True)
    acc = np.zeros(len(kb.STAGE_NAMES))
    for s in range(n_prof):
        step(first + s)
        acc += kb.kimad_debug_stage_times(ctx)
    kb.kimad_debug_enable_stage_timing(ctx, False)
    return dict(zip(kb.STAGE_NAMES, (acc / n_prof).tolist()))


def _rooflines(wl, ms_per_step, stage_ms):
    """step_roofline: the whole step on the compulsory bytes (8 B per input element: read grad and g once; packed
    output and sparse write-back are < 3 % more).  roofline: the dominant kernel on its own algorithmic bytes, and
    the same kernel time on the compulsory 8 B per element (frac_compulsory)."""
    peak, peak_kind = peaks()
    W, N = wl.n_workers, wl.N
    top = max(stage_ms, key=stage_ms.get)
    algo_b = STAGE_ALGO_BYTES.get(top, 4.0) * W * N
    achieved = algo_b / (stage_ms[top] * 1e-3) / 1e9
    tpe = NCU_TRAFFIC_BYTES_PER_ELEM.get(top)
    compulsory = 8.0 * W * N
    step_gbs = compulsory / (ms_per_step * 1e-3) / 1e9  # per GPU: every rank moves its own W * N elements
    step_roofline = {"bound": "hbm", "compulsory_bytes_per_step": compulsory, "achieved": step_gbs, "peak": peak,
                     "unit": "GB/s", "frac": step_gbs / peak, "peak_kind": f"of {peak_kind}",
                     "target_frac": TARGET_FRAC, "target_met": bool(step_gbs / peak >= TARGET_FRAC)}
    roofline = {"bound": "hbm", "kernel": top, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                "frac_compulsory": compulsory / (stage_ms[top] * 1e-3) / 1e9 / peak,
                "traffic": (tpe * W * N if tpe is not None else None),
                "algorithmic_bytes_per_launch": algo_b, "kernel_ms": stage_ms[top]}
    return step_roofline, roofline


def run_kimad(args, rank, world):
    import torch

    from paper_2312_08053_b200 import binding as kb
    from paper_2312_08053_b200 import pipeline

    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", 0)))
    torch.cuda.set_device(dev)
    wl = workloads.workload(args.config)
    W, N, L = wl.n_workers, wl.N, wl.L
    bpe = 8 if wl.value_dtype == 0 else 6
    ctx, out, grads, state, bw, cap, step, n_bufs = _time_steps(kb, torch, wl, dev, rank, args.steps, args.warmup)
    stream = torch.cuda.current_stream()
    props = torch.cuda.get_device_properties(dev)
    gpu_id = str(getattr(props, "uuid", "")) or str(dev.index)
    if "-" in gpu_id and not gpu_id.startswith("GPU-"):
        gpu_id = "GPU-" + gpu_id
    sampler = ClockSampler(gpu_id)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = kb.kimad_launch_count(ctx)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    barrier()
    torch.cuda.synchronize()
    t_wall0 = time.time()
    ev[0].record(stream)
    for s in range(args.steps):
        step(args.warmup + s)
        ev[s + 1].record(stream)
    torch.cuda.synchronize()
    barrier()
    t_wall1 = time.time()
    total_ms = ev[0].elapsed_time(ev[-1])
    per_step = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
    launches = kb.kimad_launch_count(ctx) - launches0
    total_ms = max_over_ranks(total_ms)
    ms_per_step = total_ms / args.steps
    elems_per_step = W * N * world
    value = elems_per_step / (ms_per_step * 1e-3)
    status, _ = kb.kimad_get_k(ctx)
    if status < 0:
        raise RuntimeError(f"kimad step failed on rank {rank}: {kb.kimad_strerror(status)}")
    if args.timeline and rank == 0:
        # one more step with events around every launch: which kernels ran beside each other, on which stream
        s = args.warmup + args.steps
        text = kb.kimad_debug_trace_step(ctx, grads[s % n_bufs], state, bw[s % len(bw)], wl.t_target, out, stream)
        dense = W * N * bpe
        with open(args.timeline, "w") as f:
            f.write(f"# workload {args.config}, schedule {SCHEDULE}, step {s}: budget = "
                    f"{100.0 * float(np.sum(bw[s % len(bw)])) * wl.t_target / dense:.2f} % of the dense bytes\n")
            f.write(text)

    # ---- end to end: host buffers in, packed message out, copies inside the timed region.  Two drivers of the
    # same public calls: one after the other (copy in, step, copy out), and the double-buffered driver that
    # uploads step s while step s + 1 is copied in and compressed (Section 5: the pass can be overlapped with
    # communication).  The headline e2e is the overlapped one; the serial figure is kept beside it.
    e2e_bufs = min(n_bufs, 3)
    host_grads = [g.cpu().pin_memory() for g in grads[:e2e_bufs]]
    e2e_steps = max(3, min(args.steps, 10))
    drv = pipeline.HostDriver(ctx, wl, cap, device=dev)
    e2e = {}
    for mode in ("serial", "overlapped"):
        drv.run(mode, host_grads, state, bw, 1)  # warm-up (allocations, first touches)
        barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        moved = drv.run(mode, host_grads, state, bw, e2e_steps, first_step=1)
        torch.cuda.synchronize()
        ms = max_over_ranks((time.perf_counter() - t0) * 1e3) / e2e_steps
        e2e[mode] = {"value": elems_per_step / (ms * 1e-3), "ms_per_step": ms, "d2h": int(moved / e2e_steps)}
    best = e2e["overlapped"]
    e2e_out = {"value": best["value"], "unit": UNIT, "ms_per_step": best["ms_per_step"],
               "h2d_bytes_per_step": int(W * N * 4), "d2h_bytes_per_step": best["d2h"], "driver": "overlapped",
               "serial_ms_per_step": e2e["serial"]["ms_per_step"], "serial_value": e2e["serial"]["value"]}
    del drv, host_grads

    # ---- per-stage device times (CUDA events on the launch stream) for the roofline of the top kernel
    stage_ms = _stage_times(kb, ctx, step, args.warmup, max(3, min(args.steps, 10)))
    exact_layers = kb.kimad_debug_exact_path_layers(ctx, detail=True)
    if rank == 0:
        sampler.stop()
    clocks = sampler.summary(t_wall0, t_wall1) if rank == 0 else None
    step_roofline, roofline = _rooflines(wl, ms_per_step, stage_ms)

    # ---- the other workload of 100 M parameters and more (the largest single-GPU one), device-timed only
    also = None
    other = {4: 5, 5: 4}.get(args.config)
    if other is not None and not args.no_also:
        del ctx, out, grads, state, step
        torch.cuda.empty_cache()
        wl2 = workloads.workload(other)
        k2 = max(3, min(args.steps, 10))
        ctx2, out2, grads2, state2, bw2, cap2, step2, nb2 = _time_steps(kb, torch, wl2, dev, rank, k2, 3, max_buf_bytes=40e9)
        ev2 = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        barrier()
        torch.cuda.synchronize()
        ev2[0].record(stream)
        for s in range(k2):
            step2(3 + s)
        ev2[1].record(stream)
        torch.cuda.synchronize()
        barrier()
        ms2 = max_over_ranks(ev2[0].elapsed_time(ev2[1])) / k2
        st2, _ = kb.kimad_get_k(ctx2)
        if st2 < 0:
            raise RuntimeError(f"kimad step failed on rank {rank}: {kb.kimad_strerror(st2)}")
        stage2 = _stage_times(kb, ctx2, step2, 3, k2)
        sr2, rf2 = _rooflines(wl2, ms2, stage2)
        also = {"workload": wl2.name, "cfg": wl2.cfg, "workers_per_gpu": wl2.n_workers, "elements_per_worker": wl2.N,
                "dtype": _dtype_label(wl2), "steps": k2, "warmup": 3, "gradient_buffers": nb2,
                "value": wl2.n_workers * wl2.N * world / (ms2 * 1e-3), "unit": UNIT, "ms_per_step": ms2,
                "step_roofline": sr2, "roofline": rf2, "stage_ms": stage2}
        del ctx2, out2, grads2, state2, step2
        torch.cuda.empty_cache()
    # ---- the receiving side of a round on the same workload (apply the messages, model step), device-timed
    receive = None
    if not args.no_also:
        torch.cuda.empty_cache()
        rcv = _measure_receive(args, rank, world, max(3, min(args.steps, 10)), 3)
        receive = {k: rcv[k] for k in ("metric", "value", "unit", "ms_per_step", "steps", "warmup", "roofline", "stage_ms")}
        torch.cuda.empty_cache()
    if rank != 0:
        return
    res = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": _dtype_label(wl), "data": "synthetic",
        "config": {"workload": wl.name, "cfg": wl.cfg, "workers_per_gpu": W, "layers": L, "elements_per_worker": N,
                   "ratios": len(wl.ratio_grid), "D": wl.D, "value_dtype": "bf16" if wl.value_dtype else "f32",
                   "l2": "inputs_larger_than_l2" if W * N * 4 > 200e6 else "inputs_fit_l2",
                   "budget_trace": "cycled", "gradient_buffers": n_bufs, "parallelism": f"worker-sharded x{world}",
                   "zero_rows": ZERO_ROWS},
        "step_roofline": step_roofline,
        "e2e": e2e_out, "gpu_launches": int(launches),
        "roofline": roofline,
        "stage_ms": stage_ms, "step_ms_minmax": [min(per_step), max(per_step)],
        "exact_path_layers": exact_layers,
        "clocks": clocks,
    }
    if also is not None:
        res["also"] = also
    if receive is not None:
        res["receive"] = receive
    if world == 1 and not args.no_cpu_baseline:
        res["cpu_baseline"] = cpu_baseline(args.config)
    print(json.dumps(res))


def _measure_receive(args, rank, world, steps, warmup):
    """The receiving side of one round (Algorithm 1, server lines) on the configured workload:
    kimad_apply_packed of the W workers' messages, then kimad_aggregate over the W estimators.  The
    dominant kernel is the dense model step, (W + 2) * 4 bytes per model element.  Returns the result dict."""
    import torch

    from paper_2312_08053_b200 import binding as kb

    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", 0)))
    torch.cuda.set_device(dev)
    wl = workloads.workload(args.config)
    W, N, L = wl.n_workers, wl.N, wl.L
    bw = workloads.bandwidth_trace(wl)
    bpe = 8 if wl.value_dtype == 0 else 6
    cap = int(min(N, np.max(bw) * wl.t_target / bpe + L + 1))
    ctx = kb.new_context(wl.layer_sizes, W, wl.ratio_grid, device=dev, D=wl.D, value_dtype=wl.value_dtype,
                         max_packed_elems=cap)
    n_msgs = 4
    msgs = []
    state = torch.zeros((W, N), dtype=torch.float32, device=dev)
    for s in range(n_msgs):  # messages of consecutive rounds, produced by the compression pass itself
        out = kb.Packed(ctx, device=dev)
        g = workloads.gradients(wl, 1000 * rank + s, device=dev)
        kb.kimad_step(ctx, g, state, bw[s % len(bw)], wl.t_target, out)
        torch.cuda.synchronize()
        del g
        msgs.append(out)
    est = torch.zeros((W, N), dtype=torch.float32, device=dev)
    x = torch.zeros(N, dtype=torch.float32, device=dev)
    wts = np.full(W, 1.0 / W, np.float32)
    stream = torch.cuda.current_stream()
    ev_a = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    ev_b = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    ev_c = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]

    def step(s, i=None):
        if i is not None:
            ev_a[i].record(stream)
        kb.kimad_apply_packed(ctx, msgs[s % n_msgs], est, stream)
        if i is not None:
            ev_b[i].record(stream)
        kb.kimad_aggregate(x, est, wts, 0.01, stream)
        if i is not None:
            ev_c[i].record(stream)

    for s in range(warmup):
        step(s)
    barrier()
    torch.cuda.synchronize()
    for i in range(steps):
        step(warmup + i, i)
    torch.cuda.synchronize()
    barrier()
    total_ms = max_over_ranks(ev_a[0].elapsed_time(ev_c[-1]))
    apply_ms = float(np.mean([a.elapsed_time(b) for a, b in zip(ev_a, ev_b)]))
    agg_ms = float(np.mean([b.elapsed_time(c) for b, c in zip(ev_b, ev_c)]))
    peak, peak_kind = peaks()
    ms_per_step = total_ms / steps
    algo_b = (W + 2) * 4.0 * N
    achieved = algo_b / (agg_ms * 1e-3) / 1e9
    n_entries = float(np.mean([int(m.stats_host()["n_selected"].sum()) for m in msgs]))
    return {
        "metric": "received_update_elements_per_second", "value": W * N * world / (ms_per_step * 1e-3), "unit": UNIT,
        "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": wl.name + " / receive", "cfg": wl.cfg, "senders": W, "elements_per_sender": N,
                   "packed_entries_per_step": n_entries, "l2": "inputs_larger_than_l2"},
        "gpu_launches": 2 * steps,
        "roofline": {"bound": "hbm", "kernel": "k_aggregate", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": None,
                     "algorithmic_bytes_per_launch": algo_b, "kernel_ms": agg_ms},
        "stage_ms": {"apply_packed": apply_ms, "aggregate": agg_ms}}


def run_receive(args, rank, world):
    """Secondary line (``--path receive``): the receiving side alone."""
    res = _measure_receive(args, rank, world, args.steps, args.warmup)
    if rank == 0:
        print(json.dumps(res))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=4, help="workload 1..5 (default 4: GPT-2-small shape, 4 workers)")
    ap.add_argument("--impl", default="kimad", choices=["kimad", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--schedule", type=int, default=0, choices=[0, 1, 2],
                    help="0: the library's choice (two worker groups for large steps), 1: always two groups, 2: one group")
    ap.add_argument("--zero-rows", type=float, default=0.0,
                    help="workloads 4 and 5: this fraction of the token embedding's gradient rows is exactly zero (a sparse "
                         "gradient; not the headline workload: the line says so in config.zero_rows)")
    ap.add_argument("--timeline", default=None, metavar="FILE",
                    help="after the timed steps, run one step with events around every launch and write its timeline")
    ap.add_argument("--no-also", action="store_true", help="skip the second large workload's device-timed block")
    ap.add_argument("--path", default="compress", choices=["compress", "receive"],
                    help="compress: the worker-side pass (the headline); receive: apply + aggregate on the server")
    args = ap.parse_args()
    global SCHEDULE, ZERO_ROWS
    SCHEDULE = args.schedule
    ZERO_ROWS = args.zero_rows
    if ZERO_ROWS and args.config not in (4, 5):
        ap.error("--zero-rows needs --config 4 or 5")
    args.warmup = max(args.warmup, 3) if args.impl == "kimad" else args.warmup
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    init_distributed("nccl")
    if args.path == "receive":
        run_receive(args, rank, world)
        return
    run_kimad(args, rank, world)


if __name__ == "__main__":
    main()
