#!/usr/bin/env python
"""Benchmark of the DGS push+apply+pull event loop.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload resnet50] [--impl ours|reference]

One "step" is one event (worker push, server apply, worker pull) of the chosen
workload.  Default workload: ResNet-50 shapes, 25.56 M parameters, one global 0.1 %
selection, 32 workers.  Prints ONE JSON line (rank 0).

Timed region: K consecutive events with every gradient already resident in HBM,
CUDA events on the library's stream, barrier + synchronize on both sides, max over
ranks.  Before the W warm-up events an untimed pre-roll serves every worker three times,
so that the timed events are steady-state ones (a worker's first arrival takes the
two-pass selection route).  Each event reads a different gradient, velocity and
difference vector (3 x 102 MB at the default workload, more than the L2), so no
L2 flush is needed between iterations.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

# hardware queues for the library's streams (read when the CUDA context is created; see the package)
os.environ.setdefault("CUDA_DEVICE_MAX_CONNECTIONS", "32")

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads as W  # noqa: E402

METRIC = "push+apply+pull events/sec"
UNIT = "events/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# ncu DRAM traffic of the dominant kernel: read from the tracked summary of the capture, which names the
# source state it was taken at; no number is reported once the kernel's source has changed since
TRAFFIC_SUMMARY = os.path.join(ROOT, "profiles", "k_stream_push_resnet50_traffic.txt")
KERNEL_SOURCE = os.path.join(ROOT, "paper_1910_10929_b200", "csrc", "dgs_kernels.cuh")


def stream_pass_source_hash() -> str:
    """Hash of the part of the kernel source that makes up the stream pass (everything up to the
    histogram pass), so that edits to other kernels of the same file do not invalidate the capture."""
    import hashlib
    with open(KERNEL_SOURCE) as f:
        text = f.read()
    cut = text.find("// ---- histogram of ALL elements")
    return hashlib.sha256(text[:cut if cut > 0 else len(text)].encode()).hexdigest()[:16]


def ncu_traffic(workload: str, kernel: str):
    """(bytes per launch, note) from the tracked summary if it covers this workload and kernel and was
    captured from the present source of the stream pass; else (None, why)."""
    try:
        fields = {}
        with open(TRAFFIC_SUMMARY) as f:
            for line in f:
                if ":" in line and not line.startswith("#"):
                    k, v = line.split(":", 1)
                    fields[k.strip()] = v.strip()
        if fields.get("workload") != workload or fields.get("kernel") != kernel:
            return None, "no capture for this workload and kernel"
        if fields.get("stream_pass_source_hash") != stream_pass_source_hash():
            return None, "the stream pass has changed since the capture"
        return int(fields["dram_bytes_per_launch"]), f"ncu capture at commit {fields.get('commit', '?')}"
    except Exception as e:           # no summary, or one that does not parse
        return None, f"no usable capture summary ({type(e).__name__})"


def make_workload(name: str, seed: int, workers: int = 0):
    if name not in W.BY_NAME:
        raise SystemExit(f"unknown workload {name}; choose from {sorted(W.BY_NAME)}")
    if workers:
        return W.BY_NAME[name](seed=seed, num_workers=workers)
    return W.BY_NAME[name](seed=seed)


def preroll_events(wl) -> int:
    """Untimed events before the warm-up: three rounds of the workers, so that every worker has come back,
    carried bounds and the pulls' planned ranges exist, and even a short run times steady-state events."""
    return 3 * wl.num_workers


def config_of(wl, args, world: int = 1) -> dict:
    """The `config` object both arms print: the workload and the parameters of the run, the same keys
    and values in both, so that the two lines can be matched."""
    K, Wm, R = args.steps, args.warmup, max(1, args.windows)
    return {"workload": wl.name, "n": wl.n, "workers": wl.num_workers, "K_push": wl.K_push, "K_pull": wl.K_pull,
            "segments": wl.num_segments, "lr": wl.lr, "momentum": wl.momentum, "seed": wl.seed,
            "schedule": wl.schedule_kind, "preroll_events": preroll_events(wl),
            "distinct_gradients": min(preroll_events(wl) + Wm + (R + 1) * K, args.grad_pool),
            "l2": "inputs larger than L2: every event reads a different gradient, velocity and difference vector",
            "replicas": world, "windows": R}


def algorithmic_bytes_per_event(n: int, K_push: int, K_pull: int, N: int) -> dict:
    """What the method itself must move per event (no scratch traffic counted).
    push: read u and grad, write u', write the packet.  apply: read the packet once,
    read+write one float per (entry, buffer) for theta and the N difference vectors.
    pull: read D_w, write the packet, clear the sent entries."""
    push = 12 * n + 8 * K_push
    apply_ = 8 * K_push * (N + 1) + 8 * K_push
    pull = 4 * n + 8 * K_pull + 4 * K_pull
    return {"push": push, "apply": apply_, "pull": pull, "total": push + apply_ + pull}


def hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Polls nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), [c.strip() for c in line.split(",")]))

    def window(self, t0: float, t1: float) -> None:
        """Keep the samples taken between two perf_counter readings (at least the nearest one)."""
        inside = [r for t, r in self.rows if t0 <= t <= t1]
        if not inside and self.rows:
            mid = 0.5 * (t0 + t1)
            inside = [min(self.rows, key=lambda tr: abs(tr[0] - mid))[1]]
        self.rows = inside

    def __exit__(self, *a):
        if self.proc is not None:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
            self.thread.join(timeout=2)

    def summary(self) -> dict:
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in self.rows:
            if len(r) < 8:
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for name, cell in zip(names, r[4:8]):
                if cell.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


def generate_gradients(wl, events, out_tensors) -> None:
    """Fills out_tensors[i] (pinned host float32[n]) with the gradient of events[i], in parallel."""
    def one(i):
        wl.gradient(int(events[i]), out=out_tensors[i].numpy())
    wl._scales() if wl.grad_kind == "laplace" else None
    with ThreadPoolExecutor(max_workers=min(32, os.cpu_count() or 1)) as ex:
        list(ex.map(one, range(len(events))))


def run_reference(args, wl) -> dict:
    """The CPU checker, as it stands, on the host cores: one step = one full event."""
    import oracle
    sched = wl.schedule()
    K, Wm = args.steps, args.warmup
    o = oracle.Oracle.from_workload(wl)
    # keep the whole run within a few minutes: estimate from the first warm-up event
    budget_s = 240.0
    done, t_first = 0, None
    for e in range(Wm):
        t0 = time.perf_counter()
        o.event(int(sched[e % len(sched)]), wl.gradient(e))
        t_first = time.perf_counter() - t0 if t_first is None else t_first
    if t_first is None:
        t0 = time.perf_counter()
        o.event(int(sched[0]), wl.gradient(0))
        t_first = time.perf_counter() - t0
        Wm_eff = 1
    else:
        Wm_eff = Wm
    K_eff = max(1, min(K, int(budget_s / max(t_first, 1e-6))))
    grads = None
    elapsed = 0.0
    for i in range(K_eff):
        e = Wm_eff + i
        g = wl.gradient(e)                      # input generation is outside the timed region
        t0 = time.perf_counter()
        o.event(int(sched[e % len(sched)]), g)
        elapsed += time.perf_counter() - t0
        done += 1
    value = done / elapsed
    sample = (f"{done} consecutive events of the full {wl.name} workload (n={wl.n}, {wl.num_workers} workers) "
              f"after {Wm_eff} untimed ones")
    return {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": done, "warmup": Wm_eff, "ms_per_step": 1e3 * elapsed / done, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_of(wl, args, 1),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


def cpu_baseline(wl, seconds: float = 20.0) -> dict:
    import oracle
    sched = wl.schedule()
    o = oracle.Oracle.from_workload(wl)
    elapsed, done, e = 0.0, 0, 0
    while elapsed < seconds and e < len(sched) and done < 64:
        g = wl.gradient(e)
        t0 = time.perf_counter()
        o.event(int(sched[e]), g)
        elapsed += time.perf_counter() - t0
        done += 1
        e += 1
    return {"value": done / elapsed, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"first {done} events of {wl.name} (n={wl.n}, {wl.num_workers} workers), "
                      f"{elapsed:.1f} s of single-thread CPU time on a {os.cpu_count()}-core host"}


def reduce_max_time(elapsed_s: float, events: int, dist) -> tuple:
    """Max of the elapsed time over ranks and the sum of the events all ranks served."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return elapsed_s, events
    import torch
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([elapsed_s], dtype=torch.float64, device=dev)
    c = torch.tensor([events], dtype=torch.int64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return float(t.item()), int(c.item())


def run_ours(args, wl, rank: int, world: int, local_rank: int, dist) -> dict:
    import torch

    import paper_1910_10929_b200 as dgs

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    N = wl.num_workers
    sched_full = wl.schedule()
    preroll = preroll_events(wl)
    K, Wm = args.steps, args.warmup
    R = max(1, args.windows)                     # timed windows of K events each, back to back
    total_events = preroll + Wm + (R + 1) * K    # timed windows + per-kernel timing pass
    pool = min(total_events, args.grad_pool)
    sched = np.resize(sched_full, total_events)

    # gradients: generated on the host (same generator the CPU checker is fed from), resident in HBM
    host = [torch.empty(wl.n, dtype=torch.float32).pin_memory() for _ in range(min(pool, 16))]
    grads = []
    for base in range(0, pool, len(host)):
        ids = list(range(base, min(pool, base + len(host))))
        generate_gradients(wl, ids, host[:len(ids)])
        for j in range(len(ids)):
            grads.append(host[j].to(dev, non_blocking=False))
    theta0 = torch.from_numpy(wl.theta0()).to(dev)
    ctx = dgs.Context.from_workload(wl, theta0=theta0, flags=dgs.DGS_HOST_IO)
    stream = ctx.stream

    def run_events(first: int, count: int) -> None:
        for e in range(first, first + count):
            ctx.event(int(sched[e]), grads[e % pool])

    def barrier():
        torch.cuda.synchronize(dev)
        if dist is not None and world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    window_s = []
    with ClockSampler(local_rank) as clocks:
        run_events(0, preroll)
        run_events(preroll, Wm)
        ctx.flush()
        stats0 = ctx.stats()
        reads0 = ctx.pull_read_stats()
        launches0 = ctx.launch_count()
        t_begin = time.perf_counter()
        for r in range(R):
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            barrier()
            ev0.record(stream)
            run_events(preroll + Wm + r * K, K)
            ctx.flush()
            ev1.record(stream)
            barrier()
            window_s.append(ev0.elapsed_time(ev1) * 1e-3)
        t_end = time.perf_counter()
    clocks.window(t_begin, t_end)
    elapsed = statistics.median(window_s)         # of the R windows of exactly K events each
    launches = (ctx.launch_count() - launches0) // R
    stats1 = ctx.stats()
    reads1 = ctx.pull_read_stats()
    assert ctx.status() == 0, "device status word is not clean"
    elapsed_max, events_all = reduce_max_time(elapsed, K, dist)

    # per-kernel device time, same loop continued, events around each launch
    dgs.dgs_timing_enable(ctx.handle, True)
    run_events(preroll + Wm + R * K, K)
    ktimes = dgs.dgs_timing_read(ctx.handle)
    dgs.dgs_timing_enable(ctx.handle, False)

    # end to end: host gradient in, pull packet out, every step
    Ke = min(K, len(host), 16)
    out_idx = torch.empty(wl.K_pull, dtype=torch.int32).pin_memory()
    out_val = torch.empty(wl.K_pull, dtype=torch.float32).pin_memory()
    first = preroll + Wm + (R + 1) * K
    sched_e = np.resize(sched_full, first + Ke + 3)
    for j in range(3):
        ctx.event_host(int(sched_e[first + j]), host[j % len(host)], out_idx, out_val)
    barrier()
    t0 = time.perf_counter()
    for j in range(Ke):
        ctx.event_host(int(sched_e[first + 3 + j]), host[j], out_idx, out_val)
    torch.cuda.synchronize(dev)
    e2e_elapsed = time.perf_counter() - t0
    e2e_max, e2e_events = reduce_max_time(e2e_elapsed, Ke, dist)

    # the same loop with every kernel on one stream: each kernel's own duration, nothing beside it
    ctx.close()
    del ctx
    Ks = min(K, 128)
    sctx = dgs.Context.from_workload(wl, theta0=theta0, flags=dgs.DGS_SINGLE_STREAM)
    for e in range(preroll + Wm):
        sctx.event(int(sched[e]), grads[e % pool])
    dgs.dgs_timing_enable(sctx.handle, True)
    for e in range(preroll + Wm, preroll + Wm + Ks):
        sctx.event(int(sched[e]), grads[e % pool])
    stimes = dgs.dgs_timing_read(sctx.handle)
    dgs.dgs_timing_enable(sctx.handle, False)
    assert sctx.status() == 0, "device status word is not clean"
    sctx.close()
    del sctx

    if rank != 0:
        return {}
    ab = algorithmic_bytes_per_event(wl.n, wl.K_push, wl.K_pull, N)
    peak, peak_kind = hbm_peak()
    value = events_all / elapsed_max
    eff_gbs = value / world * ab["total"] / 1e9
    # The roofline kernel is the HBM-bound pass that moves most of an event's bytes: the push stream
    # pass (12n of the 16n streamed per event).  Its time is measured live, with the other streams'
    # kernels running beside it as they do in the timed region.
    tot_ms = sum(ms for ms, _ in ktimes.values()) or 1.0
    dom = "stream_push" if ktimes["stream_push"][1] else max(ktimes, key=lambda k: ktimes[k][0])
    dom_ms, dom_cnt = stimes[dom]          # on its own (single-stream pass)
    ovl_ms, ovl_cnt = ktimes[dom]          # with the other streams' kernels beside it
    # algorithmic bytes per launch: the streaming passes move whole vectors; the apply reads the packet and
    # lowers theta (8 K read + 8 K read-modify-write); a catch-up lowers one difference vector by the packets
    # of one round of the workers (8 bytes per entry, N K entries)
    kernel_bytes = {
        "stream_push": 12 * wl.n, "finalize_push": None, "two_pass_push": 8 * wl.n,
        "scatter": 16 * wl.K_push, "stream_pull": 4 * wl.n, "finalize_pull": None, "two_pass_pull": 4 * wl.n,
        "catch_up": 8 * wl.K_push * N,
    }
    achieved = kernel_bytes[dom] / (dom_ms * 1e-3 / max(dom_cnt, 1)) / 1e9
    achieved_ovl = kernel_bytes[dom] / (ovl_ms * 1e-3 / max(ovl_cnt, 1)) / 1e9
    stot_ms = sum(ms for ms, _ in stimes.values()) or 1.0

    def kernel_gbs(k, ms, cnt):
        if not cnt or ms <= 0:
            return None
        if k == "catch_up":         # the apply's bytes of an event (N + 1 buffers) over scatter + catch-up time
            return ab["apply"] * K / ((ms + ktimes["scatter"][0]) * 1e-3) / 1e9
        return kernel_bytes[k] / (ms * 1e-3 / cnt) / 1e9 if kernel_bytes[k] else None

    traffic, traffic_note = ncu_traffic(wl.name, dom)
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": 1e3 * elapsed_max / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_of(wl, args, world),
        "cuda_device_max_connections": os.environ.get("CUDA_DEVICE_MAX_CONNECTIONS"),
        "windows": {"count": R, "events_each": K, "ms_per_step": [1e3 * t / K for t in window_s],
                    "spread": (max(window_s) - min(window_s)) / elapsed if elapsed > 0 else None,
                    "note": "value and ms_per_step are those of the median window"},
        "effective_hbm": {"algorithmic_bytes_per_event": ab, "GB/s": eff_gbs,
                          "frac_of_nominal_8TBs": eff_gbs / NOMINAL_HBM_GBS, "frac_of_peak": eff_gbs / peak,
                          "peak_GB/s": peak, "peak_kind": peak_kind},
        "selection_routes": {"selections": 2 * K * R, "single_pass": stats1[0] - stats0[0], "two_pass": stats1[1] - stats0[1],
                             "candidates_per_selection": (stats1[3] - stats0[3]) / max(1, 2 * K * R),
                             "pull_chunks_read_fraction": (reads1[1] - reads0[1]) / max(1, reads1[0] - reads0[0])},
        "kernels": {k: {"ms_total": ms, "launches": c, "us_per_launch": (1e3 * ms / c if c else None),
                        "share": ms / tot_ms,
                        "GB/s": kernel_gbs(k, ms, c)}
                    for k, (ms, c) in ktimes.items()},
        "kernels_single_stream": {k: {"launches": c, "us_per_launch": (1e3 * ms / c if c else None),
                                      "share": ms / stot_ms,
                                      "GB/s": (kernel_bytes[k] / (ms * 1e-3 / c) / 1e9
                                               if c and ms > 0 and kernel_bytes[k] else None),
                                      "frac_of_peak": (kernel_bytes[k] / (ms * 1e-3 / c) / 1e9 / peak
                                                       if c and ms > 0 and kernel_bytes[k] else None)}
                                  for k, (ms, c) in stimes.items()},
        "roofline": {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_kind": peak_kind, "traffic": traffic,
                     "traffic_note": traffic_note,
                     "algorithmic_bytes_per_launch": kernel_bytes[dom],
                     "achieved_overlapped": achieved_ovl, "frac_overlapped": achieved_ovl / peak,
                     "whole_event_frac": eff_gbs / peak,
                     "note": "achieved: CUDA events around each launch of the kernel in a pass of the same event "
                             f"loop ({Ks} events) that keeps every kernel on one stream, so the duration is the "
                             "kernel's own; achieved_overlapped: the same in the multi-stream loop, where up to "
                             "four push passes and the server-side kernels share the GPU and the bandwidth; "
                             "whole_event_frac: algorithmic bytes of a whole event over the timed region"},
        "e2e": {"value": e2e_events / e2e_max, "unit": UNIT, "steps": Ke, "h2d_bytes_per_step": 4 * wl.n,
                "d2h_bytes_per_step": 8 * wl.K_pull},
        "gpu_launches": launches,
        "clocks": clocks.summary(),
    }
    if world == 1 and N > 1 and not args.no_jitter:
        out["jittered_arrivals"] = run_jittered(wl, grads, pool, theta0, min(K, 512), dev)
    if world == 1 and N > 1 and not args.no_jitter:
        out["full_pull"] = run_full_pull(wl, sched, grads, pool, theta0, min(K, 512), dev)
    if world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(wl, args.cpu_seconds)
    return out


def run_full_pull(wl, sched, grads, pool, theta0, K, dev) -> dict:
    """The same workload with the pull that has no secondary compression (the paper's normal case): every
    pull sends all nonzero entries of the worker's difference vector (dgs_worker_pull_all) instead of the
    k largest.  Same arrival order, same gradients; push, apply and pull are three calls per event."""
    import torch

    import paper_1910_10929_b200 as dgs
    N = wl.num_workers
    # a worker's difference vector holds what arrived since its previous pull: a round of the workers in a
    # fixed cycle, now and then much more under random arrivals
    cap = int(min(wl.n, (2 if wl.schedule_kind == "cyclic" else 16) * N * wl.K_push))
    ctx = dgs.Context.from_workload(wl, theta0=theta0, pull_all_capacity=cap)
    pre = preroll_events(wl)
    sched = np.resize(sched, pre + K)

    def event(e):
        w = int(sched[e])
        pkt = ctx.worker_push(w, grads[e % pool])
        ctx.server_apply(w, pkt)
        return ctx.worker_pull_all(w)

    for e in range(pre):
        event(e)
    ctx.flush()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(dev)
    ev0.record(ctx.stream)
    last = None
    for e in range(pre, pre + K):
        last = event(e)
    ctx.flush()
    ev1.record(ctx.stream)
    torch.cuda.synchronize(dev)
    idx, _ = ctx.var_packet(last)
    status = ctx.status()
    assert status in (0, dgs.DGS_ELIMIT), "device status word is not clean"
    ctx.close()
    t = ev0.elapsed_time(ev1) * 1e-3
    return {"pull": "all nonzero entries of the difference vector (no secondary compression)", "events": K,
            "value": K / t, "unit": UNIT, "ms_per_step": 1e3 * t / K, "packet_capacity": cap,
            "entries_in_last_pull_packet": int(idx.numel()),
            "a_packet_overflowed_its_capacity": status == dgs.DGS_ELIMIT}


def run_jittered(wl, grads, pool, theta0, K, dev) -> dict:
    """The same workload with an irregular arrival order: every event is served for a worker drawn
    independently and uniformly (a worker may return at once or stay away for long), so the bounds
    carried from earlier selections fit less often.  Reports the rate and which route the selections took."""
    import torch

    import paper_1910_10929_b200 as dgs
    N = wl.num_workers
    rng = np.random.Generator(np.random.Philox(key=wl.seed + 77))
    sched = rng.integers(0, N, size=4 * N + K).astype(np.int32)
    ctx = dgs.Context.from_workload(wl, theta0=theta0)
    for e in range(4 * N):
        ctx.event(int(sched[e]), grads[e % pool])
    ctx.flush()
    s0 = ctx.stats()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(dev)
    ev0.record(ctx.stream)
    for e in range(4 * N, 4 * N + K):
        ctx.event(int(sched[e]), grads[e % pool])
    ctx.flush()
    ev1.record(ctx.stream)
    torch.cuda.synchronize(dev)
    s1 = ctx.stats()
    assert ctx.status() == 0, "device status word is not clean"
    ctx.close()
    t = ev0.elapsed_time(ev1) * 1e-3
    return {"schedule": "each event's worker drawn uniformly at random", "events": K, "value": K / t, "unit": UNIT,
            "ms_per_step": 1e3 * t / K,
            "selection_routes": {"single_pass": s1[0] - s0[0], "two_pass": s1[1] - s0[1],
                                 "candidates_per_selection": (s1[3] - s0[3]) / max(1, 2 * K)}}



def run_sweep(args) -> dict:
    """Kernel sweep on one flat vector: n = 2^16 .. 2^28 in powers of 4, density 0.01 % .. 10 %,
    values N(0,1) with 1 % of positions scaled by 100.  Times, per cell and cold (a 512 MB buffer
    is rewritten between measurements): the selection + encoding of a pull on the two-pass
    route (nothing carried over: histogram pass + stream pass + finalize) and on the single-pass
    route (bound carried over from the previous selection), and the apply of the resulting
    packet into 2 buffers (theta + 1 difference vector) and into 33 (theta + 32)."""
    import torch

    import paper_1910_10929_b200 as dgs

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peak, peak_kind = hbm_peak()
    flush_buf = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream(dev)

    def timed(fn, ctx, reps=3):
        out = []
        for _ in range(reps):
            flush_buf.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize(dev)
            e0.record(stream)
            fn()
            ctx.flush()
            e1.record(stream)
            torch.cuda.synchronize(dev)
            out.append(e0.elapsed_time(e1) * 1e3)
        return statistics.median(out)

    cells = []
    for log2n in W.SWEEP_LOG2N:
        if log2n > args.sweep_max_log2n:
            continue
        n = 1 << log2n
        x = torch.from_numpy(W.sweep_values(n, args.seed, log2n)).to(dev)
        for ppm in W.SWEEP_PPM:
            k = W.k_of(n, ppm)
            sel = dgs.Context(n, 1, 0.1, 0.9, [0], [n], [k], [k], torch.zeros(n, device=dev))

            def pull_fresh():
                sel.state_load(dgs.DGS_D, 0, x)
                return sel.worker_pull(0)
            # the first pull of a context has nothing to go by: two-pass route.  Time it on fresh contexts.
            two_pass = []
            for _ in range(3):
                c2 = dgs.Context(n, 1, 0.1, 0.9, [0], [n], [k], [k], torch.zeros(n, device=dev))
                c2.state_load(dgs.DGS_D, 0, x)
                two_pass.append(timed(lambda: c2.worker_pull(0), c2, reps=1))
                c2.close()
                del c2
            t_two = statistics.median(two_pass)
            pull_fresh()                                   # leaves a carried bound behind
            single = []
            for _ in range(3):
                sel.state_load(dgs.DGS_D, 0, x)
                single.append(timed(lambda: sel.worker_pull(0), sel, reps=1))
            t_single = statistics.median(single)
            p = pull_fresh()
            idx, val = sel.packet(p)
            idx, val = idx.clone(), val.clone()
            sel.close()
            del sel
            row = {"log2n": log2n, "density_ppm": ppm, "k": k,
                   "select_two_pass_us": t_two, "select_single_pass_us": t_single,
                   "select_two_pass_GBs": 4 * n / t_two / 1e3, "select_single_pass_GBs": 4 * n / t_single / 1e3,
                   "select_single_pass_frac_of_peak": 4 * n / t_single / 1e3 / peak}
            for nb_workers in (1, 32):
                torch.cuda.empty_cache()        # the arenas of closed contexts go back to the device
                need = dgs.dgs_arena_bytes(dgs.make_config(n, nb_workers, 0.1, 0.9, [0], [n], [k], [k]))
                free, _ = torch.cuda.mem_get_info(dev)
                if need + (8 << 30) > free:
                    continue
                ap = dgs.Context(n, nb_workers, 0.1, 0.9, [0], [n], [k], [k], torch.zeros(n, device=dev))
                fp = dgs.dgs_packet(idx.data_ptr(), val.data_ptr(), k)
                t_ap = timed(lambda: ap.server_apply(0, fp), ap)
                ap.close()
                del ap
                bytes_alg = 8 * k * (nb_workers + 1) + 8 * k
                row[f"scatter_{nb_workers + 1}buf_us"] = t_ap
                row[f"scatter_{nb_workers + 1}buf_GBs"] = bytes_alg / t_ap / 1e3
                row[f"scatter_{nb_workers + 1}buf_sector_GBs"] = 64 * k * (nb_workers + 1) / t_ap / 1e3
            cells.append(row)
            print(json.dumps(row), file=sys.stderr, flush=True)
    return {"metric": "kernel sweep: select+compact and scatter GB/s", "unit": "GB/s", "peak_GB/s": peak,
            "peak_kind": peak_kind, "data": "synthetic", "cells": cells,
            "note": "select GB/s = 4n bytes (one read of the vector) / time; scatter GB/s = 8 bytes per "
                    "(entry, buffer) + the packet / time, sector_GBs counts one 32-byte sector each way"}


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=512)
    ap.add_argument("--warmup", type=int, default=32)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet50", choices=sorted(W.BY_NAME))
    ap.add_argument("--seed", type=int, default=W.DEFAULT_SEED)
    ap.add_argument("--grad-pool", type=int, default=127, help="distinct gradients kept in HBM (reused cyclically)")
    ap.add_argument("--workers", type=int, default=0,
                    help="override the number of simulated workers (smaller state for profiler captures)")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", action="store_true", help="kernel sweep over vector sizes and densities")
    ap.add_argument("--sweep-max-log2n", type=int, default=28)
    ap.add_argument("--windows", type=int, default=5, help="timed windows of --steps events each (the median is reported)")
    ap.add_argument("--no-jitter", action="store_true", help="skip the extra pass with irregular arrivals")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.sweep:
        if rank == 0:
            print(json.dumps(run_sweep(args)), flush=True)
        return
    if args.impl == "reference":
        if rank == 0:
            print(json.dumps(run_reference(args, make_workload(args.workload, args.seed, args.workers))), flush=True)
        return

    dist = None
    if world > 1:
        import torch
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    # replicas only: the path has no exchange step, every rank runs its own workers and server
    wl = make_workload(args.workload, args.seed + rank, args.workers)
    out = run_ours(args, wl, rank, world, local_rank, dist)
    if rank == 0:
        print(json.dumps(out), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
