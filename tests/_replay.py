"""Replays a workload through the CUDA library and the CPU checker side by side."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_1910_10929_b200 as dgs


def key(x: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(x, dtype=np.float32).view(np.uint32) & np.uint32(0x7FFFFFFF)


def bits(x) -> np.ndarray:
    return np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)


def max_rel_err(a: np.ndarray, b: np.ndarray) -> float:
    """max |a-b| / max(|a|,|b|), 0 where both are 0."""
    a64, b64 = a.astype(np.float64), b.astype(np.float64)
    den = np.maximum(np.abs(a64), np.abs(b64))
    num = np.abs(a64 - b64)
    out = np.zeros_like(num)
    np.divide(num, den, out=out, where=den > 0)
    return float(out.max()) if out.size else 0.0


def packet_format(flags: int) -> int:
    """The CPU checker's packet_format for a context's flags."""
    return oracle.BF16 if flags & dgs.DGS_PACKET_BF16 else (oracle.FP16 if flags & dgs.DGS_PACKET_FP16 else oracle.FP32)


def packet_to_numpy(ctx: dgs.Context, pkt):
    idx, val = ctx.packet(pkt)
    return idx.cpu().numpy().view(np.uint32), val.cpu().numpy()


def replay_and_compare(wl, *, flags: int = 0, num_events=None, schedule=None, compare_state_every: int = 0,
                       device: str = "cuda:0"):
    """Runs events on both sides.  Packets must agree bit for bit at every event; the
    full state is compared at the end (and every `compare_state_every` events).
    Returns (ctx, oracle) for further checks."""
    keep_local = bool(flags & dgs.DGS_KEEP_LOCAL_MODEL)
    residual = bool(flags & dgs.DGS_RESIDUAL_MODE)
    theta0 = wl.theta0()
    orc = oracle.Oracle.from_workload(wl, keep_local=keep_local, residual_mode=residual, theta0=theta0,
                                      packet_format=packet_format(flags))
    ctx = dgs.Context.from_workload(wl, theta0=torch.from_numpy(theta0).to(device), flags=flags)
    sched = wl.schedule() if schedule is None else np.asarray(schedule)
    E = len(sched) if num_events is None else num_events
    for e in range(E):
        w = int(sched[e])
        g = wl.gradient(e)
        g_dev = torch.from_numpy(g).to(device)
        pkt = ctx.worker_push(w, g_dev)
        pi, pv = packet_to_numpy(ctx, pkt)
        oi, ov = orc.push(w, g)
        assert np.array_equal(pi, oi), f"event {e}: push index set differs"
        assert np.array_equal(bits(pv), bits(ov)), f"event {e}: push values differ"
        ctx.server_apply(w, pkt)
        orc.apply(w, oi, ov)
        pkt2 = ctx.worker_pull(w)
        gi, gv = packet_to_numpy(ctx, pkt2)
        qi, qv = orc.pull(w)
        assert np.array_equal(gi, qi), f"event {e}: pull index set differs"
        assert np.array_equal(bits(gv), bits(qv)), f"event {e}: pull values differ"
        assert ctx.status() == 0
        if compare_state_every and (e + 1) % compare_state_every == 0:
            compare_state(ctx, orc, wl.num_workers, keep_local)
    compare_state(ctx, orc, wl.num_workers, keep_local)
    assert dgs.dgs_stats(ctx.handle)[2] == orc.timestamp
    for q in range(wl.num_workers):
        assert dgs.dgs_prev(ctx.handle, q) == orc.prev(q)
    return ctx, orc


def compare_state(ctx, orc, num_workers: int, keep_local: bool) -> None:
    """All float32 state must agree bit for bit (the tolerance asked of the
    trajectory, 1e-6 max relative error, is checked too and is implied)."""
    def same(which_gpu, which_cpu, q, name):
        a = ctx.state(which_gpu, q).cpu().numpy()
        b = orc.state(which_cpu, q)
        assert max_rel_err(a, b) <= 1e-6, f"{name}[{q}] beyond 1e-6"
        assert np.array_equal(bits(a), bits(b)), f"{name}[{q}] not bit-identical"

    same(dgs.DGS_THETA, oracle.THETA, 0, "theta")
    for q in range(num_workers):
        same(dgs.DGS_U, oracle.U, q, "u")
        same(dgs.DGS_D, oracle.D, q, "D")
        if keep_local:
            same(dgs.DGS_THETA_LOCAL, oracle.THETA_LOCAL, q, "theta_local")


def replay_async_and_compare(wl, *, flags: int = 0, num_events=None, schedule=None, device: str = "cuda:0"):
    """Enqueues all events back to back without ever waiting (the library's streams overlap
    consecutive events), then replays the same events on the CPU checker and compares the
    whole final state and the last packets bit for bit.  Any missing dependency between the
    overlapped steps shows up as a difference."""
    keep_local = bool(flags & dgs.DGS_KEEP_LOCAL_MODEL)
    residual = bool(flags & dgs.DGS_RESIDUAL_MODE)
    theta0 = wl.theta0()
    sched = wl.schedule() if schedule is None else np.asarray(schedule)
    E = len(sched) if num_events is None else num_events
    sched = np.resize(sched, E)
    grads_host = [wl.gradient(e) for e in range(E)]
    grads = [torch.from_numpy(g).to(device) for g in grads_host]      # alive until the end
    ctx = dgs.Context.from_workload(wl, theta0=torch.from_numpy(theta0).to(device), flags=flags)
    torch.cuda.synchronize()
    last = None
    for e in range(E):
        last = ctx.event(int(sched[e]), grads[e])
    pi, pv = packet_to_numpy(ctx, last[0])
    gi, gv = packet_to_numpy(ctx, last[1])
    assert ctx.status() == 0
    orc = oracle.Oracle.from_workload(wl, keep_local=keep_local, residual_mode=residual, theta0=theta0,
                                      packet_format=packet_format(flags))
    for e in range(E):
        (oi, ov), (qi, qv) = orc.event(int(sched[e]), grads_host[e])
    assert np.array_equal(pi, oi) and np.array_equal(bits(pv), bits(ov)), "last push packet differs"
    assert np.array_equal(gi, qi) and np.array_equal(bits(gv), bits(qv)), "last pull packet differs"
    compare_state(ctx, orc, wl.num_workers, keep_local)
    return ctx, orc
