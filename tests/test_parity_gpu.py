"""Parity of the CUDA library against the CPU checker, through the C ABI.

Bar: selected index sets bit-exact (ties to the lowest index), packet values and
apply results bit-exact, all float32 state within 1e-6 max relative error after
the whole trajectory -- every step is one rounded IEEE operation in a fixed
order, so the state is in fact required to be bit-identical."""
import numpy as np
import pytest
import torch

import oracle
import paper_1910_10929_b200 as dgs
import workloads as W
from _replay import bits, key, packet_to_numpy, replay_and_compare, replay_async_and_compare

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def select_on_gpu(x: np.ndarray, seg_sizes, ks, flags=0):
    """Top-k per segment of a given vector via a pull on a one-worker context."""
    n = x.shape[0]
    off = np.concatenate([[0], np.cumsum(seg_sizes)[:-1]])
    ctx = dgs.Context(n, 1, 0.1, 0.9, off, seg_sizes, ks, ks, torch.zeros(n, device=DEV), flags=flags)
    ctx.state_load(dgs.DGS_D, 0, torch.from_numpy(x).to(DEV))
    idx, val = packet_to_numpy(ctx, ctx.worker_pull(0))
    left = ctx.state(dgs.DGS_D, 0).cpu().numpy()
    assert ctx.status() == 0
    return idx, val, left, ctx


def expect_select(x, seg_sizes, ks):
    out, base = [], 0
    for ln, k in zip(seg_sizes, ks):
        out.append(oracle.topk(x[base:base + ln], k) + base)
        base += ln
    return np.concatenate(out).astype(np.uint32)


ADVERSARIAL = [
    ("all_equal", np.ones(1500, np.float32), [1500], [37]),
    ("all_zero", np.zeros(1029, np.float32), [1029], [5]),
    ("signed_zeros", np.tile(np.array([0.0, -0.0], np.float32), 300), [600], [7]),
    ("k_is_1", np.arange(777, dtype=np.float32) - 300, [777], [1]),
    ("k_is_n", (np.arange(513, dtype=np.float32) - 77) / 3, [513], [513]),
    ("one_element", np.array([-2.5], np.float32), [1], [1]),
    ("denormals", np.concatenate([np.full(300, 1e-45, np.float32), np.zeros(300, np.float32),
                                  np.full(5, -3e-40, np.float32)]), [605], [100]),
    ("ties_across_tiles", np.tile(np.array([1, -1, 2, -2, 0.5], np.float32), 700), [3500], [1000]),
    ("ragged_segments", np.sin(np.arange(2000, dtype=np.float32)), [3, 509, 1, 700, 787], [1, 100, 1, 7, 787]),
    ("same_top_bits", (1.0 + np.arange(4096, dtype=np.float32) * 2.0 ** -20).astype(np.float32), [4096], [300]),
]


@pytest.mark.parametrize("name,x,segs,ks", ADVERSARIAL, ids=[c[0] for c in ADVERSARIAL])
def test_selection_adversarial(name, x, segs, ks):
    want = expect_select(x, segs, ks)
    idx, val, left, _ = select_on_gpu(x, segs, ks)
    assert np.array_equal(idx, want)
    assert np.array_equal(bits(val), bits(x[want]))
    # exact split: what was sent plus what stayed is the input, and the sent entries are cleared
    back = left.copy()
    assert not left[want].any()
    back[want] = val
    assert np.array_equal(bits(back), bits(x))


@pytest.mark.parametrize("flags", [0, dgs.DGS_NO_SPECULATION, dgs.DGS_KEEP_LOCAL_MODEL, dgs.DGS_RESIDUAL_MODE,
                                   dgs.DGS_SINGLE_STREAM,
                                   dgs.DGS_RESIDUAL_MODE | dgs.DGS_KEEP_LOCAL_MODEL | dgs.DGS_NO_SPECULATION])
def test_trajectory_small_ragged(flags):
    # several tiles, ragged heads and tails, tiny layers, repeated arrivals of the same worker
    wl = W.custom("ragged", [300, 7, 5000, 64, 1, 2049, 1531], 3, 30, 20_000, grad_kind="normal", grad_scale=1e-2)
    ctx, _ = replay_and_compare(wl, flags=flags, compare_state_every=7)
    single, two_pass, _, _ = ctx.stats()
    assert single + two_pass == 2 * wl.num_events
    if flags & dgs.DGS_NO_SPECULATION:
        assert single == 0
    else:
        assert single > 0


def test_trajectory_dense_limit_k_equals_n():
    wl = W.custom("dense", [700, 333], 2, 8, 1_000_000, grad_kind="normal", grad_scale=1e-2)
    assert wl.K_push == wl.n
    replay_and_compare(wl, flags=dgs.DGS_KEEP_LOCAL_MODEL)


def test_trajectory_pull_wants_more_than_is_nonzero():
    # the server sends 5 % per layer while pushes deliver 0.5 %: early pulls are filled with zeros
    wl = W.custom("zero_fill", [4000, 3000], 2, 10, 5_000, density_pull_ppm=50_000, grad_kind="laplace")
    replay_and_compare(wl)


def test_trajectory_momentum_one_and_half():
    for m in (1.0, 0.5):
        wl = W.custom("m", [3000], 2, 8, 10_000, momentum=m)
        replay_and_compare(wl)


def test_trajectory_flat_1m():
    wl = W.flat_1m()
    assert wl.K_push == 1049
    replay_and_compare(wl, flags=dgs.DGS_KEEP_LOCAL_MODEL)


def test_trajectory_resnet18_per_layer():
    wl = W.resnet18(num_workers=32, num_events=40)
    ctx, _ = replay_and_compare(wl)
    assert ctx.stats()[0] > 0          # workers that came back took the single-pass route


def test_trajectory_resnet50_global():
    wl = W.resnet50(num_workers=32, num_events=36)
    replay_and_compare(wl)


@pytest.mark.parametrize("flags", [0, dgs.DGS_KEEP_LOCAL_MODEL, dgs.DGS_RESIDUAL_MODE])
def test_overlapped_events_random_arrivals(flags):
    # i.i.d. arrivals: the same worker often comes twice in a row, ages vary, bounds fail now and then
    wl = W.custom("async", [150_000, 517, 90_000, 64, 70_001], 5, 150, 5_000, grad_kind="laplace",
                  schedule_kind="uniform")
    ctx, _ = replay_async_and_compare(wl, flags=flags)
    assert ctx.stats()[0] > 0


def test_overlapped_events_resnet50_32_workers():
    # the benchmark's configuration, three rounds of the 32 workers, nothing waited for in between
    wl = W.resnet50(num_workers=32, num_events=96)
    replay_async_and_compare(wl)


def test_overlapped_events_resnet18_per_layer():
    wl = W.resnet18(num_workers=32, num_events=80)
    replay_async_and_compare(wl)


def test_starved_worker_sees_every_packet_it_missed():
    # worker 2 arrives once, stays away for 50 events (more than the library keeps packets for), comes back
    wl = W.custom("starved", [40_000, 700, 9_001], 3, 60, 10_000, grad_kind="laplace")
    sched = [2] + [0, 1] * 25 + [2, 0, 2, 1, 2, 2, 0, 1, 2]
    replay_and_compare(wl, schedule=sched, compare_state_every=20)
    replay_async_and_compare(wl, schedule=sched, flags=dgs.DGS_KEEP_LOCAL_MODEL)


def test_pull_skips_cold_chunks_and_notices_when_they_heat_up():
    # gradients live in one third of the vector at a time and move on with growing size, so chunks of the
    # difference vectors that the pulls had stopped reading come back into the selection
    n, third = 3 * 262_144, 262_144
    wl = W.custom("moving_heat", [n], 3, 36, 2_000, grad_kind="normal", grad_scale=1e-3)
    base = wl.gradient

    def moving(e, out=None):
        g = base(e)
        phase = (e // 9) % 3
        keep = np.zeros(n, dtype=np.float32)
        keep[phase * third:(phase + 1) * third] = np.float32(1 + e // 9)
        g *= keep
        if out is not None:
            out[:] = g
            return out
        return g

    wl.gradient = moving
    ctx, _ = replay_and_compare(wl, compare_state_every=9)
    covered, read = ctx.pull_read_stats()
    assert 0 < read < covered            # some chunks were skipped, and the packets still agreed throughout
    replay_async_and_compare(wl, flags=dgs.DGS_KEEP_LOCAL_MODEL)


def test_more_workers_than_packets_kept():
    # 140 workers in a fixed cycle: every difference vector is 140 packets behind when its worker returns,
    # more than the library keeps (128 at most)
    wl = W.custom("many", [30_000, 301, 2_048], 140, 330, 10_000, grad_kind="normal", schedule_kind="cyclic")
    replay_async_and_compare(wl)


def test_catch_up_takes_a_crowded_range_in_pieces():
    # The ranges of the packet log come from the first packet: its entries lie in the first quarter
    # of the vector, so one range covers the other three quarters.  All later packets fall there,
    # and a worker that has missed a few of them finds more entries in that range than the
    # catch-up's table holds at once.
    n, N, E = 200_000, 8, 20
    wl = W.custom("moving", [n], N, E, 10_000, grad_kind="normal", grad_scale=1e-2, schedule_kind="cyclic")
    base = wl.gradient

    def gradient(e, out=None):
        g = base(e)
        lo, hi = (0, n // 4) if e == 0 else (n // 2, n)
        g[:lo] *= 1e-3
        g[hi:] *= 1e-3
        if out is not None:
            out[:] = g
            return out
        return g
    wl.gradient = gradient
    replay_and_compare(wl, compare_state_every=5)
    replay_async_and_compare(wl)


def test_more_layers_than_the_shared_memory_tables_hold():
    # 1500 layers of 40..300 elements: finalize reads its per-layer tables from global memory
    rng = np.random.default_rng(5)
    sizes = [int(v) for v in rng.integers(40, 300, size=1500)]
    wl = W.custom("many-layers", sizes, 3, 9, 50_000, grad_kind="laplace")
    replay_and_compare(wl, compare_state_every=4)


def test_selection_with_many_candidates_per_thread():
    # k = n / 2 of 2^21 values: every finalize thread owns far more candidates than it keeps in registers
    n = 1 << 21
    x = W.sweep_values(n, 7, 21)
    k = n // 2
    idx, val, left, _ = select_on_gpu(x, [n], [k])
    want = expect_select(x, [n], [k])
    assert np.array_equal(idx, want)
    assert np.array_equal(bits(val), bits(x[want]))
    assert not left[want].any()


def test_trajectory_gpt2_small_few_workers():
    wl = W.gpt2_small(num_workers=3, num_events=7)
    replay_and_compare(wl)


def test_trajectory_gpt2_small_per_layer_few_workers():
    # 148 layers from 768 to 38.6 M elements, each selected on its own
    wl = W.gpt2_small(num_workers=2, num_events=4, per_layer=True)
    replay_and_compare(wl)


# ---- pull without secondary compression (Algorithm 2 with the switch off; Eq. 3-5) ---------
def replay_full_pull(wl, *, flags=0, capacity=None, mixed=False, schedule=None):
    """push / apply / pull-all for every event on both sides; packets bit for bit at every event
    (count included), all state bit for bit at the end.  mixed: every third event takes the top-k
    pull instead, so that both kinds of pull work on the same difference vectors."""
    keep_local = bool(flags & dgs.DGS_KEEP_LOCAL_MODEL)
    theta0 = wl.theta0()
    cap = wl.n if capacity is None else capacity
    from _replay import packet_format
    orc = oracle.Oracle.from_workload(wl, keep_local=keep_local, theta0=theta0, packet_format=packet_format(flags))
    ctx = dgs.Context.from_workload(wl, theta0=torch.from_numpy(theta0).to(DEV), flags=flags, pull_all_capacity=cap)
    sched = wl.schedule() if schedule is None else np.asarray(schedule)
    for e in range(len(sched)):
        w = int(sched[e])
        g = wl.gradient(e)
        pkt = ctx.worker_push(w, torch.from_numpy(g).to(DEV))
        pi, pv = packet_to_numpy(ctx, pkt)
        oi, ov = orc.push(w, g)
        assert np.array_equal(pi, oi) and np.array_equal(bits(pv), bits(ov)), f"event {e}: push packet differs"
        ctx.server_apply(w, pkt)
        orc.apply(w, oi, ov)
        if mixed and e % 3 == 2:
            gi, gv = packet_to_numpy(ctx, ctx.worker_pull(w))
            qi, qv = orc.pull(w)
        else:
            vi, vv = ctx.var_packet(ctx.worker_pull_all(w))
            gi, gv = vi.cpu().numpy().view(np.uint32), vv.cpu().numpy()
            qi, qv, held = orc.pull_all(w, cap)
            assert held <= cap
            if not flags & (dgs.DGS_PACKET_BF16 | dgs.DGS_PACKET_FP16):
                assert not ctx.state(dgs.DGS_D, w).any()                   # Eq. 4: v_k = M after the pull
        assert np.array_equal(gi, qi), f"event {e}: pull index set differs"
        assert np.array_equal(bits(gv), bits(qv)), f"event {e}: pull values differ"
        assert ctx.status() == 0
    from _replay import compare_state
    compare_state(ctx, orc, wl.num_workers, keep_local)
    for q in range(wl.num_workers):
        assert dgs.dgs_prev(ctx.handle, q) == orc.prev(q)
    return ctx, orc


@pytest.mark.parametrize("flags,mixed", [(0, False), (dgs.DGS_KEEP_LOCAL_MODEL, False), (dgs.DGS_KEEP_LOCAL_MODEL, True),
                                         (dgs.DGS_SINGLE_STREAM, True)])
def test_full_pull_trajectory_small_ragged(flags, mixed):
    wl = W.custom("ragged", [300, 7, 5000, 64, 1, 2049, 1531], 3, 30, 20_000, grad_kind="normal", grad_scale=1e-2)
    replay_full_pull(wl, flags=flags, mixed=mixed)


# ---- 16-bit packet values ---------------------------------------------------------------------
@pytest.mark.parametrize("flags", [dgs.DGS_PACKET_BF16, dgs.DGS_PACKET_FP16,
                                   dgs.DGS_PACKET_BF16 | dgs.DGS_KEEP_LOCAL_MODEL | dgs.DGS_RESIDUAL_MODE,
                                   dgs.DGS_PACKET_FP16 | dgs.DGS_KEEP_LOCAL_MODEL | dgs.DGS_NO_SPECULATION])
def test_trajectory_with_16_bit_packet_values(flags):
    # Gradients down to 1e-6: binary16 meets its subnormal range and zero, bfloat16 only loses precision.
    # Packets (rounded values), worker state (Eq. 12 untouched, or t - q under Algorithm 1) and the server's
    # remainders (Eq. 6b) must agree with the CPU checker bit for bit.
    wl = W.custom("q16", [300, 7, 5000, 64, 1, 2049, 1531], 3, 30, 20_000, grad_kind="normal", grad_scale=1e-5)
    replay_and_compare(wl, flags=flags, compare_state_every=7)


def test_overlapped_events_with_bfloat16_packets_several_tiles():
    wl = W.custom("q16-async", [150_000, 517, 90_000, 64, 70_001], 5, 60, 5_000, grad_kind="laplace")
    replay_async_and_compare(wl, flags=dgs.DGS_PACKET_BF16 | dgs.DGS_KEEP_LOCAL_MODEL)


def test_full_pull_with_bfloat16_packets_keeps_the_remainders():
    wl = W.custom("q16-full", [40_000, 513, 9_001], 3, 15, 10_000, grad_kind="laplace")
    replay_full_pull(wl, flags=dgs.DGS_PACKET_BF16 | dgs.DGS_KEEP_LOCAL_MODEL, mixed=True)


def test_both_16_bit_formats_at_once_are_refused():
    cfg = dgs.make_config(64, 1, 0.1, 0.9, [0], [64], [1], [1], flags=dgs.DGS_PACKET_BF16 | dgs.DGS_PACKET_FP16)
    import ctypes as C
    out = C.c_uint64(0)
    assert dgs.lib().dgs_arena_bytes(C.byref(cfg), C.byref(out)) == dgs.DGS_EINVAL


def test_full_pull_many_workers_several_tiles():
    # 8 workers in a cycle over 600 K parameters: every pull sends what the seven others and the worker itself pushed
    wl = W.custom("full", [262_144, 70_001, 517, 262_144, 5_194], 8, 40, 2_000, grad_kind="laplace", schedule_kind="cyclic")
    ctx, orc = replay_full_pull(wl, capacity=8 * wl.K_push, flags=dgs.DGS_KEEP_LOCAL_MODEL)
    # Eq. 5: a worker that has just pulled holds the global model (up to the rounding of summing differences)
    w = int(wl.schedule()[-1])
    assert torch.allclose(ctx.state(dgs.DGS_THETA_LOCAL, w), ctx.state(dgs.DGS_THETA), rtol=0, atol=1e-6)


def test_full_pull_overflow_sends_the_lowest_indices_and_reports():
    wl = W.custom("overflow", [40_000, 9_001], 2, 4, 10_000, grad_kind="normal")
    cap = 300                                  # a push carries 491 entries: the first pull cannot take them all
    theta0 = wl.theta0()
    orc = oracle.Oracle.from_workload(wl, theta0=theta0)
    ctx = dgs.Context.from_workload(wl, theta0=torch.from_numpy(theta0).to(DEV), pull_all_capacity=cap)
    g = wl.gradient(0)
    pkt = ctx.worker_push(0, torch.from_numpy(g).to(DEV))
    oi, ov = orc.push(0, g)
    ctx.server_apply(0, pkt)
    orc.apply(0, oi, ov)
    vi, vv = ctx.var_packet(ctx.worker_pull_all(0))
    qi, qv, held = orc.pull_all(0, cap)
    assert held > cap and vi.numel() == cap
    assert np.array_equal(vi.cpu().numpy().view(np.uint32), qi) and np.array_equal(bits(vv.cpu().numpy()), bits(qv))
    assert ctx.status() == dgs.DGS_ELIMIT
    assert np.array_equal(bits(ctx.state(dgs.DGS_D, 0).cpu().numpy()), bits(orc.state(oracle.D, 0)))   # the rest stays
    # without a capacity the call is refused
    plain = dgs.Context.from_workload(wl)
    assert dgs.lib().dgs_worker_pull_all(plain.handle, 0, None) == dgs.DGS_EINVAL


@pytest.mark.parametrize("log2n", [16, 18, 20, 22, 24])
@pytest.mark.parametrize("ppm", W.SWEEP_PPM)
def test_sweep_selection(log2n, ppm):
    n = 1 << log2n
    x = W.sweep_values(n, index=log2n)
    k = W.k_of(n, ppm)
    want = expect_select(x, [n], [k])
    idx, val, _, _ = select_on_gpu(x, [n], [k])
    assert np.array_equal(idx, want)
    assert np.array_equal(bits(val), bits(x[want]))


@pytest.mark.parametrize("log2n,ppm", [(26, 1000), (28, 100)])
def test_sweep_selection_at_the_bandwidth_bound_sizes(log2n, ppm):
    """The two largest vectors of the kernel sweep (2^26 and 2^28 elements), where the selection is
    bound by memory bandwidth; one density each, compared with the CPU checker's selection."""
    n = 1 << log2n
    x = W.sweep_values(n, index=log2n)
    k = W.k_of(n, ppm)
    idx, val, _, ctx = select_on_gpu(x, [n], [k])
    ctx.close()
    want = expect_select(x, [n], [k])
    assert np.array_equal(idx, want)
    assert np.array_equal(bits(val), bits(x[want]))


def test_sweep_scatter_into_33_buffers_matches_the_checker():
    """The sweep's apply: the packet selected from a sweep vector (2^22 values, 1 %), given to
    dgs_server_apply as a foreign packet, is subtracted from theta and from 32 difference vectors
    (Algorithm 2, M <- M - decode(g); Eq. 3) -- compared with the CPU checker's apply, twice in a
    row so that the second subtraction meets nonzero entries."""
    n, N = 1 << 22, 32
    k = W.k_of(n, 10_000)
    x = W.sweep_values(n, index=22)
    chosen = oracle.topk(x, k).astype(np.uint32)
    vals = x[chosen]
    theta0 = W.custom("t", [n], N, 1, 10_000).theta0()
    orc = oracle.Oracle(n, N, 0.1, 0.9, [0], [n], [k], [k], theta0)
    ctx = dgs.Context(n, N, 0.1, 0.9, [0], [n], [k], [k], torch.from_numpy(theta0).to(DEV))
    idx_d = torch.from_numpy(chosen.view(np.int32)).to(DEV)
    val_d = torch.from_numpy(vals).to(DEV)
    pkt = dgs.dgs_packet(idx_d.data_ptr(), val_d.data_ptr(), k)
    for _ in range(2):
        ctx.server_apply(0, pkt)
        orc.apply(0, chosen, vals)
    assert ctx.status() == 0
    assert np.array_equal(bits(ctx.state(dgs.DGS_THETA).cpu().numpy()), bits(orc.state(oracle.THETA)))
    for q in range(N):
        assert np.array_equal(bits(ctx.state(dgs.DGS_D, q).cpu().numpy()), bits(orc.state(oracle.D, q))), f"D[{q}]"
    # the block bounds the scatter maintains still let a pull find the largest entries (Eq. 6a)
    gi, gv = packet_to_numpy(ctx, ctx.worker_pull(5))
    qi, qv = orc.pull(5)
    assert np.array_equal(gi, qi) and np.array_equal(bits(gv), bits(qv))


def test_a_wait_that_cannot_end_gives_up_and_reports():
    """Every device-side wait of the library is bounded.  With DGS_TEST_STALLED_BARRIER the barrier among
    the CTAs of the finalize kernel waits for a CTA that does not exist: each CTA must give up after its
    poll limit, return, and leave DGS_ETIMEOUT in the status word; the device stays usable."""
    import time
    wl = W.custom("stall", [70_000, 513], 2, 2, 10_000)
    ctx = dgs.Context.from_workload(wl, flags=dgs.DGS_TEST_STALLED_BARRIER)
    g = torch.from_numpy(wl.gradient(0)).to(DEV)
    t0 = time.perf_counter()
    ctx.worker_push(0, g)
    assert ctx.status() == dgs.DGS_ETIMEOUT
    ctx.worker_pull(1)
    assert ctx.status() == dgs.DGS_ETIMEOUT            # sticky
    assert time.perf_counter() - t0 < 10.0
    ctx.close()
    # a context made afterwards on the same device runs clean
    replay_and_compare(W.custom("after", [40_000, 517], 2, 4, 10_000))


def test_apply_foreign_packet_and_bad_index_is_reported():
    n = 5000
    ctx = dgs.Context(n, 2, 0.1, 0.9, [0], [n], [10], [10], torch.zeros(n, device=DEV))
    idx = torch.tensor([1, 7, 4999], dtype=torch.int32, device=DEV)
    val = torch.tensor([1.0, -2.0, 0.5], device=DEV)
    pkt = dgs.dgs_packet(idx.data_ptr(), val.data_ptr(), 3)
    ctx.server_apply(0, pkt)
    th = ctx.state(dgs.DGS_THETA).cpu().numpy()
    assert th[1] == -1.0 and th[7] == 2.0 and th[4999] == -0.5 and np.count_nonzero(th) == 3
    for q in range(2):
        assert np.array_equal(ctx.state(dgs.DGS_D, q).cpu().numpy(), th)
    assert ctx.status() == 0
    bad = torch.tensor([5000], dtype=torch.int32, device=DEV)   # out of range: skipped and flagged
    ctx.server_apply(0, dgs.dgs_packet(bad.data_ptr(), val.data_ptr(), 1))
    assert ctx.status() != 0
    assert np.array_equal(ctx.state(dgs.DGS_THETA).cpu().numpy(), th)


def test_argument_errors_on_a_live_context():
    n = 4096
    ctx = dgs.Context(n, 2, 0.1, 0.9, [0], [n], [4], [4], torch.zeros(n, device=DEV))
    g = torch.zeros(n + 1, device=DEV)
    L = dgs.lib()
    import ctypes as C
    p = dgs.dgs_packet()
    assert L.dgs_worker_push(ctx.handle, 2, g.data_ptr(), C.byref(p)) == dgs.DGS_EINVAL   # worker out of range
    assert L.dgs_worker_push(ctx.handle, 0, None, C.byref(p)) == dgs.DGS_EINVAL
    assert L.dgs_worker_push(ctx.handle, 0, g.data_ptr() + 4, C.byref(p)) == dgs.DGS_EINVAL  # misaligned
    assert L.dgs_worker_pull(ctx.handle, 5, C.byref(p)) == dgs.DGS_EINVAL
    assert L.dgs_event_host(ctx.handle, 0, None, None, None) == dgs.DGS_EINVAL            # no DGS_HOST_IO
    out = C.c_void_p()
    assert L.dgs_state_ptr(ctx.handle, dgs.DGS_THETA_LOCAL, 0, C.byref(out)) == dgs.DGS_EINVAL
    small = dgs.make_config(n, 2, 0.1, 0.9, [0], [n], [4], [4], theta0=g.data_ptr(),
                            arena=ctx.arena.data_ptr(), arena_bytes=1024)
    h = C.c_void_p()
    assert L.dgs_init(C.byref(small), C.byref(h)) == dgs.DGS_ENOMEM


def test_event_host_matches_device_path():
    wl = W.custom("host", [70_000, 513], 2, 6, 10_000, grad_kind="laplace")
    theta0 = torch.from_numpy(wl.theta0()).to(DEV)
    a = dgs.Context.from_workload(wl, theta0=theta0, flags=dgs.DGS_HOST_IO)
    b = dgs.Context.from_workload(wl, theta0=theta0)
    idx = torch.empty(wl.K_pull, dtype=torch.int32).pin_memory()
    val = torch.empty(wl.K_pull, dtype=torch.float32).pin_memory()
    for e, w in enumerate(wl.schedule()):
        g = torch.from_numpy(wl.gradient(e)).pin_memory()
        a.event_host(int(w), g, idx, val)
        _, pull = b.event(int(w), g.to(DEV))
        bi, bv = packet_to_numpy(b, pull)
        assert np.array_equal(idx.numpy().view(np.uint32), bi) and np.array_equal(bits(val.numpy()), bits(bv))
    assert torch.equal(a.state(dgs.DGS_THETA), b.state(dgs.DGS_THETA))


def test_two_runs_are_bit_identical():
    wl = W.custom("det", [100_000], 3, 12, 1000)
    outs = []
    for _ in range(2):
        ctx = dgs.Context.from_workload(wl)
        # gradients must outlive the (asynchronous) events that read them
        grads = [torch.from_numpy(wl.gradient(e)).to(DEV) for e in range(wl.num_events)]
        for e, w in enumerate(wl.schedule()):
            ctx.event(int(w), grads[e])
        outs.append([ctx.state(dgs.DGS_THETA).clone()] +
                    [ctx.state(dgs.DGS_U, q).clone() for q in range(3)] +
                    [ctx.state(dgs.DGS_D, q).clone() for q in range(3)])
    for x, y in zip(*outs):
        assert torch.equal(x.view(torch.int32), y.view(torch.int32))
