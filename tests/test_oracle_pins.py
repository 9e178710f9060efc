"""Pins for the CPU checker: each test fixes its behaviour by something other
than the checker itself -- a brute-force sort, a hand-worked trajectory, an
independent serial momentum loop, and identities the paper states."""
import os

import numpy as np
import pytest

import oracle
import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def key(x):
    return np.ascontiguousarray(x, dtype=np.float32).view(np.uint32) & np.uint32(0x7FFFFFFF)


def brute_topk(x, k):
    """Full stable sort by (|x| bit pattern descending, index ascending)."""
    ks = [int(v) for v in key(x)]
    order = sorted(range(len(ks)), key=lambda i: (-ks[i], i))
    return np.array(sorted(order[:k]), dtype=np.uint64)


# ---- TOPK against brute force ------------------------------------------------
@pytest.mark.parametrize("seed", range(20))
def test_topk_random_vs_full_sort(seed):
    r = np.random.default_rng(seed)
    n = int(r.integers(1, 65))
    k = int(r.integers(1, n + 1))
    x = r.standard_normal(n).astype(np.float32)
    # force duplicates so the boundary is often tied
    x = np.round(x * 2) / 2
    assert np.array_equal(oracle.topk(x, k), brute_topk(x, k))


def test_topk_adversarial():
    cases = [
        (np.ones(17, np.float32), 5),                      # all equal: lowest indices win
        (np.zeros(9, np.float32), 3),                      # all zero
        (np.array([0.0, -0.0, 0.0, -0.0], np.float32), 2),  # +0 and -0 tie
        (np.array([1, -1, 1, -1, 2], np.float32), 3),      # sign ignored, tie at the boundary
        (np.array([3, 1, 2], np.float32), 1),
        (np.array([3, 1, 2], np.float32), 3),              # k = len
        (np.array([5.0], np.float32), 1),                  # one element
        (np.array([1e-45, 0, -1e-45, 1e-40, 0], np.float32), 2),  # denormals are ordered, not flushed
    ]
    for x, k in cases:
        got = oracle.topk(x, k)
        assert np.array_equal(got, brute_topk(x, k)), (x, k, got)
    assert list(oracle.topk(np.ones(17, np.float32), 5)) == [0, 1, 2, 3, 4]
    assert list(oracle.topk(np.array([1, -1, 1, -1, 2], np.float32), 3)) == [0, 1, 4]
    assert list(oracle.topk(np.array([1e-45, 0, -1e-45, 1e-40, 0], np.float32), 2)) == [0, 3]


# ---- hand-worked trajectory ----------------------------------------------------
def _read_golden(path):
    head, events, cur = {}, [], None
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tok = line.split()
        if tok[0] == "event":
            cur = {"worker": int(tok[3])}
            events.append(cur)
        elif cur is None:
            head[tok[0]] = tok[1:]
        else:
            cur[tok[0]] = np.array([float(v) for v in tok[1:]])
    return head, events


@pytest.mark.parametrize("name", ["hand_example.txt", "hand_example_algorithm1.txt", "hand_example_full_pull.txt",
                                  "hand_example_bf16_packets.txt"])
def test_hand_example(name):
    head, events = _read_golden(os.path.join(GOLDEN, name))
    n, N, k = int(head["n"][0]), int(head["workers"][0]), int(head["k"][0])
    theta0 = np.array([float(v) for v in head["theta0"]], np.float32)
    residual = head.get("mode", ["momentum"])[0] == "residual"       # worker rule of Algorithm 1
    full_pull = head.get("mode", ["momentum"])[0] == "full_pull"     # Algorithm 2 without secondary compression
    fmt = oracle.BF16 if head.get("mode", ["momentum"])[0] == "bf16" else oracle.FP32
    o = oracle.Oracle(n, N, float(head["lr"][0]), float(head["momentum"][0]),
                      [0], [n], [k], [k], theta0, keep_local=True, residual_mode=residual,
                      packet_format=fmt)
    assert o.timestamp == 0 and [o.prev(q) for q in range(N)] == [-1] * N
    for ev in events:
        w = ev["worker"]
        pi, pv = o.push(w, ev["grad"].astype(np.float32))
        assert list(pi) == list(ev["push_idx"]) and list(pv) == list(ev["push_val"])
        assert list(o.state(oracle.U, w)) == list(ev["u"])
        o.apply(w, pi, pv)
        assert list(o.state(oracle.THETA)) == list(ev["theta"])
        assert list(o.state(oracle.D, 0)) == list(ev["D0_after_apply"])
        assert list(o.state(oracle.D, 1)) == list(ev["D1_after_apply"])
        if full_pull:
            gi, gv, held = o.pull_all(w)
            assert held == len(gi)
        else:
            gi, gv = o.pull(w)
        assert list(gi) == list(ev["pull_idx"]) and list(gv) == list(ev["pull_val"])
        assert list(o.state(oracle.D, 0)) == list(ev["D0"])
        assert list(o.state(oracle.D, 1)) == list(ev["D1"])
        assert list(o.state(oracle.THETA_LOCAL, w)) == list(ev["theta_local"])
        # Algorithm 2, last lines: t counts the applied packets, prev(k) = t when k has been served
        assert o.timestamp == int(ev["timestamp"][0])
        assert [o.prev(q) for q in range(N)] == [int(v) for v in ev["prev"]]
        # Eq. 3-5: every worker's copy plus what the server still owes it is the global model
        for q in range(N):
            assert np.array_equal(o.state(oracle.THETA_LOCAL, q) + o.state(oracle.D, q),
                                  o.state(oracle.THETA))


# ---- dense limit: DGS without sparsification is momentum ASGD (Eq. 4, Eq. 5) ----
def test_dense_limit_is_serial_momentum_asgd():
    n, N, E = 257, 3, 12
    lr, m = np.float32(0.1), np.float32(0.9)
    r = np.random.default_rng(7)
    theta0 = r.standard_normal(n).astype(np.float32)
    o = oracle.Oracle(n, N, lr, m, [0, 100], [100, 157], [100, 157], [100, 157], theta0,
                      keep_local=True)
    theta = theta0.copy()
    u = np.zeros((N, n), np.float32)
    sched = r.integers(0, N, E)
    for e in range(E):
        w = int(sched[e])
        g = r.standard_normal(n).astype(np.float32)
        # independent serial loop: u_w <- m u_w + eta g ; theta <- theta - u_w   (Eq. 8)
        u[w] = m * u[w] + lr * g
        theta = theta - u[w]
        (pi, pv), (gi, gv) = o.event(w, g)
        assert np.array_equal(pi, np.arange(n)) and np.array_equal(gi, np.arange(n))
        assert np.array_equal(o.state(oracle.U, w), u[w])
        assert np.array_equal(o.state(oracle.THETA), theta)
        assert not o.state(oracle.D, w).any()                       # Eq. 4: v_k = M after a pull
        # Eq. 5: theta_local = theta, up to the rounding of the sum of pulled differences
        # (theta itself moved by single subtractions, theta_local by the accumulated D)
        assert np.allclose(o.state(oracle.THETA_LOCAL, w), theta, rtol=0, atol=2e-5)


# ---- Eq. 13: an entry unsent for T-1 steps carries m*u_c + eta*sum(grad) ----------
@pytest.mark.parametrize("m", [0.5, 0.9, 0.7])
def test_telescoping_unsent_velocity(m):
    n, T, lr = 64, 9, 0.25
    r = np.random.default_rng(3)
    o = oracle.Oracle(n, 1, lr, m, [0], [n], [2], [2], np.zeros(n, np.float32))
    acc64 = np.zeros(n, np.float64)
    acc32 = np.zeros(n, np.float32)
    for t in range(T):
        g = r.standard_normal(n).astype(np.float32)
        g[0], g[1] = 1e6, -1e6            # two entries that always win k = 2
        acc64 += lr * g.astype(np.float64)
        acc32 = acc32 + np.float32(lr) * g
        pi, pv = o.push(0, g)
        assert list(pi) == [0, 1]
        u_unsent = o.state(oracle.U, 0)[2:]
        if m == 0.5:
            # 1/m = 2 and m*(2x) = x are exact: the stored value is exactly twice the
            # running float32 sum of eta*grad (u_c = 0)
            assert np.array_equal(u_unsent, np.float32(2.0) * acc32[2:])
        else:
            # pre-selection velocity t = m * u'; each step adds a few roundings
            t_unsent = u_unsent.astype(np.float64) * float(np.float32(m))
            tol = 4 * (t + 1) * 2.0 ** -24 * np.abs(acc64[2:]).max()
            assert np.max(np.abs(t_unsent - acc64[2:])) <= tol
    # the sent entries keep their velocity (Eq. 12 upper branch): geometric sum of eta*g
    expect0 = sum(lr * 1e6 * m ** j for j in range(T))
    assert abs(o.state(oracle.U, 0)[0] - expect0) <= 1e-5 * expect0


# ---- Eq. 12 and the exact split of push and pull ---------------------------------
@pytest.mark.parametrize("residual_mode", [False, True])
def test_piecewise_state_and_exact_split(residual_mode):
    wl = W.custom("mini", [300, 7, 1000, 64], 3, 10, 20_000, grad_kind="normal", grad_scale=1e-2)
    o = oracle.Oracle.from_workload(wl, keep_local=True, residual_mode=residual_mode)
    m, lr = np.float32(wl.momentum), np.float32(wl.lr)
    inv_m = np.float32(1.0) / m
    theta0 = wl.theta0()
    applied = np.zeros(wl.n, np.float64)
    theta_serial = theta0.copy()
    for e, w in enumerate(wl.schedule()):
        w = int(w)
        g = wl.gradient(e)
        u_before = o.state(oracle.U, w).copy()
        t = (u_before + lr * g) if residual_mode else (m * u_before + lr * g)
        pi, pv = o.push(w, g)
        u_after = o.state(oracle.U, w)
        sent = np.zeros(wl.n, bool)
        sent[pi] = True
        # density: exactly k per layer, ascending, inside the layer (I4)
        assert np.all(np.diff(pi.astype(np.int64)) > 0)
        for off, ln, k in zip(wl.seg_offset, wl.seg_len, wl.k_push):
            assert int(sent[int(off):int(off + ln)].sum()) == int(k)
            # threshold property (I5): nothing unsent is larger than something sent
            seg_t = key(t[int(off):int(off + ln)])
            seg_s = sent[int(off):int(off + ln)]
            if (~seg_s).any():
                assert seg_t[seg_s].min() >= seg_t[~seg_s].max()
        assert np.array_equal(pv, t[pi])
        if residual_mode:   # Algorithm 1: sent part leaves the residual, the rest stays
            assert np.array_equal(u_after[~sent], t[~sent]) and not u_after[sent].any()
        else:               # Eq. 12
            assert np.array_equal(u_after[sent], t[sent])
            assert np.array_equal(u_after[~sent], t[~sent] * inv_m)
        D_before = [o.state(oracle.D, q).copy() for q in range(wl.num_workers)]
        o.apply(w, pi, pv)
        applied[pi] += pv.astype(np.float64)
        theta_serial[pi] = theta_serial[pi] - pv
        for q in range(wl.num_workers):
            exp = D_before[q].copy()
            exp[pi] = exp[pi] - pv
            assert np.array_equal(o.state(oracle.D, q), exp)
        Dw = o.state(oracle.D, w).copy()
        gi, gv = o.pull(w)
        # exact split (sent + retained = accumulated), disjoint supports
        back = o.state(oracle.D, w).copy()
        assert not back[gi].any()
        back[gi] = gv
        assert np.array_equal(back, Dw)
        assert np.all(np.diff(gi.astype(np.int64)) > 0)
        # Eq. 2: the server model is the initial model plus everything applied
        assert np.array_equal(o.state(oracle.THETA), theta_serial)
        assert np.allclose(o.state(oracle.THETA), theta0 - applied, rtol=1e-6, atol=1e-7)
        for q in range(wl.num_workers):
            assert np.allclose(o.state(oracle.THETA_LOCAL, q) + o.state(oracle.D, q),
                               o.state(oracle.THETA), rtol=0, atol=1e-6)
    assert o.timestamp == wl.num_events


# ---- 16-bit packet values ---------------------------------------------------------------------
def test_round16_is_the_library_conversion_and_saturates():
    import torch
    r = np.random.default_rng(0)
    x = r.standard_normal(20000).astype(np.float32) * np.float32(10.0) ** r.integers(-9, 5, 20000).astype(np.float32)
    x = np.concatenate([x, np.array([0, -0.0, 1 + 2 ** -8, 1 + 2 ** -8 + 2 ** -9, 65504, 65519.99, 2 ** -24, 2 ** -25,
                                     2 ** -25 * 1.0001, 3 * 2 ** -25, 6e-8, 2 ** -14, 2 ** -14 - 2 ** -26], np.float32)])
    half = np.array([oracle.round16(v, oracle.FP16) for v in x], np.float32)
    inside = np.abs(x) < 65520
    want = x[inside].astype(np.float16).astype(np.float32)              # numpy's IEEE binary16 conversion
    assert np.array_equal(half[inside].view(np.uint32), want.view(np.uint32))
    assert np.all(np.abs(half[~inside]) == 65504) and np.array_equal(np.sign(half[~inside]), np.sign(x[~inside]))
    bf = np.array([oracle.round16(v, oracle.BF16) for v in x], np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()   # torch's bfloat16 conversion
    assert np.array_equal(bf.view(np.uint32), want.view(np.uint32))
    # by hand: ties go to the even neighbour; beyond the largest finite binary16 the value saturates
    assert oracle.round16(1 + 2 ** -8, oracle.BF16) == 1.0 and oracle.round16(1 + 3 * 2 ** -8, oracle.BF16) == 1 + 2 ** -6
    assert oracle.round16(1 + 2 ** -11, oracle.FP16) == 1.0 and oracle.round16(1 + 3 * 2 ** -11, oracle.FP16) == 1 + 2 ** -9
    assert oracle.round16(65520.0, oracle.FP16) == 65504.0 and oracle.round16(-1e9, oracle.FP16) == -65504.0
    assert oracle.round16(2 ** -25, oracle.FP16) == 0.0 and oracle.round16(3 * 2 ** -25, oracle.FP16) == 2 ** -23
    assert oracle.round16(0.1, oracle.FP32) == np.float32(0.1)


@pytest.mark.parametrize("fmt", [1, 2])
@pytest.mark.parametrize("residual_mode", [False, True])
def test_rounded_packets_keep_the_books(fmt, residual_mode):
    """With 16-bit packet values: what a packet carries is the rounded selected value; the worker's state
    follows Eq. 12 (or keeps t - q under Algorithm 1); the server's residual keeps what a pull's rounding
    left behind, so theta_k + D_k still equals theta (Eq. 3-5) up to float32 rounding."""
    wl = W.custom("mini", [300, 7, 1000, 64], 3, 12, 20_000, grad_kind="normal", grad_scale=1e-2)
    o = oracle.Oracle.from_workload(wl, keep_local=True, residual_mode=residual_mode, packet_format=fmt)
    m, lr = np.float32(wl.momentum), np.float32(wl.lr)
    for e, w in enumerate(wl.schedule()):
        w = int(w)
        g = wl.gradient(e)
        u_before = o.state(oracle.U, w).copy()
        t = (u_before + lr * g) if residual_mode else (m * u_before + lr * g)
        pi, pv = o.push(w, g)
        q = np.array([oracle.round16(v, fmt) for v in t[pi]], np.float32)
        assert np.array_equal(pv, q)
        u_after = o.state(oracle.U, w)
        assert np.array_equal(u_after[pi], (t[pi] - q) if residual_mode else t[pi])
        o.apply(w, pi, pv)
        Dw = o.state(oracle.D, w).copy()
        gi, gv = o.pull(w)
        q = np.array([oracle.round16(v, fmt) for v in Dw[gi]], np.float32)
        assert np.array_equal(gv, q)
        left = o.state(oracle.D, w)
        assert np.array_equal(left[gi], Dw[gi] - q)                       # the remainder stays with the server
        rest = np.ones(wl.n, bool)
        rest[gi] = False
        assert np.array_equal(left[rest], Dw[rest])
        assert np.all(np.abs(left[gi]) <= np.abs(Dw[gi]) * 2.0 ** -8 + 1e-45)   # at most half a step of the format
        for q_ in range(wl.num_workers):
            assert np.allclose(o.state(oracle.THETA_LOCAL, q_) + o.state(oracle.D, q_), o.state(oracle.THETA),
                               rtol=0, atol=1e-6)


# ---- pull without secondary compression: v_k = M afterwards (Eq. 4), theta_k = theta (Eq. 5) ----
def test_full_pull_sends_every_nonzero_and_leaves_nothing():
    wl = W.custom("mini", [300, 7, 1000, 64], 3, 12, 20_000, grad_kind="normal", grad_scale=1e-2)
    o = oracle.Oracle.from_workload(wl, keep_local=True)
    for e, w in enumerate(wl.schedule()):
        w = int(w)
        pi, pv = o.push(w, wl.gradient(e))
        o.apply(w, pi, pv)
        Dw = o.state(oracle.D, w).copy()
        gi, gv, held = o.pull_all(w)
        nz = np.nonzero(Dw)[0]
        assert held == len(nz) and np.array_equal(gi, nz.astype(np.uint32)) and np.array_equal(gv, Dw[nz])
        assert not o.state(oracle.D, w).any()                                   # Eq. 4: v_k = M
        # Eq. 5: the worker's model is the global one, up to the rounding of summing differences
        assert np.allclose(o.state(oracle.THETA_LOCAL, w), o.state(oracle.THETA), rtol=0, atol=1e-6)
        assert o.prev(w) == o.timestamp
    # overflow: a capacity below the number of nonzeros sends the first `cap` and keeps the rest
    pi, pv = o.push(0, wl.gradient(99))
    o.apply(0, pi, pv)
    Dw = o.state(oracle.D, 1).copy()
    nz = np.nonzero(Dw)[0]
    assert len(nz) > 3
    gi, gv, held = o.pull_all(1, cap=3)
    assert held == len(nz) and list(gi) == list(nz[:3])
    left = o.state(oracle.D, 1)
    assert not left[nz[:3]].any() and np.array_equal(left[nz[3:]], Dw[nz[3:]])


def test_fewer_nonzeros_than_k_fills_with_lowest_zero_indices():
    n = 32
    o = oracle.Oracle(n, 2, 1.0, 0.5, [0], [n], [2], [5], np.zeros(n, np.float32))
    g = np.zeros(n, np.float32)
    g[10], g[20] = 3.0, -4.0
    (pi, pv), (gi, gv) = o.event(0, g)
    assert list(pi) == [10, 20]
    assert list(gi) == [0, 1, 2, 10, 20] and list(gv) == [0, 0, 0, -3, 4]


def test_determinism_same_seed_same_bytes():
    outs = []
    for _ in range(2):
        wl = W.custom("mini", [500, 12], 2, 6, 10_000)
        o = oracle.Oracle.from_workload(wl)
        acc = []
        for e, w in enumerate(wl.schedule()):
            (pi, pv), (gi, gv) = o.event(int(w), wl.gradient(e))
            acc += [pi.tobytes(), pv.tobytes(), gi.tobytes(), gv.tobytes()]
        acc.append(o.state(oracle.THETA).tobytes())
        outs.append(b"".join(acc))
    assert outs[0] == outs[1]
