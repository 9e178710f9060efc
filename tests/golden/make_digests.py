#!/usr/bin/env python
"""Writes tests/golden/digests_<workload>.json: what the CPU checker computes for a whole
workload at its stated size, reduced to hashes.

    python tests/golden/make_digests.py resnet18 resnet50 gpt2 [--events E]

The script imports only the CPU checker (``oracle``) and the input generators
(``workloads``); nothing of the CUDA library is touched, so the stored values are the
checker's own.  For every event it stores a hash of the push packet and of the pull packet
(index bytes followed by value bytes), and after the last event one hash per state vector
(theta, every u_q, every D_q).  The GPU tests replay the same seeded events through the
library and compare every hash; a full run of the checker (minutes to half an hour, tens of
GB of host memory for the largest workload) is then not needed inside the test.

Hashing (BLAKE2b, 8-byte digests) is bookkeeping, not part of the method.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import sys
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import oracle  # noqa: E402
import workloads as W  # noqa: E402


def digest(*arrays: np.ndarray) -> str:
    h = hashlib.blake2b(digest_size=8)
    for a in arrays:
        h.update(np.ascontiguousarray(a).view(np.uint8).data)
    return h.hexdigest()


def run(name: str, events: int, threads: int) -> dict:
    wl = W.BY_NAME[name]()
    E = wl.num_events if events <= 0 else min(events, wl.num_events)
    sched = wl.schedule()
    o = oracle.Oracle.from_workload(wl)
    push, pull = [], []
    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=threads) as ex:
        ahead = {}
        nxt = 0
        for e in range(E):
            while nxt < E and nxt < e + 2 * threads:        # gradients are generated a few events ahead
                ahead[nxt] = ex.submit(wl.gradient, nxt)
                nxt += 1
            g = ahead.pop(e).result()
            (pi, pv), (gi, gv) = o.event(int(sched[e]), g)
            push.append(digest(pi, pv))
            pull.append(digest(gi, gv))
            if (e + 1) % 32 == 0:
                print(f"{name}: {e + 1}/{E} events, {time.perf_counter() - t0:.0f} s", file=sys.stderr, flush=True)
        N = wl.num_workers
        state = {"theta": digest(o.state(oracle.THETA))}
        state["u"] = list(ex.map(lambda q: digest(o.state(oracle.U, q)), range(N)))
        state["D"] = list(ex.map(lambda q: digest(o.state(oracle.D, q)), range(N)))
    out = {
        "workload": wl.name, "constructor": name, "seed": wl.seed, "n": wl.n, "workers": wl.num_workers,
        "segments": wl.num_segments, "K_push": wl.K_push, "K_pull": wl.K_pull, "lr": wl.lr,
        "momentum": wl.momentum, "events": E, "events_of_workload": wl.num_events,
        "hash": "blake2b-64 over index bytes then value bytes (packets), over the float32 bytes (state)",
        "written_by": "tests/golden/make_digests.py (CPU checker only)",
        "timestamp_after": o.timestamp, "prev_after": [o.prev(q) for q in range(N)],
        "push": push, "pull": pull, "state": state,
    }
    o.close()
    return out


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("workloads", nargs="+", choices=sorted(W.BY_NAME))
    ap.add_argument("--events", type=int, default=0, help="only the first E events (default: the whole workload)")
    ap.add_argument("--threads", type=int, default=max(1, min(6, (os.cpu_count() or 2) - 1)))
    args = ap.parse_args()
    for name in args.workloads:
        out = run(name, args.events, args.threads)
        path = os.path.join(HERE, f"digests_{name}.json")
        with open(path, "w") as f:
            json.dump(out, f, indent=0)
            f.write("\n")
        print(f"wrote {path}: {out['events']} events", file=sys.stderr, flush=True)


if __name__ == "__main__":
    main()
