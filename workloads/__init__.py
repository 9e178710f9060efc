"""Seeded synthetic inputs for the DGS push/apply/pull loop.

This module only *makes inputs*: parameter-segment tables, initial models,
arrival schedules and per-event gradients.  It contains none of the method's
arithmetic (no momentum update, no selection, no scatter) and is the one module
that both the CPU checker and the CUDA path are fed from, so that both always
see byte-identical inputs.  Everything is generated with numpy on the host from
one master seed; sub-streams are keyed by (purpose, event number) so that the
gradient of event ``e`` does not depend on how many other events were drawn.

The paper trains ResNet-18/50 on CIFAR-10 and an LSTM on AN4 (Section
"Dataset and Models").  Those datasets are not used here: the workloads below
take only the parameter *shapes* of the named architectures and draw the
gradients from fixed distributions.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

from . import shapes as _shapes

_STREAM_THETA0 = 1
_STREAM_SCHEDULE = 2
_STREAM_SCALES = 3
_STREAM_GRAD = 4
_STREAM_SWEEP = 5

DEFAULT_SEED = 1910


def _rng(seed: int, stream: int, index: int = 0) -> np.random.Generator:
    ss = np.random.SeedSequence(entropy=int(seed), spawn_key=(int(stream), int(index)))
    return np.random.Generator(np.random.Philox(ss))


def k_of(length: int, density_ppm: int) -> int:
    """Entries kept out of ``length`` at a density given in parts per million:
    the ceiling of length*density, and never fewer than one."""
    return max(1, (int(length) * int(density_ppm) + 999_999) // 1_000_000)


@dataclass
class Workload:
    name: str
    n: int
    num_workers: int
    num_events: int
    lr: float
    momentum: float
    seg_offset: np.ndarray            # uint64[S]
    seg_len: np.ndarray               # uint64[S]
    k_push: np.ndarray                # uint32[S]
    k_pull: np.ndarray                # uint32[S]
    grad_kind: str                    # "normal" | "laplace" | "student_t" | "sweep"
    tensor_sizes: List[int] = field(default_factory=list)
    schedule_kind: str = "uniform"    # "uniform" | "cyclic"
    seed: int = DEFAULT_SEED
    grad_scale: float = 1.0
    zero_rows: Optional[tuple] = None  # (tensor index, rows, cols, keep probability)
    _scale_vec: Optional[np.ndarray] = field(default=None, repr=False)

    # ---- static tables -------------------------------------------------
    @property
    def num_segments(self) -> int:
        return int(self.seg_len.shape[0])

    @property
    def K_push(self) -> int:
        return int(self.k_push.sum())

    @property
    def K_pull(self) -> int:
        return int(self.k_pull.sum())

    def theta0(self) -> np.ndarray:
        """Initial model, N(0, 0.05^2), float32[n]."""
        r = _rng(self.seed, _STREAM_THETA0)
        x = r.standard_normal(self.n, dtype=np.float32)
        x *= np.float32(0.05)
        return x

    def schedule(self) -> np.ndarray:
        """Arrival order: ``schedule[e]`` is the worker served at event ``e``."""
        r = _rng(self.seed, _STREAM_SCHEDULE)
        N, E = self.num_workers, self.num_events
        if self.schedule_kind == "uniform":
            return r.integers(0, N, size=E, dtype=np.int64).astype(np.int32)
        # Staleness capped at N-1 other events between two arrivals of a worker.
        # With N workers served one per event the mean gap is N, so a cap of N-1
        # leaves exactly one order: a fixed cycle through a seeded permutation
        # (every arrival after the first round has staleness N-1).
        perm = r.permutation(N).astype(np.int32)
        return np.resize(perm, E)

    # ---- gradients -----------------------------------------------------
    def _scales(self) -> np.ndarray:
        """Per-element Laplace scale: b_l = 10^(-5+3U) per tensor, repeated."""
        if self._scale_vec is None:
            r = _rng(self.seed, _STREAM_SCALES)
            b = np.power(10.0, -5.0 + 3.0 * r.random(len(self.tensor_sizes))).astype(np.float32)
            self._scale_vec = np.repeat(b, self.tensor_sizes)
            assert self._scale_vec.shape[0] == self.n
        return self._scale_vec

    def gradient(self, e: int, out: Optional[np.ndarray] = None) -> np.ndarray:
        """Stochastic gradient handed to the worker served at event ``e``, float32[n]."""
        r = _rng(self.seed, _STREAM_GRAD, e)
        n = self.n
        if out is None:
            out = np.empty(n, dtype=np.float32)
        assert out.dtype == np.float32 and out.shape == (n,)
        if self.grad_kind == "normal":
            r.standard_normal(n, dtype=np.float32, out=out)
            out *= np.float32(self.grad_scale)
        elif self.grad_kind == "laplace":
            r.standard_exponential(n, dtype=np.float32, out=out)
            out *= self._scales()
            s = r.random(n, dtype=np.float32)
            s -= np.float32(0.5)
            np.copysign(out, s, out=out)
        elif self.grad_kind == "student_t":
            self._student_t(r, out)
        elif self.grad_kind == "sweep":
            sweep_values(n, self.seed, e, out=out)
        else:
            raise ValueError(self.grad_kind)
        return out

    def _student_t(self, r: np.random.Generator, out: np.ndarray) -> None:
        # t_3 = Z / sqrt(chi2_3 / 3), chi2_3 = 2*Gamma(3/2); rows of the one
        # "zero_rows" tensor are all-zero except with the keep probability.
        def fill(dst: np.ndarray) -> None:
            m = dst.shape[0]
            z = r.standard_normal(m, dtype=np.float32)
            g = r.standard_gamma(1.5, size=m, dtype=np.float32)
            g *= np.float32(2.0 / 3.0)
            np.sqrt(g, out=g)
            np.divide(z, g, out=dst)
            dst *= np.float32(self.grad_scale)

        if self.zero_rows is None:
            fill(out)
            return
        t_idx, rows, cols, keep = self.zero_rows
        start = int(sum(self.tensor_sizes[:t_idx]))
        stop = start + rows * cols
        live = np.nonzero(r.random(rows) < keep)[0]
        emb = out[start:stop].reshape(rows, cols)
        emb[:] = 0.0
        buf = np.empty(live.shape[0] * cols, dtype=np.float32)
        fill(buf)
        emb[live] = buf.reshape(-1, cols)
        if start > 0:
            fill(out[:start])
        fill(out[stop:])


def sweep_values(n: int, seed: int = DEFAULT_SEED, index: int = 0,
                 out: Optional[np.ndarray] = None) -> np.ndarray:
    """Kernel-sweep vector: N(0,1) with a seeded 1 % of positions scaled by 100."""
    r = _rng(seed, _STREAM_SWEEP, index)
    if out is None:
        out = np.empty(n, dtype=np.float32)
    r.standard_normal(n, dtype=np.float32, out=out)
    hot = r.random(n, dtype=np.float32) < np.float32(0.01)
    out[hot] *= np.float32(100.0)
    return out


# ---- workload constructors --------------------------------------------------
def _segments_from_sizes(sz: Sequence[int], ppm_push: int, ppm_pull: int):
    ln = np.asarray(sz, dtype=np.uint64)
    off = np.concatenate([[0], np.cumsum(ln)[:-1]]).astype(np.uint64)
    kp = np.asarray([k_of(x, ppm_push) for x in sz], dtype=np.uint32)
    kl = np.asarray([k_of(x, ppm_pull) for x in sz], dtype=np.uint32)
    return off, ln, kp, kl


def custom(name: str, seg_sizes: Sequence[int], num_workers: int, num_events: int,
           density_ppm: int, *, density_pull_ppm: Optional[int] = None, lr: float = 0.1,
           momentum: float = 0.9, grad_kind: str = "normal", grad_scale: float = 1e-3,
           schedule_kind: str = "uniform", seed: int = DEFAULT_SEED,
           tensor_sizes: Optional[Sequence[int]] = None,
           zero_rows: Optional[tuple] = None) -> Workload:
    """A workload over segments of the given sizes, each selected on its own."""
    pull = density_ppm if density_pull_ppm is None else density_pull_ppm
    off, ln, kp, kl = _segments_from_sizes(seg_sizes, density_ppm, pull)
    n = int(ln.sum())
    return Workload(name, n, num_workers, num_events, lr, momentum, off, ln, kp, kl,
                    grad_kind, list(tensor_sizes if tensor_sizes is not None else seg_sizes),
                    schedule_kind, seed, grad_scale, zero_rows)


def flat_1m(num_workers: int = 4, num_events: int = 16, seed: int = DEFAULT_SEED) -> Workload:
    """Flat vector n = 2^20, Gaussian gradients, density 0.1 % (k = 1049)."""
    return custom("flat-2^20", [1 << 20], num_workers, num_events, 1000,
                  grad_kind="normal", grad_scale=1e-3, schedule_kind="uniform", seed=seed)


def resnet18(num_workers: int = 32, num_events: int = 256, seed: int = DEFAULT_SEED) -> Workload:
    """ResNet-18 shapes, per-layer Laplace gradients, 1 % density per layer."""
    sz = _shapes.sizes(_shapes.resnet18_shapes())
    assert sum(sz) == 11_689_512 and len(sz) == 62
    return custom("resnet18-per-layer", sz, num_workers, num_events, 10_000,
                  grad_kind="laplace", schedule_kind="cyclic", seed=seed)


def resnet50(num_workers: int = 32, num_events: int = 1024, seed: int = DEFAULT_SEED) -> Workload:
    """ResNet-50 shapes, per-layer Laplace scales, one global 0.1 % selection."""
    sz = _shapes.sizes(_shapes.resnet50_shapes())
    assert sum(sz) == 25_557_032 and len(sz) == 161
    return custom("resnet50-global", [sum(sz)], num_workers, num_events, 1000,
                  grad_kind="laplace", schedule_kind="cyclic", seed=seed, tensor_sizes=sz)


def gpt2_small(num_workers: int = 32, num_events: int = 512, seed: int = DEFAULT_SEED,
               per_layer: bool = False) -> Workload:
    """GPT-2-small shapes, 1e-4 * Student-t(3) gradients, 99 % of embedding rows zero."""
    sz = _shapes.sizes(_shapes.gpt2_small_shapes())
    assert sum(sz) == 124_439_808 and len(sz) == 148
    segs = sz if per_layer else [sum(sz)]
    return custom("gpt2-small-" + ("per-layer" if per_layer else "global"), segs, num_workers,
                  num_events, 1000, grad_kind="student_t", grad_scale=1e-4,
                  schedule_kind="cyclic", seed=seed, tensor_sizes=sz,
                  zero_rows=(0, 50257, 768, 0.01))


def sweep(log2n: int, density_ppm: int, seed: int = DEFAULT_SEED) -> Workload:
    """One cell of the kernel sweep: flat vector of 2^log2n values, one selection."""
    return custom(f"sweep-2^{log2n}-{density_ppm}ppm", [1 << log2n], 1, 1, density_ppm,
                  grad_kind="sweep", seed=seed)


SWEEP_LOG2N = (16, 18, 20, 22, 24, 26, 28)
SWEEP_PPM = (100, 1000, 10_000, 100_000)

BY_NAME = {
    "flat1m": flat_1m,
    "resnet18": resnet18,
    "resnet50": resnet50,
    "gpt2": gpt2_small,
    "gpt2-layerwise": lambda **kw: gpt2_small(per_layer=True, **kw),   # one selection per tensor (148 layers)
}


def staleness(schedule: np.ndarray, num_workers: int) -> np.ndarray:
    """For each event, how many other events were served since that worker's
    previous arrival (-1 for a worker's first arrival)."""
    last = -np.ones(num_workers, dtype=np.int64)
    out = np.empty(len(schedule), dtype=np.int64)
    for e, w in enumerate(schedule):
        out[e] = -1 if last[w] < 0 else e - last[w] - 1
        last[w] = e
    return out
