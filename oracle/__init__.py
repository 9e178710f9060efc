"""ctypes front end of the CPU checker (``dgs_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
CPU-baseline leg of the benchmark, never by the CUDA package.  The arithmetic
lives in the C++ file; this wrapper only builds it and marshals numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import hashlib
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dgs_oracle.cpp")
_LIB = os.path.join(_HERE, "libdgs_oracle.so")
_lib = None


_FLAGS = ["-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC"]


def _source_hash() -> str:
    h = hashlib.sha256(" ".join(_FLAGS).encode())
    with open(_SRC, "rb") as f:
        h.update(f.read())
    return h.hexdigest()


def build(force: bool = False) -> str:
    """Compile the checker (g++, no FMA contraction, no fast-math).  Rebuilt whenever the source or the
    flags differ from those the library beside it was built from (a hash is stored with it)."""
    stamp = _LIB + ".hash"
    digest = _source_hash()
    fresh = os.path.exists(_LIB) and os.path.exists(stamp) and open(stamp).read().strip() == digest
    if force or not fresh:
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["g++"] + _FLAGS + ["-o", tmp, _SRC])
        os.replace(tmp, _LIB)
        with open(stamp, "w") as f:
            f.write(digest + "\n")
    return _LIB


def _load():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        u64, u32, f32, vp = C.c_uint64, C.c_uint32, C.c_float, C.c_void_p
        L.dgs_oracle_topk.argtypes = [vp, u64, u64, vp]
        L.dgs_oracle_topk.restype = None
        L.dgs_oracle_create.argtypes = [u64, u32, f32, f32, u32, vp, vp, vp, vp, vp, C.c_int, C.c_int, C.c_int]
        L.dgs_oracle_round16.argtypes = [f32, C.c_int]
        L.dgs_oracle_round16.restype = f32
        L.dgs_oracle_create.restype = vp
        L.dgs_oracle_free.argtypes = [vp]
        L.dgs_oracle_free.restype = None
        L.dgs_oracle_push.argtypes = [vp, u32, vp, vp, vp]
        L.dgs_oracle_push.restype = u64
        L.dgs_oracle_apply.argtypes = [vp, u32, vp, vp, u64]
        L.dgs_oracle_apply.restype = None
        L.dgs_oracle_pull.argtypes = [vp, u32, vp, vp]
        L.dgs_oracle_pull.restype = u64
        L.dgs_oracle_pull_all.argtypes = [vp, u32, vp, vp, u64]
        L.dgs_oracle_pull_all.restype = u64
        L.dgs_oracle_state.argtypes = [vp, C.c_int, u32]
        L.dgs_oracle_state.restype = vp
        L.dgs_oracle_timestamp.argtypes = [vp]
        L.dgs_oracle_timestamp.restype = u64
        L.dgs_oracle_prev.argtypes = [vp, u32]
        L.dgs_oracle_prev.restype = C.c_int64
        _lib = L
    return _lib


def _p(a: np.ndarray) -> int:
    return a.ctypes.data


def topk(x: np.ndarray, k: int) -> np.ndarray:
    """Positions (ascending) of the k entries of largest |x|, ties to the lowest index."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(k, dtype=np.uint64)
    _load().dgs_oracle_topk(_p(x), x.shape[0], k, _p(out))
    return out


def round16(x: float, fmt: int) -> np.float32:
    """A packet value in the 16-bit format fmt (1: bfloat16, 2: binary16 saturating at 65504), as float32."""
    return np.float32(_load().dgs_oracle_round16(np.float32(x), int(fmt)))


THETA, U, D, THETA_LOCAL = 0, 1, 2, 3
FP32, BF16, FP16 = 0, 1, 2


class Oracle:
    """N workers + server replayed on the CPU, one call per step of an event."""

    def __init__(self, n: int, num_workers: int, lr: float, momentum: float,
                 seg_offset, seg_len, k_push, k_pull, theta0: np.ndarray,
                 keep_local: bool = False, residual_mode: bool = False, packet_format: int = 0):
        L = _load()
        self.n, self.N = int(n), int(num_workers)
        so = np.ascontiguousarray(seg_offset, dtype=np.uint64)
        sl = np.ascontiguousarray(seg_len, dtype=np.uint64)
        kp = np.ascontiguousarray(k_push, dtype=np.uint32)
        kl = np.ascontiguousarray(k_pull, dtype=np.uint32)
        th = np.ascontiguousarray(theta0, dtype=np.float32)
        assert th.shape == (self.n,)
        self.K_push, self.K_pull = int(kp.sum()), int(kl.sum())
        self._h = L.dgs_oracle_create(self.n, self.N, np.float32(lr), np.float32(momentum),
                                      so.shape[0], _p(so), _p(sl), _p(kp), _p(kl), _p(th),
                                      int(keep_local), int(residual_mode), int(packet_format))
        self._L = L

    @classmethod
    def from_workload(cls, wl, keep_local: bool = False, residual_mode: bool = False,
                      theta0: Optional[np.ndarray] = None, packet_format: int = 0) -> "Oracle":
        return cls(wl.n, wl.num_workers, wl.lr, wl.momentum, wl.seg_offset, wl.seg_len,
                   wl.k_push, wl.k_pull, wl.theta0() if theta0 is None else theta0,
                   keep_local, residual_mode, packet_format)

    def push(self, w: int, grad: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
        g = np.ascontiguousarray(grad, dtype=np.float32)
        assert g.shape == (self.n,)
        idx = np.empty(self.K_push, dtype=np.uint32)
        val = np.empty(self.K_push, dtype=np.float32)
        c = self._L.dgs_oracle_push(self._h, w, _p(g), _p(idx), _p(val))
        assert c == self.K_push
        return idx, val

    def apply(self, w: int, idx: np.ndarray, val: np.ndarray) -> None:
        idx = np.ascontiguousarray(idx, dtype=np.uint32)
        val = np.ascontiguousarray(val, dtype=np.float32)
        self._L.dgs_oracle_apply(self._h, w, _p(idx), _p(val), idx.shape[0])

    def pull(self, w: int) -> Tuple[np.ndarray, np.ndarray]:
        idx = np.empty(self.K_pull, dtype=np.uint32)
        val = np.empty(self.K_pull, dtype=np.float32)
        c = self._L.dgs_oracle_pull(self._h, w, _p(idx), _p(val))
        assert c == self.K_pull
        return idx, val

    def pull_all(self, w: int, cap: Optional[int] = None) -> Tuple[np.ndarray, np.ndarray, int]:
        """Pull without secondary compression: every nonzero entry of D_w, ascending, then cleared.
        Returns (idx, val, held) where held is how many nonzeros D_w had (> cap means overflow)."""
        cap = self.n if cap is None else int(cap)
        idx = np.empty(cap, dtype=np.uint32)
        val = np.empty(cap, dtype=np.float32)
        held = int(self._L.dgs_oracle_pull_all(self._h, w, _p(idx), _p(val), cap))
        m = min(held, cap)
        return idx[:m].copy(), val[:m].copy(), held

    def event(self, w: int, grad: np.ndarray):
        """push -> apply -> pull for worker w; returns both packets."""
        pi, pv = self.push(w, grad)
        self.apply(w, pi, pv)
        gi, gv = self.pull(w)
        return (pi, pv), (gi, gv)

    def state(self, which: int, w: int = 0) -> np.ndarray:
        """A read-only numpy view of theta / u[w] / D[w] / theta_local[w]."""
        ptr = self._L.dgs_oracle_state(self._h, which, w)
        if not ptr:
            raise ValueError("state not kept")
        a = np.ctypeslib.as_array(C.cast(ptr, C.POINTER(C.c_float)), shape=(self.n,))
        a.flags.writeable = False
        return a

    @property
    def timestamp(self) -> int:
        return int(self._L.dgs_oracle_timestamp(self._h))

    def prev(self, w: int) -> int:
        return int(self._L.dgs_oracle_prev(self._h, w))

    def close(self) -> None:
        if self._h:
            self._L.dgs_oracle_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
