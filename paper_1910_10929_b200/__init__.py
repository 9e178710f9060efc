"""DGS push / apply / pull loop on one B200: Python binding of the C ABI in include/dgs.h.

The functions ``dgs_*`` below carry the names and meaning of the C entry points and
only marshal arguments; every step of the path runs in the CUDA library
``libdgs.so``.  There is no CPU path: if the library is missing or cannot be
loaded, importing the binding raises.  PyTorch is used for device memory (the
arena handed to ``dgs_init``) and for the stream.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence, Tuple

# The library spreads its kernels over eleven CUDA streams.  The driver maps streams onto a fixed
# number of hardware queues (8 unless told otherwise) and streams that share a queue run one after
# the other; the variable is read when the process creates its CUDA context, so it has to be in
# place before that.  A value the user has set is left alone.
os.environ.setdefault("CUDA_DEVICE_MAX_CONNECTIONS", "32")

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdgs.so")

DGS_OK, DGS_EINVAL, DGS_ENOMEM, DGS_ECUDA, DGS_ETIMEOUT, DGS_ESTATE = 0, -1, -2, -3, -4, -5
DGS_KEEP_LOCAL_MODEL, DGS_RESIDUAL_MODE, DGS_HOST_IO, DGS_NO_SPECULATION, DGS_SINGLE_STREAM = 1, 2, 4, 8, 16
DGS_TEST_STALLED_BARRIER = 32
DGS_PACKET_BF16, DGS_PACKET_FP16 = 64, 128
DGS_THETA, DGS_U, DGS_D, DGS_THETA_LOCAL = 0, 1, 2, 3

EXPORTS = (
    "dgs_arena_bytes", "dgs_init", "dgs_worker_push", "dgs_server_apply", "dgs_worker_pull", "dgs_worker_pull_all",
    "dgs_event", "dgs_flush", "dgs_event_host", "dgs_state_ptr", "dgs_state_load", "dgs_status", "dgs_stats", "dgs_pull_read_stats",
    "dgs_prev", "dgs_launch_count", "dgs_last_cuda_error", "dgs_free", "dgs_error_string",
    "dgs_timing_enable", "dgs_timing_read", "dgs_timing_trace", "dgs_topk_encode_static",
    "dgs_topk_encode_static_status", "dgs_hardware_queues",
)
DGS_ELIMIT = -6
DGS_STATIC_MAX_N = 1 << 20
DGS_NUM_KERNELS = 8
KERNEL_NAMES = ("stream_push", "finalize_push", "two_pass_push", "scatter", "stream_pull", "finalize_pull",
                "two_pass_pull", "catch_up")


class dgs_segment(C.Structure):
    _fields_ = [("offset", C.c_uint64), ("len", C.c_uint64), ("k_push", C.c_uint32), ("k_pull", C.c_uint32)]


class dgs_packet(C.Structure):
    _fields_ = [("idx", C.c_void_p), ("val", C.c_void_p), ("count", C.c_uint32)]


class dgs_var_packet(C.Structure):
    _fields_ = [("idx", C.c_void_p), ("val", C.c_void_p), ("count", C.c_void_p), ("capacity", C.c_uint32)]


class dgs_config(C.Structure):
    _fields_ = [("n", C.c_uint64), ("num_workers", C.c_uint32), ("lr", C.c_float), ("momentum", C.c_float),
                ("num_segments", C.c_uint32), ("segments", C.POINTER(dgs_segment)), ("theta0", C.c_void_p),
                ("arena", C.c_void_p), ("arena_bytes", C.c_uint64), ("stream", C.c_void_p), ("flags", C.c_uint32),
                ("pull_all_capacity", C.c_uint32)]


class DgsError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {lib().dgs_error_string(code).decode()} ({code})")


_lib = None


def lib() -> C.CDLL:
    """The loaded CUDA library.  Raises if it has not been built (python -m paper_1910_10929_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_1910_10929_b200.build` "
                              "(nvcc, sm_100a); there is no fallback path")
        L = C.CDLL(LIB_PATH)
        vp, u32, i32 = C.c_void_p, C.c_uint32, C.c_int
        L.dgs_arena_bytes.argtypes = [C.POINTER(dgs_config), C.POINTER(C.c_uint64)]
        L.dgs_init.argtypes = [C.POINTER(dgs_config), C.POINTER(vp)]
        L.dgs_worker_push.argtypes = [vp, u32, vp, C.POINTER(dgs_packet)]
        L.dgs_server_apply.argtypes = [vp, u32, C.POINTER(dgs_packet)]
        L.dgs_worker_pull.argtypes = [vp, u32, C.POINTER(dgs_packet)]
        L.dgs_worker_pull_all.argtypes = [vp, u32, C.POINTER(dgs_var_packet)]
        L.dgs_event.argtypes = [vp, u32, vp, C.POINTER(dgs_packet), C.POINTER(dgs_packet)]
        L.dgs_flush.argtypes = [vp]
        L.dgs_event_host.argtypes = [vp, u32, vp, vp, vp]
        L.dgs_state_ptr.argtypes = [vp, i32, u32, C.POINTER(vp)]
        L.dgs_state_load.argtypes = [vp, i32, u32, vp]
        L.dgs_status.argtypes = [vp, C.POINTER(i32)]
        L.dgs_stats.argtypes = [vp, C.POINTER(C.c_uint64)]
        L.dgs_pull_read_stats.argtypes = [vp, C.POINTER(C.c_uint64)]
        L.dgs_prev.argtypes = [vp, u32, C.POINTER(C.c_int64)]
        L.dgs_launch_count.argtypes = [vp, C.POINTER(C.c_uint64)]
        L.dgs_last_cuda_error.argtypes = [vp]
        L.dgs_topk_encode_static.argtypes = [vp, u32, u32, vp, vp, vp]
        L.dgs_topk_encode_static_status.argtypes = [vp, C.POINTER(i32)]
        L.dgs_hardware_queues.argtypes = [C.POINTER(i32), C.POINTER(i32)]
        L.dgs_timing_enable.argtypes = [vp, i32]
        L.dgs_timing_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_uint64)]
        L.dgs_timing_trace.argtypes = [vp, u32, C.POINTER(C.c_float), C.POINTER(C.c_float), C.POINTER(C.c_int32),
                                       C.POINTER(C.c_int32), C.POINTER(u32)]
        L.dgs_free.argtypes = [vp]
        L.dgs_error_string.argtypes = [i32]
        L.dgs_error_string.restype = C.c_char_p
        for name in EXPORTS:
            if name != "dgs_error_string":
                getattr(L, name).restype = i32
        _lib = L
    return _lib


def _check(rc: int, where: str) -> None:
    if rc != DGS_OK:
        raise DgsError(rc, where)


def make_config(n: int, num_workers: int, lr: float, momentum: float, seg_offset: Sequence[int],
                seg_len: Sequence[int], k_push: Sequence[int], k_pull: Sequence[int], *, theta0: int = 0,
                arena: int = 0, arena_bytes: int = 0, stream: int = 0, flags: int = 0,
                pull_all_capacity: int = 0) -> dgs_config:
    """Fills a dgs_config; pointers are plain integers (device addresses)."""
    S = len(seg_len)
    segs = (dgs_segment * S)()
    for s in range(S):
        segs[s] = dgs_segment(int(seg_offset[s]), int(seg_len[s]), int(k_push[s]), int(k_pull[s]))
    cfg = dgs_config(int(n), int(num_workers), float(lr), float(momentum), S, segs, theta0 or None,
                     arena or None, int(arena_bytes), stream or None, int(flags), int(pull_all_capacity))
    cfg._segs_keepalive = segs
    return cfg


def dgs_arena_bytes(cfg: dgs_config) -> int:
    out = C.c_uint64(0)
    _check(lib().dgs_arena_bytes(C.byref(cfg), C.byref(out)), "dgs_arena_bytes")
    return int(out.value)


def dgs_init(cfg: dgs_config) -> int:
    h = C.c_void_p(None)
    _check(lib().dgs_init(C.byref(cfg), C.byref(h)), "dgs_init")
    return int(h.value)


def dgs_worker_push(ctx: int, worker: int, grad_ptr: int) -> dgs_packet:
    p = dgs_packet()
    _check(lib().dgs_worker_push(ctx, worker, grad_ptr, C.byref(p)), "dgs_worker_push")
    return p


def dgs_server_apply(ctx: int, worker: int, pkt: dgs_packet) -> None:
    _check(lib().dgs_server_apply(ctx, worker, C.byref(pkt)), "dgs_server_apply")


def dgs_worker_pull(ctx: int, worker: int) -> dgs_packet:
    p = dgs_packet()
    _check(lib().dgs_worker_pull(ctx, worker, C.byref(p)), "dgs_worker_pull")
    return p


def dgs_worker_pull_all(ctx: int, worker: int) -> dgs_var_packet:
    p = dgs_var_packet()
    _check(lib().dgs_worker_pull_all(ctx, worker, C.byref(p)), "dgs_worker_pull_all")
    return p


def dgs_event(ctx: int, worker: int, grad_ptr: int) -> Tuple[dgs_packet, dgs_packet]:
    p, g = dgs_packet(), dgs_packet()
    _check(lib().dgs_event(ctx, worker, grad_ptr, C.byref(p), C.byref(g)), "dgs_event")
    return p, g


def dgs_flush(ctx: int) -> None:
    _check(lib().dgs_flush(ctx), "dgs_flush")


def dgs_event_host(ctx: int, worker: int, grad_host_ptr: int, out_idx_ptr: int = 0, out_val_ptr: int = 0) -> None:
    _check(lib().dgs_event_host(ctx, worker, grad_host_ptr, out_idx_ptr or None, out_val_ptr or None),
           "dgs_event_host")


def dgs_state_ptr(ctx: int, which: int, worker: int = 0) -> int:
    out = C.c_void_p(None)
    _check(lib().dgs_state_ptr(ctx, which, worker, C.byref(out)), "dgs_state_ptr")
    return int(out.value)


def dgs_state_load(ctx: int, which: int, worker: int, src_ptr: int) -> None:
    _check(lib().dgs_state_load(ctx, which, worker, src_ptr), "dgs_state_load")


def dgs_status(ctx: int) -> int:
    out = C.c_int(0)
    _check(lib().dgs_status(ctx, C.byref(out)), "dgs_status")
    return int(out.value)


def dgs_stats(ctx: int) -> Tuple[int, int, int, int]:
    out = (C.c_uint64 * 4)()
    _check(lib().dgs_stats(ctx, out), "dgs_stats")
    return tuple(int(v) for v in out)


def dgs_pull_read_stats(ctx: int) -> Tuple[int, int]:
    """(chunks of D covered by the pulls' stream passes, chunks actually read)."""
    out = (C.c_uint64 * 2)()
    _check(lib().dgs_pull_read_stats(ctx, out), "dgs_pull_read_stats")
    return int(out[0]), int(out[1])


def dgs_prev(ctx: int, worker: int) -> int:
    out = C.c_int64(0)
    _check(lib().dgs_prev(ctx, worker, C.byref(out)), "dgs_prev")
    return int(out.value)


def dgs_launch_count(ctx: int) -> int:
    out = C.c_uint64(0)
    _check(lib().dgs_launch_count(ctx, C.byref(out)), "dgs_launch_count")
    return int(out.value)


def dgs_timing_enable(ctx: int, on: bool) -> None:
    _check(lib().dgs_timing_enable(ctx, int(bool(on))), "dgs_timing_enable")


def dgs_timing_read(ctx: int):
    """{kernel name: (milliseconds, launches)} since the last read."""
    ms = (C.c_double * DGS_NUM_KERNELS)()
    cnt = (C.c_uint64 * DGS_NUM_KERNELS)()
    _check(lib().dgs_timing_read(ctx, ms, cnt), "dgs_timing_read")
    return {KERNEL_NAMES[i]: (float(ms[i]), int(cnt[i])) for i in range(DGS_NUM_KERNELS)}


def dgs_timing_trace(ctx: int, cap: int = 65536):
    """[(start_ms, stop_ms, kernel name, stream index)] of the launches recorded since the last read."""
    a, b = (C.c_float * cap)(), (C.c_float * cap)()
    k, s = (C.c_int32 * cap)(), (C.c_int32 * cap)()
    cnt = C.c_uint32(0)
    _check(lib().dgs_timing_trace(ctx, cap, a, b, k, s, C.byref(cnt)), "dgs_timing_trace")
    return [(float(a[i]), float(b[i]), KERNEL_NAMES[k[i]], int(s[i])) for i in range(cnt.value)]


def dgs_topk_encode_static(x_ptr: int, n: int, k: int, out_idx_ptr: int, out_val_ptr: int, stream: int = 0) -> None:
    """Top-k + encode of a flat device vector with no allocation anywhere (scratch is a
    fixed array inside the library, n <= DGS_STATIC_MAX_N).  Enqueues on `stream`."""
    _check(lib().dgs_topk_encode_static(x_ptr, n, k, out_idx_ptr, out_val_ptr, stream or None),
           "dgs_topk_encode_static")


def dgs_topk_encode_static_status(stream: int = 0) -> int:
    """Waits for `stream`; 0 if the packets of the static selections enqueued so far are complete."""
    out = C.c_int(0)
    _check(lib().dgs_topk_encode_static_status(stream or None, C.byref(out)), "dgs_topk_encode_static_status")
    return int(out.value)


def dgs_hardware_queues() -> Tuple[int, int]:
    """(hardware queues the library's streams want, queues the process asked the driver for)."""
    a, b = C.c_int(0), C.c_int(0)
    _check(lib().dgs_hardware_queues(C.byref(a), C.byref(b)), "dgs_hardware_queues")
    return int(a.value), int(b.value)


def dgs_free(ctx: int) -> None:
    _check(lib().dgs_free(ctx), "dgs_free")


from .context import Context  # noqa: E402  (torch-backed convenience holder of arena + handle)

__all__ = [n for n in dir() if n.startswith(("dgs_", "DGS_"))] + ["Context", "DgsError", "lib", "make_config"]
