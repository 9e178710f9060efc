"""A context whose arena is a torch CUDA tensor.  Marshalling only."""
from __future__ import annotations

from typing import Optional, Tuple

import torch

import paper_1910_10929_b200 as dgs


class Context:
    """Owns the arena tensor and the C handle; methods mirror the C entry points."""

    def __init__(self, n: int, num_workers: int, lr: float, momentum: float, seg_offset, seg_len, k_push, k_pull,
                 theta0: torch.Tensor, flags: int = 0, device: Optional[torch.device] = None,
                 stream: Optional[torch.cuda.Stream] = None, pull_all_capacity: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required: this library has no CPU path")
        self.device = torch.device(device if device is not None else theta0.device)
        if self.device.type != "cuda":
            raise RuntimeError("theta0 must live on a CUDA device")
        self.n, self.num_workers = int(n), int(num_workers)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        theta0 = theta0.to(device=self.device, dtype=torch.float32).contiguous()
        assert theta0.numel() == self.n
        cfg = dgs.make_config(n, num_workers, lr, momentum, seg_offset, seg_len, k_push, k_pull, flags=flags,
                              pull_all_capacity=pull_all_capacity)
        self.arena_bytes = dgs.dgs_arena_bytes(cfg)
        with torch.cuda.device(self.device):
            self.arena = torch.empty(self.arena_bytes, dtype=torch.uint8, device=self.device)
            cfg.theta0 = theta0.data_ptr()
            cfg.arena = self.arena.data_ptr()
            cfg.arena_bytes = self.arena_bytes
            cfg.stream = self.stream.cuda_stream
            with torch.cuda.stream(self.stream):
                self.handle = dgs.dgs_init(cfg)
        self.K_push = int(sum(int(k) for k in k_push))
        self.K_pull = int(sum(int(k) for k in k_pull))
        self.flags = flags

    @classmethod
    def from_workload(cls, wl, theta0: Optional[torch.Tensor] = None, flags: int = 0,
                      device: str = "cuda:0", pull_all_capacity: int = 0) -> "Context":
        if theta0 is None:
            theta0 = torch.from_numpy(wl.theta0()).to(device)
        return cls(wl.n, wl.num_workers, wl.lr, wl.momentum, wl.seg_offset, wl.seg_len, wl.k_push, wl.k_pull,
                   theta0, flags=flags, device=theta0.device, pull_all_capacity=pull_all_capacity)

    # ---- the three steps of an event ---------------------------------------------
    def worker_push(self, worker: int, grad: torch.Tensor) -> "dgs.dgs_packet":
        assert grad.is_cuda and grad.dtype == torch.float32 and grad.is_contiguous() and grad.numel() == self.n
        return dgs.dgs_worker_push(self.handle, worker, grad.data_ptr())

    def server_apply(self, worker: int, pkt: "dgs.dgs_packet") -> None:
        dgs.dgs_server_apply(self.handle, worker, pkt)

    def worker_pull(self, worker: int) -> "dgs.dgs_packet":
        return dgs.dgs_worker_pull(self.handle, worker)

    def worker_pull_all(self, worker: int) -> "dgs.dgs_var_packet":
        return dgs.dgs_worker_pull_all(self.handle, worker)

    def var_packet(self, pkt: "dgs.dgs_var_packet") -> Tuple[torch.Tensor, torch.Tensor]:
        """(idx, val) of a packet whose count lives on the device: flushes, reads the count (this waits
        for the stream), returns views of the valid entries."""
        self.flush()
        count = int(self._view(pkt.count, 1, torch.int32).item())
        return self._view(pkt.idx, count, torch.int32), self._view(pkt.val, count, torch.float32)

    def event(self, worker: int, grad: torch.Tensor) -> Tuple["dgs.dgs_packet", "dgs.dgs_packet"]:
        assert grad.is_cuda and grad.dtype == torch.float32 and grad.is_contiguous() and grad.numel() == self.n
        return dgs.dgs_event(self.handle, worker, grad.data_ptr())

    def event_host(self, worker: int, grad_host: torch.Tensor, out_idx: Optional[torch.Tensor] = None,
                   out_val: Optional[torch.Tensor] = None) -> None:
        assert not grad_host.is_cuda and grad_host.dtype == torch.float32 and grad_host.numel() == self.n
        dgs.dgs_event_host(self.handle, worker, grad_host.data_ptr(),
                           out_idx.data_ptr() if out_idx is not None else 0,
                           out_val.data_ptr() if out_val is not None else 0)

    # ---- reading results ---------------------------------------------------------
    def _view(self, ptr: int, count: int, dtype: torch.dtype) -> torch.Tensor:
        """A tensor over `count` 4-byte elements at a device address inside the arena."""
        off = ptr - self.arena.data_ptr()
        assert 0 <= off and off + 4 * count <= self.arena_bytes
        return self.arena[off:off + 4 * count].view(dtype)

    def flush(self) -> None:
        """Orders the context's stream after all work enqueued so far."""
        dgs.dgs_flush(self.handle)

    def packet(self, pkt: "dgs.dgs_packet") -> Tuple[torch.Tensor, torch.Tensor]:
        """(idx int32 view holding uint32 bits, val float32) views of a packet slot, readable on
        the context's stream (flushes first)."""
        self.flush()
        return self._view(pkt.idx, pkt.count, torch.int32), self._view(pkt.val, pkt.count, torch.float32)

    def state(self, which: int, worker: int = 0) -> torch.Tensor:
        return self._view(dgs.dgs_state_ptr(self.handle, which, worker), self.n, torch.float32)

    def state_load(self, which: int, worker: int, src: torch.Tensor) -> None:
        assert src.is_cuda and src.dtype == torch.float32 and src.is_contiguous() and src.numel() == self.n
        dgs.dgs_state_load(self.handle, which, worker, src.data_ptr())

    def status(self) -> int:
        return dgs.dgs_status(self.handle)

    def stats(self):
        return dgs.dgs_stats(self.handle)

    def pull_read_stats(self):
        return dgs.dgs_pull_read_stats(self.handle)

    def launch_count(self) -> int:
        return dgs.dgs_launch_count(self.handle)

    def close(self) -> None:
        if getattr(self, "handle", None):
            dgs.dgs_free(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
