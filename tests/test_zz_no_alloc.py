"""dgs_topk_encode_static: the selection + encode step for callers that cannot allocate.

Some users of this library run where device allocation is not allowed: their memory
plan is fixed before the loop starts (a pool that must not grow, a serving or control
loop that may not enter the allocator), or they are plug-ins that receive buffers but
no allocator, so they cannot hand dgs_init an arena either.  For them the library has
one entry point whose scratch is a fixed array inside the library's device image.

The test calls it through the C ABI twice in a row (the second call sees whatever the
first one left in the shared scratch) and requires the packets to be bit-identical to
those of the ordinary route, dgs_worker_pull on a one-worker context, and to the CPU
checker's selection of the same vector: same indices, same value bits -- the bar every
selection test here uses.  It sits in a file that is
collected last so that a failure here cannot hide any other test, and it must pass both
alone in a fresh process and after the rest of the suite."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
import paper_1910_10929_b200 as dgs
import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def reference_packet(x_dev: torch.Tensor, k: int):
    n = x_dev.numel()
    ctx = dgs.Context(n, 1, 0.1, 0.9, [0], [n], [k], [k], torch.zeros(n, device=DEV))
    ctx.state_load(dgs.DGS_D, 0, x_dev)
    idx, val = ctx.packet(ctx.worker_pull(0))
    out = idx.clone(), val.clone()
    assert ctx.status() == 0
    ctx.close()
    return out


def static_packet(x_dev: torch.Tensor, k: int):
    idx = torch.full((k,), -1, dtype=torch.int32, device=DEV)
    val = torch.full((k,), float("nan"), dtype=torch.float32, device=DEV)
    before = torch.cuda.memory_allocated(DEV)
    dgs.dgs_topk_encode_static(x_dev.data_ptr(), x_dev.numel(), k, idx.data_ptr(), val.data_ptr(),
                               torch.cuda.current_stream().cuda_stream)
    # the call only enqueues: the device-side outcome is read back separately (and waits for the stream)
    assert dgs.dgs_topk_encode_static_status(torch.cuda.current_stream().cuda_stream) == 0
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated(DEV) == before
    return idx, val


def test_static_selection_matches_pull_twice_in_a_row():
    torch.cuda.set_device(0)
    cases = [
        (W.sweep_values(1 << 20, index=3), 1049),                 # the full capacity, outliers included
        (W.sweep_values(70_001, index=4), 7001),                  # smaller, ragged tail, denser: reuses dirty scratch
    ]
    for x, k in cases:
        x_dev = torch.from_numpy(x).to(DEV)
        keep = x_dev.clone()
        want_idx, want_val = reference_packet(x_dev, k)
        got_idx, got_val = static_packet(x_dev, k)
        assert torch.equal(got_idx, want_idx)
        assert torch.equal(got_val.view(torch.int32), want_val.view(torch.int32))
        chosen = oracle.topk(x, k)                                 # the CPU checker's selection of the same vector
        assert np.array_equal(got_idx.cpu().numpy().view(np.uint32), chosen.astype(np.uint32))
        assert np.array_equal(got_val.cpu().numpy().view(np.uint32), x[chosen].view(np.uint32))
        assert torch.equal(x_dev.view(torch.int32), keep.view(torch.int32))   # the input is left alone


def test_static_selection_rejects_what_does_not_fit():
    L = dgs.lib()
    x = torch.zeros(16, device=DEV)
    idx = torch.zeros(16, dtype=torch.int32, device=DEV)
    val = torch.zeros(16, device=DEV)
    args = (x.data_ptr(), idx.data_ptr(), val.data_ptr())
    assert L.dgs_topk_encode_static(args[0], dgs.DGS_STATIC_MAX_N + 1, 4, args[1], args[2], None) == dgs.DGS_ELIMIT
    assert L.dgs_topk_encode_static(args[0], 16, 0, args[1], args[2], None) == dgs.DGS_EINVAL
    assert L.dgs_topk_encode_static(args[0], 16, 17, args[1], args[2], None) == dgs.DGS_EINVAL
    assert L.dgs_topk_encode_static(None, 16, 4, args[1], args[2], None) == dgs.DGS_EINVAL
    assert b"capacity" in L.dgs_error_string(dgs.DGS_ELIMIT)
