"""Host-side checks that need no GPU: the library loads, exports every symbol the
header declares, and its argument validation and sizing logic behave."""
import os
import re

import pytest

import paper_1910_10929_b200 as dgs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "dgs.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dgs_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert "dgs_init" in names and "dgs_worker_push" in names and "dgs_server_apply" in names
    assert "dgs_worker_pull" in names and "dgs_free" in names
    L = dgs.lib()
    for name in names:
        assert hasattr(L, name), name
    assert sorted(dgs.EXPORTS) == names


def test_error_strings():
    L = dgs.lib()
    assert L.dgs_error_string(0) == b"ok"
    for code in (-1, -2, -3, -4, -5):
        assert L.dgs_error_string(code) not in (b"ok", b"unknown error")
    assert L.dgs_error_string(-99) == b"unknown error"


def cfg(**kw):
    base = dict(n=1000, num_workers=2, lr=0.1, momentum=0.9, seg_offset=[0, 300], seg_len=[300, 700],
                k_push=[3, 7], k_pull=[3, 7])
    base.update(kw)
    return dgs.make_config(**base)


def test_arena_sizing_scales_with_workers_and_flags():
    a2 = dgs.dgs_arena_bytes(cfg())
    a4 = dgs.dgs_arena_bytes(cfg(num_workers=4))
    # two more workers: two more velocity and two more difference vectors, at least
    assert a4 - a2 >= 4 * 1000 * 4
    assert dgs.dgs_arena_bytes(cfg(flags=dgs.DGS_KEEP_LOCAL_MODEL)) - a2 >= 2 * 1000 * 4
    assert dgs.dgs_arena_bytes(cfg(flags=dgs.DGS_HOST_IO)) - a2 >= 1000 * 4
    big = dgs.make_config(25_557_032, 32, 0.1, 0.9, [0], [25_557_032], [25_558], [25_558])
    need = dgs.dgs_arena_bytes(big)
    state = (2 * 32 + 1) * 25_557_032 * 4
    # four spare velocity vectors, ten scratch sets (one per stream that selects) with two candidate buffers
    # of capacity n each, packet slots and the packet log
    assert state < need < 1.45 * state


@pytest.mark.parametrize("bad", [
    dict(momentum=0.0), dict(momentum=1.5), dict(momentum=float("nan")), dict(lr=float("inf")),
    dict(num_workers=0), dict(n=0), dict(n=1 << 32, seg_len=[300, (1 << 32) - 300]),
    dict(seg_offset=[0, 301]), dict(seg_len=[300, 699]), dict(k_push=[0, 7]), dict(k_push=[301, 7]),
    dict(k_pull=[3, 0]), dict(k_pull=[3, 701]), dict(seg_len=[0, 1000], seg_offset=[0, 0]),
])
def test_bad_configs_are_rejected(bad):
    with pytest.raises(dgs.DgsError) as e:
        dgs.dgs_arena_bytes(cfg(**bad))
    assert e.value.code == dgs.DGS_EINVAL


def test_momentum_one_is_legal():
    assert dgs.dgs_arena_bytes(cfg(momentum=1.0)) > 0


def test_null_arguments():
    L = dgs.lib()
    assert L.dgs_arena_bytes(None, None) == dgs.DGS_EINVAL
    assert L.dgs_init(None, None) == dgs.DGS_EINVAL
    assert L.dgs_worker_push(None, 0, None, None) == dgs.DGS_ESTATE
    assert L.dgs_server_apply(None, 0, None) == dgs.DGS_ESTATE
    assert L.dgs_worker_pull(None, 0, None) == dgs.DGS_ESTATE
    assert L.dgs_free(None) == dgs.DGS_ESTATE


def test_init_without_arena_is_rejected_before_any_gpu_work():
    import ctypes as C
    c = cfg()
    h = C.c_void_p(None)
    assert dgs.lib().dgs_init(C.byref(c), C.byref(h)) == dgs.DGS_EINVAL
    assert h.value is None


def test_hardware_queues_reports_what_the_environment_says(monkeypatch):
    needed, configured = dgs.dgs_hardware_queues()
    assert needed == 12                      # eleven streams of the library and the caller's
    monkeypatch.setenv("CUDA_DEVICE_MAX_CONNECTIONS", "5")
    assert dgs.dgs_hardware_queues() == (12, 5)
    monkeypatch.delenv("CUDA_DEVICE_MAX_CONNECTIONS")
    assert dgs.dgs_hardware_queues() == (12, 8)
