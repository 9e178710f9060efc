"""The seeded input generators: sizes, selection counts, schedules, determinism."""
import numpy as np

import workloads as W
from workloads import shapes


def test_architecture_totals():
    assert sum(shapes.sizes(shapes.resnet18_shapes())) == 11_689_512
    assert len(shapes.resnet18_shapes()) == 62
    assert sum(shapes.sizes(shapes.resnet50_shapes())) == 25_557_032
    assert len(shapes.resnet50_shapes()) == 161
    assert sum(shapes.sizes(shapes.gpt2_small_shapes())) == 124_439_808
    assert len(shapes.gpt2_small_shapes()) == 148


def test_k_rule():
    assert W.k_of(1 << 20, 1000) == 1049
    assert W.k_of(64, 10_000) == 1
    assert W.k_of(100, 10_000) == 1 and W.k_of(101, 10_000) == 2
    assert W.flat_1m().K_push == 1049
    assert W.resnet18().K_push == 116_928
    assert W.resnet50().K_push == 25_558
    assert W.gpt2_small().K_push == 124_440


def test_segments_tile_the_vector():
    for wl in (W.flat_1m(), W.resnet18(), W.resnet50()):
        end = wl.seg_offset + wl.seg_len
        assert wl.seg_offset[0] == 0 and end[-1] == wl.n
        assert np.array_equal(end[:-1], wl.seg_offset[1:])
        assert np.all(wl.k_push <= wl.seg_len) and np.all(wl.k_push >= 1)


def test_cyclic_schedule_caps_staleness():
    wl = W.resnet18()
    s = wl.schedule()
    st = W.staleness(s, wl.num_workers)
    assert st.max() == wl.num_workers - 1
    assert sorted(s[:wl.num_workers].tolist()) == list(range(wl.num_workers))
    assert np.array_equal(s, W.resnet18().schedule())
    assert not np.array_equal(s, W.resnet18(seed=7).schedule())


def test_uniform_schedule_has_repeats():
    s = W.flat_1m().schedule()
    assert len(s) == 16 and s.min() >= 0 and s.max() < 4


def test_gradients_are_keyed_by_event():
    wl = W.custom("mini", [1000, 24], 2, 4, 10_000, grad_kind="laplace")
    a, b = wl.gradient(3), wl.gradient(3)
    assert a.dtype == np.float32 and np.array_equal(a, b)
    assert not np.array_equal(a, wl.gradient(2))
    out = np.empty(wl.n, np.float32)
    assert wl.gradient(3, out=out) is out and np.array_equal(out, a)


def test_student_t_rows_mostly_zero():
    wl = W.custom("mini-t", [400 * 8, 300], 2, 2, 10_000, grad_kind="student_t", grad_scale=1e-4,
                  tensor_sizes=[400 * 8, 300], zero_rows=(0, 400, 8, 0.05))
    g = wl.gradient(0)
    rows = g[:3200].reshape(400, 8)
    live = np.any(rows != 0, axis=1)
    assert 0 < live.sum() < 60 and np.all(rows[live] != 0)
    assert np.all(g[3200:] != 0)


def test_sweep_values_have_outliers():
    x = W.sweep_values(1 << 16)
    assert 0.005 < np.mean(np.abs(x) > 10) < 0.02
