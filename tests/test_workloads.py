"""Shapes and structure of the seeded synthetic streams (no GPU)."""
import numpy as np

from paper_2609_34653_b200 import workloads as wl


def _check_table(units, total=None):
    assert units.dtype == np.int32 and units.shape[1] == 6
    assert np.all(units[:, 1] > 0)
    assert np.array_equal(units[:, 0], np.concatenate([[0], np.cumsum(units[:, 1])[:-1]]))
    assert np.all(np.diff(units[:, 3]) >= 0)
    if total is not None:
        assert int(units[:, 1].sum()) == total


def test_tiny_shapes():
    w = wl.tiny()
    _check_table(w.units, 2048)
    assert len(w.units) == 12 and w.t == 256 and w.units[0, 4] == 0
    assert w.q.shape == (256, 4, 64) and w.k_hist.shape == (2048, 1, 64) and w.q.dtype == np.float32
    assert (w.budget, w.page_size, w.n_recent_events) == (1024, 16, 1)
    w2 = wl.tiny()
    assert np.array_equal(w.k_hist, w2.k_hist) and w.biased_unit == w2.biased_unit   # seeded


def test_layer_and_long_stream_structure():
    w = wl.layer_8b(draw_values=False)
    _check_table(w.units, 16384)
    assert w.units[0, 1] == 16 and w.units[0, 2] == wl.MOD_TEXT and w.units[0, 4] == 0
    assert w.t == 690 and (w.budget, w.page_size) == (4096, 64)
    assert {640, 50, 32, 16} >= set(np.unique(w.units[2:, 1]).tolist()) >= {640, 50, 32}
    w = wl.long_stream(draw_values=False)
    _check_table(w.units, 80000)
    assert w.t == 2354 and (w.budget, w.page_size) == (8192, 64)
    assert (w.units[:, 1] == 2304).sum() >= 33
    w = wl.sweep_cell(1024, 0.125, 64, draw_values=False)
    _check_table(w.units, 131072)
    assert w.t == 1024 and w.budget == 16384


def test_bf16_rounding_helpers():
    x = np.array([1.0, 1.00390625, 1.01171875, -3.3, 1e-3, 65504.0], dtype=np.float32)
    r = wl.round_to_bf16(x)
    assert np.all((r.view(np.uint32) & 0xFFFF) == 0)
    assert r[1] == 1.0 and r[2] == np.float32(1.015625)          # ties to even, both directions
    assert np.array_equal(wl.bf16_bits_to_f32(wl.bf16_bits(r)), r)
    big = np.random.default_rng(0).standard_normal(1 << 17).astype(np.float32)
    u = big.view(np.uint32)
    ref = ((u + (((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF))) & np.uint32(0xFFFF0000)).view(np.float32)
    assert np.array_equal(wl.round_to_bf16(big), ref)      # the large-array path rounds identically


def test_loop_schedule_and_small_mixed():
    sched = wl.loop_schedule(20)
    assert len(sched) == 20
    for c, cu in enumerate(sched):
        assert cu[0, 1] in (640, 1280, 2304) and 20 <= cu[1, 1] <= 50 and np.all(cu[:, 3] == c + 1)
    w = wl.small_mixed(5)
    _check_table(w.units)
    assert w.q.shape == (w.t, w.h_q, w.d) and w.k_hist.shape[0] == w.n_hist
