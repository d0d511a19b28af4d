"""Parity at the full sizes of the benchmark configurations, through the same entry point and launch
configuration that bench.py times.  Integer results (selection given the scores, compaction, append)
are compared whole; attention on sampled outputs the oracle evaluates one by one; unit scores on one
KV group evaluated whole by the oracle, tied to the full launch by an identity (the full-geometry
mass is the mean of the per-group masses)."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import omni_oracle as oc
from paper_2609_34653_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def H():
    from tests import gpu_helpers
    return gpu_helpers


@pytest.fixture(scope="module")
def ob():
    from paper_2609_34653_b200 import binding
    return binding


@pytest.fixture(scope="module")
def P():
    from tests import test_gpu_parity
    return test_gpu_parity


def _kv_group(w, g):
    """The workload restricted to KV group g (its G query heads and one KV head)."""
    G = w.h_q // w.h_kv
    return dataclasses.replace(
        w, h_q=G, h_kv=1, q=np.ascontiguousarray(w.q[:, g * G:(g + 1) * G]),
        k_hist=np.ascontiguousarray(w.k_hist[:, g:g + 1]), v_hist=np.ascontiguousarray(w.v_hist[:, g:g + 1]),
        k_chunk=np.ascontiguousarray(w.k_chunk[:, g:g + 1]), v_chunk=np.ascontiguousarray(w.v_chunk[:, g:g + 1]))


def _sample_rows(w, rng, n_random=48):
    """(query row, head) pairs: tile edges, the first and last rows, and random ones."""
    T = w.t
    fixed_i = sorted({0, 1, 127, 128, 129, T // 2, T - 129, T - 128, T - 2, T - 1} & set(range(T)))
    rows = [(i, h) for i in fixed_i for h in (0, w.h_q // 2 + 1, w.h_q - 1)]
    rows += [(int(rng.integers(T)), int(rng.integers(w.h_q))) for _ in range(n_random)]
    return rows


def _check_integer_path_and_sampled_attention(H, ob, P, w, res, rng):
    n_new = res["n_hist"] - w.t
    nu = res["n_units"] - len(w.chunk_units)
    again = oc.select_units(w.units, res["scores"], w.budget, w.n_recent_events, w.modality_cap)
    assert np.array_equal(again["units_out"], res["units"][:nu])
    # no unit is split and the budget holds for everything but the protected groups
    assert res["info"]["n_kept"] == int(again["keep_mask"].sum()) == n_new
    raw_k = H.bytes_of(ob.to_device(w.k_hist, w.dtype)).reshape(w.n_hist, -1)
    raw_v = H.bytes_of(ob.to_device(w.v_hist, w.dtype)).reshape(w.n_hist, -1)
    cp = oc.compact_pack(raw_k, raw_v, again["keep_mask"], w.page_size, again["units_out"])
    assert res["info"]["span_pages"] == cp["span_pages"] and res["info"]["rows_moved"] == cp["rows_moved"]
    assert res["info"]["part_begin"] == cp["part_begin"].tolist()
    assert res["info"]["span_pages"] * w.page_size - n_new < w.page_size
    assert np.array_equal(H.bytes_of(res["k"][:n_new]).reshape(n_new, -1), cp["k"])
    assert np.array_equal(H.bytes_of(res["v"][:n_new]).reshape(n_new, -1), cp["v"])
    kc_bits = H.bytes_of(res["k"][n_new:n_new + w.t]).reshape(w.t, -1).view(np.uint16).reshape(w.t, w.h_kv, w.d)
    assert np.array_equal(kc_bits, wl.bf16_bits(w.k_chunk))
    assert np.array_equal(res["units"][:res["n_units"]], oc.append_chunk(again["units_out"], n_new, w.chunk_units))
    keep = again["keep_mask"].astype(bool)
    rows = _sample_rows(w, rng)
    o_ref, _ = oc.chunk_attention(w.q, w.k_hist[keep], w.v_hist[keep], w.k_chunk, w.v_chunk, rows=rows)
    o_gpu = np.stack([res["o"][i, h] for i, h in rows])
    assert np.isfinite(res["o"]).all()
    err = np.abs(o_gpu - o_ref)
    assert err.max() <= P.ATT_MAX_ABS, err.max()
    assert err.mean() <= P.ATT_MEAN_ABS, err.mean()
    return again


def _check_scores_by_group(H, ob, P, w, full_scores, oracle_groups):
    """mass(full geometry) == mean over KV groups of mass(group); the listed groups against the oracle."""
    masses = []
    for g in range(w.h_kv):
        wg = _kv_group(w, g)
        ctx = H.make_ctx(wg)
        s_g, m_g = H.gpu_score(ctx, wg)
        ctx.close()
        masses.append(m_g.astype(np.float64))
        if g in oracle_groups:
            s_ref, m_ref = oc.score_units(wg.q, wg.k_hist, wg.units, wg.w_modality)
            P._check_scores(s_g, m_g, s_ref, m_ref)
    mass_mean = np.mean(masses, axis=0)
    lens = w.units[:, 1].astype(np.float64)
    wmod = np.array([w.w_modality[m] for m in w.units[:, 2]])
    score_from_groups = wmod * mass_mean * w.n_hist / lens
    rel = np.abs(full_scores - score_from_groups) / np.maximum(np.abs(score_from_groups), 1e-3 * np.abs(score_from_groups).max())
    assert rel.max() <= 2e-5, rel.max()
    assert abs(mass_mean.sum() - 1.0) < 1e-4


def test_long_stream_full_size(H, ob, P):
    """Config 3 (80,000-token history, 2,354-token chunk): the workload bench.py times."""
    w = wl.long_stream()
    assert w.n_hist == 80000 and w.t == 2354
    res = P._run_step(H, ob, w)
    rng = np.random.Generator(np.random.PCG64(77))
    again = _check_integer_path_and_sampled_attention(H, ob, P, w, res, rng)
    assert res["info"]["n_kept"] <= w.n_hist and res["info"]["n_kept"] >= min(w.budget, w.n_hist) - 2304 - 64
    _check_scores_by_group(H, ob, P, w, res["scores"], oracle_groups=(3,))
    # the whole selection against the oracle's own scores of the sampled group is not defined (scores average
    # all groups); the decision rule itself is checked exactly above, given the GPU's scores
    assert again["unit_keep"].sum() > 0


@pytest.mark.parametrize("t,ratio,page,cell,oracle_groups", [
    (256, 0.05, 16, 0, (0,)),
    (1024, 0.25, 256, 1, (5,)),
    (4096, 0.5, 64, 2, ()),
])
def test_sweep_cells_full_size(H, ob, P, t, ratio, page, cell, oracle_groups):
    """Config 5 sub-grid (131,072-token history, heavy-tailed key scales): one cell per chunk size."""
    w = wl.sweep_cell(t, ratio, page, cell=cell)
    assert w.n_hist == 131072 and w.t == t
    res = P._run_step(H, ob, w)
    rng = np.random.Generator(np.random.PCG64(78 + cell))
    _check_integer_path_and_sampled_attention(H, ob, P, w, res, rng)
    assert res["info"]["span_pages"] * page >= res["info"]["n_kept"]
    _check_scores_by_group(H, ob, P, w, res["scores"], oracle_groups=oracle_groups)


def test_stream_loop_short(H, ob, P):
    """Config 4 shape: chunks of one frame from {640, 1280, 2304} tokens plus 2 s of audio at 10-25 tok/s,
    32/8 heads of 128, bf16, one layer, the cache carried on the device from chunk to chunk.  The budget
    is scaled down so that eviction starts within a few chunks.  Every step is compared with the oracle
    advanced from the same state: scores within tolerance, selection by the oracle's rule on the GPU's
    scores, cache bytes and unit table exactly, attention within tolerance."""
    sched = wl.loop_schedule(n_chunks=7)
    budget, page, R, caps, w_mod = 3000, 64, 1, (-1, -1, -1), (1.0, 2.0, 2.0)
    h_q, h_kv, d = 32, 8, 128
    s_cap, u_cap, t_cap = 12288, 64, 2400
    ctx = ob.Context(h_q, h_kv, d, "bf16", s_cap, u_cap, t_cap)
    rng = np.random.Generator(np.random.PCG64(4242))
    draw = lambda shape: wl.round_to_bf16(rng.standard_normal(shape, dtype=np.float32))
    units = wl.loop_prefix_units()
    k_cache, v_cache = draw((16, h_kv, d)), draw((16, h_kv, d))
    dev = lambda a: ob.to_device(a, "bf16")
    k_a = torch.zeros((s_cap, h_kv, d), dtype=torch.bfloat16, device="cuda")
    v_a = torch.zeros_like(k_a)
    k_b, v_b = torch.full_like(k_a, float("nan")), torch.full_like(v_a, float("nan"))
    k_a[:16], v_a[:16] = dev(k_cache), dev(v_cache)
    units_a = ob.units_to_device(units, u_cap)
    units_b = torch.zeros_like(units_a)
    n_hist_a, n_units_a = H.i32(16), H.i32(len(units))
    n_hist_b, n_units_b = H.i32(-1), H.i32(-1)
    params = ob.select_params(budget, R, caps)
    evicted = False
    for c, cu in enumerate(sched):
        T = int(cu[:, 1].sum())
        n, U = len(k_cache), len(units)
        zs = np.exp(0.5 * rng.standard_normal(len(cu))).astype(np.float32)
        q, v_chunk = draw((T, h_q, d)), draw((T, h_kv, d))
        k_chunk = wl.round_to_bf16(rng.standard_normal((T, h_kv, d), dtype=np.float32) * np.repeat(zs, cu[:, 1])[:, None, None])
        o = torch.full((T, h_q, d), float("nan"), dtype=torch.float32, device="cuda")
        info = torch.zeros((8,), dtype=torch.int32, device="cuda")
        qd = dev(q)
        ctx.chunk_step(qd, dev(k_chunk), dev(v_chunk), T, ob.units_to_device(cu), len(cu), k_a, v_a, n_hist_a, n, units_a,
                       n_units_a, U, w_mod, params, page, 0.0, k_b, v_b, units_b, n_hist_b, n_units_b, o, ob.DTYPE_FP32,
                       info_out=info)
        torch.cuda.synchronize()
        assert ctx.poll_status() == 0
        # the scores the step used (the work buffers are not part of the ABI: the scoring call is repeated)
        scores = torch.zeros((U,), dtype=torch.float32, device="cuda")
        ctx.score_units(qd, T, k_a, n_hist_a, n, units_a, n_units_a, U, w_mod, 0.0, scores, None)
        torch.cuda.synchronize()
        gpu_scores = scores.cpu().numpy()
        s_ref, _ = oc.score_units(q, k_cache, units, w_mod)
        rel = np.abs(gpu_scores - s_ref) / np.maximum(np.abs(s_ref), 1e-3 * np.abs(s_ref).max())
        assert rel.max() <= P.SCORE_REL, (c, rel.max())
        st = oc.stream_step(q, k_cache, v_cache, units, k_chunk, v_chunk, cu, w_mod, budget, R, caps, page,
                            scores_override=gpu_scores)
        P._selection_matches(units, st["select"]["unit_keep"], gpu_scores, s_ref, budget, R, caps)
        n_new = len(st["k_cache"])
        assert int(n_hist_b.item()) == n_new and int(n_units_b.item()) == len(st["units"])
        assert np.array_equal(units_b[:len(st["units"])].cpu().numpy(), st["units"])
        got = ob.info_to_dict(info)
        cp = st["compact"]
        assert got["n_kept"] == cp["n_kept"] and got["span_pages"] == cp["span_pages"] and got["rows_moved"] == cp["rows_moved"]
        assert got["span_pages"] * page - got["n_kept"] < page
        for gpu_c, ref_c in ((k_b, st["k_cache"]), (v_b, st["v_cache"])):
            bits = H.bytes_of(gpu_c[:n_new]).reshape(n_new, -1).view(np.uint16).reshape(n_new, h_kv, d)
            assert np.array_equal(bits, wl.bf16_bits(ref_c))
        P._check_attention(o.cpu().numpy(), None, st["o"], None)
        evicted |= cp["n_kept"] < n
        # advance both states
        k_cache, v_cache, units = st["k_cache"], st["v_cache"], st["units"]
        k_a, k_b, v_a, v_b = k_b, k_a, v_b, v_a
        units_a, units_b = units_b, units_a
        n_hist_a, n_hist_b, n_units_a, n_units_b = n_hist_b, n_hist_a, n_units_b, n_units_a
    assert evicted, "the schedule never exceeded the budget: the test did not exercise eviction"
    ctx.close()


def test_stream_loop_structural_short(H, ob, P):
    """The score-free pass (structural plan -> unit-granular compaction with sink prefixes -> attention -> append)
    carried on the device over nine chunks of the config-4 schedule, with a text span added to every other chunk so
    that the text budget matters; every step against the oracle advanced from the same state: unit table, counts
    and cache bytes exactly, attention within tolerance."""
    sched = wl.loop_schedule(n_chunks=9)
    Hw, Lw, R, sink, Tb, page = 4000, 3000, 2, (48, 6, 0), 40, 64
    h_q, h_kv, d = 32, 8, 128
    s_cap, u_cap, t_cap = 12288, 96, 2432
    ctx = ob.Context(h_q, h_kv, d, "bf16", s_cap, u_cap, t_cap)
    rng = np.random.Generator(np.random.PCG64(4343))
    draw = lambda shape: wl.round_to_bf16(rng.standard_normal(shape, dtype=np.float32))
    units = wl.loop_prefix_units()
    k_cache, v_cache = draw((16, h_kv, d)), draw((16, h_kv, d))
    dev = lambda a: ob.to_device(a, "bf16")
    k_a = torch.zeros((s_cap, h_kv, d), dtype=torch.bfloat16, device="cuda")
    v_a = torch.zeros_like(k_a)
    k_b, v_b = torch.full_like(k_a, float("nan")), torch.full_like(v_a, float("nan"))
    k_a[:16], v_a[:16] = dev(k_cache), dev(v_cache)
    units_a = ob.units_to_device(units, u_cap)
    units_b = torch.zeros_like(units_a)
    n_hist_a, n_units_a = H.i32(16), H.i32(len(units))
    n_hist_b, n_units_b = H.i32(-1), H.i32(-1)
    params = ob.structural_params(Hw, Lw, R, sink, Tb)
    saw_sink = saw_drop = False
    for c, cu in enumerate(sched):
        if c % 2 == 1:                                       # a text query behind the audio of every other chunk
            tx = wl.make_units([(int(rng.integers(16, 40)), wl.MOD_TEXT, c + 1)], group_of_first=None)
            tx[0, 0] = int(cu[:, 1].sum())
            cu = np.concatenate([cu, tx], axis=0)
        T = int(cu[:, 1].sum())
        n, U = len(k_cache), len(units)
        q, k_chunk, v_chunk = draw((T, h_q, d)), draw((T, h_kv, d)), draw((T, h_kv, d))
        o = torch.full((T, h_q, d), float("nan"), dtype=torch.float32, device="cuda")
        info = torch.zeros((8,), dtype=torch.int32, device="cuda")
        ctx.chunk_step_structural(dev(q), dev(k_chunk), dev(v_chunk), T, ob.units_to_device(cu), len(cu), k_a, v_a, n_hist_a, n,
                                  units_a, n_units_a, U, params, page, 0.0, k_b, v_b, units_b, n_hist_b, n_units_b, o,
                                  ob.DTYPE_FP32, info_out=info)
        torch.cuda.synchronize()
        assert ctx.poll_status() == 0
        st = oc.stream_step_structural(q, k_cache, v_cache, units, k_chunk, v_chunk, cu, Hw, Lw, R, sink, Tb, page)
        n_new = len(st["k_cache"])
        assert int(n_hist_b.item()) == n_new and int(n_units_b.item()) == len(st["units"])
        assert np.array_equal(units_b[:len(st["units"])].cpu().numpy(), st["units"])
        got, cp = ob.info_to_dict(info), st["compact"]
        assert (got["n_kept"], got["span_pages"], got["rows_moved"]) == (cp["n_kept"], cp["span_pages"], cp["rows_moved"])
        assert got["part_begin"] == cp["part_begin"].tolist()
        for gpu_c, ref_c in ((k_b, st["k_cache"]), (v_b, st["v_cache"])):
            bits = H.bytes_of(gpu_c[:n_new]).reshape(n_new, -1).view(np.uint16).reshape(n_new, h_kv, d)
            assert np.array_equal(bits, wl.bf16_bits(ref_c))
        P._check_attention(o.cpu().numpy(), None, st["o"], None)
        saw_sink |= bool((st["plan"]["unit_keep"] == 1).any())
        saw_drop |= bool((st["plan"]["unit_keep"] == 0).any())
        k_cache, v_cache, units = st["k_cache"], st["v_cache"], st["units"]
        k_a, k_b, v_a, v_b = k_b, k_a, v_b, v_a
        units_a, units_b = units_b, units_a
        n_hist_a, n_hist_b, n_units_a, n_units_b = n_hist_b, n_hist_a, n_units_b, n_units_a
    assert saw_sink and saw_drop, "the schedule must exercise sink prefixes and dropped spans"
    ctx.close()
