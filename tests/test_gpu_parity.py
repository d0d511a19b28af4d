"""Parity of the CUDA path (through the C ABI) against the CPU oracle, element by element."""
import math

import numpy as np
import pytest
import torch

from oracle import omni_oracle as oc
from paper_2609_34653_b200 import workloads as wl

pytestmark = pytest.mark.gpu

ATT_MAX_ABS, ATT_MEAN_ABS = 1e-2, 1e-3       # attention tolerance on fp32 outputs
SCORE_REL = 1e-3                              # unit scores, relative
TIE_REL = 1e-4                                # score gap below which the selected set may differ


@pytest.fixture(scope="module")
def H():
    from tests import gpu_helpers
    return gpu_helpers


@pytest.fixture(scope="module")
def ob():
    from paper_2609_34653_b200 import binding
    return binding


@pytest.fixture(scope="module")
def cfg2():
    return wl.layer_8b()


# ------------------------------------------------------------------------------------ compaction
@pytest.mark.parametrize("S,rowshape,dtype,page,density", [
    (1, (1, 64), torch.float32, 16, 1.0),
    (17, (1, 64), torch.float32, 16, 0.5),
    (2048, (1, 64), torch.float32, 16, 0.5),
    (1000, (8, 128), torch.bfloat16, 64, 0.3),
    (5000, (2, 64), torch.bfloat16, 256, 0.9),
    (16384, (8, 128), torch.bfloat16, 64, 0.25),
    (80000, (8, 128), torch.bfloat16, 64, 0.1),
])
@pytest.mark.parametrize("in_place", [False, True])
def test_compact_bit_exact(H, ob, S, rowshape, dtype, page, density, in_place):
    rng = np.random.default_rng(S + 7 * in_place)
    mask = (rng.random(S) < density).astype(np.uint8)
    es = 2 if dtype == torch.bfloat16 else 4
    raw = rng.integers(0, 256, size=(2, S, rowshape[0] * rowshape[1] * es), dtype=np.uint8)
    k = torch.from_numpy(raw[0]).cuda().view(dtype).view(S, *rowshape).contiguous()
    v = torch.from_numpy(raw[1]).cuda().view(dtype).view(S, *rowshape).contiguous()
    exp = oc.compact_pack(raw[0], raw[1], mask, page)
    ctx = ob.Context(4 * rowshape[0], rowshape[0], rowshape[1], "bf16" if es == 2 else "fp32", S + 64, 8, 16)
    got = H.gpu_compact(ctx, k, v, mask, page, in_place=in_place, s_span_max=S + 40)
    n = exp["n_kept"]
    assert (got["n_kept"], got["span_pages"], got["rows_moved"]) == (n, exp["span_pages"], exp["rows_moved"])
    assert np.array_equal(got["slot_map"], exp["slot_map"])
    assert np.array_equal(H.bytes_of(got["k"][:n]).reshape(n, -1), exp["k"])
    assert np.array_equal(H.bytes_of(got["v"][:n]).reshape(n, -1), exp["v"])
    n_pages = (S + 40 + page - 1) // page
    exp_pc = np.full(n_pages, 255, np.uint8)
    exp_pc[:len(exp["page_class"])] = exp["page_class"]
    assert np.array_equal(got["page_class"], exp_pc)
    ctx.close()


def test_compact_edges_and_partitions(H, ob):
    rng = np.random.default_rng(1)
    S = 300
    k = torch.from_numpy(rng.standard_normal((S, 2, 64)).astype(np.float32)).cuda()
    v = torch.from_numpy(rng.standard_normal((S, 2, 64)).astype(np.float32)).cuda()
    ctx = ob.Context(4, 2, 64, "fp32", 512, 16, 16)
    # none kept / all kept
    got = H.gpu_compact(ctx, k, v, np.zeros(S, np.uint8), 16)
    assert (got["n_kept"], got["span_pages"], got["rows_moved"]) == (0, 0, 0) and np.all(got["slot_map"] == -1)
    assert np.all(got["page_class"] == 255)
    got = H.gpu_compact(ctx, k, v, np.ones(S, np.uint8), 16)
    assert (got["n_kept"], got["span_pages"], got["rows_moved"]) == (S, 19, 0)
    assert torch.equal(got["k"], k) and torch.equal(got["v"], v)
    # partitions and page classes from the compacted unit table
    units_out = np.array([[0, 20, 2, 0, 0, 0], [20, 30, 0, 1, 1, 0], [50, 14, 1, 1, 1, 0], [64, 25, 0, 9, 2, 0]], np.int32)
    mask = np.zeros(S, np.uint8)
    mask[np.arange(89) + np.arange(89) // 3] = 1
    exp = oc.compact_pack(H.bytes_of(k).reshape(S, -1), H.bytes_of(v).reshape(S, -1), mask, 16, units_out)
    got = H.gpu_compact(ctx, k, v, mask, 16, units_out_np=units_out)
    assert got["part_begin"] == exp["part_begin"].tolist() == [0, 20, 64, 89]
    assert np.array_equal(got["page_class"], exp["page_class"])
    # idempotence: compacting the packed cache moves nothing
    mask2 = np.zeros(S, np.uint8)
    mask2[:89] = 1
    got2 = H.gpu_compact(ctx, got["k"], got["v"], mask2, 16)
    assert got2["rows_moved"] == 0 and torch.equal(got2["k"][:89], got["k"][:89])
    # determinism: same inputs twice give identical bytes
    got3 = H.gpu_compact(ctx, k, v, mask, 16, units_out_np=units_out)
    assert torch.equal(got3["k"][:89], got["k"][:89]) and np.array_equal(got3["slot_map"], got["slot_map"])
    # host-side argument errors
    with pytest.raises(ob.OmniTideError):
        ctx.compact(k, v, k, v, None, None, S, 16, None, None, 1, None, None, None)
    with pytest.raises(ob.OmniTideError):
        ctx.compact(k, v, torch.empty_like(k), torch.empty_like(v), torch.zeros(4096, dtype=torch.uint8, device="cuda"),
                    None, 4000, 16, None, None, 1, None, None, None)      # above s_cap
    ctx.close()


@pytest.mark.parametrize("U,max_len,rowshape,dtype,page,density,seed", [
    (1, 40, (1, 64), torch.float32, 16, 1.0, 0),
    (12, 300, (2, 64), torch.bfloat16, 16, 0.5, 1),
    (70, 2400, (8, 128), torch.bfloat16, 64, 0.15, 2),
    (600, 90, (8, 128), torch.bfloat16, 256, 0.5, 3),         # more units than threads in a CTA
    (37, 1000, (8, 128), torch.bfloat16, 64, 0.0, 4),          # nothing kept
])
@pytest.mark.parametrize("in_place", [False, True])
def test_compact_units_bit_exact(H, ob, U, max_len, rowshape, dtype, page, density, seed, in_place):
    """The unit-granular entry point equals the oracle's pack of the equivalent token mask, bit for bit."""
    rng = np.random.default_rng(100 + seed)
    units = _random_table(rng, U) if U > 1 else wl.make_units([(int(max_len), 0, 0)])
    if U > 1:
        units[:, 1] = rng.integers(1, max_len + 1, size=U)
        units[:, 0] = np.concatenate([[0], np.cumsum(units[:-1, 1])])
    S = int(units[:, 1].sum())
    keep_u = np.where(rng.random(U) < density, 2, 0).astype(np.uint8)
    mask = np.repeat(keep_u != 0, units[:, 1]).astype(np.uint8)
    es = 2 if dtype == torch.bfloat16 else 4
    raw = rng.integers(0, 256, size=(2, S, rowshape[0] * rowshape[1] * es), dtype=np.uint8)
    k = torch.from_numpy(raw[0]).cuda().view(dtype).view(S, *rowshape).contiguous()
    v = torch.from_numpy(raw[1]).cuda().view(dtype).view(S, *rowshape).contiguous()
    # the survivors' table as the selection step writes it (start = kept tokens before the unit)
    kept_idx = np.nonzero(keep_u)[0]
    units_out = units[kept_idx].copy()
    if len(units_out):
        units_out[:, 0] = np.concatenate([[0], np.cumsum(units_out[:-1, 1])])
        idx = np.arange(len(units_out))
        units_out[:, 4] = np.where(idx == 0, 0, np.where(idx < (2 * len(units_out)) // 3, 1, 2))   # ordered groups
    exp = oc.compact_pack(raw[0], raw[1], mask, page, units_out if len(units_out) else None)
    ctx = ob.Context(4 * rowshape[0], rowshape[0], rowshape[1], "bf16" if es == 2 else "fp32", S + 64, U + 8, 16)
    got = H.gpu_compact_units(ctx, k, v, units, keep_u, page, units_out_np=units_out, in_place=in_place, s_span_max=S + 40,
                              u_max=U + 5)
    assert got["status"] == 0
    n = exp["n_kept"]
    assert (got["n_kept"], got["span_pages"], got["rows_moved"]) == (n, exp["span_pages"], exp["rows_moved"])
    assert np.array_equal(got["slot_map"], exp["slot_map"])
    if n:
        assert np.array_equal(H.bytes_of(got["k"][:n]).reshape(n, -1), exp["k"])
        assert np.array_equal(H.bytes_of(got["v"][:n]).reshape(n, -1), exp["v"])
    if len(units_out):
        assert got["part_begin"] == exp["part_begin"].tolist()
    n_pages = (S + 40 + page - 1) // page
    exp_pc = np.full(n_pages, 255, np.uint8)
    exp_pc[:len(exp["page_class"])] = exp["page_class"]
    assert np.array_equal(got["page_class"], exp_pc)
    # and it agrees with the mask entry point on the same decision
    if not in_place:
        got_m = H.gpu_compact(ctx, k, v, mask, page, units_out_np=units_out if len(units_out) else None)
        assert np.array_equal(H.bytes_of(got_m["k"][:n]), H.bytes_of(got["k"][:n]))
        assert np.array_equal(H.bytes_of(got_m["v"][:n]), H.bytes_of(got["v"][:n]))
    ctx.close()


@pytest.mark.parametrize("n_layers,U,max_len,density,seed", [(1, 9, 200, 0.5, 0), (3, 40, 700, 0.3, 1), (5, 70, 300, 0.9, 2),
                                                             (4, 12, 500, 0.0, 3)])
def test_compact_units_batched_bit_exact(H, ob, n_layers, U, max_len, density, seed):
    """Cross-layer batching: every layer's packed cache equals the oracle's pack of that layer with the shared mask."""
    rng = np.random.default_rng(200 + seed)
    units = _random_table(rng, U)
    units[:, 1] = rng.integers(1, max_len + 1, size=U)
    units[:, 0] = np.concatenate([[0], np.cumsum(units[:-1, 1])])
    S = int(units[:, 1].sum())
    keep_u = np.where(rng.random(U) < density, 2, 0).astype(np.uint8)
    mask = np.repeat(keep_u != 0, units[:, 1]).astype(np.uint8)
    rowshape, page = (8, 128), 64
    raw = rng.integers(0, 256, size=(n_layers, 2, S, rowshape[0] * rowshape[1] * 2), dtype=np.uint8)
    ks = [torch.from_numpy(raw[l, 0]).cuda().view(torch.bfloat16).view(S, *rowshape).contiguous() for l in range(n_layers)]
    vs = [torch.from_numpy(raw[l, 1]).cuda().view(torch.bfloat16).view(S, *rowshape).contiguous() for l in range(n_layers)]
    kd = [torch.zeros_like(k) for k in ks]
    vd = [torch.zeros_like(v) for v in vs]
    ptrs = lambda ts: torch.tensor([t.data_ptr() for t in ts], dtype=torch.int64, device="cuda")
    ctx = ob.Context(32, 8, 128, "bf16", S + 64, U + 8, 16)
    du = ob.units_to_device(units, U + 4)
    keep = torch.full((U + 20,), 2, dtype=torch.uint8, device="cuda")
    keep[:U] = torch.from_numpy(keep_u).cuda()
    slot_map = torch.full((S + 16,), -5, dtype=torch.int32, device="cuda")
    info = torch.full((8,), -5, dtype=torch.int32, device="cuda")
    ctx.compact_units_batched(ptrs(ks), ptrs(vs), ptrs(kd), ptrs(vd), n_layers, du, H.i32(U), U + 4, keep, S, page, None, None,
                              slot_map, info, None)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    got = ob.info_to_dict(info)
    for l in range(n_layers):
        exp = oc.compact_pack(raw[l, 0], raw[l, 1], mask, page)
        n = exp["n_kept"]
        assert (got["n_kept"], got["span_pages"], got["rows_moved"]) == (n, exp["span_pages"], exp["rows_moved"])
        if n:
            assert np.array_equal(H.bytes_of(kd[l][:n]).reshape(n, -1), exp["k"]), l
            assert np.array_equal(H.bytes_of(vd[l][:n]).reshape(n, -1), exp["v"]), l
        assert np.array_equal(slot_map[:S].cpu().numpy(), exp["slot_map"])
    ctx.close()


def test_compact_units_rejects_bad_tables(H, ob):
    rng = np.random.default_rng(5)
    units = wl.make_units([(100, 0, 0), (50, 1, 1), (70, 0, 2)])
    S = 220
    k = torch.from_numpy(rng.standard_normal((S, 2, 64)).astype(np.float32)).cuda()
    v = torch.from_numpy(rng.standard_normal((S, 2, 64)).astype(np.float32)).cuda()
    ctx = ob.Context(4, 2, 64, "fp32", 512, 16, 16)
    bad = units.copy()
    bad[2, 1] = 4000                                          # reaches outside the span: flagged, treated as dropped
    got = H.gpu_compact_units(ctx, k, v, bad, np.array([2, 0, 2], np.uint8), 16, s_span_max=S)
    assert got["status"] & 2 and got["n_kept"] == 100
    with pytest.raises(ob.OmniTideError):
        ctx.compact_units(k, v, torch.empty_like(k), torch.empty_like(v), None, None, 3, None, S, 16, None, None, None,
                          None, None)
    ctx.close()


# ------------------------------------------------------------------------------------- selection
def _random_table(rng, U):
    lens = rng.integers(1, 400, size=U)
    mods = rng.integers(0, 3, size=U)
    events = np.cumsum(rng.integers(0, 2, size=U))
    spans = list(zip(lens.tolist(), mods.tolist(), events.tolist()))
    units = wl.make_units(spans, group_of_first=0 if rng.random() < 0.7 else None)
    return units


def test_select_exact_given_scores(H, ob):
    rng = np.random.default_rng(77)
    ctx = ob.Context(4, 2, 64, "bf16", 1 << 20, 2048, 16)
    for trial in range(60):
        U = int(rng.choice([1, 2, 3, 7, 31, 32, 33, 100, 257, 1500]))
        units = _random_table(rng, U)
        scores = rng.random(U).astype(np.float32)
        if trial % 3 == 0:
            scores = np.round(scores * 4) / 4                   # many exact ties
        if trial % 5 == 0:
            scores[rng.integers(U)] = np.nan
            scores[rng.integers(U)] = -0.0
        n = int(units[:, 1].sum())
        budget = int(rng.integers(1, n + 50))
        R = int(rng.integers(0, 4))
        caps = tuple(int(c) for c in rng.choice([-1, 200, 1000, 5000], size=3))
        exp = oc.select_units(units, scores, budget, R, caps)
        got = H.gpu_select(ctx, units, scores, budget, R, caps)
        assert got["status"] == 0
        assert np.array_equal(got["unit_keep"], exp["unit_keep"]), (trial, U)
        assert got["n_kept"] == exp["n_kept"] and got["n_units_out"] == len(exp["units_out"])
        assert np.array_equal(got["keep_mask"], exp["keep_mask"])
        assert np.array_equal(got["units_out"], exp["units_out"])
    # malformed tables are reported, not trusted
    bad = wl.make_units([(5, 0, 3), (5, 0, 2)], group_of_first=None)
    got = H.gpu_select(ctx, bad, np.zeros(2, np.float32), 5, 1, (-1, -1, -1))
    assert got["status"] & ob.DEV_BAD_UNITS
    ctx.close()


# -------------------------------------------------------------------------------------- attention
def _check_attention(o, lse, o_ref, lse_ref):
    err = np.abs(o - o_ref)
    assert np.isfinite(o).all()
    assert err.max() <= ATT_MAX_ABS, err.max()
    assert err.mean() <= ATT_MEAN_ABS, err.mean()
    if lse is not None:
        # the tensor-core path normalises with the bf16-rounded weights it multiplies by, so its
        # log-sum-exp carries their rounding (2^-9 relative on a dominant weight)
        assert np.abs(lse - lse_ref).max() <= 5e-3


def test_attention_tiny_fp32(H, ob):
    w = wl.tiny()
    ctx = H.make_ctx(w)
    kh, vh = ob.to_device(w.k_hist, "fp32"), ob.to_device(w.v_hist, "fp32")
    for n in (1024, 1000, 0):
        o, lse = H.gpu_attention(ctx, w, kh[:max(n, 1)], vh[:max(n, 1)], n)
        o_ref, lse_ref = oc.chunk_attention(w.q, w.k_hist[:n], w.v_hist[:n], w.k_chunk, w.v_chunk)
        _check_attention(o, lse, o_ref, lse_ref)
    ctx.close()


@pytest.mark.parametrize("seed,d,t,n_hist", [(1, 64, 200, None), (2, 32, 77, None), (3, 256, 40, None)])
def test_attention_cuda_core_bf16(H, ob, seed, d, t, n_hist):
    w = wl.small_mixed(seed, d=d, t=t)
    ctx = H.make_ctx(w)
    kh, vh = ob.to_device(w.k_hist, "bf16"), ob.to_device(w.v_hist, "bf16")
    o, lse = H.gpu_attention(ctx, w, kh, vh, w.n_hist)
    o_ref, lse_ref = oc.chunk_attention(w.q, w.k_hist, w.v_hist, w.k_chunk, w.v_chunk)
    _check_attention(o, lse, o_ref, lse_ref)
    ctx.close()


@pytest.mark.parametrize("t,n_hist,h_q,h_kv", [
    (128, 128, 4, 2),       # one full tile, one full history block
    (50, 77, 4, 1),         # ragged everything, single pair with one active tile
    (300, 1000, 8, 2),      # 3 tiles (second pair half empty), ragged history tail
    (256, 0, 4, 4),         # no history: plain causal self-attention
    (690, 4080, 8, 2),      # config-2 chunk and kept-history sizes
    (1, 1, 4, 2),
    # few queries: the GQA-packed tile (all query heads of a KV group in one 128-row tile)
    (1, 8191, 32, 8),       # decode over the config-3 retained history
    (1, 0, 8, 2),           # decode with an empty history: the token attends to itself
    (4, 5000, 32, 8),       # 4 tokens x 4 heads = 16 rows of the tile
    (32, 1000, 32, 8),      # exactly fills the packed tile
    (33, 1000, 32, 8),      # one token too many: falls back to one tile per head
    (16, 300, 8, 1),        # G = 8
    (5, 129, 12, 4),        # G = 3 is not a power of two: not packed
])
def test_attention_tensor_core(H, ob, t, n_hist, h_q, h_kv):
    rng = np.random.default_rng(t * 7 + n_hist)
    units = wl.make_units([(max(n_hist, 1), 0, 0)], group_of_first=None)
    chunk_units = wl.make_units([(t, 0, 1)], group_of_first=None)
    q, kh, vh, kc, vc = wl.random_layer_inputs(rng, units, chunk_units, h_q, h_kv, 128, "bf16")
    kh, vh = kh[:n_hist], vh[:n_hist]
    w = wl.Workload("tc", h_q, h_kv, 128, "bf16", units, chunk_units, 1, 64, 1, q=q, k_hist=kh, v_hist=vh,
                    k_chunk=kc, v_chunk=vc)
    ctx = ob.Context(h_q, h_kv, 128, "bf16", n_hist + 300, 8, t)
    # device buffers longer than the history, tail poisoned with NaN: must not leak into the output
    pad = 200
    khd = torch.full((n_hist + pad, h_kv, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    vhd = torch.full((n_hist + pad, h_kv, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    if n_hist:
        khd[:n_hist] = ob.to_device(kh, "bf16")
        vhd[:n_hist] = ob.to_device(vh, "bf16")
    o_ref, lse_ref = oc.chunk_attention(q, kh, vh, kc, vc)
    o, lse = H.gpu_attention(ctx, w, khd, vhd, n_hist, n_hist_max=n_hist + pad)
    _check_attention(o, lse, o_ref, lse_ref)
    # bf16 output is the fp32 result rounded to nearest even
    o16, _ = H.gpu_attention(ctx, w, khd, vhd, n_hist, out_fp32=False, n_hist_max=n_hist + pad)
    assert np.array_equal(o16, wl.round_to_bf16(o))
    # the CUDA-core kernels agree as a second implementation
    ctx.set_option(ob.OPT_FORCE_CUDA_CORES, 1)
    o2, lse2 = H.gpu_attention(ctx, w, khd, vhd, n_hist, n_hist_max=n_hist + pad)
    _check_attention(o2, lse2, o_ref, lse_ref)
    ctx.close()


# ---------------------------------------------------------------------------------------- scoring
def _check_scores(score, mass, score_ref, mass_ref):
    assert np.isfinite(score).all()
    assert np.abs(mass - mass_ref).max() <= SCORE_REL * max(mass_ref.max(), 1e-30)
    rel = np.abs(score - score_ref) / np.maximum(np.abs(score_ref), 1e-3 * np.abs(score_ref).max())
    assert rel.max() <= SCORE_REL, rel.max()
    assert abs(mass.sum() - 1.0) < 1e-4


def test_score_tiny_and_small(H, ob):
    w = wl.tiny()
    ctx = H.make_ctx(w)
    s, m = H.gpu_score(ctx, w)
    s_ref, m_ref = oc.score_units(w.q, w.k_hist, w.units, w.w_modality)
    _check_scores(s, m, s_ref, m_ref)
    ctx.close()
    for seed, d in [(4, 64), (5, 128), (6, 128)]:
        w = wl.small_mixed(seed, d=d, n_units=11, max_len=500, t=333)
        ctx = H.make_ctx(w)
        s, m = H.gpu_score(ctx, w, use_dev_counts=(seed % 2 == 0))
        s_ref, m_ref = oc.score_units(w.q, w.k_hist, w.units, w.w_modality)
        _check_scores(s, m, s_ref, m_ref)
        ctx.close()


def test_score_closed_form_identical_keys(H, ob):
    """All history keys equal: every unit's score is exactly its modality weight."""
    w = wl.small_mixed(9, d=128, n_units=7, max_len=300, t=130)
    w.k_hist[:] = w.k_hist[0:1]
    ctx = H.make_ctx(w)
    wm = (1.0, 2.5, 0.75)
    s, m = H.gpu_score(ctx, w, w_mod=wm)
    exp = np.array([wm[mod] for mod in w.units[:, 2]])
    assert np.abs(s - exp).max() < 1e-3
    ctx.close()


def test_score_config2(H, ob, cfg2):
    w = cfg2
    ctx = H.make_ctx(w)
    s, m = H.gpu_score(ctx, w)
    s_ref, m_ref = oc.score_units(w.q, w.k_hist, w.units, w.w_modality)
    _check_scores(s, m, s_ref, m_ref)
    ctx.close()


# ------------------------------------------------------------------------------ the whole pass
def _selection_matches(units, gpu_keep, gpu_scores, ref_scores, budget, R, caps):
    """The selected set equals the oracle's, except where the oracle's score gap at a decision is
    below TIE_REL: (i) the oracle's integer rule applied to the GPU's scores reproduces the GPU set
    exactly, and (ii) the two rankings differ only by swaps of units whose oracle scores are
    within TIE_REL of each other."""
    again = oc.select_units(units, gpu_scores, budget, R, caps)
    assert np.array_equal(again["unit_keep"], gpu_keep)
    ref = oc.select_units(units, ref_scores.astype(np.float32), budget, R, caps)
    if np.array_equal(ref["unit_keep"], gpu_keep):
        return
    pos_ref = {u: i for i, u in enumerate(ref["order"])}
    for a, b in zip(again["order"], again["order"][1:]):
        if pos_ref[a] > pos_ref[b]:
            gap = abs(ref_scores[a] - ref_scores[b]) / max(abs(ref_scores[a]), abs(ref_scores[b]), 1e-30)
            assert gap < TIE_REL, (a, b, gap)


def _run_step(H, ob, w, host=False):
    N, T, U = w.n_hist, w.t, len(w.units)
    s_cap = N + T + 64
    u_cap = U + len(w.chunk_units) + 4
    ctx = ob.Context(w.h_q, w.h_kv, w.d, w.dtype, s_cap, u_cap, T)
    tdt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    kc_in = torch.zeros((s_cap, w.h_kv, w.d), dtype=tdt, device="cuda")
    vc_in = torch.zeros_like(kc_in)
    kc_in[:N] = ob.to_device(w.k_hist, w.dtype)
    vc_in[:N] = ob.to_device(w.v_hist, w.dtype)
    kc_out = torch.full_like(kc_in, float("nan"))
    vc_out = torch.full_like(vc_in, float("nan"))
    units_in = ob.units_to_device(w.units, u_cap)
    units_out = torch.zeros((u_cap, 6), dtype=torch.int32, device="cuda")
    n_hist_out, n_units_out = H.i32(-1), H.i32(-1)
    info = torch.zeros((8,), dtype=torch.int32, device="cuda")
    params = ob.select_params(w.budget, w.n_recent_events, w.modality_cap)
    if host:
        conv = (lambda a: torch.from_numpy(a).to(tdt).contiguous().pin_memory())
        q, kc, vc = conv(w.q), conv(w.k_chunk), conv(w.v_chunk)
        cu = np.ascontiguousarray(w.chunk_units, dtype=np.int32)
        o = torch.empty((T, w.h_q, w.d), dtype=torch.float32).pin_memory()
        ctx.chunk_step_host(q, kc, vc, T, cu, len(cu), kc_in, vc_in, H.i32(N), N, units_in, H.i32(U), U, w.w_modality,
                            params, w.page_size, 0.0, kc_out, vc_out, units_out, n_hist_out, n_units_out, o,
                            ob.DTYPE_FP32, info_out=info)
    else:
        q, kc, vc = (ob.to_device(a, w.dtype) for a in (w.q, w.k_chunk, w.v_chunk))
        cu = ob.units_to_device(w.chunk_units)
        o = torch.full((T, w.h_q, w.d), float("nan"), dtype=torch.float32, device="cuda")
        ctx.chunk_step(q, kc, vc, T, cu, len(w.chunk_units), kc_in, vc_in, H.i32(N), N, units_in, H.i32(U), U,
                       w.w_modality, params, w.page_size, 0.0, kc_out, vc_out, units_out, n_hist_out, n_units_out, o,
                       ob.DTYPE_FP32, info_out=info)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    res = dict(o=o.cpu().numpy(), info=ob.info_to_dict(info), n_hist=int(n_hist_out.item()),
               n_units=int(n_units_out.item()), k=kc_out, v=vc_out, units=units_out.cpu().numpy(),
               scores=None, launches=ctx.launch_count())
    # the work buffers are not part of the ABI; re-run the scoring call to look at the scores
    res["scores"], _ = H.gpu_score(ctx, w)
    ctx.close()
    return res


def _check_step(H, ob, w, res):
    s_ref, _ = oc.score_units(w.q, w.k_hist, w.units, w.w_modality)
    n_new = res["n_hist"] - w.t
    nu = res["n_units"] - len(w.chunk_units)
    kept_units = res["units"][:nu]
    again = oc.select_units(w.units, res["scores"], w.budget, w.n_recent_events, w.modality_cap)
    assert np.array_equal(again["units_out"], kept_units)
    gpu_keep = again["unit_keep"]
    _selection_matches(w.units, gpu_keep, res["scores"], s_ref, w.budget, w.n_recent_events, w.modality_cap)
    # compaction: bit-exact given the GPU's keep mask
    es = 2 if w.dtype == "bf16" else 4
    raw_k = H.bytes_of(ob.to_device(w.k_hist, w.dtype)).reshape(w.n_hist, -1)
    raw_v = H.bytes_of(ob.to_device(w.v_hist, w.dtype)).reshape(w.n_hist, -1)
    cp = oc.compact_pack(raw_k, raw_v, again["keep_mask"], w.page_size, again["units_out"])
    assert res["info"]["n_kept"] == cp["n_kept"] == n_new
    assert res["info"]["span_pages"] == cp["span_pages"] and res["info"]["rows_moved"] == cp["rows_moved"]
    assert res["info"]["part_begin"] == cp["part_begin"].tolist()
    assert res["info"]["span_pages"] * w.page_size - n_new < w.page_size
    assert np.array_equal(H.bytes_of(res["k"][:n_new]).reshape(n_new, -1), cp["k"])
    assert np.array_equal(H.bytes_of(res["v"][:n_new]).reshape(n_new, -1), cp["v"])
    # appended chunk rows and units
    kc_bytes = H.bytes_of(res["k"][n_new:n_new + w.t]).reshape(w.t, -1)
    assert np.array_equal(kc_bytes.view(np.uint16 if es == 2 else np.uint32).reshape(w.t, w.h_kv, w.d),
                          (wl.bf16_bits(w.k_chunk) if es == 2 else w.k_chunk.view(np.uint32)))
    assert np.array_equal(res["units"][:res["n_units"]], oc.append_chunk(again["units_out"], n_new, w.chunk_units))
    # attention over the GPU's retained set
    keep_rows = again["keep_mask"].astype(bool)
    o_ref, _ = oc.chunk_attention(w.q, w.k_hist[keep_rows], w.v_hist[keep_rows], w.k_chunk, w.v_chunk)
    _check_attention(res["o"], None, o_ref, None)


def test_chunk_step_tiny(H, ob):
    w = wl.tiny()
    res = _run_step(H, ob, w)
    _check_step(H, ob, w, res)
    assert res["launches"] >= 5


def test_chunk_step_small_mixed_and_host_entry(H, ob):
    for seed, d in [(11, 64), (12, 128)]:
        w = wl.small_mixed(seed, d=d, n_units=12, max_len=400, t=300)
        _check_step(H, ob, w, _run_step(H, ob, w))
        _check_step(H, ob, w, _run_step(H, ob, w, host=True))


def test_chunk_step_host_pipelined_stream(H, ob):
    """Five chunks through omnitide_chunk_step_host_pipelined back to back, nothing waited for in between: every output
    and the final cache equal, bit for bit, what the device entry point gives one call at a time.  Each chunk has its own
    host buffers and values, so a staging buffer reused too early or a download taken too early shows."""
    w = wl.small_mixed(31, d=128, n_units=10, max_len=350, t=280)
    N, T, U = w.n_hist, w.t, len(w.units)
    n_steps = 5
    s_cap, u_cap = N + n_steps * T + 64, U + n_steps * len(w.chunk_units) + 4
    rng = np.random.default_rng(5)
    tdt = torch.bfloat16
    params = ob.select_params(w.budget, w.n_recent_events, w.modality_cap)
    chunks = []
    for i in range(n_steps):
        conv = lambda a: torch.from_numpy(a + 0.25 * rng.standard_normal(a.shape).astype(a.dtype)).to(tdt).contiguous()
        cu = np.ascontiguousarray(w.chunk_units, dtype=np.int32).copy()
        cu[:, oc.U_EVENT] += i                                  # later chunks are later events
        chunks.append((conv(w.q), conv(w.k_chunk), conv(w.v_chunk), cu))

    def run(pipelined):
        ctx = ob.Context(w.h_q, w.h_kv, w.d, w.dtype, s_cap, u_cap, T)
        caches = [[torch.zeros((s_cap, w.h_kv, w.d), dtype=tdt, device="cuda") for _ in range(2)] for _ in range(2)]
        caches[0][0][:N] = ob.to_device(w.k_hist, w.dtype)
        caches[0][1][:N] = ob.to_device(w.v_hist, w.dtype)
        units = [ob.units_to_device(w.units, u_cap), torch.zeros((u_cap, 6), dtype=torch.int32, device="cuda")]
        n_hist = [H.i32(N), H.i32(-1)]
        n_units = [H.i32(U), H.i32(-1)]
        outs, pinned = [], []
        for i, (q, kc, vc, cu) in enumerate(chunks):
            a, b = i & 1, (i + 1) & 1
            if pipelined:
                o = torch.empty((T, w.h_q, w.d), dtype=torch.float32).pin_memory()
                pinned.append((q.pin_memory(), kc.pin_memory(), vc.pin_memory()))      # alive until host_wait
                ctx.chunk_step_host_pipelined(*pinned[-1], T, cu, len(cu), caches[a][0], caches[a][1],
                                              n_hist[a], s_cap - T, units[a], n_units[a], u_cap - len(cu), w.w_modality, params,
                                              w.page_size, 0.0, caches[b][0], caches[b][1], units[b], n_hist[b], n_units[b], o,
                                              ob.DTYPE_FP32)
            else:
                o = torch.empty((T, w.h_q, w.d), dtype=torch.float32, device="cuda")
                ctx.chunk_step(q.cuda(), kc.cuda(), vc.cuda(), T, torch.from_numpy(cu).cuda(), len(cu), caches[a][0], caches[a][1],
                               n_hist[a], s_cap - T, units[a], n_units[a], u_cap - len(cu), w.w_modality, params, w.page_size, 0.0,
                               caches[b][0], caches[b][1], units[b], n_hist[b], n_units[b], o, ob.DTYPE_FP32)
                torch.cuda.synchronize()
            outs.append(o)
        if pipelined:
            ctx.host_wait()
        torch.cuda.synchronize()
        assert ctx.poll_status() == 0
        last = n_steps & 1
        nh = int(n_hist[last].item())
        res = ([o.cpu().numpy().copy() for o in outs], nh, H.bytes_of(caches[last][0][:nh]).copy(), H.bytes_of(caches[last][1][:nh]).copy(),
               units[last].cpu().numpy().copy(), int(n_units[last].item()))
        ctx.close()
        return res

    ref, got = run(False), run(True)
    assert got[1] == ref[1] and got[5] == ref[5]
    for i in range(n_steps):
        assert np.array_equal(got[0][i], ref[0][i]), f"output of chunk {i}"
    assert np.array_equal(got[2], ref[2]) and np.array_equal(got[3], ref[3]) and np.array_equal(got[4][:got[5]], ref[4][:ref[5]])


def test_chunk_step_config2(H, ob, cfg2):
    res = _run_step(H, ob, cfg2)
    _check_step(H, ob, cfg2, res)
    assert res["info"]["n_kept"] <= cfg2.budget


def test_budget_covers_history_is_full_attention(H, ob):
    """No eviction when the budget covers the cache: output equals dense causal attention."""
    w = wl.small_mixed(21, d=128, n_units=8, max_len=300, t=260)
    w.budget = w.n_hist
    res = _run_step(H, ob, w)
    assert res["info"]["rows_moved"] == 0 and res["info"]["n_kept"] == w.n_hist
    o_ref, _ = oc.chunk_attention(w.q, w.k_hist, w.v_hist, w.k_chunk, w.v_chunk)
    _check_attention(res["o"], None, o_ref, None)


# ------------------------------------------------------- structural (score-free) retention plan
def test_plan_structural_exact(H, ob):
    """omnitide_plan_structural equals the oracle's plan on random streams: codes, kept lengths, mask, table."""
    from tests.test_oracle_pins import _random_stream, _toy_stream
    rng = np.random.default_rng(616)
    ctx = ob.Context(4, 1, 64, "fp32", 4096, 64, 16)
    cases = [(_toy_stream(), 40, 45, 2, (2, 1, 0), 4), (_toy_stream(), 40, 30, 2, (2, 1, 0), 4),
             (_toy_stream(), 74, 10, 1, (0, 0, 0), 0), (_toy_stream(), 40, 5, 2, (2, 1, 0), 4)]
    for _ in range(120):
        u = _random_stream(rng, int(rng.integers(1, 10)), with_prefix=rng.random() < 0.8)
        n = int(u[:, 1].sum())
        Hw = int(rng.integers(0, n + 10))
        cases.append((u, Hw, int(rng.integers(0, Hw + 1)), int(rng.integers(0, 4)),
                      (int(rng.integers(0, 12)), int(rng.integers(0, 12)), 0), int(rng.integers(0, 60))))
    for i, (u, Hw, Lw, R, sink, Tb) in enumerate(cases):
        exp = oc.plan_structural(u, Hw, Lw, R, sink, Tb)
        got = H.gpu_plan_structural(ctx, u, Hw, Lw, R, sink, Tb, use_dev_count=(i % 2 == 0))
        assert got["status"] == 0
        assert np.array_equal(got["unit_keep"], exp["unit_keep"]), i
        assert np.array_equal(got["unit_kept_len"], exp["unit_kept_len"]), i
        assert np.array_equal(got["keep_mask"], exp["keep_mask"]), i
        assert got["n_kept"] == exp["n_kept"] and np.array_equal(got["units_out"], exp["units_out"]), i
    # a malformed table is flagged and yields an empty plan
    bad = _toy_stream()
    bad[3, 0] += 1
    got = H.gpu_plan_structural(ctx, bad, 0, 0, 1, (1, 1, 0), 0)
    assert got["status"] & 2 and got["n_kept"] == 0
    ctx.close()


def test_structural_plan_then_compaction_bit_exact(H, ob):
    """The plan's sink prefixes through the unit-granular compaction equal the oracle's pack of the plan's mask."""
    rng = np.random.default_rng(717)
    w = wl.layer_8b(n_hist=6000, budget=2000)
    u = w.units
    n = w.n_hist
    exp_plan = oc.plan_structural(u, 3000, 2500, 2, (24, 8, 0), 64)
    assert (exp_plan["unit_keep"] == 1).any(), "the case must contain sink prefixes"
    ctx = H.make_ctx(w)
    plan = H.gpu_plan_structural(ctx, u, 3000, 2500, 2, (24, 8, 0), 64)
    assert np.array_equal(plan["unit_kept_len"], exp_plan["unit_kept_len"])
    k, v = ob.to_device(w.k_hist, w.dtype), ob.to_device(w.v_hist, w.dtype)
    raw_k, raw_v = H.bytes_of(k).reshape(n, -1), H.bytes_of(v).reshape(n, -1)
    exp = oc.compact_pack(raw_k, raw_v, exp_plan["keep_mask"], w.page_size, exp_plan["units_out"])
    got = H.gpu_compact_units(ctx, k, v, u, plan["unit_keep"], w.page_size, units_out_np=plan["units_out"],
                              kept_len_np=plan["unit_kept_len"])
    m = exp["n_kept"]
    assert (got["n_kept"], got["span_pages"], got["rows_moved"]) == (m, exp["span_pages"], exp["rows_moved"])
    assert got["part_begin"] == exp["part_begin"].tolist()
    assert np.array_equal(got["slot_map"], exp["slot_map"])
    assert np.array_equal(H.bytes_of(got["k"][:m]).reshape(m, -1), exp["k"])
    assert np.array_equal(H.bytes_of(got["v"][:m]).reshape(m, -1), exp["v"])
    ctx.close()


# ------------------------------------------------------------- RoPE re-index fused into the pack
@pytest.mark.parametrize("n_dims,base", [(128, 10000.0), (64, 1000000.0)])
def test_compact_units_rope(H, ob, n_dims, base):
    """Keys re-rotated to their new positions while they are packed: within one bf16 step of the float64 oracle on
    every element and bit-identical on all but a sliver (fp32 rotation vs float64); V rows and integers exact."""
    rng = np.random.default_rng(919)
    w = wl.layer_8b(n_hist=9000, budget=3000)
    u, n = w.units, w.n_hist
    keep_u = np.where(rng.random(len(u)) < 0.4, 2, 0).astype(np.uint8)
    keep_u[0] = 2
    mask = np.repeat(keep_u != 0, u[:, 1]).astype(np.uint8)
    ctx = H.make_ctx(w)
    k, v = ob.to_device(w.k_hist, "bf16"), ob.to_device(w.v_hist, "bf16")
    kd, vd = torch.zeros_like(k), torch.zeros_like(v)
    du = ob.units_to_device(u)
    keep = torch.from_numpy(keep_u).cuda()
    info = torch.zeros((8,), dtype=torch.int32, device="cuda")
    ctx.compact_units_rope(k, v, kd, vd, du, H.i32(len(u)), len(u), keep, n, w.page_size, None, None, None, info, None, base,
                           n_dims)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    k_ref, v_ref, delta = oc.compact_pack_rope(w.k_hist, w.v_hist, mask, base, n_dims)
    m = len(delta)
    assert ob.info_to_dict(info)["n_kept"] == m and (delta < 0).any()
    assert np.array_equal(H.bytes_of(vd[:m]).reshape(m, -1), H.bytes_of(v[torch.from_numpy(np.nonzero(mask)[0]).cuda()]).reshape(m, -1))
    got = kd[:m].float().cpu().numpy().astype(np.float64)
    ref16 = wl.round_to_bf16(k_ref.astype(np.float32)).astype(np.float64)
    # one bf16 step at the value's binade, plus the fp32 rounding of the two products when they cancel
    # (x cos - y sin near zero: absolute error up to about 2^-22 of the operands, whatever the result's size)
    step = np.abs(ref16) * 2.0 ** -7 + np.abs(w.k_hist).max() * 2.0 ** -21
    assert (np.abs(got - ref16) <= step).all()
    assert (got != ref16).mean() < 2e-3, (got != ref16).mean()
    # rows that do not move (the leading kept run) are copied bit for bit
    lead = int(np.argmin(mask)) if not mask.all() else m
    assert np.array_equal(H.bytes_of(kd[:lead]), H.bytes_of(k[:lead]))
    ctx.close()


def test_chunk_step_with_observation_window(H, ob, cfg2):
    """OMNI_OPT_SCORE_WINDOW: the pass scores with the last W queries only; the scores equal the oracle's on
    that row range and the selection follows the oracle's rule on them."""
    w = cfg2
    W = 128
    N, T, U = w.n_hist, w.t, len(w.units)
    ctx = ob.Context(w.h_q, w.h_kv, w.d, w.dtype, N + T + 64, U + 8, T)
    ctx.set_option(ob.OPT_SCORE_WINDOW, W)
    kc_in = torch.zeros((N + T + 64, w.h_kv, w.d), dtype=torch.bfloat16, device="cuda")
    vc_in = torch.zeros_like(kc_in)
    kc_in[:N], vc_in[:N] = ob.to_device(w.k_hist, "bf16"), ob.to_device(w.v_hist, "bf16")
    kc_out, vc_out = torch.zeros_like(kc_in), torch.zeros_like(vc_in)
    units_out = torch.zeros((U + 8, 6), dtype=torch.int32, device="cuda")
    n_hist_out, n_units_out = H.i32(-1), H.i32(-1)
    o = torch.zeros((T, w.h_q, w.d), dtype=torch.float32, device="cuda")
    q = ob.to_device(w.q, "bf16")
    ctx.chunk_step(q, ob.to_device(w.k_chunk, "bf16"), ob.to_device(w.v_chunk, "bf16"), T, ob.units_to_device(w.chunk_units),
                   len(w.chunk_units), kc_in, vc_in, H.i32(N), N, ob.units_to_device(w.units, U + 8), H.i32(U), U,
                   w.w_modality, ob.select_params(w.budget, w.n_recent_events, w.modality_cap), w.page_size, 0.0, kc_out,
                   vc_out, units_out, n_hist_out, n_units_out, o, ob.DTYPE_FP32)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    # the scores of the window, through the scoring entry point on the same row range, against the oracle
    win = dataclasses_replace_q(w, W)
    s_gpu, m_gpu = H.gpu_score(ctx, win)
    s_ref, m_ref = oc.score_units(win.q, w.k_hist, w.units, w.w_modality)
    _check_scores(s_gpu, m_gpu, s_ref, m_ref)
    sel = oc.select_units(w.units, s_gpu, w.budget, w.n_recent_events, w.modality_cap)
    nu = int(n_units_out.item()) - len(w.chunk_units)
    assert np.array_equal(units_out[:nu].cpu().numpy(), sel["units_out"])
    assert int(n_hist_out.item()) == sel["n_kept"] + T
    # and the window changes the decision input: scores of all queries differ from scores of the window
    s_all, _ = oc.score_units(w.q, w.k_hist, w.units, w.w_modality)
    assert np.abs(s_all - s_ref).max() > 1e-3
    ctx.close()


@pytest.mark.parametrize("above", [False, True])
def test_chunk_step_with_high_watermark(H, ob, cfg2, above):
    """OMNI_OPT_HIGH_WATERMARK: a call whose history bound is at most the watermark keeps the whole history (the
    selection rule with a budget that covers everything, Section 5.1 hysteresis) and launches no scoring kernel;
    above it the pass is the ordinary one."""
    w = cfg2
    N, T, U = w.n_hist, w.t, len(w.units)
    ctx = ob.Context(w.h_q, w.h_kv, w.d, w.dtype, N + T + 64, U + 8, T)
    kc_in = torch.zeros((N + T + 64, w.h_kv, w.d), dtype=torch.bfloat16, device="cuda")
    vc_in = torch.zeros_like(kc_in)
    kc_in[:N], vc_in[:N] = ob.to_device(w.k_hist, "bf16"), ob.to_device(w.v_hist, "bf16")
    kc_out, vc_out = torch.zeros_like(kc_in), torch.zeros_like(vc_in)
    units_out = torch.zeros((U + 8, 6), dtype=torch.int32, device="cuda")
    n_hist_out, n_units_out = H.i32(-1), H.i32(-1)
    o = torch.zeros((T, w.h_q, w.d), dtype=torch.float32, device="cuda")
    def step():
        before = ctx.launch_count()
        ctx.chunk_step(ob.to_device(w.q, "bf16"), ob.to_device(w.k_chunk, "bf16"), ob.to_device(w.v_chunk, "bf16"), T,
                       ob.units_to_device(w.chunk_units), len(w.chunk_units), kc_in, vc_in, H.i32(N), N,
                       ob.units_to_device(w.units, U + 8), H.i32(U), U, w.w_modality,
                       ob.select_params(w.budget, w.n_recent_events, w.modality_cap), w.page_size, 0.0, kc_out, vc_out,
                       units_out, n_hist_out, n_units_out, o, ob.DTYPE_FP32)
        torch.cuda.synchronize()
        assert ctx.poll_status() == 0
        return ctx.launch_count() - before
    ctx.set_option(ob.OPT_HIGH_WATERMARK, 0)
    launches_full = step()
    ctx.set_option(ob.OPT_HIGH_WATERMARK, N - 1 if above else N)
    launches = step()
    if above:
        s_gpu, _ = H.gpu_score(ctx, w)
        sel = oc.select_units(w.units, s_gpu, w.budget, w.n_recent_events, w.modality_cap)
        assert sel["n_kept"] < N
    else:
        sel = oc.select_units(w.units, np.zeros(U, np.float32), N, w.n_recent_events, (-1, -1, -1))
        assert sel["n_kept"] == N                                   # a budget that covers the history keeps all of it
        assert launches < launches_full                             # no scoring kernels
    nk = sel["n_kept"]
    nu = int(n_units_out.item()) - len(w.chunk_units)
    assert np.array_equal(units_out[:nu].cpu().numpy(), sel["units_out"])
    assert int(n_hist_out.item()) == nk + T
    exp = oc.compact_pack(H.bytes_of(kc_in[:N]).reshape(N, -1), H.bytes_of(vc_in[:N]).reshape(N, -1), sel["keep_mask"], w.page_size)
    assert np.array_equal(H.bytes_of(kc_out[:nk]).reshape(nk, -1), exp["k"][:nk])
    assert np.array_equal(H.bytes_of(vc_out[:nk]).reshape(nk, -1), exp["v"][:nk])
    keep = sel["keep_mask"].astype(bool)
    o_ref, _ = oc.chunk_attention(w.q, w.k_hist[keep], w.v_hist[keep], w.k_chunk, w.v_chunk)
    _check_attention(o.cpu().numpy(), None, o_ref, None)
    ctx.close()


def dataclasses_replace_q(w, W):
    import dataclasses
    return dataclasses.replace(w, q=np.ascontiguousarray(w.q[-W:]))


# ------------------------------------------------------------------ attention over a history with holes
@pytest.mark.parametrize("t,n_hist,h_q,h_kv,pattern", [
    (128, 1000, 8, 2, "random50"),      # holes in every block
    (200, 3000, 8, 2, "blocks"),        # whole blocks dead (skipped), others partly live
    (77, 517, 4, 1, "random10"),        # sparse, ragged tail
    (64, 2048, 4, 2, "all_dead"),       # the history contributes nothing
    (64, 1300, 4, 2, "all_live"),       # equals the dense call
    (1, 4000, 32, 8, "random50"),       # decode over holes (GQA-packed tile)
    (690, 16384, 32, 8, "sinks"),       # config-2 sizes: kept units whole, others reduced to short prefixes
])
def test_attention_masked_tensor_core(H, ob, t, n_hist, h_q, h_kv, pattern):
    rng = np.random.default_rng(t + n_hist)
    units = wl.make_units([(n_hist, 0, 0)], group_of_first=None)
    chunk_units = wl.make_units([(t, 0, 1)], group_of_first=None)
    q, kh, vh, kc, vc = wl.random_layer_inputs(rng, units, chunk_units, h_q, h_kv, 128, "bf16")
    if pattern.startswith("random"):
        keep = (rng.random(n_hist) < int(pattern[6:]) / 100.0).astype(np.uint8)
    elif pattern == "blocks":
        keep = np.repeat((rng.random((n_hist + 127) // 128) < 0.5), 128)[:n_hist].astype(np.uint8)
        keep &= (rng.random(n_hist) < 0.8).astype(np.uint8)
        keep[128:256] = 0
    elif pattern == "all_dead":
        keep = np.zeros(n_hist, np.uint8)
    elif pattern == "all_live":
        keep = np.ones(n_hist, np.uint8)
    else:                                                    # 'sinks'
        keep = np.zeros(n_hist, np.uint8)
        for s0 in range(0, n_hist, 690):
            keep[s0:s0 + (690 if rng.random() < 0.2 else 24)] = 1
    w = wl.Workload("m", h_q, h_kv, 128, "bf16", units, chunk_units, 1, 64, 1, q=q, k_hist=kh, v_hist=vh, k_chunk=kc, v_chunk=vc)
    ctx = ob.Context(h_q, h_kv, 128, "bf16", n_hist + 300, 8, t)
    pad = 200
    khd = torch.full((n_hist + pad, h_kv, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    vhd = torch.full((n_hist + pad, h_kv, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    khd[:n_hist], vhd[:n_hist] = ob.to_device(kh, "bf16"), ob.to_device(vh, "bf16")
    mask = torch.full((n_hist + pad + 16,), 1, dtype=torch.uint8, device="cuda")        # stale ones beyond the span
    mask[:n_hist] = torch.from_numpy(keep).cuda()
    o = torch.full((t, h_q, 128), float("nan"), dtype=torch.float32, device="cuda")
    lse = torch.full((t, h_q), float("nan"), dtype=torch.float32, device="cuda")
    ctx.chunk_attention_masked(ob.to_device(q, "bf16"), t, khd, vhd, mask, H.i32(n_hist), n_hist + pad, ob.to_device(kc, "bf16"),
                               ob.to_device(vc, "bf16"), 0.0, o, ob.DTYPE_FP32, lse)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    o_ref, lse_ref = oc.chunk_attention_masked(q, kh, vh, keep, kc, vc)
    _check_attention(o.cpu().numpy(), lse.cpu().numpy(), o_ref, lse_ref)
    if pattern == "all_live":
        o2, _ = H.gpu_attention(ctx, w, khd, vhd, n_hist, n_hist_max=n_hist + pad)
        assert np.array_equal(o2, o.cpu().numpy())
    ctx.close()


def test_attention_masked_cuda_cores(H, ob):
    w = wl.tiny()
    rng = np.random.default_rng(77)
    keep = (rng.random(w.n_hist) < 0.4).astype(np.uint8)
    ctx = H.make_ctx(w)
    mask = torch.zeros((w.n_hist + 16,), dtype=torch.uint8, device="cuda")
    mask[:w.n_hist] = torch.from_numpy(keep).cuda()
    o = torch.zeros((w.t, w.h_q, w.d), dtype=torch.float32, device="cuda")
    ctx.chunk_attention_masked(ob.to_device(w.q, "fp32"), w.t, ob.to_device(w.k_hist, "fp32"), ob.to_device(w.v_hist, "fp32"), mask,
                               None, w.n_hist, ob.to_device(w.k_chunk, "fp32"), ob.to_device(w.v_chunk, "fp32"), 0.0, o,
                               ob.DTYPE_FP32)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    o_ref, _ = oc.chunk_attention_masked(w.q, w.k_hist, w.v_hist, keep, w.k_chunk, w.v_chunk)
    _check_attention(o.cpu().numpy(), None, o_ref, None)
    ctx.close()


# ------------------------------------------------------------------ ordered-suffix migration
@pytest.mark.parametrize("S,page,theta,pattern,seed", [
    (1000, 16, 1, "tail_sparse", 0),
    (5000, 64, 2, "tail_sparse", 1),
    (16384, 64, 4, "sinks", 2),
    (3000, 256, 1, "random", 3),
    (2048, 64, 1, "dense", 4),          # nothing qualifies: nothing moves
    (2043, 16, 3, "dense", 7),          # the same with a span that is not a multiple of 16
    (777, 64, 40, "random", 8),         # a threshold no suffix can meet
    (80000, 64, 8, "sinks", 5),
    (777, 16, 3, "random", 6),
])
def test_migrate_suffix_bit_exact(H, ob, S, page, theta, pattern, seed):
    """omnipage_migrate_suffix equals the oracle: chosen suffix, new mask and span, slot map, and every row of the
    cache up to the new span, bit for bit; then attention over the migrated layout is unchanged."""
    rng = np.random.default_rng(300 + seed)
    if pattern == "tail_sparse":
        keep = np.ones(S, np.uint8)
        keep[S // 2:] = (rng.random(S - S // 2) < 0.3).astype(np.uint8)
    elif pattern == "sinks":
        keep = np.zeros(S, np.uint8)
        for s0 in range(0, S, 690):
            keep[s0:s0 + (690 if rng.random() < 0.3 else 24)] = 1
        keep[:16] = 1
    elif pattern == "random":
        keep = (rng.random(S) < 0.5).astype(np.uint8)
    else:
        keep = np.ones(S, np.uint8)
    rowshape = (2, 128)
    raw = rng.integers(0, 256, size=(2, S, rowshape[0] * rowshape[1] * 2), dtype=np.uint8)
    k = torch.from_numpy(raw[0]).cuda().view(torch.bfloat16).view(S, *rowshape).contiguous()
    v = torch.from_numpy(raw[1]).cuda().view(torch.bfloat16).view(S, *rowshape).contiguous()
    exp = oc.migrate_suffix(raw[0], raw[1], keep, page, theta)
    ctx = ob.Context(8, 2, 128, "bf16", S + 64, 8, 16)
    mask = torch.zeros((S + 48,), dtype=torch.uint8, device="cuda")
    mask[:S] = torch.from_numpy(keep).cuda()
    mask[S:S + 40] = 1                                        # stale bytes beyond the span
    span = H.i32(S)
    slot_map = torch.full((S + 48,), -5, dtype=torch.int32, device="cuda")
    info = torch.full((8,), -5, dtype=torch.int32, device="cuda")
    ctx.migrate_suffix(k, v, mask, span, S + 40, page, theta, slot_map, info)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    got = ob.info_to_dict(info)
    ns = exp["new_span"]
    assert got["part_begin"] == [exp["start"], ns, exp["pages_saved"], S]
    assert got["n_kept"] == int(keep.sum()) and got["rows_moved"] == exp["rows_moved"] and int(span.item()) == ns
    assert np.array_equal(mask[:S].cpu().numpy(), exp["keep_mask"])
    assert np.array_equal(slot_map[:S].cpu().numpy(), exp["slot_map"])
    assert np.array_equal(H.bytes_of(k[:ns]).reshape(ns, -1), exp["k"][:ns])
    assert np.array_equal(H.bytes_of(v[:ns]).reshape(ns, -1), exp["v"][:ns])
    if pattern == "dense" or theta >= 40:
        assert exp["start"] == -1 and got["rows_moved"] == 0
    else:
        assert exp["start"] >= 0
    ctx.close()


# ------------------------------------------------------------------ class-aware selective migration
def _class_case(rng, S, page, pattern):
    """A layout after a structural retention round: a must-keep head, older units reduced to short marked prefixes
    (selected-history), unmarked survivors, recent units whole (recent-context)."""
    keep = np.zeros(S, np.uint8)
    cls = np.zeros(S, np.uint8)
    head = min(S // 8, 3 * page + 5)
    keep[:head] = 1                                              # must-keep, class 0
    recent0 = S - S // 6
    pos = head
    while pos < recent0:
        n = int(rng.integers(40, 700))
        end = min(recent0, pos + n)
        r = rng.random()
        if pattern == "random":
            m = rng.random(end - pos) < 0.3
            keep[pos:end] = m
            cls[pos:end] = np.where(m, rng.choice([1, 2]) | np.where(rng.random(end - pos) < 0.7, 0x80, 0), 0)
        elif r < 0.65:                                           # sink prefix of a partially evicted unit
            pre = min(end - pos, int(rng.choice([4, 8, 24])))
            keep[pos:pos + pre] = 1
            cls[pos:pos + pre] = 1 | 0x80
        elif r < 0.8:                                            # kept whole: not a candidate
            keep[pos:end] = 1
            cls[pos:end] = 1
        pos = end
    keep[recent0:] = 1
    cls[recent0:] = 2
    if pattern == "no_holes":
        keep[:] = 1
        cls[head:recent0] = 1 | 0x80
    return keep, np.where(keep == 1, cls, 0).astype(np.uint8)


@pytest.mark.parametrize("S,page,sub,pattern,promote,seed", [
    (1000, 16, 8, "random", 1, 0),
    (5000, 64, 32, "sinks", 1, 1),
    (16384, 64, 32, "random", 1, 2),
    (3000, 256, 64, "sinks", 0, 3),
    (2048, 64, 64, "no_holes", 1, 4),      # no empty slot anywhere: no plan
    (80000, 64, 32, "sinks", 1, 5),
    (80000, 16, 16, "random", 1, 6),
    (777, 16, 2, "random", 1, 7),
    (37, 16, 4, "random", 1, 8),
])
def test_migrate_class_bit_exact(H, ob, S, page, sub, pattern, promote, seed):
    """omnipage_migrate_class equals the oracle: the plan move by move, the accept decision and its four counts, the new
    mask, classes and page labels, and every live row of the cache, bit for bit."""
    rng = np.random.default_rng(500 + seed)
    keep, cls = _class_case(rng, S, page, pattern)
    rowshape = (2, 128)
    raw = rng.integers(0, 256, size=(2, S, rowshape[0] * rowshape[1] * 2), dtype=np.uint8)
    k = torch.from_numpy(raw[0]).cuda().view(torch.bfloat16).view(S, *rowshape).contiguous()
    v = torch.from_numpy(raw[1]).cuda().view(torch.bfloat16).view(S, *rowshape).contiguous()
    exp = oc.migrate_class(raw[0], raw[1], keep, cls, page, sub, promote=bool(promote))
    ctx = ob.Context(8, 2, 128, "bf16", S + 64, 8, 16)
    mask = torch.zeros((S + 48,), dtype=torch.uint8, device="cuda")
    mask[:S] = torch.from_numpy(keep).cuda()
    mask[S:S + 40] = 1                                        # stale bytes beyond the span
    sc = torch.zeros((S + 48,), dtype=torch.uint8, device="cuda")
    sc[:S] = torch.from_numpy(cls).cuda()
    n_pages = -(-S // page)
    moves = torch.full((2 * (S + 48),), -5, dtype=torch.int32, device="cuda")
    labels = torch.full((n_pages + 4,), 77, dtype=torch.uint8, device="cuda")
    info = torch.full((8,), -5, dtype=torch.int32, device="cuda")
    ctx.migrate_class(k, v, mask, sc, H.i32(S), S + 40, page, sub, promote, moves, labels, info)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    acc, n_moves, n_cand, pb, pa, sb, sa, _ = info.cpu().tolist()
    assert bool(acc) == exp["accepted"] and n_moves == len(exp["moves"]) and n_cand == exp["n_candidates"]
    assert (pb, pa, sb, sa) == (exp["pages_before"], exp["pages_after"], exp["subblocks_before"], exp["subblocks_after"])
    if exp["accepted"]:
        assert moves[:2 * n_moves].cpu().numpy().reshape(-1, 2).tolist() == [list(m) for m in exp["moves"]]
    new_mask = mask[:S].cpu().numpy()
    assert np.array_equal(new_mask, exp["keep_mask"]) and bool((mask[S:S + 40] == 1).all())
    live = new_mask == 1
    assert np.array_equal(sc[:S].cpu().numpy()[live], exp["slot_class"][live])
    vacated = (keep == 1) & ~live
    assert not sc[:S].cpu().numpy()[vacated].any()
    assert np.array_equal(labels[:n_pages].cpu().numpy(), exp["page_class"]) and bool((labels[n_pages:] == 77).all())
    assert np.array_equal(H.bytes_of(k).reshape(S, -1)[live], exp["k"][live])
    assert np.array_equal(H.bytes_of(v).reshape(S, -1)[live], exp["v"][live])
    if pattern == "no_holes":
        assert not exp["accepted"] and n_moves == 0
    elif S >= 777:
        assert exp["accepted"] and n_moves > 0          # the cases are meant to exercise the move path
    ctx.close()


def test_migrate_class_argument_and_device_errors(H, ob):
    """Host-side refusals (null pointers, a subblock that does not divide the page, a span above the capacity) and the
    device-side one (a class value outside 0..2 sets OMNI_DEV_BAD_UNITS and moves nothing)."""
    S = 512
    ctx = ob.Context(8, 2, 128, "bf16", S + 64, 8, 16)
    k = torch.zeros((S, 2, 128), dtype=torch.bfloat16, device="cuda")
    v = torch.zeros_like(k)
    mask = torch.ones(S + 16, dtype=torch.uint8, device="cuda")
    mask[10:200] = 0
    mask[230:256] = 0                                      # 30 entries left in page 3: moving them to page 0 empties it
    cls = torch.full((S + 16,), 1 | 0x80, dtype=torch.uint8, device="cuda")
    info = torch.full((8,), -5, dtype=torch.int32, device="cuda")
    with pytest.raises(ob.OmniTideError):
        ctx.migrate_class(k, v, None, cls, None, S, 64, 32, 1, None, None, info)
    with pytest.raises(ob.OmniTideError):
        ctx.migrate_class(k, v, mask, cls, None, S, 64, 48, 1, None, None, info)        # 48 does not divide 64
    with pytest.raises(ob.OmniTideError):
        ctx.migrate_class(k, v, mask, cls, None, S + 4096, 64, 32, 1, None, None, info)  # above s_cap
    with pytest.raises(ob.OmniTideError):
        ctx.migrate_class(k, v, mask, cls, None, S, 64, 32, 1, None, None, None)        # the outcome has to go somewhere
    assert int(info[0].item()) == -5                       # nothing was launched
    cls[300] = 3
    before = mask.clone()
    ctx.migrate_class(k, v, mask, cls, None, S, 64, 32, 1, None, None, info)
    torch.cuda.synchronize()
    assert ctx.poll_status() & ob.DEV_BAD_UNITS
    assert info.cpu().tolist() == [0] * 8 and torch.equal(mask, before)
    # a device span above the host bound is refused on the device
    cls[300] = 1
    ctx.migrate_class(k, v, mask, cls, H.i32(S + 1), S, 64, 32, 1, None, None, info)
    torch.cuda.synchronize()
    assert ctx.poll_status() & ob.DEV_BAD_COUNT and torch.equal(mask, before)
    # and the same call with a valid span works afterwards: the context is still usable
    ctx.migrate_class(k, v, mask, cls, H.i32(S), S, 64, 32, 1, None, None, info)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0 and info.cpu().tolist()[:2] == [1, 30] and not bool(mask[192:256].any())
    ctx.close()


def test_migrate_class_then_attention(H, ob, cfg2):
    """Attention over the class-migrated layout equals attention over the layout with its original holes: the migration
    changes where entries are stored, not the history (Section 6.2)."""
    w = cfg2
    N, T = w.n_hist, w.t
    plan = oc.plan_structural(w.units, 0, 6000, 2, (24, 8, 0), 64)
    keep = plan["keep_mask"]
    kept_len = plan["unit_kept_len"]
    cls = np.zeros(N, np.uint8)
    for u, (st, ln) in enumerate(zip(w.units[:, oc.U_START].tolist(), w.units[:, oc.U_LEN].tolist())):
        part = 0 < kept_len[u] < ln
        cls[st:st + ln] = (1 | 0x80) if part else 2
    cls = np.where(keep == 1, cls, 0).astype(np.uint8)
    o_ref, _ = oc.chunk_attention_masked(w.q, w.k_hist, w.v_hist, keep, w.k_chunk, w.v_chunk)
    exp = oc.migrate_class(None, None, keep, cls, w.page_size, w.page_size // 2)
    ctx = H.make_ctx(w)
    q, kc, vc = (ob.to_device(a, "bf16") for a in (w.q, w.k_chunk, w.v_chunk))
    k, v = ob.to_device(w.k_hist, "bf16").clone(), ob.to_device(w.v_hist, "bf16").clone()
    mask = torch.zeros((N + 16,), dtype=torch.uint8, device="cuda")
    mask[:N] = torch.from_numpy(keep).cuda()
    sc = torch.from_numpy(cls).cuda()
    info = torch.zeros((8,), dtype=torch.int32, device="cuda")
    ctx.migrate_class(k, v, mask, sc, None, N, w.page_size, w.page_size // 2, 1, None, None, info)
    o = torch.zeros((T, w.h_q, w.d), dtype=torch.float32, device="cuda")
    ctx.chunk_attention_masked(q, T, k, v, mask, H.i32(N), N, kc, vc, 0.0, o, ob.DTYPE_FP32)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    got = info.cpu().tolist()
    assert bool(got[0]) == exp["accepted"] and got[1] == len(exp["moves"]) and got[4] == exp["pages_after"]
    assert np.array_equal(mask[:N].cpu().numpy(), exp["keep_mask"])
    _check_attention(o.cpu().numpy(), None, o_ref, None)
    ctx.close()


def test_native_suffix_eager_layouts_attend_alike(H, ob, cfg2):
    """The three layouts of the paper's ablation (native holes, ordered-suffix migration, eager pack) present the same
    live rows: attention over each of them matches the oracle, and the spans shrink in that order."""
    w = cfg2
    rng = np.random.default_rng(31)
    N, T = w.n_hist, w.t
    plan = oc.plan_structural(w.units, 0, 6000, 2, (24, 8, 0), 64)
    keep = plan["keep_mask"]
    o_ref, _ = oc.chunk_attention_masked(w.q, w.k_hist, w.v_hist, keep, w.k_chunk, w.v_chunk)
    ctx = H.make_ctx(w)
    q, kc, vc = (ob.to_device(a, "bf16") for a in (w.q, w.k_chunk, w.v_chunk))
    k, v = ob.to_device(w.k_hist, "bf16").clone(), ob.to_device(w.v_hist, "bf16").clone()
    mask = torch.zeros((N + 16,), dtype=torch.uint8, device="cuda")
    mask[:N] = torch.from_numpy(keep).cuda()
    span = H.i32(N)
    o = torch.zeros((T, w.h_q, w.d), dtype=torch.float32, device="cuda")
    # native: holes left in place
    ctx.chunk_attention_masked(q, T, k, v, mask, span, N, kc, vc, 0.0, o, ob.DTYPE_FP32)
    torch.cuda.synchronize()
    _check_attention(o.cpu().numpy(), None, o_ref, None)
    # ordered suffix
    info = torch.zeros((8,), dtype=torch.int32, device="cuda")
    ctx.migrate_suffix(k, v, mask, span, N, w.page_size, 4, None, info)
    ctx.chunk_attention_masked(q, T, k, v, mask, span, N, kc, vc, 0.0, o, ob.DTYPE_FP32)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    _check_attention(o.cpu().numpy(), None, o_ref, None)
    span_suffix = int(span.item())
    # eager
    got = H.gpu_compact(ctx, ob.to_device(w.k_hist, "bf16"), ob.to_device(w.v_hist, "bf16"), keep, w.page_size)
    o3, _ = H.gpu_attention(ctx, w, got["k"], got["v"], got["n_kept"], n_hist_max=N, want_lse=False)
    _check_attention(o3, None, o_ref, None)
    assert got["n_kept"] <= span_suffix < N
    ctx.close()


@pytest.mark.parametrize("h_q,h_kv", [(32, 8), (8, 1), (64, 8), (8, 8), (4, 2)])
def test_decode_attention_many_lengths(H, ob, h_q, h_kv):
    """One token against histories of many lengths (every alignment of the split and batch boundaries), for group
    sizes 1, 2, 4 and 8, through the split-KV decode kernel; fp32 and bf16 outputs, log-sum-exp."""
    rng = np.random.default_rng(h_q * 10 + h_kv)
    n_max = 2600
    units = wl.make_units([(n_max, 0, 0)], group_of_first=None)
    chunk_units = wl.make_units([(1, 0, 1)], group_of_first=None)
    q, kh, vh, kc, vc = wl.random_layer_inputs(rng, units, chunk_units, h_q, h_kv, 128, "bf16")
    ctx = ob.Context(h_q, h_kv, 128, "bf16", n_max + 64, 8, 4)
    khd, vhd = ob.to_device(kh, "bf16"), ob.to_device(vh, "bf16")
    qd, kcd, vcd = ob.to_device(q, "bf16"), ob.to_device(kc, "bf16"), ob.to_device(vc, "bf16")
    lengths = [0, 1, 2, 15, 16, 17, 63, 64, 65, 127, 128, 129, 500, 1023, 1024, 1025, 2048, 2599, 2600] + \
        [int(x) for x in rng.integers(1, n_max, size=12)]
    for n in lengths:
        o = torch.full((1, h_q, 128), float("nan"), dtype=torch.float32, device="cuda")
        lse = torch.full((1, h_q), float("nan"), dtype=torch.float32, device="cuda")
        ctx.chunk_attention(qd, 1, khd, vhd, H.i32(n), n_max, kcd, vcd, 0.0, o, ob.DTYPE_FP32, lse)
        torch.cuda.synchronize()
        assert ctx.poll_status() == 0
        o_ref, lse_ref = oc.chunk_attention(q, kh[:n], vh[:n], kc, vc)
        _check_attention(o.cpu().numpy(), lse.cpu().numpy(), o_ref, lse_ref)
    o16 = torch.zeros((1, h_q, 128), dtype=torch.bfloat16, device="cuda")
    ctx.chunk_attention(qd, 1, khd, vhd, H.i32(777), n_max, kcd, vcd, 0.0, o16, ob.DTYPE_BF16)
    ctx.chunk_attention(qd, 1, khd, vhd, H.i32(777), n_max, kcd, vcd, 0.0, o, ob.DTYPE_FP32)
    torch.cuda.synchronize()
    assert np.array_equal(o16.float().cpu().numpy(), wl.round_to_bf16(o.cpu().numpy()))
    ctx.close()


@pytest.mark.parametrize("h_q,h_kv", [(32, 8), (8, 1), (64, 8), (8, 8), (4, 2)])
def test_decode_attention_staged_long_histories(H, ob, h_q, h_kv):
    """The same against a long cache bound (the split count is at its maximum): actual lengths from empty to the bound,
    around the multiples of the split count and of the batch a warp takes per step."""
    rng = np.random.default_rng(h_q * 100 + h_kv)
    n_max = 21000
    units = wl.make_units([(n_max, 0, 0)], group_of_first=None)
    chunk_units = wl.make_units([(1, 0, 1)], group_of_first=None)
    q, kh, vh, kc, vc = wl.random_layer_inputs(rng, units, chunk_units, h_q, h_kv, 128, "bf16")
    ctx = ob.Context(h_q, h_kv, 128, "bf16", n_max + 64, 8, 4)
    khd, vhd = ob.to_device(kh, "bf16"), ob.to_device(vh, "bf16")
    qd, kcd, vcd = ob.to_device(q, "bf16"), ob.to_device(kc, "bf16"), ob.to_device(vc, "bf16")
    n_split = min(64, max(1, 148 // h_kv))
    lengths = [0, 1, 127, 128, 129, n_split - 1, n_split, n_split * 128 - 1, n_split * 128, n_split * 128 + 1, n_split * 384 - 1,
               n_split * 384, n_split * 384 + 1, 8191, 16384, n_max - 1, n_max] + [int(x) for x in rng.integers(1, n_max, size=10)]
    for n in lengths:
        n = min(n, n_max)
        o = torch.full((1, h_q, 128), float("nan"), dtype=torch.float32, device="cuda")
        lse = torch.full((1, h_q), float("nan"), dtype=torch.float32, device="cuda")
        ctx.chunk_attention(qd, 1, khd, vhd, H.i32(n), n_max, kcd, vcd, 0.0, o, ob.DTYPE_FP32, lse)
        torch.cuda.synchronize()
        assert ctx.poll_status() == 0
        o_ref, lse_ref = oc.chunk_attention(q, kh[:n], vh[:n], kc, vc)
        _check_attention(o.cpu().numpy(), lse.cpu().numpy(), o_ref, lse_ref)
    o16 = torch.zeros((1, h_q, 128), dtype=torch.bfloat16, device="cuda")
    ctx.chunk_attention(qd, 1, khd, vhd, H.i32(9999), n_max, kcd, vcd, 0.0, o16, ob.DTYPE_BF16)
    ctx.chunk_attention(qd, 1, khd, vhd, H.i32(9999), n_max, kcd, vcd, 0.0, o, ob.DTYPE_FP32)
    torch.cuda.synchronize()
    assert np.array_equal(o16.float().cpu().numpy(), wl.round_to_bf16(o.cpu().numpy()))
    ctx.close()


def test_shared_plan_over_layers_equals_per_layer_steps(H, ob, cfg2):
    """One structural plan and one batched compaction for the caches of two layers, then attention and append per layer
    (the paper's executor: one map shared by all layers, Section 6.2), against omnitide_chunk_step_structural run on each
    layer by itself: outputs, caches, unit table and counts bit for bit."""
    w = cfg2
    N, T, U = w.n_hist, w.t, len(w.units)
    s_cap, u_cap = N + T + 64, U + len(w.chunk_units) + 4
    sp = ob.structural_params(6000, 4000, 2, (24, 8, 0), 64)
    rng = np.random.default_rng(8)
    tdt = torch.bfloat16
    mk = lambda a: torch.from_numpy(wl.round_to_bf16(a + 0.5 * rng.standard_normal(a.shape).astype(np.float32))).to(tdt).cuda()
    layers = [dict(k=mk(w.k_hist), v=mk(w.v_hist), q=mk(w.q), kc=mk(w.k_chunk), vc=mk(w.v_chunk)) for _ in range(2)]
    cu = ob.units_to_device(w.chunk_units)

    def fresh_cache(L):
        k = torch.zeros((s_cap, w.h_kv, w.d), dtype=tdt, device="cuda")
        v = torch.zeros_like(k)
        k[:N], v[:N] = L["k"], L["v"]
        return k, v

    # ---- reference: the fused per-layer entry point
    ref = []
    ctx = ob.Context(w.h_q, w.h_kv, w.d, w.dtype, s_cap, u_cap, T)
    for L in layers:
        k_in, v_in = fresh_cache(L)
        k_out, v_out = torch.zeros_like(k_in), torch.zeros_like(v_in)
        units_out = torch.zeros((u_cap, 6), dtype=torch.int32, device="cuda")
        nh, nu = H.i32(-1), H.i32(-1)
        o = torch.zeros((T, w.h_q, w.d), dtype=torch.float32, device="cuda")
        ctx.chunk_step_structural(L["q"], L["kc"], L["vc"], T, cu, len(w.chunk_units), k_in, v_in, H.i32(N), N,
                                  ob.units_to_device(w.units, u_cap), H.i32(U), U, sp, w.page_size, 0.0, k_out, v_out, units_out,
                                  nh, nu, o, ob.DTYPE_FP32)
        torch.cuda.synchronize()
        ref.append(dict(o=o.cpu().numpy(), nh=int(nh.item()), nu=int(nu.item()), k=k_out, v=v_out, units=units_out.cpu().numpy()))
    assert ctx.poll_status() == 0 and ref[0]["nh"] < N + T                     # the plan evicts
    # ---- one plan, one batched compaction, then per layer attention + append
    ins = [fresh_cache(L) for L in layers]
    outs = [(torch.zeros_like(a), torch.zeros_like(b)) for a, b in ins]
    ptrs = lambda ts: torch.tensor([t_.data_ptr() for t_ in ts], dtype=torch.int64, device="cuda")
    units_in = ob.units_to_device(w.units, u_cap)
    keep = torch.zeros(u_cap + 16, dtype=torch.uint8, device="cuda")
    klen = torch.zeros(u_cap + 16, dtype=torch.int32, device="cuda")
    n_kept, n_uk = H.i32(-1), H.i32(-1)
    kept_units = torch.zeros((u_cap, 6), dtype=torch.int32, device="cuda")
    info = torch.zeros(8, dtype=torch.int32, device="cuda")
    ctx.plan_structural(units_in, H.i32(U), U, sp, keep, klen, None, N, n_kept, kept_units, n_uk)
    ctx.compact_units_batched(ptrs([a for a, _ in ins]), ptrs([b for _, b in ins]), ptrs([a for a, _ in outs]),
                              ptrs([b for _, b in outs]), 2, units_in, H.i32(U), U, keep, N, w.page_size, kept_units, n_uk, None,
                              info, None, unit_kept_len=klen)
    for i, L in enumerate(layers):
        o = torch.zeros((T, w.h_q, w.d), dtype=torch.float32, device="cuda")
        ctx.chunk_attention(L["q"], T, outs[i][0], outs[i][1], n_kept, N, L["kc"], L["vc"], 0.0, o, ob.DTYPE_FP32)
        table = kept_units.clone()
        nh, nu = H.i32(-1), H.i32(-1)
        ctx.append(outs[i][0], outs[i][1], n_kept, L["kc"], L["vc"], T, table, n_uk, cu, len(w.chunk_units), nh, nu)
        torch.cuda.synchronize()
        assert ctx.poll_status() == 0
        assert (int(nh.item()), int(nu.item())) == (ref[i]["nh"], ref[i]["nu"])
        assert np.array_equal(o.cpu().numpy(), ref[i]["o"])
        n_new = ref[i]["nh"]
        assert torch.equal(outs[i][0][:n_new], ref[i]["k"][:n_new]) and torch.equal(outs[i][1][:n_new], ref[i]["v"][:n_new])
        assert np.array_equal(table[:ref[i]["nu"]].cpu().numpy(), ref[i]["units"][:ref[i]["nu"]])
    ctx.close()
