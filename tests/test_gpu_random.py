"""Seeded random shapes through the C ABI against the oracle: sizes that are not multiples of anything, empty
inputs, every group size -- the cases nobody thought of writing down (one such run found an alignment fault in the
empty-suffix path of omnipage_migrate_suffix)."""
import numpy as np
import pytest

from oracle import omni_oracle as oc
from paper_2609_34653_b200 import workloads as wl

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ob():
    from paper_2609_34653_b200 import binding
    return binding


@pytest.fixture(scope="module")
def H():
    from tests import gpu_helpers
    return gpu_helpers


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_attention_shapes(H, ob, seed):
    rng = np.random.default_rng(seed)
    for _ in range(30):
        h_kv = int(rng.choice([1, 2, 4, 8]))
        h_q = min(32, h_kv * int(rng.choice([1, 2, 4, 8])))
        t = int(rng.choice([1, 3, 17, 64, 128, 129, 300, 511, 700]))
        n_hist = int(rng.choice([0, 1, 63, 128, 500, 1000, 2048, 3333, 6000]))
        masked = bool(rng.random() < 0.5) and n_hist > 0
        units = wl.make_units([(max(n_hist, 1), 0, 0)], group_of_first=None)
        chunk_units = wl.make_units([(t, 0, 1)], group_of_first=None)
        q, kh, vh, kc, vc = wl.random_layer_inputs(rng, units, chunk_units, h_q, h_kv, 128, "bf16")
        kh, vh = kh[:n_hist], vh[:n_hist]
        q = wl.round_to_bf16((q * float(rng.choice([1.0, 1.0, 3.0, 8.0]))).astype(np.float32))      # peaky rows too
        keep = (rng.random(n_hist) < rng.choice([0.1, 0.5, 0.9, 1.0])).astype(np.uint8)
        pad = int(rng.integers(0, 200))
        ctx = ob.Context(h_q, h_kv, 128, "bf16", n_hist + pad + 64, 8, t)
        khd = torch.zeros((n_hist + pad + 1, h_kv, 128), dtype=torch.bfloat16, device="cuda")
        vhd = torch.zeros_like(khd)
        if n_hist:
            khd[:n_hist], vhd[:n_hist] = ob.to_device(kh, "bf16"), ob.to_device(vh, "bf16")
        o = torch.full((t, h_q, 128), float("nan"), dtype=torch.float32, device="cuda")
        lse = torch.full((t, h_q), float("nan"), dtype=torch.float32, device="cuda")
        args = (ob.to_device(kc, "bf16"), ob.to_device(vc, "bf16"), 0.0, o, ob.DTYPE_FP32, lse)
        if masked:
            mask = torch.ones(n_hist + pad + 32, dtype=torch.uint8, device="cuda")
            mask[:n_hist] = torch.from_numpy(keep).cuda()
            ctx.chunk_attention_masked(ob.to_device(q, "bf16"), t, khd, vhd, mask, H.i32(n_hist), n_hist + pad, *args)
            o_ref, lse_ref = oc.chunk_attention_masked(q, kh, vh, keep, kc, vc)
        else:
            ctx.chunk_attention(ob.to_device(q, "bf16"), t, khd, vhd, H.i32(n_hist), n_hist + pad, *args)
            o_ref, lse_ref = oc.chunk_attention(q, kh, vh, kc, vc)
        torch.cuda.synchronize()
        assert ctx.poll_status() == 0
        err = np.abs(o.cpu().numpy() - o_ref)
        case = (t, n_hist, h_q, h_kv, masked, pad)
        assert np.isfinite(err).all() and err.max() <= 1e-2 and err.mean() <= 1e-3, case
        assert np.abs(lse.cpu().numpy() - lse_ref).max() <= 2e-2, case
        ctx.close()


def _random_rows(rng, S):
    raw = rng.integers(0, 256, size=(2, S, 512), dtype=np.uint8)
    k = torch.from_numpy(raw[0]).cuda().view(torch.bfloat16).view(S, 2, 128).contiguous()
    v = torch.from_numpy(raw[1]).cuda().view(torch.bfloat16).view(S, 2, 128).contiguous()
    return raw, k, v


@pytest.mark.parametrize("seed", [21, 22])
def test_random_layout_maintenance(H, ob, seed):
    """Token-mask pack, ordered-suffix and class-aware migration on random spans, densities, page and subblock sizes."""
    rng = np.random.default_rng(seed)
    for _ in range(12):                                      # class-aware
        P = int(rng.choice([16, 32, 64, 128, 256]))
        B = int(rng.choice([b for b in (2, 4, 8, 16, 32, 64) if P % b == 0]))
        S = int(rng.integers(1, 20000))
        keep = (rng.random(S) < rng.random()).astype(np.uint8)
        cls = np.zeros(S, np.uint8)
        pos = int(rng.integers(0, max(1, S // 4)))
        while pos < S:
            n = int(rng.integers(1, 5 * P))
            cls[pos:pos + n] = rng.choice([1, 2])
            pos += n
        cls |= np.where(rng.random(S) < rng.random(), 0x80, 0).astype(np.uint8)
        cls = np.where(keep == 1, cls, 0).astype(np.uint8)
        raw, k, v = _random_rows(rng, S)
        promote = int(rng.random() < 0.7)
        exp = oc.migrate_class(raw[0], raw[1], keep, cls, P, B, promote=bool(promote))
        ctx = ob.Context(8, 2, 128, "bf16", S + 64, 8, 16)
        mask = torch.zeros(S + 48, dtype=torch.uint8, device="cuda")
        mask[:S] = torch.from_numpy(keep).cuda()
        sc = torch.zeros(S + 48, dtype=torch.uint8, device="cuda")
        sc[:S] = torch.from_numpy(cls).cuda()
        n_pages = -(-S // P)
        moves = torch.full((2 * (S + 48),), -5, dtype=torch.int32, device="cuda")
        labels = torch.full((n_pages + 4,), 77, dtype=torch.uint8, device="cuda")
        info = torch.full((8,), -5, dtype=torch.int32, device="cuda")
        ctx.migrate_class(k, v, mask, sc, H.i32(S), S + 40, P, B, promote, moves, labels, info)
        torch.cuda.synchronize()
        assert ctx.poll_status() == 0
        inf = info.cpu().tolist()
        case = (S, P, B, promote)
        assert (bool(inf[0]), inf[1], inf[2]) == (exp["accepted"], len(exp["moves"]), exp["n_candidates"]), case
        assert tuple(inf[3:7]) == (exp["pages_before"], exp["pages_after"], exp["subblocks_before"], exp["subblocks_after"]), case
        live = mask[:S].cpu().numpy() == 1
        assert np.array_equal(live.astype(np.uint8), exp["keep_mask"]), case
        assert np.array_equal(sc[:S].cpu().numpy()[live], exp["slot_class"][live]), case
        assert np.array_equal(labels[:n_pages].cpu().numpy(), exp["page_class"]), case
        assert np.array_equal(H.bytes_of(k).reshape(S, -1)[live], exp["k"][live]), case
        assert np.array_equal(H.bytes_of(v).reshape(S, -1)[live], exp["v"][live]), case
        if exp["accepted"]:
            assert moves[:2 * inf[1]].cpu().numpy().reshape(-1, 2).tolist() == [list(m) for m in exp["moves"]], case
        ctx.close()
    for _ in range(12):                                      # ordered suffix
        P = int(rng.choice([16, 64, 256]))
        S = int(rng.integers(1, 20000))
        theta = int(rng.integers(1, 6))
        keep = (rng.random(S) < rng.random()).astype(np.uint8)
        if rng.random() < 0.5:
            keep[:S // 2] = 1
        raw, k, v = _random_rows(rng, S)
        exp = oc.migrate_suffix(raw[0], raw[1], keep, P, theta)
        ctx = ob.Context(8, 2, 128, "bf16", S + 64, 8, 16)
        mask = torch.zeros(S + 48, dtype=torch.uint8, device="cuda")
        mask[:S] = torch.from_numpy(keep).cuda()
        mask[S:S + 40] = 1
        span = H.i32(S)
        slot_map = torch.full((S + 48,), -5, dtype=torch.int32, device="cuda")
        info = torch.full((8,), -5, dtype=torch.int32, device="cuda")
        ctx.migrate_suffix(k, v, mask, span, S + 40, P, theta, slot_map, info)
        torch.cuda.synchronize()
        assert ctx.poll_status() == 0
        ns, case = exp["new_span"], (S, P, theta)
        assert int(span.item()) == ns and np.array_equal(mask[:S].cpu().numpy(), exp["keep_mask"]), case
        assert np.array_equal(slot_map[:S].cpu().numpy(), exp["slot_map"]), case
        assert np.array_equal(H.bytes_of(k[:ns]).reshape(ns, -1), exp["k"][:ns]), case
        assert np.array_equal(H.bytes_of(v[:ns]).reshape(ns, -1), exp["v"][:ns]), case
        ctx.close()
    for _ in range(12):                                      # token-mask pack
        P = int(rng.choice([16, 64, 256]))
        S = int(rng.integers(1, 30000))
        keep = (rng.random(S) < rng.random()).astype(np.uint8)
        raw, k, v = _random_rows(rng, S)
        exp = oc.compact_pack(raw[0], raw[1], keep, P)
        ctx = ob.Context(8, 2, 128, "bf16", S + 64, 8, 16)
        got = H.gpu_compact(ctx, k, v, keep, P)
        n = exp["n_kept"]
        assert got["n_kept"] == n and np.array_equal(got["slot_map"], exp["slot_map"]), (S, P)
        assert np.array_equal(H.bytes_of(got["k"][:n]).reshape(n, -1), exp["k"][:n]), (S, P)
        assert np.array_equal(H.bytes_of(got["v"][:n]).reshape(n, -1), exp["v"][:n]), (S, P)
        ctx.close()


def _random_units(rng, n_units, max_len):
    spans = [(int(rng.integers(1, 40)), wl.MOD_TEXT, 0)]
    ev = 1
    while len(spans) < n_units:
        for mod in (wl.MOD_VIDEO, wl.MOD_AUDIO, wl.MOD_TEXT):
            if len(spans) < n_units and rng.random() < 0.8:
                spans.append((int(rng.integers(1, max_len)), mod, ev))
        ev += 1
    return wl.make_units(spans)


@pytest.mark.parametrize("seed", [31, 32])
def test_random_structural_plans_and_unit_compaction(H, ob, seed):
    rng = np.random.default_rng(seed)
    for _ in range(25):
        units = _random_units(rng, int(rng.integers(1, 120)), int(rng.choice([8, 60, 400])))
        n = int(units[:, 1].sum())
        Hw = int(rng.integers(0, n + 50))
        Lw, R = int(rng.integers(0, Hw + 1)), int(rng.integers(0, 4))
        sink = (int(rng.integers(0, 40)), int(rng.integers(0, 12)), int(rng.integers(0, 8)))
        Tb, P = int(rng.integers(0, 300)), int(rng.choice([16, 64, 256]))
        exp = oc.plan_structural(units, Hw, Lw, R, sink, Tb)
        ctx = ob.Context(8, 2, 128, "bf16", n + 64, len(units) + 8, 16)
        got = H.gpu_plan_structural(ctx, units, Hw, Lw, R, sink, Tb)
        case = (len(units), n, Hw, Lw, R, sink, Tb, P)
        assert got["status"] == 0, case
        for key in ("unit_keep", "unit_kept_len", "keep_mask", "units_out"):
            assert np.array_equal(got[key], exp[key]), (key, case)
        raw, k, v = _random_rows(rng, n)
        expc = oc.compact_pack(raw[0], raw[1], exp["keep_mask"], P, exp["units_out"])
        gc = H.gpu_compact_units(ctx, k, v, units, exp["unit_keep"], P, units_out_np=exp["units_out"], kept_len_np=exp["unit_kept_len"])
        nk = expc["n_kept"]
        assert gc["status"] == 0 and gc["n_kept"] == nk and gc["part_begin"] == expc["part_begin"].tolist(), case
        assert np.array_equal(gc["slot_map"], expc["slot_map"]), case
        assert np.array_equal(H.bytes_of(gc["k"][:nk]).reshape(nk, -1), expc["k"][:nk]), case
        assert np.array_equal(H.bytes_of(gc["v"][:nk]).reshape(nk, -1), expc["v"][:nk]), case
        ctx.close()
