"""Pins for the CPU oracle: what the paper prints, closed forms, invariants, library
routines on special cases and brute force on tiny inputs.  No GPU needed."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import omni_oracle as oc
from paper_2609_34653_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_span_arithmetic.txt")


def _golden_rows():
    rows = {}
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, useful, before, after, page, note = line.split()
            rows[name] = (int(useful), int(before), int(after), int(page), note)
    return rows


# ---------------------------------------------------------------- compaction
def test_compact_paper_span_qwen_fig12():
    """2,778 useful cells scattered over a 3,840-slot span pack to 44 pages = 2,816 slots (Fig. 12)."""
    useful, before, after, page, _ = _golden_rows()["qwen_32k"]
    rng = np.random.default_rng(7)
    mask = np.zeros(before, dtype=np.uint8)
    idx = rng.choice(before - 1, size=useful - 1, replace=False)
    mask[idx] = 1
    mask[before - 1] = 1                       # the span really is `before` slots long
    k = rng.integers(0, 2**16, size=(before, 2, 4), dtype=np.uint16)
    res = oc.compact_pack(k, k[::-1].copy(), mask, page)
    assert res["n_kept"] == useful
    assert res["span_pages"] * page == after
    assert abs(1 - after / before - 0.267) < 5e-4


def test_compact_paper_span_minicpm_and_eager_ratio():
    g = _golden_rows()
    useful, before, after, page, _ = g["minicpm_32k"]
    mask = np.zeros(before, dtype=np.uint8)
    mask[np.linspace(0, before - 1, useful).astype(int)] = 1
    n = int(mask.sum())
    res = oc.compact_pack(None, None, mask, page)
    # eager packing reaches the page-rounded optimum, which is below the paper's selective result
    assert res["span_pages"] * page == -(-n // page) * page <= after
    assert abs(1 - after / before - 0.10) < 1e-3
    useful, before, after, page, _ = g["eager_60chunk"]
    mask = np.zeros(before, dtype=np.uint8)
    mask[np.arange(useful) * before // useful] = 1
    res = oc.compact_pack(None, None, mask, page)
    assert res["span_pages"] * page == after and before / after == 2.25


def test_compact_definition_and_invariants():
    rng = np.random.default_rng(3)
    for S, P in [(1, 16), (17, 16), (200, 16), (1000, 64), (777, 256)]:
        mask = (rng.random(S) < 0.37).astype(np.uint8)
        k = rng.integers(0, 2**16, size=(S, 3, 8), dtype=np.uint16)
        v = rng.integers(0, 2**16, size=(S, 3, 8), dtype=np.uint16)
        res = oc.compact_pack(k, v, mask, P)
        n = int(mask.sum())
        assert res["n_kept"] == n and res["span_pages"] == -(-n // P)
        # span never exceeds the kept count rounded up to a page, and wastes less than one page
        assert 0 <= res["span_pages"] * P - n < P
        # written out independently: the j-th kept slot lands at j, bytes intact, order preserved
        kept_slots = [s for s in range(S) if mask[s]]
        for j, s in enumerate(kept_slots):
            assert res["slot_map"][s] == j
            assert res["k"][j].tobytes() == k[s].tobytes() and res["v"][j].tobytes() == v[s].tobytes()
        assert all(res["slot_map"][s] == -1 for s in range(S) if not mask[s])
        assert res["rows_moved"] == sum(1 for j, s in enumerate(kept_slots) if j != s)
        # idempotence: compacting the packed cache moves nothing
        mask2 = np.zeros(S, dtype=np.uint8)
        mask2[:n] = 1
        res2 = oc.compact_pack(res["k"], res["v"], mask2[:n], P)
        assert res2["rows_moved"] == 0 and res2["n_kept"] == n
    # all keep = identity, none keep = empty
    k = np.arange(40, dtype=np.float32).reshape(10, 4)
    res = oc.compact_pack(k, k, np.ones(10, np.uint8), 4)
    assert res["rows_moved"] == 0 and np.array_equal(res["k"], k) and res["span_pages"] == 3
    res = oc.compact_pack(k, k, np.zeros(10, np.uint8), 4)
    assert res["n_kept"] == 0 and res["span_pages"] == 0 and np.all(res["page_class"] == 255)


def test_compact_partitions_and_page_classes():
    # groups 0,1,1,2 with lens 20, 30, 14, 25 -> n = 89, P = 16
    units_out = np.array([[0, 20, 2, 0, 0, 0], [20, 30, 0, 1, 1, 0], [50, 14, 1, 1, 1, 0],
                          [64, 25, 0, 9, 2, 0]], dtype=np.int32)
    mask = np.zeros(160, dtype=np.uint8)
    mask[np.arange(89) + np.arange(89) // 3] = 1
    res = oc.compact_pack(None, None, mask, 16, units_out)
    assert res["part_begin"].tolist() == [0, 20, 64, 89]
    # pages 0,1 hold must-keep rows; 2..4 are full -> promoted; page 5 partial -> recent; rest empty
    assert res["page_class"].tolist() == [0, 0, 1, 1, 1, 2, 255, 255, 255, 255]
    with pytest.raises(ValueError):
        oc.compact_pack(None, None, mask, 16, units_out[[1, 0, 2, 3]])


# ----------------------------------------------------------------- attention
def _brute_attention(q, kh, vh, kc, vc, scale):
    T, Hq, D = q.shape
    G = Hq // kc.shape[1]
    o = np.zeros((T, Hq, D))
    lse = np.zeros((T, Hq))
    for i in range(T):
        for h in range(Hq):
            g = h // G
            keys = [kh[j, g] for j in range(kh.shape[0])] + [kc[j, g] for j in range(i + 1)]
            vals = [vh[j, g] for j in range(vh.shape[0])] + [vc[j, g] for j in range(i + 1)]
            s = [scale * sum(float(a) * float(b) for a, b in zip(q[i, h], kk)) for kk in keys]
            m = max(s)
            e = [math.exp(x - m) for x in s]
            z = sum(e)
            for d in range(D):
                o[i, h, d] = sum(e[j] * float(vals[j][d]) for j in range(len(e))) / z
            lse[i, h] = m + math.log(z)
    return o, lse


def test_attention_brute_force_tiny():
    rng = np.random.default_rng(11)
    T, Hq, Hkv, D, N = 5, 4, 2, 8, 7
    q = rng.standard_normal((T, Hq, D)).astype(np.float32)
    kh, vh = rng.standard_normal((2, N, Hkv, D)).astype(np.float32)
    kc, vc = rng.standard_normal((2, T, Hkv, D)).astype(np.float32)
    o, lse = oc.chunk_attention(q, kh, vh, kc, vc)
    ob, lb = _brute_attention(q, kh, vh, kc, vc, 1 / math.sqrt(D))
    assert np.allclose(o, ob, atol=1e-12) and np.allclose(lse, lb, atol=1e-12)
    # a non-default scale and the sampled-rows form agree too
    o2, l2 = oc.chunk_attention(q, kh, vh, kc, vc, scale=0.3, rows=[(4, 3), (0, 0), (2, 1)])
    ob2, lb2 = _brute_attention(q, kh, vh, kc, vc, 0.3)
    assert np.allclose(o2, [ob2[4, 3], ob2[0, 0], ob2[2, 1]], atol=1e-12)
    assert np.allclose(l2, [lb2[4, 3], lb2[0, 0], lb2[2, 1]], atol=1e-12)


def test_attention_equals_library_causal_attention():
    """History + chunk attention is plain causal attention of the last T rows of the joined
    sequence (dense attention keeps every preceding token): compare with torch SDPA."""
    import torch
    rng = np.random.default_rng(5)
    T, Hq, Hkv, D, N = 33, 4, 2, 16, 70
    q = rng.standard_normal((T, Hq, D)).astype(np.float32)
    kh, vh = rng.standard_normal((2, N, Hkv, D)).astype(np.float32)
    kc, vc = rng.standard_normal((2, T, Hkv, D)).astype(np.float32)
    o, _ = oc.chunk_attention(q, kh, vh, kc, vc)
    G = Hq // Hkv
    K = torch.from_numpy(np.concatenate([kh, kc])).double().permute(1, 0, 2).repeat_interleave(G, 0)
    V = torch.from_numpy(np.concatenate([vh, vc])).double().permute(1, 0, 2).repeat_interleave(G, 0)
    Q = torch.from_numpy(q).double().permute(1, 0, 2)
    mask = torch.ones(T, N + T, dtype=torch.bool).tril(diagonal=N)
    ref = torch.nn.functional.scaled_dot_product_attention(Q[None], K[None], V[None], attn_mask=mask)[0]
    assert np.allclose(o, ref.permute(1, 0, 2).numpy(), atol=1e-10)


def test_attention_closed_forms():
    rng = np.random.default_rng(9)
    T, Hq, Hkv, D, N = 6, 2, 1, 8, 10
    q = rng.standard_normal((T, Hq, D)).astype(np.float32)
    vh = rng.standard_normal((N, Hkv, D)).astype(np.float32)
    vc = rng.standard_normal((T, Hkv, D)).astype(np.float32)
    kconst = rng.standard_normal(D).astype(np.float32)
    kh = np.broadcast_to(kconst, (N, Hkv, D)).copy()
    kc = np.broadcast_to(kconst, (T, Hkv, D)).copy()
    o, lse = oc.chunk_attention(q, kh, vh, kc, vc)
    # equal keys -> uniform weights -> running mean of the values; lse = s + log(count)
    for i in range(T):
        mean = (vh[:, 0].astype(np.float64).sum(0) + vc[:i + 1, 0].astype(np.float64).sum(0)) / (N + i + 1)
        for h in range(Hq):
            assert np.allclose(o[i, h], mean, atol=1e-12)
            s = float(np.dot(q[i, h].astype(np.float64), kconst.astype(np.float64))) / math.sqrt(D)
            assert abs(lse[i, h] - (s + math.log(N + i + 1))) < 1e-12
    # permuting history rows does not change the output
    kh = rng.standard_normal((N, Hkv, D)).astype(np.float32)
    kc = rng.standard_normal((T, Hkv, D)).astype(np.float32)
    o1, l1 = oc.chunk_attention(q, kh, vh, kc, vc)
    perm = rng.permutation(N)
    o2, l2 = oc.chunk_attention(q, kh[perm], vh[perm], kc, vc)
    assert np.allclose(o1, o2, atol=1e-12) and np.allclose(l1, l2, atol=1e-12)
    # splitting the history and merging the halves by their log-sum-exp reproduces the result
    oa, la = oc.chunk_attention(q, kh[:4], vh[:4], kc, vc)
    # second half: history only, no chunk -> emulate with a chunk whose keys never win
    s_b = np.einsum("ihd,jd->ihj", q.astype(np.float64), kh[4:, 0].astype(np.float64)) / math.sqrt(D)
    lb = np.log(np.exp(s_b).sum(-1))
    ob = np.einsum("ihj,jd->ihd", np.exp(s_b - lb[..., None]), vh[4:, 0].astype(np.float64))
    wa, wb = np.exp(la - np.logaddexp(la, lb)), np.exp(lb - np.logaddexp(la, lb))
    assert np.allclose(o1, wa[..., None] * oa + wb[..., None] * ob, atol=1e-12)
    # empty history is plain causal self-attention: row 0 returns v_chunk[0]
    o0, _ = oc.chunk_attention(q, kh[:0], vh[:0], kc, vc)
    assert np.allclose(o0[0, 0], vc[0, 0], atol=1e-12)


# ------------------------------------------------------------------- scoring
def _units(lens, mods=None, events=None, groups=None):
    mods = mods or [0] * len(lens)
    events = events or list(range(len(lens)))
    u = wl.make_units(list(zip(lens, mods, events)), group_of_first=None)
    if groups is not None:
        u[:, 4] = groups
    return u


def test_score_closed_form_identical_keys():
    rng = np.random.default_rng(2)
    units = _units([5, 9, 2, 16], mods=[2, 0, 1, 0])
    N = 32
    q = rng.standard_normal((7, 4, 8)).astype(np.float32)
    k = np.broadcast_to(rng.standard_normal(8).astype(np.float32), (N, 2, 8)).copy()
    w = (1.0, 2.5, 0.75)
    score, mass = oc.score_units(q, k, units, w)
    assert np.allclose(mass, np.array([5, 9, 2, 16]) / N, atol=1e-14)
    assert np.allclose(score, [w[2], w[0], w[1], w[0]], atol=1e-13)


def test_score_invariants_and_permutation():
    rng = np.random.default_rng(4)
    lens = [5, 9, 2, 16, 7]
    units = _units(lens, mods=[2, 0, 1, 0, 1])
    N = sum(lens)
    q = rng.standard_normal((6, 4, 8)).astype(np.float32)
    k = rng.standard_normal((N, 2, 8)).astype(np.float32)
    score, mass = oc.score_units(q, k, units, (1, 1, 1))
    assert abs(mass.sum() - 1) < 1e-13
    assert abs((score * np.array(lens)).sum() - N) < 1e-11
    # re-ordering whole units permutes the scores
    order = [3, 0, 4, 1, 2]
    k2 = np.concatenate([k[units[u, 0]:units[u, 0] + units[u, 1]] for u in order])
    units2 = _units([lens[u] for u in order], mods=[int(units[u, 2]) for u in order])
    w = (1.0, 2.0, 3.0)
    s1, m1 = oc.score_units(q, k, units, w)
    s2, m2 = oc.score_units(q, k2, units2, w)
    assert np.allclose(s2, s1[order], atol=1e-13) and np.allclose(m2, m1[order], atol=1e-14)
    # one key strongly aligned with every query draws all the mass to its unit
    qpos = np.abs(q)
    kb = k.copy()
    kb[20] = 50.0
    _, mb = oc.score_units(qpos, kb, units, (1, 1, 1))
    assert mb[3] > 1 - 1e-9


def test_score_single_row_is_textbook_softmax():
    from scipy.special import softmax
    rng = np.random.default_rng(8)
    lens = [3, 4, 6]
    units = _units(lens)
    q = rng.standard_normal((1, 1, 16)).astype(np.float32)
    k = rng.standard_normal((13, 1, 16)).astype(np.float32)
    _, mass = oc.score_units(q, k, units, (1, 1, 1))
    a = softmax((k[:, 0].astype(np.float64) @ q[0, 0].astype(np.float64)) / 4.0)
    assert np.allclose(mass, [a[0:3].sum(), a[3:7].sum(), a[7:13].sum()], atol=1e-14)


def test_score_brute_force_tiny():
    rng = np.random.default_rng(13)
    lens = [4, 1, 7, 3]
    mods = [2, 0, 1, 0]
    units = _units(lens, mods=mods)
    N, T, Hq, Hkv, D = sum(lens), 5, 4, 2, 6
    q = rng.standard_normal((T, Hq, D)).astype(np.float32)
    k = rng.standard_normal((N, Hkv, D)).astype(np.float32)
    w = (1.0, 2.0, 0.5)
    imp = [0.0] * N
    for h in range(Hq):
        for i in range(T):
            s = [sum(float(q[i, h, d]) * float(k[j, h // 2, d]) for d in range(D)) / math.sqrt(D)
                 for j in range(N)]
            m = max(s)
            e = [math.exp(x - m) for x in s]
            z = sum(e)
            for j in range(N):
                imp[j] += e[j] / z / (Hq * T)
    exp_score, pos = [], 0
    for ln, mod in zip(lens, mods):
        exp_score.append(w[mod] * sum(imp[pos:pos + ln]) * N / ln)
        pos += ln
    score, _ = oc.score_units(q, k, units, w)
    assert np.allclose(score, exp_score, atol=1e-12)


# ----------------------------------------------------------------- selection
def _check_select_invariants(units, scores, budget, R, caps, res):
    U = len(units)
    keep = res["unit_keep"]
    events = units[:, 3]
    distinct = sorted(set(events.tolist()))
    recent = set(distinct[-R:]) if R > 0 else set()
    prot = [u for u in range(U) if units[u, 4] == 0 or events[u] in recent]
    assert all(keep[u] == 2 for u in prot)                                     # I1
    prot_len = int(units[prot, 1].sum())
    n_kept = int(units[keep != 0, 1].sum())
    assert res["n_kept"] == n_kept
    if prot_len >= budget:
        assert sorted(np.nonzero(keep)[0].tolist()) == sorted(prot)            # I2 (target, not bound)
    else:
        assert n_kept <= budget
    mask = res["keep_mask"]
    for u in range(U):                                                         # I3 no unit split
        seg = mask[units[u, 0]:units[u, 0] + units[u, 1]]
        assert np.all(seg == (1 if keep[u] else 0))
    # re-indexing: new start = kept tokens before the unit; labels preserved
    uo = res["units_out"]
    kept_idx = [u for u in range(U) if keep[u]]
    assert len(uo) == len(kept_idx)
    pos = 0
    for row, u in zip(uo, kept_idx):
        assert row[0] == pos and row[1] == units[u, 1] and row[2] == units[u, 2] and row[3] == units[u, 3]
        assert row[4] == (0 if units[u, 4] == 0 else (2 if events[u] in recent else 1))
        pos += units[u, 1]
    for m in range(3):
        if caps[m] >= 0:
            cand_kept = [u for u in kept_idx if u not in prot and units[u, 2] == m]
            assert int(units[cand_kept, 1].sum()) <= caps[m]


def test_select_invariants_random():
    rng = np.random.default_rng(21)
    for trial in range(200):
        U = int(rng.integers(1, 14))
        lens = rng.integers(1, 50, size=U).tolist()
        mods = rng.integers(0, 3, size=U).tolist()
        events = np.cumsum(rng.integers(0, 2, size=U)).tolist()
        groups = [0 if (i == 0 and rng.random() < 0.7) else 2 for i in range(U)]
        units = _units(lens, mods, events, groups)
        scores = rng.random(U).astype(np.float32)
        if rng.random() < 0.3:
            scores[rng.integers(U)] = scores[rng.integers(U)]        # exact ties
        budget = int(rng.integers(1, sum(lens) + 20))
        R = int(rng.integers(0, 5))
        caps = tuple(int(c) for c in rng.choice([-1, 10, 40, 100], size=3))
        res = oc.select_units(units, scores, budget, R, caps)
        _check_select_invariants(units, scores, budget, R, caps, res)
        # I4 greedy maximality: replay -- every rejected candidate was a misfit at its turn
        prot = [u for u in range(U) if res["unit_keep"][u] and u not in res["order"]]
        used = int(units[prot, 1].sum())
        cap_rem = list(caps)
        prev = None
        for u in res["order"]:
            if prev is not None:     # order is by score desc, ties by recency
                assert (scores[prev] > scores[u]) or (scores[prev] == scores[u] and prev > u)
            prev = u
            fits = units[u, 1] <= budget - used and (cap_rem[units[u, 2]] < 0 or units[u, 1] <= cap_rem[units[u, 2]])
            assert bool(res["unit_keep"][u]) == bool(fits)
            if fits:
                used += int(units[u, 1])
                if cap_rem[units[u, 2]] >= 0:
                    cap_rem[units[u, 2]] -= int(units[u, 1])


def test_select_special_cases():
    units = _units([16, 100, 20, 100, 20, 100, 20], mods=[2, 0, 1, 0, 1, 0, 1],
                   events=[0, 1, 1, 2, 2, 3, 3], groups=[0, 2, 2, 2, 2, 2, 2])
    N = int(units[:, 1].sum())
    # I5 budget >= history: nothing is evicted ("no-slide")
    res = oc.select_units(units, np.zeros(7, np.float32), N, 1)
    assert np.all(res["unit_keep"] == 2) and res["n_kept"] == N and np.all(res["keep_mask"] == 1)
    # I6 score = recency reduces to unit-level FIFO: the newest units that fit survive
    res = oc.select_units(units, np.arange(7, dtype=np.float32), 16 + 120 + 120, 1)
    assert res["unit_keep"].tolist() == [2, 0, 0, 2, 2, 2, 2]
    # a misfit does not end the walk: the frame of event 1 does not fit, its audio does
    res = oc.select_units(units, np.array([0, 9, 1, 8, 7, 0, 0], np.float32), 16 + 120 + 100 + 30, 1)
    assert res["unit_keep"].tolist() == [2, 0, 2, 2, 0, 2, 2] or res["unit_keep"].tolist() == [2, 2, 0, 0, 2, 2, 2]
    # the exact expected walk: cand order 1(9),3(8),4(7),2(1): 1 fits (100<=130), 3 no (100>30), 4 yes (20<=30), 2 no (20>10)
    assert res["unit_keep"].tolist() == [2, 2, 0, 0, 2, 2, 2]
    # protected set alone above budget: kept = protected exactly (trimming target, not a bound)
    res = oc.select_units(units, np.ones(7, np.float32), 50, 2)
    assert res["unit_keep"].tolist() == [2, 0, 0, 2, 2, 2, 2] and res["n_kept"] == 256
    # fewer events than the recent window: every event is recent, nothing is evicted
    two = _units([26, 178], mods=[2, 0], events=[0, 1], groups=[2, 2])
    res = oc.select_units(two, np.array([0.8, 0.5], np.float32), 92, 3)
    assert res["unit_keep"].tolist() == [2, 2] and res["n_kept"] == 204
    # NaN scores go last; ties go to the more recent unit
    sc = np.array([0, np.nan, 1, 1, 1, 0, 0], np.float32)
    res = oc.select_units(units, sc, 16 + 120 + 40, 1)
    assert res["order"] == [4, 3, 2, 1] and res["unit_keep"].tolist() == [2, 0, 2, 0, 2, 2, 2]
    # modality caps bound candidates only
    res = oc.select_units(units, np.arange(7, dtype=np.float32), N, 1, (100, -1, -1))
    assert res["unit_keep"].tolist() == [2, 0, 2, 2, 2, 2, 2]
    with pytest.raises(ValueError):
        oc.select_units(_units([1, 1], events=[3, 2]), np.zeros(2, np.float32), 5)


def test_select_brute_force_orderings():
    """On <= 5 candidates, the rule's result equals a replay written independently:
    enumerate every permutation, keep the one sorted by (score desc, index desc), walk it."""
    rng = np.random.default_rng(33)
    for trial in range(60):
        U = int(rng.integers(2, 7))
        lens = rng.integers(1, 30, size=U).tolist()
        units = _units(lens, events=list(range(U)), groups=[0] + [2] * (U - 1))
        scores = rng.integers(0, 3, size=U).astype(np.float32)   # many ties
        budget = int(rng.integers(lens[0] + lens[-1], sum(lens) + 1))
        res = oc.select_units(units, scores, budget, 1)
        cand = list(range(1, U - 1))
        best = None
        for perm in itertools.permutations(cand):
            ok = all((scores[a] > scores[b]) or (scores[a] == scores[b] and a > b)
                     for a, b in zip(perm, perm[1:]))
            if ok:
                assert best is None
                best = perm
        used = lens[0] + lens[-1]
        exp = {0, U - 1}
        for u in best:
            if lens[u] <= budget - used:
                exp.add(u)
                used += lens[u]
        assert set(np.nonzero(res["unit_keep"])[0].tolist()) == exp


# ------------------------------------------------------------ whole pass
def test_stream_step_budget_covers_history_is_full_attention():
    """With the budget covering the whole cache the pass is brute-force full attention."""
    w = wl.small_mixed(3, n_units=6, h_q=2, h_kv=1, d=8, dtype="fp32", max_len=12, t=9)
    N = w.n_hist
    res = oc.stream_step(w.q, w.k_hist, w.v_hist, w.units, w.k_chunk, w.v_chunk, w.chunk_units,
                         w.w_modality, budget=N, n_recent_events=1, modality_cap=(-1, -1, -1), page_size=4)
    ob, _ = _brute_attention(w.q, w.k_hist, w.v_hist, w.k_chunk, w.v_chunk, 1 / math.sqrt(8))
    assert res["compact"]["rows_moved"] == 0 and res["compact"]["n_kept"] == N
    assert np.allclose(res["o"], ob, atol=1e-12)
    assert len(res["units"]) == len(w.units) + len(w.chunk_units)
    assert res["units"][-1, 0] + res["units"][-1, 1] == N + w.t


def test_tiny_config_ranking_is_nontrivial():
    """Config 1: the biased video unit must out-score the other old video units and survive."""
    w = wl.tiny()
    score, mass = oc.score_units(w.q, w.k_hist, w.units, w.w_modality)
    vids = [u for u in range(len(w.units)) if w.units[u, 2] == 0 and u != 0 and w.units[u, 3] != 3]
    assert max(vids, key=lambda u: score[u]) == w.biased_unit
    sel = oc.select_units(w.units, score, w.budget, w.n_recent_events)
    assert sel["unit_keep"][w.biased_unit] == 2 and sel["unit_keep"][0] == 2
    assert sel["n_kept"] <= w.budget
    cp = oc.compact_pack(w.k_hist, w.v_hist, sel["keep_mask"], w.page_size, sel["units_out"])
    assert 0 <= cp["span_pages"] * w.page_size - cp["n_kept"] < w.page_size


# ------------------------------------------------------------------ structural retention planning
def _toy_stream():
    """4-token protected prefix, then four events of (video 10, audio 6[, text 3])."""
    return np.array([[0, 4, 2, 0, 0, 0],
                     [4, 10, 0, 1, 2, 0], [14, 6, 1, 1, 2, 0], [20, 3, 2, 1, 2, 0],
                     [23, 10, 0, 2, 2, 0], [33, 6, 1, 2, 2, 0], [39, 3, 2, 2, 2, 0],
                     [42, 10, 0, 3, 2, 0], [52, 6, 1, 3, 2, 0],
                     [58, 10, 0, 4, 2, 0], [68, 6, 1, 4, 2, 0]], dtype=np.int32)


def test_plan_structural_hand_worked():
    """Section 5.1 worked by hand on an 11-span stream of 74 tokens: the two newest events stay whole, older
    image/audio spans shrink to sink prefixes of 2 / 1 tokens, older text is kept oldest first under a shared
    budget of 4 (the first 3-token span fits, the second does not), then whole events go, oldest first."""
    u = _toy_stream()
    # no drop phase needed: 4 + (2+1+3) + (2+1+0) + 16 + 16 = 45 <= 45
    r = oc.plan_structural(u, 40, 45, 2, (2, 1, 0), 4)
    assert r["unit_kept_len"].tolist() == [4, 2, 1, 3, 2, 1, 0, 10, 6, 10, 6]
    assert r["unit_keep"].tolist() == [2, 1, 1, 2, 1, 1, 0, 2, 2, 2, 2]
    assert r["n_kept"] == 45
    assert r["units_out"][:, 0].tolist() == [0, 4, 6, 7, 10, 12, 13, 23, 29, 39]
    assert r["units_out"][:, 4].tolist() == [0, 1, 1, 1, 1, 1, 2, 2, 2, 2]           # must-keep | selected | recent
    mask = r["keep_mask"]
    assert mask[:4].all() and mask[4:6].all() and not mask[6:14].any()               # image span keeps its first 2 tokens
    assert mask[14] and not mask[15:20].any() and mask[20:23].all()                  # audio sink, then the text span
    assert not mask[39:42].any() and mask[42:].all()
    # target 40: one partially retained event (the oldest) is dropped, 45 - 6 = 39
    r = oc.plan_structural(u, 40, 40, 2, (2, 1, 0), 4)
    assert r["unit_kept_len"].tolist() == [4, 0, 0, 0, 2, 1, 0, 10, 6, 10, 6] and r["n_kept"] == 39
    # target 30: both partially retained events go (36 left), then complete events oldest first: 20
    r = oc.plan_structural(u, 40, 30, 2, (2, 1, 0), 4)
    assert r["unit_kept_len"].tolist() == [4, 0, 0, 0, 0, 0, 0, 0, 0, 10, 6] and r["n_kept"] == 20
    # target 5 cannot be met: the walk stops when one event remains; the prefix is never dropped
    r = oc.plan_structural(u, 40, 5, 2, (2, 1, 0), 4)
    assert r["unit_kept_len"].tolist() == [4, 0, 0, 0, 0, 0, 0, 0, 0, 10, 6]
    # below the high watermark nothing happens
    r = oc.plan_structural(u, 74, 10, 1, (0, 0, 0), 0)
    assert r["unit_kept_len"].tolist() == u[:, 1].tolist() and r["keep_mask"].all() and (r["unit_keep"] == 2).all()
    # a boundary span of an older event is kept whole while its event survives
    ub = u.copy()
    ub[1, 5] = oc.FLAG_BOUNDARY
    r = oc.plan_structural(ub, 40, 60, 2, (2, 1, 0), 4)
    assert r["unit_kept_len"].tolist() == [4, 10, 1, 3, 2, 1, 0, 10, 6, 10, 6]


def _random_stream(rng, n_events, with_prefix=True):
    spans = [(int(rng.integers(1, 9)), 2, 0)] if with_prefix else []
    for e in range(1, n_events + 1):
        for mod in (0, 1, 2):
            if rng.random() < (0.9, 0.8, 0.4)[mod]:
                spans.append((int(rng.integers(1, 40)), mod, e))
        if not spans or spans[-1][2] != e:
            spans.append((int(rng.integers(1, 40)), 0, e))
    u = wl.make_units(spans, group_of_first=0 if with_prefix else None)
    for i in range(len(u)):
        if rng.random() < 0.1 and u[i, 4] != 0:
            u[i, 5] |= oc.FLAG_BOUNDARY
    return u


def _token_level_replay(u, H, L, R, sink, Tb):
    """The same rules replayed per TOKEN with array operations (a second derivation, no shared code)."""
    lens = u[:, 1]
    n = int(lens.sum())
    tok_unit = np.repeat(np.arange(len(u)), lens)
    tok_off = np.arange(n) - np.repeat(u[:, 0], lens)
    if n <= H:
        return np.ones(n, dtype=bool)
    ev = u[tok_unit, 3]
    mod = u[tok_unit, 2]
    must = u[tok_unit, 4] == 0
    bnd = (u[tok_unit, 5] & 1) == 1
    ids = np.unique(u[:, 3])
    recent_ids = ids[max(0, len(ids) - R):] if R > 0 else ids[:0]
    rec = np.isin(ev, recent_ids)
    keep = must | rec | (~must & ~rec & bnd)
    older = ~must & ~rec & ~bnd
    for m in (0, 1):
        keep |= older & (mod == m) & (tok_off < sink[m])
    # text: cumulative length of older text spans in time order, span by span
    t_units = [i for i in range(len(u)) if u[i, 2] == 2 and u[i, 4] != 0 and u[i, 3] not in recent_ids and not (u[i, 5] & 1)]
    csum = np.cumsum([int(u[i, 1]) for i in t_units]) if t_units else np.array([], dtype=int)
    fits = csum <= Tb
    if len(fits) and not fits.all():
        fits[np.argmin(fits):] = False
    for i, ok in zip(t_units, fits):
        if ok:
            keep[tok_unit == i] = True
    # whole events, oldest first, partially retained ones before complete ones
    full = np.array([keep[(tok_unit == i)].all() for i in range(len(u))])
    droppable = lambda e: (ev == e) & ~must
    alive = [e for e in ids if keep[droppable(e)].any()]
    part = [e for e in alive if not all(full[i] for i in range(len(u)) if u[i, 3] == e and u[i, 4] != 0)]
    comp = [e for e in alive if e not in part]
    left = len(alive)
    for e in part + comp:
        if keep.sum() <= L or left <= 1:
            break
        keep[droppable(e)] = False
        left -= 1
    return keep


def test_plan_structural_matches_token_level_replay_and_invariants():
    rng = np.random.default_rng(515)
    for trial in range(300):
        u = _random_stream(rng, int(rng.integers(1, 9)), with_prefix=rng.random() < 0.8)
        n = int(u[:, 1].sum())
        H = int(rng.integers(0, n + 10))
        L = int(rng.integers(0, H + 1))
        R = int(rng.integers(0, 4))
        sink = (int(rng.integers(0, 12)), int(rng.integers(0, 12)), 0)
        Tb = int(rng.integers(0, 60))
        r = oc.plan_structural(u, H, L, R, sink, Tb)
        ref = _token_level_replay(u, H, L, R, sink, Tb)
        assert np.array_equal(r["keep_mask"].astype(bool), ref), trial
        kept, lens = r["unit_kept_len"], u[:, 1]
        # a span survives as a prefix of itself; the mask is that prefix
        assert ((kept >= 0) & (kept <= lens)).all()
        for i in range(len(u)):
            st = int(u[i, 0])
            assert r["keep_mask"][st:st + kept[i]].all() and not r["keep_mask"][st + kept[i]:st + lens[i]].any()
        # the protected prefix always survives whole
        assert (kept[u[:, 4] == 0] == lens[u[:, 4] == 0]).all()
        # survivors are re-indexed contiguously, in order, with their new lengths
        uo = r["units_out"]
        assert uo[:, 1].tolist() == [int(k) for k in kept if k > 0]
        assert uo[:, 0].tolist() == np.concatenate([[0], np.cumsum(uo[:-1, 1])]).astype(int).tolist() if len(uo) else True
        assert r["n_kept"] == int(kept.sum()) == int(r["keep_mask"].sum())
        if n > H:
            # stop rule: the target is met, or a single event is left beside the prefix
            ev_alive = {int(u[i, 3]) for i in range(len(u)) if kept[i] > 0 and u[i, 4] != 0}
            assert r["n_kept"] <= L or len(ev_alive) <= 1
            # an older image/audio span keeps nothing or exactly its sink prefix
            ids = np.unique(u[:, 3])
            rec = set(ids[max(0, len(ids) - R):].tolist()) if R > 0 else set()
            for i in range(len(u)):
                if u[i, 4] != 0 and int(u[i, 3]) not in rec and not (u[i, 5] & 1) and u[i, 2] in (0, 1):
                    assert kept[i] in (0, min(int(lens[i]), sink[int(u[i, 2])]))


# ------------------------------------------------------------------ RoPE position re-index
def _rope_textbook(x, pos, base, nd):
    """RoPE from its complex-number definition: (x_i + j x_{i+nd/2}) * exp(j pos theta_i)."""
    half = nd // 2
    z = x[..., :half] + 1j * x[..., half:nd]
    theta = base ** (-2.0 * np.arange(half) / nd)
    z = z * np.exp(1j * np.asarray(pos, dtype=np.float64)[:, None, None] * theta[None, None, :])
    out = np.array(x, dtype=np.float64, copy=True)
    out[..., :half], out[..., half:nd] = z.real, z.imag
    return out


def test_rope_reindex_against_definition_and_group_properties():
    rng = np.random.default_rng(818)
    n, hkv, d = 37, 2, 16
    x = rng.standard_normal((n, hkv, d))
    pos = rng.integers(0, 5000, size=n)
    delta = -rng.integers(0, 3000, size=n)
    for nd in (16, 8):
        keyed = _rope_textbook(x, pos, 10000.0, nd)                      # keys as cached at their old positions
        moved = oc.rope_reindex(keyed, delta, 10000.0, nd)
        assert np.allclose(moved, _rope_textbook(x, pos + delta, 10000.0, nd), rtol=0, atol=1e-9)   # == keys at the new positions
        assert np.array_equal(moved[..., nd:], keyed[..., nd:])         # dimensions beyond n_dims untouched
        # zero shift is the identity, a shift and its inverse compose to the identity, norms are preserved
        assert np.array_equal(oc.rope_reindex(keyed, np.zeros(n, dtype=int), 10000.0, nd), keyed)
        assert np.allclose(oc.rope_reindex(moved, -delta, 10000.0, nd), keyed, rtol=0, atol=1e-9)
        assert np.allclose(np.linalg.norm(moved, axis=-1), np.linalg.norm(keyed, axis=-1))
    # the dot product of a query and a key depends on their distance only: shifting both leaves it unchanged
    q = _rope_textbook(rng.standard_normal((n, hkv, d)), pos + 7, 500000.0, d)
    k = _rope_textbook(x, pos, 500000.0, d)
    before = (q * k).sum(-1)
    after = (oc.rope_reindex(q, delta, 500000.0) * oc.rope_reindex(k, delta, 500000.0)).sum(-1)
    assert np.allclose(before, after, atol=1e-9)
    # packed form: delta = new slot - old slot
    mask = rng.random(n) < 0.5
    kk, vv, dl = oc.compact_pack_rope(x, x + 1, mask, 10000.0)
    assert np.array_equal(dl, np.arange(mask.sum()) - np.nonzero(mask)[0]) and np.array_equal(vv, (x + 1)[mask])
    assert np.allclose(kk, oc.rope_reindex(x[mask], dl, 10000.0))


# ------------------------------------------------------------------ ordered-suffix migration
def test_migrate_suffix_brute_force_and_invariants():
    rng = np.random.default_rng(929)
    for trial in range(400):
        P = int(rng.choice([4, 8, 16]))
        S = int(rng.integers(1, 200))
        dens = rng.random()
        keep = (rng.random(S) < dens).astype(np.uint8)
        if rng.random() < 0.3:                                   # a dense head and a sparse tail, the case the mode is for
            keep[:S // 2] = 1
        theta = int(rng.integers(1, 4))
        k = rng.integers(0, 1 << 30, size=(S, 3))
        v = rng.integers(0, 1 << 30, size=(S, 3))
        r = oc.migrate_suffix(k, v, keep, P, theta)
        pages = lambda n: -(-n // P)
        # brute force over every page-aligned start: the chosen one is the largest that saves >= theta pages
        ok = [p for p in range(0, S, P) if pages(S) - pages(p + int(keep[p:].sum())) >= theta]
        assert r["start"] == (max(ok) if ok else -1)
        if not ok:
            assert r["rows_moved"] == 0 and np.array_equal(r["keep_mask"], keep) and np.array_equal(r["k"], k)
            continue
        p = r["start"]
        assert p % P == 0 and r["pages_saved"] >= theta and r["new_span"] == p + int(keep[p:].sum())
        # everything before the suffix is untouched: contents and holes
        assert np.array_equal(r["k"][:p], k[:p]) and np.array_equal(r["keep_mask"][:p], keep[:p])
        # the suffix is packed in order: the live rows after the move are the live rows before it, same order
        live_before = np.nonzero(keep)[0]
        live_after = np.nonzero(r["keep_mask"])[0]
        assert np.array_equal(r["k"][live_after], k[live_before]) and np.array_equal(r["v"][live_after], v[live_before])
        assert np.array_equal(r["slot_map"][live_before], live_after) and (r["slot_map"][keep == 0] == -1).all()
        assert r["keep_mask"][p:r["new_span"]].all() and not r["keep_mask"][r["new_span"]:].any()
        assert r["rows_moved"] == int((live_before != live_after).sum())
    # worked by hand: 12 slots, pages of 4, live slots {0, 2, 3, 6, 8, 11}.  Packing [8, 12) gives span 10 (3 pages, none
    # saved); packing [4, 12) gives span 7 (2 pages, one saved): the scan stops there; nothing saves two pages.
    keep = np.array([1, 0, 1, 1, 0, 0, 1, 0, 1, 0, 0, 1], dtype=np.uint8)
    r = oc.migrate_suffix(np.arange(12), np.arange(12) + 100, keep, 4, 1)
    assert r["start"] == 4 and r["new_span"] == 7 and r["pages_saved"] == 1 and r["rows_moved"] == 3
    assert r["k"][:7].tolist() == [0, 1, 2, 3, 6, 8, 11] and r["keep_mask"].tolist() == [1, 0, 1, 1, 1, 1, 1, 0, 0, 0, 0, 0]
    assert oc.migrate_suffix(np.arange(12), np.arange(12) + 100, keep, 4, 2)["start"] == -1


def test_attention_masked_is_attention_over_live_rows():
    w = wl.tiny()
    rng = np.random.default_rng(939)
    keep = (rng.random(w.n_hist) < 0.6).astype(np.uint8)
    o, lse = oc.chunk_attention_masked(w.q, w.k_hist, w.v_hist, keep, w.k_chunk, w.v_chunk)
    # brute force for a few outputs: explicit -inf on the dead slots of the FULL history
    for i, h in [(0, 0), (17, 3), (255, 1)]:
        keys = np.concatenate([w.k_hist[:, 0], w.k_chunk[:i + 1, 0]]).astype(np.float64)
        vals = np.concatenate([w.v_hist[:, 0], w.v_chunk[:i + 1, 0]]).astype(np.float64)
        s = keys @ w.q[i, h].astype(np.float64) / math.sqrt(w.d)
        s[:w.n_hist][keep == 0] = -np.inf
        p = np.exp(s - s.max())
        assert np.allclose(o[i, h], (p @ vals) / p.sum(), atol=1e-12)
    # a suffix migration does not change what attention sees
    m = oc.migrate_suffix(w.k_hist, w.v_hist, keep, 16, 1)
    assert m["start"] >= 0
    o2, _ = oc.chunk_attention_masked(w.q, m["k"], m["v"], m["keep_mask"], w.k_chunk, w.v_chunk)
    assert np.allclose(o, o2, atol=1e-12)


# ---------------------------------------------------------------------------------------------------------------
# class-aware selective migration (Section 6.2 "packing scattered entries" / "checking layout improvement")
def _class_layout(spec):
    """'M' must-keep, 's'/'r' selected / recent, 'S'/'R' the same as candidates, '.' a hole."""
    code = {"M": 0, "s": 1, "r": 2, "S": 1 | 0x80, "R": 2 | 0x80}
    spec = spec.replace(" ", "")
    keep = np.array([ch != "." for ch in spec], dtype=np.uint8)
    cls = np.array([code.get(ch, 0) for ch in spec], dtype=np.uint8)
    return keep, cls


def test_migrate_class_hand_worked():
    # pages of 4, subblocks of 2.  Candidates in physical order: 4 (no earlier hole: stays), 7 -> 5, 9 -> 6,
    # 15 -> 7 (the slot vacated by the first move; page 1 holds class selected only).  Pages 4 -> 3, subblocks 7 -> 5.
    keep, cls = _class_layout("MMMM S..S .S.. r..S")
    ids = np.arange(16)
    r = oc.migrate_class(ids, ids + 100, keep, cls, 4, 2)
    assert r["accepted"] and r["moves"] == [(7, 5), (9, 6), (15, 7)]
    assert (r["pages_before"], r["pages_after"], r["subblocks_before"], r["subblocks_after"]) == (4, 3, 7, 5)
    assert r["keep_mask"].tolist() == [1, 1, 1, 1, 1, 1, 1, 1, 0, 0, 0, 0, 1, 0, 0, 0]
    assert r["k"][[4, 5, 6, 7, 12]].tolist() == [4, 7, 9, 15, 12] and r["v"][[5, 6, 7]].tolist() == [107, 109, 115]
    assert r["page_class"].tolist() == [0, 1, oc.PAGE_EMPTY, 2] and r["n_candidates"] == 4
    assert r["slot_class"][4:8].tolist() == [0x81] * 4                       # the moved entries keep class and mark

    # destination pages must be empty or of the same class: the hole in the must-keep page (slot 2) and the holes
    # of the page that holds a recent entry (5, 6) are closed to a selected-history candidate; page 2 is empty.
    keep, cls = _class_layout("MM.M r..r .... ..S. ...S")
    r = oc.migrate_class(ids.repeat(2)[:20], ids.repeat(2)[:20], keep, cls, 4, 2)
    assert r["moves"] == [(14, 8), (19, 9)] and r["accepted"]
    assert (r["pages_before"], r["pages_after"]) == (4, 3) and (r["subblocks_before"], r["subblocks_after"]) == (6, 5)
    # a recent-context candidate may use the holes of the recent page, not the others
    keep, cls = _class_layout("MM.M r..r .... ..R.")
    assert oc.migrate_class(None, None, keep, cls, 4, 2)["moves"] == [(14, 5)]

    # moving an entry between two pages that both stay active is not an improvement: rejected, nothing moves
    keep, cls = _class_layout("S... sS..")
    r = oc.migrate_class(np.arange(8), np.arange(8), keep, cls, 4, 2)
    assert not r["accepted"] and r["moves"] == [] and np.array_equal(r["keep_mask"], keep)
    assert np.array_equal(r["k"], np.arange(8)) and (r["pages_after"], r["subblocks_after"]) == (2, 2)
    # ... but with the candidate alone in its subblock the subblock count drops: accepted although both pages stay
    keep, cls = _class_layout("S... s..S")
    r = oc.migrate_class(np.arange(8), np.arange(8), keep, cls, 4, 2)
    assert r["accepted"] and r["moves"] == [(7, 1)] and (r["pages_after"], r["subblocks_after"]) == (2, 2)
    assert (r["pages_before"], r["subblocks_before"]) == (2, 3)

    # full pages stay in place: the candidates of page 1 do not move although page 0 has holes; the one of page 2 does
    keep, cls = _class_layout("s... SSSS S...")
    r = oc.migrate_class(None, None, keep, cls, 4, 2)
    assert r["moves"] == [(8, 1)] and r["n_candidates"] == 1

    # promotion: a page packed full of recent / selected entries becomes selected-history; a full page that holds
    # must-keep entries does not; nothing is promoted when the plan is rejected
    keep, cls = _class_layout("Rr.r .R.. MMMM")
    r = oc.migrate_class(None, None, keep, cls, 4, 2)
    assert r["moves"] == [(5, 2)] and r["accepted"]
    assert r["slot_class"][:4].tolist() == [0x81, 1, 0x81, 1] and r["page_class"].tolist() == [1, oc.PAGE_EMPTY, 0]
    r = oc.migrate_class(None, None, keep, cls, 4, 2, promote=False)
    assert r["slot_class"][:4].tolist() == [0x82, 2, 0x82, 2] and r["page_class"].tolist() == [2, oc.PAGE_EMPTY, 0]
    keep, cls = _class_layout("rrrr rR..")                                   # no hole before the candidate: no plan
    r = oc.migrate_class(None, None, keep, cls, 4, 2)
    assert not r["accepted"] and r["slot_class"][:4].tolist() == [2, 2, 2, 2] and r["page_class"].tolist() == [2, 2]


def test_migrate_class_replay_minimality_and_invariants():
    rng = np.random.default_rng(4711)
    n_acc = n_rej = 0
    for trial in range(300):
        P = int(rng.choice([4, 8, 16])); B = int(rng.choice([b for b in (2, 4, 8, 16) if P % b == 0]))
        S = int(rng.integers(1, 160))
        keep = (rng.random(S) < rng.random()).astype(np.uint8)
        # classes in runs (must-keep head, then selected / recent mixed by runs), candidates at random
        cls = np.zeros(S, np.uint8)
        pos = int(rng.integers(0, max(1, S // 4)))
        while pos < S:
            n = int(rng.integers(1, 3 * P)); cls[pos:pos + n] = rng.choice([1, 2]); pos += n
        cls |= np.where(rng.random(S) < rng.random(), 0x80, 0).astype(np.uint8)
        cls = np.where(keep == 1, cls, 0).astype(np.uint8)
        ids = rng.permutation(S) + 1
        r = oc.migrate_class(ids, -ids, keep, cls, P, B)
        # independent replay with sets: every move went to the smallest empty compatible slot before its source
        live = {s: (int(ids[s]), int(cls[s])) for s in range(S) if keep[s]}
        full0 = {p for p in range(-(-S // P)) if all((s in live) for s in range(p * P, min(S, (p + 1) * P)))}
        planned = []
        for s in sorted(s for s in live if live[s][1] & 0x80 and s // P not in full0):
            c = live[s][1] & 3
            best = None
            for d in range(s):
                if d in live:
                    continue
                if all((live[x][1] & 3) == c for x in range(d // P * P, min(S, (d // P + 1) * P)) if x in live):
                    best = d
                    break
            if best is not None:
                live[best] = live.pop(s)
                planned.append((s, best))
        act = lambda slots, size: len({s // size for s in slots})
        before = set(np.nonzero(keep)[0].tolist())
        improves = bool(planned) and (act(live, P) < act(before, P) or act(live, B) < act(before, B))
        assert r["accepted"] == improves
        assert (r["pages_before"], r["subblocks_before"]) == (act(before, P), act(before, B))
        if not improves:
            n_rej += 1
            assert r["moves"] == [] and np.array_equal(r["keep_mask"], keep) and np.array_equal(r["k"], ids)
            assert np.array_equal(r["slot_class"], cls)
            continue
        n_acc += 1
        assert r["moves"] == planned
        assert (r["pages_after"], r["subblocks_after"]) == (act(live, P), act(live, B))
        assert set(np.nonzero(r["keep_mask"])[0].tolist()) == set(live)
        for s, (i, c) in live.items():
            assert r["k"][s] == i and r["v"][s] == -i and (r["slot_class"][s] & 0x80) == (c & 0x80)
            promoted = s // P * P + P <= S and all(x in live and (live[x][1] & 3) >= 1 for x in range(s // P * P, s // P * P + P))
            assert (r["slot_class"][s] & 3) == (1 if promoted else (c & 3))
        # the history is the same set of entries: nothing lost, nothing duplicated, non-candidates did not move
        assert sorted(i for i, _ in live.values()) == sorted(int(ids[s]) for s in before)
        moved_from = {s for s, _ in planned}
        assert all(cls[s] & 0x80 for s in moved_from) and all(d < s for s, d in planned)
    assert n_acc > 50 and n_rej > 20


def test_migrate_class_leaves_attention_unchanged():
    rng = np.random.default_rng(77)
    S, P, B, hq, hkv, d, t = 96, 8, 4, 4, 2, 16, 5
    keep = (rng.random(S) < 0.35).astype(np.uint8)
    cls = np.where(keep == 1, rng.choice([1, 2], size=S) | np.where(rng.random(S) < 0.6, 0x80, 0), 0).astype(np.uint8)
    k = rng.standard_normal((S, hkv, d)); v = rng.standard_normal((S, hkv, d))
    q = rng.standard_normal((t, hq, d)); kc = rng.standard_normal((t, hkv, d)); vc = rng.standard_normal((t, hkv, d))
    r = oc.migrate_class(k, v, keep, cls, P, B)
    assert r["accepted"] and len(r["moves"]) > 5
    a0 = oc.chunk_attention_masked(q, k, v, keep, kc, vc)
    a1 = oc.chunk_attention_masked(q, r["k"], r["v"], r["keep_mask"], kc, vc)
    out0 = a0[0] if isinstance(a0, tuple) else a0
    out1 = a1[0] if isinstance(a1, tuple) else a1
    assert np.allclose(out0, out1, rtol=0, atol=1e-12)
