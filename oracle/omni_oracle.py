"""CPU oracle for the per-chunk hot path: score -> select -> compact -> attend.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the
CUDA kernels are checked against.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import it; the product path never does.  It
shares no code with the CUDA path and imports nothing from the package.

Arithmetic: inputs are taken exactly as stored (bf16 or fp32 values widened to
float64); every product, sum, exponential and division is float64 (numpy).
Integer steps are plain integer arithmetic.

What follows the paper and what does not
----------------------------------------
* compact_pack      -- eager compaction exactly as the paper defines it
                       (Section 6, "Compaction-movement trade-off": all
                       retained entries packed into a contiguous prefix), the
                       allocation classes and page promotion rule of
                       Section 6.1, the page-rounded span of Section 6.2.
                       Pinned by the definition, by the span arithmetic the
                       paper prints for Fig. 12 and Fig. 8, and by invariants.
* chunk_attention   -- dense causal attention of the new chunk over the
                       retained history (Section 2.1 prefill; Section 3 "Dense
                       attention").  Pinned by brute force, by a library
                       attention routine and by closed forms.
* select_units      -- the paper's structural rules that are fixed (protected
                       prefix, most recent events kept whole, whole-span
                       boundaries, low watermark as a trimming target,
                       re-indexing of survivors: Sections 5.1-5.2) plus a
                       score-ordered greedy fill that the paper does NOT
                       define.  PARITY UNPINNED for the greedy order; pinned
                       only by invariants, special cases and brute force.
* plan_structural   -- OmniPick as the paper describes it (Section 5.1): no
                       scores; recent events whole, older events reduced to
                       boundary spans, per-modality sink prefixes and text under
                       a shared budget, then whole events dropped oldest first
                       (partially retained before complete) down to the low
                       watermark.  Prefix lengths, budgets and what counts as a
                       boundary span are parameters the paper leaves open;
                       pinned by a hand-worked example, an independent
                       token-level replay and invariants.
* migrate_suffix    -- OmniPage's ordered-suffix migration, the mode the paper uses
                       on CUDA (Section 6.2 "Checking layout improvement"): scan
                       backward for the smallest suffix whose packing shortens
                       the page-rounded span by at least a configured number of
                       pages, pack only that suffix in order, leave the rest in
                       place; no migration if no suffix qualifies.  Page
                       alignment of the suffix start and the default threshold
                       are readings.  Pinned by brute force over every suffix
                       start and by invariants.  Attention over the resulting
                       layout with holes is attention over the live rows.
* migrate_class     -- OmniPage's class-aware selective migration (Section 6.2
                       "Packing scattered entries", "Checking layout
                       improvement"; classes and promotion of Section 6.1):
                       candidates (entries kept from partially evicted units,
                       outside full pages) go, in physical order, to the earliest
                       empty slot of a page that is empty or of their class; the
                       plan is simulated and accepted only if the active pages
                       or the active subblocks decrease; full pages are promoted
                       to selected-history.  Readings: what "earlier empty slot"
                       means while the plan is being simulated (vacated slots
                       count), the mark that makes an entry a candidate, which
                       full pages are promoted.  PARITY UNPINNED by the paper
                       (it prints no example); pinned by hand-worked layouts,
                       an independent set-based replay that checks every move
                       is to the smallest admissible slot, and invariants.
* rope_reindex      -- the position shift the runtime applies to cached keys after
                       logical deletion (Section 5.2): a kept token's position
                       drops by the number of deleted tokens before it and its
                       key is re-rotated by that amount.  The paper names RoPE
                       only; the pairing (half-split), the base and the number
                       of rotated dimensions are parameters.  Pinned against
                       the complex-number definition of RoPE and by group
                       properties (composition, inverse, norm).
* score_units       -- the paper's OmniPick collects no attention scores at
                       run time; the statistic scored here is the one its
                       design study measures offline (attention weight from
                       later queries to each span, averaged; Section 5 "Key
                       insight"), weighted per modality ("Modality-asymmetric
                       attention").  PARITY UNPINNED by the paper; pinned only
                       by closed forms, invariants and brute force.
"""
from __future__ import annotations

import math

import numpy as np

# unit-table columns
U_START, U_LEN, U_MOD, U_EVENT, U_GROUP, U_FLAGS = range(6)
GRP_MUST_KEEP, GRP_SELECTED, GRP_RECENT = 0, 1, 2
KEEP_DROPPED, KEEP_SINK_PREFIX, KEEP_WHOLE = 0, 1, 2
FLAG_BOUNDARY = 1                         # unit.flags bit 0: a boundary span (kept whole while its event survives)
MOD_VIDEO, MOD_AUDIO, MOD_TEXT = 0, 1, 2
PAGE_EMPTY = 255


def _f64(a):
    return np.asarray(a, dtype=np.float64)


# ---------------------------------------------------------------------------
# S -- unit scoring
# ---------------------------------------------------------------------------
def score_units(q, k_hist, units, w_modality, scale=None):
    """Modality-weighted mean attention lift of the chunk's queries on each history unit.

    q [T, Hq, D], k_hist [N, Hkv, D], units [U, 6] covering slots 0..N-1 in order.
    For head h, query i, history key j:
        s_hij = scale * <q[i,h,:], k[j, h // G, :]>,     G = Hq / Hkv
        a_hij = softmax over j in [0, N) of s_hij        (history keys only)
    token importance  I_j    = mean over (h, i) of a_hij            (sums to 1 over j)
    unit mass         mass_u = sum of I_j over the unit's tokens
    unit score        score_u = w[modality_u] * mass_u * N / len_u  (1.0*w means "uniform attention")
    Returns (score[U], mass[U]) as float64.
    """
    q = _f64(q)
    k = _f64(k_hist)
    units = np.asarray(units)
    T, Hq, D = q.shape
    N, Hkv, _ = k.shape
    G = Hq // Hkv
    if scale is None or scale <= 0:
        scale = 1.0 / math.sqrt(D)
    importance = np.zeros(N, dtype=np.float64)
    for h in range(Hq):
        s = (q[:, h, :] @ k[:, h // G, :].T) * scale              # [T, N]
        s -= s.max(axis=1, keepdims=True)
        a = np.exp(s)
        a /= a.sum(axis=1, keepdims=True)
        importance += a.sum(axis=0)
    importance /= float(Hq * T)
    U = len(units)
    mass = np.zeros(U, dtype=np.float64)
    score = np.zeros(U, dtype=np.float64)
    for u in range(U):
        st, ln, mod = int(units[u, U_START]), int(units[u, U_LEN]), int(units[u, U_MOD])
        mass[u] = importance[st:st + ln].sum()
        score[u] = float(w_modality[mod]) * mass[u] * N / ln if ln > 0 else 0.0
    return score, mass


# ---------------------------------------------------------------------------
# L -- budgeted unit selection
# ---------------------------------------------------------------------------
def select_units(units, scores, budget, n_recent_events=1, modality_cap=(-1, -1, -1)):
    """Choose which whole units of the history survive.

    1. Protected set: units in the must-keep group (protected system prefix,
       Section 5.1) and every unit of the `n_recent_events` newest events
       (recent units kept in full, never cut at a token position).
    2. If the protected set alone reaches the budget, keep exactly it: the
       budget is a trimming target, not a strict bound (Section 5.1).
    3. Remaining units are candidates, visited by descending score (ties: the
       more recent unit first; NaN scores last).  A candidate is taken iff it
       fits the remaining budget and its modality's remaining cap; a misfit
       does not end the walk.
    4. Survivors are re-indexed: a kept token's new position is the number of
       kept tokens before it (Section 5.2); unit records keep modality, event
       and flags; group becomes must-keep / recent-context / selected-history.

    `scores` is compared in float32 (the precision the CUDA path ranks in).
    Returns dict(unit_keep[U] u8, keep_mask[N] u8, n_kept, units_out[U', 6], order[list]).
    """
    units = np.asarray(units, dtype=np.int64)
    U = len(units)
    scores = np.asarray(scores, dtype=np.float32)
    events = units[:, U_EVENT]
    if U > 1 and np.any(np.diff(events) < 0):
        raise ValueError("event ids must be non-decreasing in unit order")
    distinct = sorted(set(int(e) for e in events))
    recent = set(distinct[max(0, len(distinct) - n_recent_events):]) if n_recent_events > 0 else set()

    protected = [u for u in range(U)
                 if units[u, U_GROUP] == GRP_MUST_KEEP or int(events[u]) in recent]
    keep = np.zeros(U, dtype=np.uint8)
    for u in protected:
        keep[u] = KEEP_WHOLE
    used = int(sum(units[u, U_LEN] for u in protected))
    order = []
    if used < budget:
        cand = [u for u in range(U) if keep[u] == 0]

        def key(u):
            s = scores[u]
            if np.isnan(s):
                return (1, 0.0, -u)
            return (0, -float(s), -u)
        cand.sort(key=key)
        order = cand
        cap_rem = [int(c) if c >= 0 else None for c in modality_cap]
        for u in cand:
            ln, mod = int(units[u, U_LEN]), int(units[u, U_MOD])
            if ln > budget - used:
                continue
            if cap_rem[mod] is not None and ln > cap_rem[mod]:
                continue
            keep[u] = KEEP_WHOLE
            used += ln
            if cap_rem[mod] is not None:
                cap_rem[mod] -= ln

    n_hist = int(units[:, U_LEN].sum())
    keep_mask = np.zeros(n_hist, dtype=np.uint8)
    units_out = []
    pos = 0
    for u in range(U):
        if keep[u]:
            st, ln = int(units[u, U_START]), int(units[u, U_LEN])
            keep_mask[st:st + ln] = 1
            if units[u, U_GROUP] == GRP_MUST_KEEP:
                g = GRP_MUST_KEEP
            elif int(events[u]) in recent:
                g = GRP_RECENT
            else:
                g = GRP_SELECTED
            units_out.append((pos, ln, int(units[u, U_MOD]), int(events[u]), g, int(units[u, U_FLAGS])))
            pos += ln
    units_out = np.asarray(units_out, dtype=np.int32).reshape(-1, 6)
    return dict(unit_keep=keep, keep_mask=keep_mask, n_kept=pos, units_out=units_out, order=order)


# ---------------------------------------------------------------------------
# P -- structure-aware, score-free retention planning (OmniPick as written)
# ---------------------------------------------------------------------------
def plan_structural(units, high_watermark, low_watermark, n_recent_events, sink_prefix, text_budget):
    """The paper's retention plan, from unit metadata alone (Section 5.1).

    An *event* (the paper's "unit": one input chunk or one response) is the run
    of typed spans (rows of `units`) that share an event id.

    0. Retention starts only when the history exceeds the high watermark;
       otherwise everything is kept.
    1. Spans of the must-keep group (the protected system prefix) are kept
       whole and never dropped.  The `n_recent_events` newest events are kept
       whole ("keeping recent units intact").
    2. Older events, oldest to newest ("selecting spans from older units"):
       a boundary span is kept whole; an image/video or audio span keeps only
       its first `sink_prefix[modality]` tokens (a candidate sink); text spans
       are kept whole, oldest to newest, until their shared token budget is
       exhausted (the first text span that does not fit and all later ones of
       the older events are dropped).
    3. If the selection still exceeds the low watermark, whole events are
       dropped oldest first, partially retained events before complete ones;
       the walk stops when the target is met or only one event remains: the
       low watermark is a trimming target, not a strict bound.
    4. Survivors are re-indexed as in `select_units` (Section 5.2); a shortened
       span keeps its modality, event and flags with its new length.

    Returns dict(unit_keep[U] u8 (0 dropped, 1 sink prefix only, 2 whole),
    unit_kept_len[U] i32, keep_mask[N] u8, n_kept, units_out[U', 6]).
    """
    units = np.asarray(units, dtype=np.int64)
    U = len(units)
    lens = units[:, U_LEN]
    events = units[:, U_EVENT]
    if U > 1 and np.any(np.diff(events) < 0):
        raise ValueError("event ids must be non-decreasing in unit order")
    n_hist = int(lens.sum())
    kept = lens.copy()
    must = units[:, U_GROUP] == GRP_MUST_KEEP
    distinct = sorted(set(int(e) for e in events))
    recent = set(distinct[max(0, len(distinct) - n_recent_events):]) if n_recent_events > 0 else set()
    is_recent = np.array([int(e) in recent for e in events], dtype=bool)

    if n_hist > high_watermark:
        text_used = 0
        text_open = True
        for u in range(U):                                   # oldest to newest
            if must[u] or is_recent[u]:
                continue
            mod = int(units[u, U_MOD])
            if int(units[u, U_FLAGS]) & FLAG_BOUNDARY:
                continue                                     # kept whole
            if mod == MOD_TEXT:
                if text_open and text_used + int(lens[u]) <= text_budget:
                    text_used += int(lens[u])
                else:
                    text_open = False
                    kept[u] = 0
            else:
                kept[u] = min(int(lens[u]), int(sink_prefix[mod]))
        total = int(kept.sum())
        if total > low_watermark:
            # events that can be dropped, with what they hold outside the protected prefix
            ev_units = {e: [u for u in range(U) if int(events[u]) == e and not must[u]] for e in distinct}
            alive = [e for e in distinct if sum(int(kept[u]) for u in ev_units[e]) > 0]
            partial = [e for e in alive if any(kept[u] < lens[u] for u in ev_units[e])]
            complete = [e for e in alive if e not in partial]
            n_alive = len(alive)
            for e in partial + complete:                     # oldest first within each class
                if total <= low_watermark or n_alive <= 1:
                    break
                for u in ev_units[e]:
                    total -= int(kept[u])
                    kept[u] = 0
                n_alive -= 1

    keep = np.where(kept == 0, KEEP_DROPPED, np.where(kept == lens, KEEP_WHOLE, KEEP_SINK_PREFIX)).astype(np.uint8)
    keep_mask = np.zeros(n_hist, dtype=np.uint8)
    units_out = []
    pos = 0
    for u in range(U):
        k = int(kept[u])
        if k > 0:
            st = int(units[u, U_START])
            keep_mask[st:st + k] = 1
            g = GRP_MUST_KEEP if must[u] else (GRP_RECENT if is_recent[u] else GRP_SELECTED)
            units_out.append((pos, k, int(units[u, U_MOD]), int(events[u]), g, int(units[u, U_FLAGS])))
            pos += k
    units_out = np.asarray(units_out, dtype=np.int32).reshape(-1, 6)
    return dict(unit_keep=keep, unit_kept_len=kept.astype(np.int32), keep_mask=keep_mask, n_kept=pos, units_out=units_out)


# ---------------------------------------------------------------------------
# C -- eager compaction into the retention-partitioned page layout
# ---------------------------------------------------------------------------
def compact_pack(k_cache, v_cache, keep_mask, page_size, units_out=None):
    """Pack every retained KV row into a contiguous prefix, order preserved.

    k_cache, v_cache: [S, ...] arrays of any dtype (rows are copied bit for bit).
    keep_mask [S_span] u8.  As-if semantics: all reads precede all writes.
    Returns dict with
      k, v         packed rows [n_kept, ...]
      slot_map     [S_span] int32, destination slot or -1
      n_kept, span_pages (= ceil(n_kept / P): the page-rounded span), rows_moved
      part_begin   [4]: first slot of must-keep / selected-history / recent-context / end
      page_class   [ceil(S_span / P)] u8: 0 page holds a must-keep row; else 1 if it holds P
                   kept rows (fully packed page promoted to selected-history); else 2 if
                   partially filled (stays recent-context); else 255 (empty, reusable).
    `units_out` (the compacted unit table) supplies the groups for the partitions; because
    units are in logical order and group rank grows with recency, the stable pack IS the
    partitioned order -- this is asserted, not assumed.
    """
    keep_mask = np.asarray(keep_mask, dtype=np.uint8)
    S = len(keep_mask)
    P = int(page_size)
    slot_map = np.full(S, -1, dtype=np.int32)
    n = 0
    src = []
    for s in range(S):
        if keep_mask[s]:
            slot_map[s] = n
            src.append(s)
            n += 1
    src = np.asarray(src, dtype=np.int64)
    k_out = np.array(np.asarray(k_cache)[src], copy=True) if k_cache is not None else None
    v_out = np.array(np.asarray(v_cache)[src], copy=True) if v_cache is not None else None
    rows_moved = int(np.sum(src != np.arange(n)))
    span_pages = (n + P - 1) // P

    part_begin = np.array([0, 0, 0, n], dtype=np.int32)
    if units_out is not None and len(units_out):
        uo = np.asarray(units_out, dtype=np.int64)
        groups = uo[:, U_GROUP]
        if np.any(np.diff(groups) < 0):
            raise ValueError("retention groups are not ordered must-keep <= selected-history <= recent-context")
        if int(uo[:, U_LEN].sum()) != n:
            raise ValueError("compacted unit table does not cover the kept rows")
        n0 = int(uo[groups == GRP_MUST_KEEP, U_LEN].sum())
        n1 = int(uo[groups == GRP_SELECTED, U_LEN].sum())
        part_begin = np.array([0, n0, n0 + n1, n], dtype=np.int32)

    n_pages = (S + P - 1) // P
    page_class = np.full(n_pages, PAGE_EMPTY, dtype=np.uint8)
    for p in range(n_pages):
        lo, hi = p * P, min((p + 1) * P, n)
        if hi <= lo:
            continue
        if lo < part_begin[1]:
            page_class[p] = GRP_MUST_KEEP
        elif hi - lo == P:
            page_class[p] = GRP_SELECTED
        else:
            page_class[p] = GRP_RECENT
    return dict(k=k_out, v=v_out, slot_map=slot_map, n_kept=n, span_pages=span_pages,
                rows_moved=rows_moved, part_begin=part_begin, page_class=page_class)


# ---------------------------------------------------------------------------
# a5 -- append the chunk behind the compacted history
# ---------------------------------------------------------------------------
def append_chunk(units_kept, n_kept, chunk_units):
    """New entries enter the recent-context class behind the kept history (Section 6.1)."""
    cu = np.array(chunk_units, dtype=np.int32, copy=True).reshape(-1, 6)
    cu[:, U_START] += int(n_kept)
    cu[:, U_GROUP] = GRP_RECENT
    uk = np.asarray(units_kept, dtype=np.int32).reshape(-1, 6)
    return np.concatenate([uk, cu], axis=0)


# ---------------------------------------------------------------------------
# A -- GQA chunk-prefill attention
# ---------------------------------------------------------------------------
def chunk_attention(q, k_hist, v_hist, k_chunk, v_chunk, scale=None, rows=None):
    """o[i,h] = sum_j softmax_j(scale * <q_ih, k_j>) v_j over the kept history rows followed by
    chunk rows 0..i (causal inside the chunk, diagonal included); kv head of h is h // G.

    rows: optional iterable of (i, h) pairs to evaluate only those outputs.
    Returns (o [T, Hq, D] float64, lse [T, Hq] float64) or, with rows, (o [R, D], lse [R]).
    """
    q = _f64(q)
    kh, vh, kc, vc = _f64(k_hist), _f64(v_hist), _f64(k_chunk), _f64(v_chunk)
    T, Hq, D = q.shape
    Hkv = kc.shape[1]
    G = Hq // Hkv
    Nh = kh.shape[0]
    if scale is None or scale <= 0:
        scale = 1.0 / math.sqrt(D)

    if rows is not None:
        rows = list(rows)
        o = np.zeros((len(rows), D), dtype=np.float64)
        lse = np.zeros(len(rows), dtype=np.float64)
        for r, (i, h) in enumerate(rows):
            g = h // G
            keys = np.concatenate([kh[:, g, :], kc[:i + 1, g, :]], axis=0)
            vals = np.concatenate([vh[:, g, :], vc[:i + 1, g, :]], axis=0)
            s = (keys @ q[i, h, :]) * scale
            m = s.max()
            p = np.exp(s - m)
            z = p.sum()
            o[r] = (p @ vals) / z
            lse[r] = m + math.log(z)
        return o, lse

    o = np.zeros((T, Hq, D), dtype=np.float64)
    lse = np.zeros((T, Hq), dtype=np.float64)
    causal = np.tril(np.ones((T, T), dtype=bool))
    for h in range(Hq):
        g = h // G
        s_h = (q[:, h, :] @ kh[:, g, :].T) * scale if Nh else np.zeros((T, 0))
        s_c = (q[:, h, :] @ kc[:, g, :].T) * scale
        s_c = np.where(causal, s_c, -np.inf)
        s = np.concatenate([s_h, s_c], axis=1)                    # [T, Nh + T]
        m = s.max(axis=1, keepdims=True)
        p = np.exp(s - m)
        z = p.sum(axis=1, keepdims=True)
        o[:, h, :] = (p[:, :Nh] @ vh[:, g, :] + p[:, Nh:] @ vc[:, g, :]) / z
        lse[:, h] = (m + np.log(z))[:, 0]
    return o, lse


# ---------------------------------------------------------------------------
# M -- selective migration, ordered-suffix mode
# ---------------------------------------------------------------------------
def migrate_suffix(k_cache, v_cache, keep_mask, page_size, min_pages_saved=1):
    """Pack only a suffix of the cache (Section 6.2, ordered-suffix mode).

    keep_mask [S] marks the live slots of the span [0, S).  Among the page-aligned suffix starts
    p = 0, P, 2P, ... the LARGEST one (the smallest suffix, found by scanning backward from the end)
    is taken whose packing shortens the page-rounded span by at least `min_pages_saved` pages:
        new_span(p) = p + #live slots in [p, S);   saved(p) = ceil(S / P) - ceil(new_span(p) / P).
    The live rows of [p, S) are packed, in order, to slots p, p+1, ...; every slot before p keeps its
    content and its hole pattern.  If no suffix qualifies nothing moves.  As-if semantics: all reads
    precede all writes.
    Returns dict(start (p, or -1 when nothing moves), k, v (caches of S rows after the move; rows at
    and beyond new_span are unspecified and returned unchanged), keep_mask (the new one), new_span,
    pages_saved, rows_moved, slot_map [S] (new slot of every live row, -1 for dead ones)).
    """
    keep = np.asarray(keep_mask).astype(bool)
    S, P = len(keep), int(page_size)
    pages = lambda n: (n + P - 1) // P
    start = -1
    for p in range(((S - 1) // P) * P if S else -P, -1, -P):            # backward from the last page
        live = int(keep[p:].sum())
        if pages(S) - pages(p + live) >= min_pages_saved:
            start = p
            break
    k = np.array(k_cache, copy=True) if k_cache is not None else None
    v = np.array(v_cache, copy=True) if v_cache is not None else None
    new_mask = keep.copy()
    slot_map = np.where(keep, np.arange(S), -1).astype(np.int32)
    if start < 0:
        return dict(start=-1, k=k, v=v, keep_mask=new_mask.astype(np.uint8), new_span=S, pages_saved=0, rows_moved=0,
                    slot_map=slot_map)
    src = start + np.nonzero(keep[start:])[0]
    dst = start + np.arange(len(src))
    if k is not None:
        k[dst] = np.asarray(k_cache)[src]
        v[dst] = np.asarray(v_cache)[src]
    new_mask[start:] = False
    new_mask[dst] = True
    slot_map[src] = dst
    new_span = start + len(src)
    return dict(start=start, k=k, v=v, keep_mask=new_mask.astype(np.uint8), new_span=new_span,
                pages_saved=pages(S) - pages(new_span), rows_moved=int((src != dst).sum()), slot_map=slot_map)


CLASS_MUST_KEEP, CLASS_SELECTED, CLASS_RECENT = 0, 1, 2      # allocation classes (Section 6.1)
CLASS_CANDIDATE = 0x80                                       # slot_class bit 7: entry retained from a partially evicted unit
PAGE_MIXED = 254


def migrate_class(k_cache, v_cache, keep_mask, slot_class, page_size, subblock, promote=True):
    """Class-aware selective migration (Section 6.2, "packing scattered entries" and "checking layout
    improvement"; the allocation classes are those of Section 6.1).

    keep_mask [S] marks the live slots after the logical deletion; slot_class [S] gives, for a live slot,
    its allocation class in the low two bits (0 must-keep, 1 selected-history, 2 recent-context) and in
    bit 7 whether the entry was retained from a partially evicted unit (a candidate).  Pages are P
    consecutive slots, subblocks B consecutive slots (B divides P).

    Plan.  Candidates are the live slots with bit 7 set whose page is not full when the plan starts (full
    pages stay in place), visited in ascending physical order.  A candidate at slot s of class c goes to the
    smallest slot d < s that is empty in the simulated layout at that moment (a hole of the starting layout not
    yet filled, or a slot vacated by an earlier move of the plan) and whose page, in that simulated layout, is
    empty or holds entries of class c only; if there is none it stays.  Entries that are not candidates never
    move, and no entry moves twice.  A destination may be the source of an earlier move, so the copies are
    as-if all sources were read before any destination is written.
    Accept test.  The moves are simulated; a page (subblock) is active if it holds a live entry; the plan is
    accepted iff the number of active pages or the number of active subblocks decreases.  A rejected plan
    moves nothing.
    Promotion (Section 6.1): after an accepted plan every full page whose entries are all of the classes
    selected-history / recent-context becomes selected-history (its entries' class is rewritten to 1).

    Returns dict(accepted, moves [(src, dst)], k, v, keep_mask, slot_class (of the new layout; dead slots 0),
    page_class [n_pages] (class of a page's entries, PAGE_MIXED, PAGE_EMPTY), pages_before, pages_after,
    subblocks_before, subblocks_after, n_candidates).
    """
    keep = np.asarray(keep_mask).astype(bool).copy()
    cls = np.where(keep, np.asarray(slot_class).astype(np.uint8), 0).astype(np.uint8)
    S, P, B = len(keep), int(page_size), int(subblock)
    assert P % B == 0
    n_pages = (S + P - 1) // P
    page_of = np.arange(S) // P

    def active(mask, size):
        n = (S + size - 1) // size
        return int(np.count_nonzero(np.bincount(np.arange(S)[mask] // size, minlength=n))) if S else 0

    pages_before, sub_before = active(keep, P), active(keep, B)
    # simulated layout
    live = keep.copy()
    c_now = cls.copy()
    page_fill0 = np.bincount(page_of[keep], minlength=n_pages)
    page_len = np.minimum(P, S - np.arange(n_pages) * P)            # the last page may be short
    cnt = np.zeros((n_pages, 3), np.int64)                          # live entries per page and class
    for c in range(3):
        cnt[:, c] = np.bincount(page_of[keep & ((cls & 3) == c)], minlength=n_pages)
    cand = [s for s in np.nonzero(keep & ((cls & CLASS_CANDIDATE) != 0))[0] if page_fill0[s // P] < page_len[s // P]]
    moves = []
    for s in cand:
        c = int(cls[s] & 3)
        others = cnt.sum(axis=1) - cnt[:, c]
        ok_page = others == 0                                       # empty, or class c only
        dst_ok = ~live[:s] & ok_page[page_of[:s]]
        hit = np.nonzero(dst_ok)[0]
        if len(hit) == 0:
            continue
        d = int(hit[0])
        moves.append((int(s), d))
        live[s], live[d] = False, True
        c_now[d], c_now[s] = c_now[s], 0
        cnt[s // P, c] -= 1
        cnt[d // P, c] += 1
    pages_after, sub_after = active(live, P), active(live, B)
    accepted = bool(moves) and (pages_after < pages_before or sub_after < sub_before)
    k = np.array(k_cache, copy=True) if k_cache is not None else None
    v = np.array(v_cache, copy=True) if v_cache is not None else None
    if not accepted:
        live, c_now, moves_done = keep, cls, []
        pages_after, sub_after = pages_before, sub_before
    else:
        moves_done = moves
        if k is not None and moves:
            src = np.array([m[0] for m in moves]); dst = np.array([m[1] for m in moves])
            k[dst] = np.asarray(k_cache)[src]                       # sources are read from the starting layout
            v[dst] = np.asarray(v_cache)[src]
    c_out = c_now.copy()
    page_class = np.full(n_pages, PAGE_EMPTY, np.uint8)
    for p in range(n_pages):
        sl = slice(p * P, min(S, (p + 1) * P))
        m = live[sl]
        if not m.any():
            continue
        kinds = np.unique(c_out[sl][m] & 3)
        if accepted and promote and m.all() and len(m) == P and kinds.min() >= CLASS_SELECTED:
            c_out[sl] = (c_out[sl] & ~np.uint8(3)) | np.uint8(CLASS_SELECTED)
            kinds = np.array([CLASS_SELECTED])
        page_class[p] = kinds[0] if len(kinds) == 1 else PAGE_MIXED
    return dict(accepted=accepted, moves=moves_done, k=k, v=v, keep_mask=live.astype(np.uint8), slot_class=c_out,
                page_class=page_class, pages_before=pages_before, pages_after=pages_after,
                subblocks_before=sub_before, subblocks_after=sub_after, n_candidates=len(cand))


def chunk_attention_masked(q, k_cache, v_cache, keep_mask, k_chunk, v_chunk, scale=None, rows=None):
    """Attention over a history with holes: only the live slots are visible (Section 6, "Fragmentation
    after logical eviction": masked entries are not attended to).  By definition this is dense
    attention over the live rows in order."""
    live = np.asarray(keep_mask).astype(bool)
    n = len(live)
    return chunk_attention(q, np.asarray(k_cache)[:n][live], np.asarray(v_cache)[:n][live], k_chunk, v_chunk, scale, rows)


# ---------------------------------------------------------------------------
# R -- RoPE position re-index of moved keys
# ---------------------------------------------------------------------------
def rope_reindex(k_rows, delta, theta_base=10000.0, n_dims=None):
    """Rotate key rows by a position shift (Section 5.2: "the runtime applies the corresponding RoPE
    adjustment to cached keys").

    k_rows [n, Hkv, D]; delta [n] integer position shifts (new position - old position).  Half-split
    pairing: dimension i pairs with i + n_dims/2, i < n_dims/2, angle delta * theta_base**(-2i/n_dims);
    dimensions >= n_dims are left alone.  float64 arithmetic; returns float64 [n, Hkv, D].
    """
    k = _f64(k_rows).copy()
    n, hkv, d = k.shape
    nd = d if n_dims is None else int(n_dims)
    half = nd // 2
    inv_freq = float(theta_base) ** (-2.0 * np.arange(half, dtype=np.float64) / nd)
    ang = np.asarray(delta, dtype=np.float64)[:, None] * inv_freq[None, :]            # [n, half]
    c, s_ = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    x, y = k[:, :, :half].copy(), k[:, :, half:nd].copy()
    k[:, :, :half] = x * c - y * s_
    k[:, :, half:nd] = x * s_ + y * c
    return k


def compact_pack_rope(k_cache, v_cache, keep_mask, theta_base=10000.0, n_dims=None):
    """Eager pack with the keys re-rotated to their new positions (position == slot index before and
    after): returns (k [n, Hkv, D] float64 before storage rounding, v rows unchanged, delta [n])."""
    keep = np.asarray(keep_mask).astype(bool)
    src = np.nonzero(keep)[0]
    delta = np.arange(len(src)) - src
    return rope_reindex(np.asarray(k_cache)[src], delta, theta_base, n_dims), np.asarray(v_cache)[src], delta


# ---------------------------------------------------------------------------
# one pass of the whole path
# ---------------------------------------------------------------------------
def stream_step(q, k_cache, v_cache, units, k_chunk, v_chunk, chunk_units, w_modality, budget,
                n_recent_events, modality_cap, page_size, scale=None, scores_override=None):
    """score -> select -> compact -> append -> attend, for one chunk and one layer.
    k_cache/v_cache hold exactly the history rows [N, Hkv, D]."""
    units = np.asarray(units)
    n_hist = int(units[:, U_LEN].sum())
    if scores_override is None:
        score, mass = score_units(q, k_cache[:n_hist], units, w_modality, scale)
    else:
        score, mass = np.asarray(scores_override), None
    sel = select_units(units, score, budget, n_recent_events, modality_cap)
    cp = compact_pack(k_cache[:n_hist], v_cache[:n_hist], sel["keep_mask"], page_size, sel["units_out"])
    o, lse = chunk_attention(q, cp["k"], cp["v"], k_chunk, v_chunk, scale)
    units_new = append_chunk(sel["units_out"], cp["n_kept"], chunk_units)
    k_new = np.concatenate([cp["k"], np.asarray(k_chunk)], axis=0)
    v_new = np.concatenate([cp["v"], np.asarray(v_chunk)], axis=0)
    return dict(score=score, mass=mass, select=sel, compact=cp, o=o, lse=lse,
                units=units_new, k_cache=k_new, v_cache=v_new)


def stream_step_structural(q, k_cache, v_cache, units, k_chunk, v_chunk, chunk_units, high_watermark, low_watermark,
                           n_recent_events, sink_prefix, text_budget, page_size, scale=None):
    """The pass as the paper runs it: plan from metadata -> compact -> append -> attend (no scoring)."""
    units = np.asarray(units)
    n_hist = int(units[:, U_LEN].sum())
    plan = plan_structural(units, high_watermark, low_watermark, n_recent_events, sink_prefix, text_budget)
    cp = compact_pack(k_cache[:n_hist], v_cache[:n_hist], plan["keep_mask"], page_size, plan["units_out"])
    o, lse = chunk_attention(q, cp["k"], cp["v"], k_chunk, v_chunk, scale)
    units_new = append_chunk(plan["units_out"], cp["n_kept"], chunk_units)
    k_new = np.concatenate([cp["k"], np.asarray(k_chunk)], axis=0)
    v_new = np.concatenate([cp["v"], np.asarray(v_chunk)], axis=0)
    return dict(plan=plan, compact=cp, o=o, lse=lse, units=units_new, k_cache=k_new, v_cache=v_new)
