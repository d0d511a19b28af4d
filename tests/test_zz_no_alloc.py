"""The context-free scoring entry point, for hosts that may not call cudaMalloc (a serving runtime
whose KV pool owns all of HBM, or a loop that cannot afford cudaMalloc's device-wide sync).

Collected last on purpose: a failure here must not hide any other test in a run that stops at the
first failure.  It calls the new entry point through the C ABI twice in a row, on different inputs,
and checks each result against the existing omnitide_score_units within the scoring tolerance used
by the other GPU tests; the second call proves that the shared, fixed scratch array is cleared.
"""
import numpy as np
import pytest
import torch

from paper_2609_34653_b200 import workloads as wl

pytestmark = pytest.mark.gpu
SCORE_REL = 1e-3


def _existing(ob, w):
    ctx = ob.Context(w.h_q, w.h_kv, w.d, w.dtype, w.n_hist + 64, len(w.units) + 4, w.t)
    q, k = ob.to_device(w.q, w.dtype), ob.to_device(w.k_hist, w.dtype)
    du = ob.units_to_device(w.units)
    U = len(w.units)
    s = torch.zeros(U, dtype=torch.float32, device="cuda")
    m = torch.zeros(U, dtype=torch.float32, device="cuda")
    ctx.score_units(q, w.t, k, None, w.n_hist, du, None, U, w.w_modality, 0.0, s, m)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    ctx.close()
    return s.cpu().numpy(), m.cpu().numpy()


def _no_alloc(ob, w):
    q, k = ob.to_device(w.q, w.dtype), ob.to_device(w.k_hist, w.dtype)
    du = ob.units_to_device(w.units)
    U = len(w.units)
    s = torch.full((U,), -3.0, dtype=torch.float32, device="cuda")
    m = torch.full((U,), -3.0, dtype=torch.float32, device="cuda")
    before = torch.cuda.memory_allocated()
    ob.score_units_noalloc(w.h_q, w.h_kv, w.d, w.dtype, q, w.t, k, w.n_hist, du, U, w.w_modality, 0.0, s, m)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before
    return s.cpu().numpy(), m.cpu().numpy()


def _close(a, ref):
    return np.abs(a - ref).max() <= SCORE_REL * max(np.abs(ref).max(), 1e-30)


def test_no_alloc_scoring_matches_existing_entry_point_twice():
    from paper_2609_34653_b200 import binding as ob
    first = wl.small_mixed(41, d=128, n_units=13, max_len=350, t=140)            # tensor-core path as the reference
    second = wl.small_mixed(42, d=64, n_units=6, max_len=200, t=90, dtype="fp32")  # fewer units: stale sums would show
    for w in (first, second):
        s_ref, m_ref = _existing(ob, w)
        s, m = _no_alloc(ob, w)
        assert _close(s, s_ref) and _close(m, m_ref)
        assert abs(m.sum() - 1.0) < 1e-4
    # same inputs again: the array kept the previous sums, the call must have cleared them
    s2, m2 = _no_alloc(ob, second)
    s_ref, m_ref = _existing(ob, second)
    assert _close(s2, s_ref) and _close(m2, m_ref)


def test_no_alloc_rejects_more_units_than_the_fixed_scratch():
    from paper_2609_34653_b200 import binding as ob
    w = wl.small_mixed(43, d=64, n_units=5, max_len=50, t=16)
    q, k = ob.to_device(w.q, w.dtype), ob.to_device(w.k_hist, w.dtype)
    du = ob.units_to_device(w.units, ob.NOALLOC_MAX_UNITS + 8)
    s = torch.zeros(ob.NOALLOC_MAX_UNITS + 8, dtype=torch.float32, device="cuda")
    with pytest.raises(ob.OmniTideError, match="CAPACITY"):
        ob.score_units_noalloc(w.h_q, w.h_kv, w.d, w.dtype, q, w.t, k, w.n_hist, du, ob.NOALLOC_MAX_UNITS + 1,
                               w.w_modality, 0.0, s)
