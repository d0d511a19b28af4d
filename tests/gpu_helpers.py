"""Helpers shared by the GPU parity tests: move a workload to the device and call the C ABI."""
import numpy as np
import torch

from paper_2609_34653_b200 import binding as ob


def make_ctx(w, s_cap=None, u_cap=None, t_cap=None):
    return ob.Context(w.h_q, w.h_kv, w.d, w.dtype, s_cap or max(w.n_hist + w.t, 16),
                      u_cap or (len(w.units) + len(w.chunk_units) + 4), t_cap or w.t)


def i32(v):
    return torch.tensor([int(v)], dtype=torch.int32, device="cuda")


def gpu_score(ctx, w, q=None, k=None, units=None, n_units=None, use_dev_counts=True, w_mod=None):
    q = ob.to_device(w.q, w.dtype) if q is None else q
    k = ob.to_device(w.k_hist, w.dtype) if k is None else k
    units_np = w.units if units is None else units
    U = len(units_np)
    n = int(units_np[:, 1].sum())
    du = ob.units_to_device(units_np)
    scores = torch.full((U,), -7.0, dtype=torch.float32, device="cuda")
    mass = torch.full((U,), -7.0, dtype=torch.float32, device="cuda")
    ctx.score_units(q, q.shape[0], k, i32(n) if use_dev_counts else None, n, du, i32(U) if use_dev_counts else None, U,
                    w_mod or w.w_modality, 0.0, scores, mass)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    return scores.cpu().numpy(), mass.cpu().numpy()


def gpu_select(ctx, units_np, scores_np, budget, R, caps, n_hist_cap=None):
    U = len(units_np)
    n = int(units_np[:, 1].sum())
    du = ob.units_to_device(units_np)
    ds = torch.from_numpy(np.asarray(scores_np, dtype=np.float32)).cuda()
    unit_keep = torch.full((U + 16,), 9, dtype=torch.uint8, device="cuda")
    cap = n_hist_cap or n
    keep_mask = torch.full((cap + 16,), 9, dtype=torch.uint8, device="cuda")
    n_kept = i32(-1)
    n_units_out = i32(-1)
    units_out = torch.zeros((U, 6), dtype=torch.int32, device="cuda")
    ctx.select_units(du, i32(U), U, ds, ob.select_params(budget, R, caps), unit_keep, keep_mask, cap, n_kept,
                     units_out, n_units_out)
    torch.cuda.synchronize()
    status = ctx.poll_status()
    nu = int(n_units_out.item())
    return dict(unit_keep=unit_keep[:U].cpu().numpy(), keep_mask=keep_mask[:n].cpu().numpy(),
                n_kept=int(n_kept.item()), units_out=units_out[:max(nu, 0)].cpu().numpy(), n_units_out=nu,
                status=status, keep_mask_dev=keep_mask, units_out_dev=units_out, n_units_out_dev=n_units_out)


def gpu_compact(ctx, k, v, mask_np, page, units_out_np=None, in_place=False, s_span_max=None, want_pages=True):
    S = len(mask_np)
    smax = s_span_max or S
    mask = torch.zeros((smax + 16,), dtype=torch.uint8, device="cuda")
    mask[:S] = torch.from_numpy(np.asarray(mask_np, dtype=np.uint8)).cuda()
    if smax > S:
        mask[S:smax] = 1           # stale bytes beyond the device-side span must be ignored
    kd = k if in_place else torch.full_like(k, 0)
    vd = v if in_place else torch.full_like(v, 0)
    slot_map = torch.full((smax + 16,), -5, dtype=torch.int32, device="cuda")
    info = torch.full((8,), -5, dtype=torch.int32, device="cuda")
    n_pages = (smax + page - 1) // page
    page_class = torch.full((n_pages + 16,), 7, dtype=torch.uint8, device="cuda") if want_pages else None
    du = nu = None
    U = 0
    if units_out_np is not None and len(units_out_np):
        U = len(units_out_np)
        du = ob.units_to_device(units_out_np)
        nu = i32(U)
    ctx.compact(k, v, kd, vd, mask, i32(S), smax, page, du, nu, max(U, 1), slot_map, info, page_class)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    out = ob.info_to_dict(info)
    out.update(k=kd, v=vd, slot_map=slot_map[:S].cpu().numpy(),
               page_class=page_class[:n_pages].cpu().numpy() if want_pages else None)
    return out


def gpu_attention(ctx, w, k_hist, v_hist, n_hist, out_fp32=True, n_hist_max=None, q=None, k_chunk=None, v_chunk=None,
                  want_lse=True):
    q = ob.to_device(w.q, w.dtype) if q is None else q
    kc = ob.to_device(w.k_chunk, w.dtype) if k_chunk is None else k_chunk
    vc = ob.to_device(w.v_chunk, w.dtype) if v_chunk is None else v_chunk
    T = q.shape[0]
    o = torch.full((T, w.h_q, w.d), float("nan"), dtype=torch.float32 if out_fp32 else torch.bfloat16, device="cuda")
    lse = torch.full((T, w.h_q), float("nan"), dtype=torch.float32, device="cuda") if want_lse else None
    nmax = n_hist if n_hist_max is None else n_hist_max
    ctx.chunk_attention(q, T, k_hist, v_hist, i32(n_hist) if n_hist_max is not None else None, nmax, kc, vc, 0.0, o,
                        ob.DTYPE_FP32 if out_fp32 else ob.DTYPE_BF16, lse)
    torch.cuda.synchronize()
    assert ctx.poll_status() == 0
    return o.float().cpu().numpy(), (lse.cpu().numpy() if want_lse else None)


def bytes_of(t):
    return t.contiguous().view(torch.uint8).cpu().numpy()


def gpu_compact_units(ctx, k, v, units_np, unit_keep_np, page, units_out_np=None, in_place=False, s_span_max=None,
                      u_max=None, want_slot_map=True, kept_len_np=None):
    """omnipage_compact_units on a history unit table and one keep code per unit."""
    U = len(units_np)
    S = int(units_np[:, 1].sum()) if U else 0
    smax = s_span_max or S
    umax = u_max or max(U, 1)
    du = ob.units_to_device(units_np, umax)
    keep = torch.full((umax + 16,), 2, dtype=torch.uint8, device="cuda")      # stale codes beyond n_units are ignored
    if U:
        keep[:U] = torch.from_numpy(np.asarray(unit_keep_np, dtype=np.uint8)).cuda()
    kd = k if in_place else torch.full_like(k, 0)
    vd = v if in_place else torch.full_like(v, 0)
    slot_map = torch.full((smax + 16,), -5, dtype=torch.int32, device="cuda") if want_slot_map else None
    info = torch.full((8,), -5, dtype=torch.int32, device="cuda")
    n_pages = (smax + page - 1) // page
    page_class = torch.full((n_pages + 16,), 7, dtype=torch.uint8, device="cuda")
    dk = nk = None
    if units_out_np is not None and len(units_out_np):
        dk = ob.units_to_device(units_out_np, umax)
        nk = i32(len(units_out_np))
    klen = None
    if kept_len_np is not None:
        klen = torch.full((umax + 16,), 10 ** 6, dtype=torch.int32, device="cuda")      # stale entries beyond n_units are ignored
        klen[:U] = torch.from_numpy(np.asarray(kept_len_np, dtype=np.int32)).cuda()
    ctx.compact_units(k, v, kd, vd, du, i32(U), umax, keep, smax, page, dk, nk, slot_map, info, page_class, unit_kept_len=klen)
    torch.cuda.synchronize()
    status = ctx.poll_status()
    out = ob.info_to_dict(info)
    out.update(k=kd, v=vd, slot_map=slot_map[:S].cpu().numpy() if want_slot_map else None,
               page_class=page_class[:n_pages].cpu().numpy(), status=status)
    return out


def gpu_plan_structural(ctx, units_np, H_, L_, R, sink, Tb, want_mask=True, use_dev_count=True):
    U = len(units_np)
    n = int(units_np[:, 1].sum())
    du = ob.units_to_device(units_np, U + 3)
    unit_keep = torch.full((U + 19,), 9, dtype=torch.uint8, device="cuda")
    kept_len = torch.full((U + 19,), -9, dtype=torch.int32, device="cuda")
    keep_mask = torch.full((n + 32,), 9, dtype=torch.uint8, device="cuda") if want_mask else None
    n_kept, n_units_out = i32(-1), i32(-1)
    units_out = torch.zeros((U + 3, 6), dtype=torch.int32, device="cuda")
    ctx.plan_structural(du, i32(U) if use_dev_count else None, U if not use_dev_count else U + 3,
                        ob.structural_params(H_, L_, R, sink, Tb), unit_keep, kept_len, keep_mask, n, n_kept, units_out,
                        n_units_out)
    torch.cuda.synchronize()
    nu = int(n_units_out.item())
    return dict(unit_keep=unit_keep[:U].cpu().numpy(), unit_kept_len=kept_len[:U].cpu().numpy(),
                keep_mask=keep_mask[:n].cpu().numpy() if want_mask else None, n_kept=int(n_kept.item()),
                units_out=units_out[:max(nu, 0)].cpu().numpy(), status=ctx.poll_status(),
                unit_keep_dev=unit_keep, kept_len_dev=kept_len, units_out_dev=units_out, n_units_out_dev=n_units_out)
