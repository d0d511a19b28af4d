"""ctypes binding of libomnitide.so: argument marshalling only.

Every step of the path runs in the library's CUDA kernels; this module only turns torch CUDA
tensors into raw device pointers, passes the current stream, and raises on a non-zero status.
There is no fallback: if the shared library is missing the import of this module fails.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libomnitide.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_CUDA, ERR_TIMEOUT, ERR_CAPACITY = range(6)
DEV_TIMEOUT, DEV_BAD_UNITS, DEV_BAD_COUNT = 1, 2, 4
DTYPE_BF16, DTYPE_FP32 = 0, 1
OPT_FORCE_CUDA_CORES = 1
OPT_SCORE_WINDOW = 2
OPT_HIGH_WATERMARK = 3
_STATUS_NAMES = {1: "INVALID_ARG", 2: "UNSUPPORTED", 3: "CUDA_ERROR", 4: "TIMEOUT", 5: "CAPACITY"}


class Geometry(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("h_q", "h_kv", "d", "dtype", "s_cap", "u_cap", "t_cap")]


class SelectParams(C.Structure):
    _fields_ = [("budget", C.c_int32), ("n_recent_events", C.c_int32), ("modality_cap", C.c_int32 * 3)]


class StructuralParams(C.Structure):
    _fields_ = [("high_watermark", C.c_int32), ("low_watermark", C.c_int32), ("n_recent_events", C.c_int32),
                ("sink_prefix", C.c_int32 * 3), ("text_budget", C.c_int32)]


class RopeParams(C.Structure):
    _fields_ = [("theta_base", C.c_float), ("n_dims", C.c_int32)]


class CompactInfo(C.Structure):
    _fields_ = [("n_kept", C.c_int32), ("span_pages", C.c_int32), ("rows_moved", C.c_int32),
                ("part_begin", C.c_int32 * 4), ("reserved", C.c_int32)]


class ClassInfo(C.Structure):
    _fields_ = [("accepted", C.c_int32), ("n_moves", C.c_int32), ("n_candidates", C.c_int32),
                ("pages_before", C.c_int32), ("pages_after", C.c_int32),
                ("subblocks_before", C.c_int32), ("subblocks_after", C.c_int32), ("reserved", C.c_int32)]


EXPORTS = [
    "omnitide_create", "omnitide_destroy", "omnitide_poll_status", "omnitide_last_error",
    "omnitide_score_units", "omnitide_select_units", "omnitide_plan_structural", "omnipage_compact", "omnipage_migrate_suffix", "omnipage_migrate_class", "omnipage_compact_units", "omnipage_compact_units_rope", "omnipage_compact_units_batched", "omnipage_append",
    "omnitide_chunk_attention", "omnitide_chunk_attention_masked", "omnitide_chunk_step", "omnitide_chunk_step_host", "omnitide_chunk_step_host_pipelined", "omnitide_host_wait", "omnitide_chunk_step_structural",
    "omnitide_set_option", "omnitide_launch_count", "omnitide_score_units_noalloc",
]
NOALLOC_MAX_UNITS = 1024


def load_library(path: str = LIB_PATH) -> C.CDLL:
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python -m paper_2609_34653_b200.build` "
            "(there is no CPU or PyTorch fallback for the OmniTide hot path)")
    lib = C.CDLL(path)
    vp, i32, f32 = C.c_void_p, C.c_int32, C.c_float
    lib.omnitide_create.argtypes = [C.POINTER(vp), C.POINTER(Geometry)]
    lib.omnitide_destroy.argtypes = [vp]
    lib.omnitide_poll_status.argtypes = [vp, vp, C.POINTER(i32)]
    lib.omnitide_last_error.argtypes = [vp]
    lib.omnitide_last_error.restype = C.c_char_p
    lib.omnitide_set_option.argtypes = [vp, i32, i32]
    lib.omnitide_launch_count.argtypes = [vp]
    lib.omnitide_launch_count.restype = C.c_int64
    lib.omnitide_score_units.argtypes = [vp, vp, vp, i32, vp, vp, i32, vp, vp, i32, C.POINTER(f32), f32, vp, vp]
    lib.omnitide_select_units.argtypes = [vp, vp, vp, vp, i32, vp, C.POINTER(SelectParams), vp, vp, i32, vp, vp, vp]
    lib.omnipage_compact.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, vp, vp, i32, vp, vp, vp]
    lib.omnitide_plan_structural.argtypes = [vp, vp, vp, vp, i32, C.POINTER(StructuralParams), vp, vp, vp, i32, vp, vp, vp]
    lib.omnipage_migrate_suffix.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, vp, vp]
    lib.omnipage_migrate_class.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, vp, vp, vp]
    lib.omnipage_compact_units.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, vp, i32, i32, vp, vp, vp, vp, vp]
    lib.omnipage_compact_units_rope.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, vp, i32, i32, vp, vp, vp, vp, vp,
                                                C.POINTER(RopeParams)]
    lib.omnipage_compact_units_batched.argtypes = [vp, vp, vp, vp, vp, vp, i32, vp, vp, i32, vp, vp, i32, i32, vp, vp, vp,
                                                   vp, vp]
    lib.omnipage_append.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, vp, vp, vp, i32, vp, vp]
    lib.omnitide_chunk_attention.argtypes = [vp, vp, vp, i32, vp, vp, vp, i32, vp, vp, f32, vp, i32, vp]
    lib.omnitide_chunk_attention_masked.argtypes = [vp, vp, vp, i32, vp, vp, vp, vp, i32, vp, vp, f32, vp, i32, vp]
    lib.omnitide_score_units_noalloc.argtypes = [vp, i32, i32, i32, i32, vp, i32, vp, i32, vp, i32, C.POINTER(f32), f32,
                                                 vp, vp]
    step = [vp, vp, vp, vp, vp, i32, vp, i32, vp, vp, vp, i32, vp, vp, i32, C.POINTER(f32),
            C.POINTER(SelectParams), i32, f32, vp, vp, vp, vp, vp, vp, i32, vp]
    lib.omnitide_chunk_step.argtypes = step
    lib.omnitide_chunk_step_structural.argtypes = [vp, vp, vp, vp, vp, i32, vp, i32, vp, vp, vp, i32, vp, vp, i32,
                                                   C.POINTER(StructuralParams), i32, f32, vp, vp, vp, vp, vp, vp, i32, vp]
    lib.omnitide_chunk_step_host.argtypes = step
    lib.omnitide_chunk_step_host_pipelined.argtypes = step
    lib.omnitide_host_wait.argtypes = [vp]
    for name in EXPORTS:
        fn = getattr(lib, name)
        if name not in ("omnitide_last_error", "omnitide_launch_count"):
            fn.restype = i32
    return lib


class OmniTideError(RuntimeError):
    pass


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        if not t.is_cuda:
            raise ValueError("expected a CUDA tensor")
        if not t.is_contiguous():
            raise ValueError("expected a contiguous tensor")
        return C.c_void_p(t.data_ptr())
    return C.c_void_p(int(t))


def _host_ptr(a):
    if isinstance(a, torch.Tensor):
        if a.is_cuda or not a.is_contiguous():
            raise ValueError("expected a contiguous host tensor")
        return C.c_void_p(a.data_ptr())
    if isinstance(a, np.ndarray):
        if not a.flags["C_CONTIGUOUS"]:
            raise ValueError("expected a contiguous host array")
        return C.c_void_p(a.ctypes.data)
    return C.c_void_p(int(a))


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def structural_params(high_watermark, low_watermark, n_recent_events, sink_prefix, text_budget) -> StructuralParams:
    sp = [int(x) for x in sink_prefix] + [0] * (3 - len(sink_prefix))
    return StructuralParams(int(high_watermark), int(low_watermark), int(n_recent_events), (C.c_int32 * 3)(*sp[:3]),
                            int(text_budget))


def select_params(budget, n_recent_events=1, modality_cap=(-1, -1, -1)) -> SelectParams:
    return SelectParams(int(budget), int(n_recent_events), (C.c_int32 * 3)(*[int(c) for c in modality_cap]))


class Context:
    """One geometry on the current CUDA device.  Methods mirror the C entry points by name."""

    def __init__(self, h_q, h_kv, d, dtype, s_cap, u_cap, t_cap):
        self.lib = load_library()
        self.geometry = Geometry(h_q, h_kv, d, DTYPE_BF16 if dtype in ("bf16", DTYPE_BF16) else DTYPE_FP32,
                                 s_cap, u_cap, t_cap)
        self._ctx = C.c_void_p()
        st = self.lib.omnitide_create(C.byref(self._ctx), C.byref(self.geometry))
        if st != OK:
            raise OmniTideError(f"omnitide_create failed: {_STATUS_NAMES.get(st, st)}")

    def close(self):
        if self._ctx:
            self.lib.omnitide_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st, what):
        if st != OK:
            msg = self.lib.omnitide_last_error(self._ctx)
            raise OmniTideError(f"{what}: {_STATUS_NAMES.get(st, st)}: {msg.decode() if msg else ''}")

    def poll_status(self) -> int:
        out = C.c_int32(0)
        self._check(self.lib.omnitide_poll_status(self._ctx, _stream(), C.byref(out)), "omnitide_poll_status")
        return out.value

    def set_option(self, option, value):
        self._check(self.lib.omnitide_set_option(self._ctx, option, value), "omnitide_set_option")

    def launch_count(self) -> int:
        return int(self.lib.omnitide_launch_count(self._ctx))

    def score_units(self, q, t, k_cache, n_hist_dev, n_hist_max, units, n_units_dev, n_units_max, w_modality,
                    scale, scores_out, mass_out=None):
        w = (C.c_float * 3)(*[float(x) for x in w_modality])
        self._check(self.lib.omnitide_score_units(self._ctx, _stream(), _ptr(q), t, _ptr(k_cache), _ptr(n_hist_dev),
                                                  n_hist_max, _ptr(units), _ptr(n_units_dev), n_units_max, w,
                                                  float(scale), _ptr(scores_out), _ptr(mass_out)),
                    "omnitide_score_units")

    def select_units(self, units, n_units_dev, n_units_max, scores, params, unit_keep_out, keep_mask_out,
                     n_hist_max, n_kept_out, units_out, n_units_out):
        self._check(self.lib.omnitide_select_units(self._ctx, _stream(), _ptr(units), _ptr(n_units_dev), n_units_max,
                                                   _ptr(scores), C.byref(params), _ptr(unit_keep_out),
                                                   _ptr(keep_mask_out), n_hist_max, _ptr(n_kept_out), _ptr(units_out),
                                                   _ptr(n_units_out)), "omnitide_select_units")

    def plan_structural(self, units, n_units_dev, n_units_max, params, unit_keep_out, unit_kept_len_out, keep_mask_out,
                        n_hist_max, n_kept_out, units_out, n_units_out):
        self._check(self.lib.omnitide_plan_structural(self._ctx, _stream(), _ptr(units), _ptr(n_units_dev), n_units_max,
                                                      C.byref(params), _ptr(unit_keep_out), _ptr(unit_kept_len_out),
                                                      _ptr(keep_mask_out), n_hist_max, _ptr(n_kept_out), _ptr(units_out),
                                                      _ptr(n_units_out)), "omnitide_plan_structural")

    def compact(self, k_src, v_src, k_dst, v_dst, keep_mask, s_span_dev, s_span_max, page_size, units_kept,
                n_units_kept_dev, n_units_max, slot_map_out, info_out, page_class_out, mode=0):
        self._check(self.lib.omnipage_compact(self._ctx, _stream(), _ptr(k_src), _ptr(v_src), _ptr(k_dst), _ptr(v_dst),
                                              _ptr(keep_mask), _ptr(s_span_dev), s_span_max, page_size, mode,
                                              _ptr(units_kept), _ptr(n_units_kept_dev), n_units_max,
                                              _ptr(slot_map_out), _ptr(info_out), _ptr(page_class_out)),
                    "omnipage_compact")

    def migrate_suffix(self, k_cache, v_cache, keep_mask, s_span_dev, s_span_max, page_size, min_pages_saved, slot_map_out,
                       info_out):
        self._check(self.lib.omnipage_migrate_suffix(self._ctx, _stream(), _ptr(k_cache), _ptr(v_cache), _ptr(keep_mask),
                                                     _ptr(s_span_dev), s_span_max, page_size, min_pages_saved,
                                                     _ptr(slot_map_out), _ptr(info_out)), "omnipage_migrate_suffix")

    def migrate_class(self, k_cache, v_cache, keep_mask, slot_class, s_span_dev, s_span_max, page_size, subblock,
                      promote, moves_out, page_class_out, info_out):
        self._check(self.lib.omnipage_migrate_class(self._ctx, _stream(), _ptr(k_cache), _ptr(v_cache), _ptr(keep_mask),
                                                    _ptr(slot_class), _ptr(s_span_dev), s_span_max, page_size, subblock,
                                                    int(bool(promote)), _ptr(moves_out), _ptr(page_class_out),
                                                    _ptr(info_out)), "omnipage_migrate_class")

    def compact_units(self, k_src, v_src, k_dst, v_dst, units, n_units_dev, n_units_max, unit_keep, s_span_max,
                      page_size, units_kept, n_units_kept_dev, slot_map_out, info_out, page_class_out, unit_kept_len=None):
        self._check(self.lib.omnipage_compact_units(self._ctx, _stream(), _ptr(k_src), _ptr(v_src), _ptr(k_dst),
                                                    _ptr(v_dst), _ptr(units), _ptr(n_units_dev), n_units_max,
                                                    _ptr(unit_keep), _ptr(unit_kept_len), s_span_max, page_size, _ptr(units_kept),
                                                    _ptr(n_units_kept_dev), _ptr(slot_map_out), _ptr(info_out),
                                                    _ptr(page_class_out)),
                    "omnipage_compact_units")

    def compact_units_rope(self, k_src, v_src, k_dst, v_dst, units, n_units_dev, n_units_max, unit_keep, s_span_max,
                           page_size, units_kept, n_units_kept_dev, slot_map_out, info_out, page_class_out, theta_base,
                           n_dims, unit_kept_len=None):
        rp = RopeParams(float(theta_base), int(n_dims))
        self._check(self.lib.omnipage_compact_units_rope(
            self._ctx, _stream(), _ptr(k_src), _ptr(v_src), _ptr(k_dst), _ptr(v_dst), _ptr(units), _ptr(n_units_dev),
            n_units_max, _ptr(unit_keep), _ptr(unit_kept_len), s_span_max, page_size, _ptr(units_kept),
            _ptr(n_units_kept_dev), _ptr(slot_map_out), _ptr(info_out), _ptr(page_class_out), C.byref(rp)),
            "omnipage_compact_units_rope")

    def compact_units_batched(self, k_src_ptrs, v_src_ptrs, k_dst_ptrs, v_dst_ptrs, n_layers, units, n_units_dev,
                              n_units_max, unit_keep, s_span_max, page_size, units_kept, n_units_kept_dev, slot_map_out,
                              info_out, page_class_out, unit_kept_len=None):
        """k_src_ptrs ...: int64 CUDA tensors holding n_layers device pointers each."""
        self._check(self.lib.omnipage_compact_units_batched(
            self._ctx, _stream(), _ptr(k_src_ptrs), _ptr(v_src_ptrs), _ptr(k_dst_ptrs), _ptr(v_dst_ptrs), n_layers,
            _ptr(units), _ptr(n_units_dev), n_units_max, _ptr(unit_keep), _ptr(unit_kept_len), s_span_max, page_size,
            _ptr(units_kept), _ptr(n_units_kept_dev), _ptr(slot_map_out), _ptr(info_out), _ptr(page_class_out)),
            "omnipage_compact_units_batched")

    def append(self, k_cache, v_cache, n_kept_dev, k_chunk, v_chunk, t, units, n_units_dev, chunk_units,
               n_chunk_units, n_hist_out, n_units_out):
        self._check(self.lib.omnipage_append(self._ctx, _stream(), _ptr(k_cache), _ptr(v_cache), _ptr(n_kept_dev),
                                             _ptr(k_chunk), _ptr(v_chunk), t, _ptr(units), _ptr(n_units_dev),
                                             _ptr(chunk_units), n_chunk_units, _ptr(n_hist_out), _ptr(n_units_out)),
                    "omnipage_append")

    def chunk_attention(self, q, t, k_hist, v_hist, n_hist_dev, n_hist_max, k_chunk, v_chunk, scale, o_out,
                        out_dtype, lse_out=None):
        self._check(self.lib.omnitide_chunk_attention(self._ctx, _stream(), _ptr(q), t, _ptr(k_hist), _ptr(v_hist),
                                                      _ptr(n_hist_dev), n_hist_max, _ptr(k_chunk), _ptr(v_chunk),
                                                      float(scale), _ptr(o_out), out_dtype, _ptr(lse_out)),
                    "omnitide_chunk_attention")

    def chunk_attention_masked(self, q, t, k_hist, v_hist, hist_keep_mask, s_span_dev, s_span_max, k_chunk, v_chunk, scale,
                               o_out, out_dtype, lse_out=None):
        self._check(self.lib.omnitide_chunk_attention_masked(self._ctx, _stream(), _ptr(q), t, _ptr(k_hist), _ptr(v_hist),
                                                             _ptr(hist_keep_mask), _ptr(s_span_dev), s_span_max,
                                                             _ptr(k_chunk), _ptr(v_chunk), float(scale), _ptr(o_out),
                                                             out_dtype, _ptr(lse_out)),
                    "omnitide_chunk_attention_masked")

    def _step(self, fn, name, hp, q, k_chunk, v_chunk, t, chunk_units, n_chunk_units, k_cache, v_cache, n_hist_dev,
              n_hist_max, units, n_units_dev, n_units_max, w_modality, params, page_size, scale, k_cache_out,
              v_cache_out, units_out, n_hist_out, n_units_out, o_out, out_dtype, info_out):
        w = (C.c_float * 3)(*[float(x) for x in w_modality])
        self._check(fn(self._ctx, _stream(), hp(q), hp(k_chunk), hp(v_chunk), t, hp(chunk_units), n_chunk_units,
                       _ptr(k_cache), _ptr(v_cache), _ptr(n_hist_dev), n_hist_max, _ptr(units), _ptr(n_units_dev),
                       n_units_max, w, C.byref(params), page_size, float(scale), _ptr(k_cache_out), _ptr(v_cache_out),
                       _ptr(units_out), _ptr(n_hist_out), _ptr(n_units_out), hp(o_out), out_dtype, _ptr(info_out)),
                    name)

    def chunk_step_structural(self, q, k_chunk, v_chunk, t, chunk_units, n_chunk_units, k_cache, v_cache, n_hist_dev,
                              n_hist_max, units, n_units_dev, n_units_max, params, page_size, scale, k_cache_out,
                              v_cache_out, units_out, n_hist_out, n_units_out, o_out, out_dtype, info_out=None):
        self._check(self.lib.omnitide_chunk_step_structural(
            self._ctx, _stream(), _ptr(q), _ptr(k_chunk), _ptr(v_chunk), t, _ptr(chunk_units), n_chunk_units,
            _ptr(k_cache), _ptr(v_cache), _ptr(n_hist_dev), n_hist_max, _ptr(units), _ptr(n_units_dev), n_units_max,
            C.byref(params), page_size, float(scale), _ptr(k_cache_out), _ptr(v_cache_out), _ptr(units_out),
            _ptr(n_hist_out), _ptr(n_units_out), _ptr(o_out), out_dtype, _ptr(info_out)),
            "omnitide_chunk_step_structural")

    def chunk_step(self, *a, info_out=None):
        self._step(self.lib.omnitide_chunk_step, "omnitide_chunk_step", _ptr, *a, info_out)

    def chunk_step_host(self, *a, info_out=None):
        self._step(self.lib.omnitide_chunk_step_host, "omnitide_chunk_step_host", _host_ptr, *a, info_out)

    def chunk_step_host_pipelined(self, *a, info_out=None):
        self._step(self.lib.omnitide_chunk_step_host_pipelined, "omnitide_chunk_step_host_pipelined", _host_ptr, *a, info_out)

    def host_wait(self):
        self._check(self.lib.omnitide_host_wait(self._ctx), "omnitide_host_wait")


def score_units_noalloc(h_q, h_kv, d, dtype, q, t, k_cache, n_hist, units, n_units, w_modality, scale, scores_out,
                        mass_out=None, lib=None):
    """Context-free scoring for hosts that may not call cudaMalloc: the accumulators live in a fixed
    array inside the library (at most NOALLOC_MAX_UNITS units).  Calls sharing a device must not
    overlap on the GPU.  Argument marshalling only."""
    lib = lib or load_library()
    w = (C.c_float * 3)(*[float(x) for x in w_modality])
    st = lib.omnitide_score_units_noalloc(_stream(), h_q, h_kv, d, DTYPE_BF16 if dtype in ("bf16", DTYPE_BF16) else DTYPE_FP32,
                                          _ptr(q), t, _ptr(k_cache), n_hist, _ptr(units), n_units, w, float(scale),
                                          _ptr(scores_out), _ptr(mass_out))
    if st == ERR_CAPACITY:
        raise OmniTideError(f"omnitide_score_units_noalloc: CAPACITY: {n_units} units exceed the fixed scratch of "
                            f"{NOALLOC_MAX_UNITS} units")
    if st != OK:
        raise OmniTideError(f"omnitide_score_units_noalloc: {_STATUS_NAMES.get(st, st)}")


# ---- small helpers for tests and the benchmark (device memory plumbing only) -------------------
def units_to_device(units: np.ndarray, capacity: int | None = None) -> torch.Tensor:
    u = np.ascontiguousarray(units, dtype=np.int32).reshape(-1, 6)
    cap = capacity or len(u)
    out = torch.zeros((cap, 6), dtype=torch.int32, device="cuda")
    if len(u):
        out[:len(u)] = torch.from_numpy(u).cuda()
    return out


def to_device(x: np.ndarray, dtype: str) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(x))
    return t.cuda().to(torch.bfloat16 if dtype == "bf16" else torch.float32).contiguous()


def info_to_dict(info_tensor: torch.Tensor) -> dict:
    v = info_tensor.cpu().numpy().astype(np.int32).reshape(-1)
    return dict(n_kept=int(v[0]), span_pages=int(v[1]), rows_moved=int(v[2]), part_begin=v[3:7].tolist())
