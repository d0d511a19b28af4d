"""Seeded synthetic multimodal streams (inputs only).

This module builds the *inputs* that both the CUDA path and the CPU oracle
consume: unit tables and Q/K/V tensors shaped like the paper's streaming
workloads (640- and 2,304-token image frames and 10-25 tok/s audio, Table 1;
an ~80K-token history, Section 2.2).  It holds none of the method's
arithmetic (no scoring, selection, compaction or attention) and imports
neither the CUDA binding nor the oracle.

Unit table: int32 array [U, 6], one row per typed span, in logical (time)
order.  Columns (same order as the C struct ``omni_unit``):
  0 start     first token (history units: cache slot; chunk units: row in chunk)
  1 len       tokens
  2 modality  0 = video/image, 1 = audio, 2 = text
  3 event     id of the streaming event the span belongs to, non-decreasing
  4 group     0 = must-keep, 1 = selected-history, 2 = recent-context
  5 flags     opaque, carried through

Floating-point tensors are returned as float32 arrays whose values are
exactly representable in the workload's storage dtype (bf16 or fp32), so that
converting them to the storage dtype on either side is lossless.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

MOD_VIDEO, MOD_AUDIO, MOD_TEXT = 0, 1, 2
GRP_MUST_KEEP, GRP_SELECTED, GRP_RECENT = 0, 1, 2
UNIT_FIELDS = ("start", "len", "modality", "event", "group", "flags")
SEED_BASE = 34653 * 100


# --------------------------------------------------------------------------
# storage-dtype helpers (data preparation only)
# --------------------------------------------------------------------------
def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); returns float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if x.size >= (1 << 16):
        import torch  # same rounding, much faster than numpy integer ops on large arrays
        return torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    u = x.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    r = (u + bias) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are already bf16-representable."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------
# workload container
# --------------------------------------------------------------------------
@dataclass
class Workload:
    name: str
    h_q: int
    h_kv: int
    d: int
    dtype: str                 # "bf16" or "fp32"
    units: np.ndarray          # [U, 6] int32, history units
    chunk_units: np.ndarray    # [Uc, 6] int32, units of the incoming chunk (start relative to chunk)
    budget: int
    page_size: int
    n_recent_events: int
    w_modality: tuple = (1.0, 2.0, 2.0)
    modality_cap: tuple = (-1, -1, -1)
    q: np.ndarray = field(default=None, repr=False)        # [T, h_q, d]
    k_hist: np.ndarray = field(default=None, repr=False)   # [N, h_kv, d]
    v_hist: np.ndarray = field(default=None, repr=False)
    k_chunk: np.ndarray = field(default=None, repr=False)  # [T, h_kv, d]
    v_chunk: np.ndarray = field(default=None, repr=False)

    @property
    def n_hist(self) -> int:
        return int(self.units[:, 1].sum()) if len(self.units) else 0

    @property
    def t(self) -> int:
        return int(self.chunk_units[:, 1].sum())


def make_units(spans, group_of_first=GRP_MUST_KEEP, default_group=GRP_RECENT) -> np.ndarray:
    """spans: list of (len, modality, event).  Returns the [U, 6] table with running starts."""
    u = np.zeros((len(spans), 6), dtype=np.int32)
    pos = 0
    for i, (ln, mod, ev) in enumerate(spans):
        u[i] = (pos, ln, mod, ev, default_group, 0)
        pos += ln
    if len(spans) and group_of_first is not None:
        u[0, 4] = group_of_first
    return u


def _trim_oldest(spans, total, first_trimmable=1):
    """Shorten/remove the oldest non-prefix spans until the lengths sum to `total`."""
    spans = [list(s) for s in spans]
    excess = sum(s[0] for s in spans) - total
    i = first_trimmable
    while excess > 0:
        take = min(excess, spans[i][0])
        spans[i][0] -= take
        excess -= take
        i += 1
    return [tuple(s) for s in spans if s[0] > 0]


def _draw_qkv(rng, n, t, h_q, h_kv, d, dtype, key_scale_hist=None, key_scale_chunk=None,
              head_scale=None):
    def draw(shape):
        return rng.standard_normal(shape, dtype=np.float32)
    q = draw((t, h_q, d))
    k_hist = draw((n, h_kv, d))
    v_hist = draw((n, h_kv, d))
    k_chunk = draw((t, h_kv, d))
    v_chunk = draw((t, h_kv, d))
    if key_scale_hist is not None:
        k_hist *= key_scale_hist[:, None, None].astype(np.float32)
    if key_scale_chunk is not None:
        k_chunk *= key_scale_chunk[:, None, None].astype(np.float32)
    if head_scale is not None:
        k_hist *= head_scale[None, :, None].astype(np.float32)
        k_chunk *= head_scale[None, :, None].astype(np.float32)
    if dtype == "bf16":
        q, k_hist, v_hist, k_chunk, v_chunk = (round_to_bf16(a) for a in (q, k_hist, v_hist, k_chunk, v_chunk))
    return q, k_hist, v_hist, k_chunk, v_chunk


def _per_token_scale(units, per_unit):
    return np.repeat(per_unit, units[:, 1])


# --------------------------------------------------------------------------
# config 1: Tiny (fp32)
# --------------------------------------------------------------------------
def tiny(seed: int = SEED_BASE + 1) -> Workload:
    rng = np.random.Generator(np.random.PCG64(seed))
    spans = []
    for ev in range(4):
        spans += [(128, MOD_VIDEO, ev), (128, MOD_VIDEO, ev), (256, MOD_AUDIO, ev)]
    units = make_units(spans)
    chunk_units = make_units([(128, MOD_VIDEO, 4), (128, MOD_AUDIO, 4)], group_of_first=None)
    q, k_hist, v_hist, k_chunk, v_chunk = _draw_qkv(rng, 2048, 256, 4, 1, 64, "fp32")
    # sink tokens and one "important" older video unit get a +2.0 key bias
    k_hist[0:4] += np.float32(2.0)
    newest = units[:, 3].max()
    cand = [i for i in range(len(units))
            if units[i, 2] == MOD_VIDEO and i != 0 and units[i, 3] != newest]
    pick = cand[int(rng.integers(len(cand)))]
    s, ln = units[pick, 0], units[pick, 1]
    k_hist[s:s + ln] += np.float32(2.0)
    wl = Workload("tiny", 4, 1, 64, "fp32", units, chunk_units, budget=1024, page_size=16,
                  n_recent_events=1, q=q, k_hist=k_hist, v_hist=v_hist, k_chunk=k_chunk, v_chunk=v_chunk)
    wl.biased_unit = pick
    return wl


# --------------------------------------------------------------------------
# configs 2, 3, 5: one 32/8-head, head_dim-128 bf16 layer
# --------------------------------------------------------------------------
def _av_stream_spans(rng, frame, audio, total, text_every=None, text_len=32, text_poisson=None,
                     text_range=(16, 64), prefix=16):
    """Prefix text unit, then (video frame, audio segment) events with optional text events,
    generated until at least `total` tokens, then trimmed at the old end to exactly `total`."""
    spans = []
    ev = 0
    if prefix:
        spans.append((prefix, MOD_TEXT, ev))
        ev += 1
    n = prefix
    frames = 0
    while n < total:
        spans += [(frame, MOD_VIDEO, ev), (audio, MOD_AUDIO, ev)]
        n += frame + audio
        ev += 1
        frames += 1
        if text_every and frames % text_every == 0:
            spans.append((text_len, MOD_TEXT, ev))
            n += text_len
            ev += 1
        if text_poisson:
            for _ in range(int(rng.poisson(text_poisson))):
                ln = int(rng.integers(text_range[0], text_range[1] + 1))
                spans.append((ln, MOD_TEXT, ev))
                n += ln
                ev += 1
    return _trim_oldest(spans, total, first_trimmable=1 if prefix else 0)


def _layer_workload(name, rng, spans, chunk_spans, budget, page, sigma=0.5, head_t_nu=None,
                    h_q=32, h_kv=8, d=128, draw_values=True):
    units = make_units(spans, group_of_first=GRP_MUST_KEEP if spans[0][1] == MOD_TEXT else None)
    next_ev = int(units[:, 3].max()) + 1
    chunk_units = make_units([(ln, mod, next_ev) for ln, mod in chunk_spans], group_of_first=None)
    wl = Workload(name, h_q, h_kv, d, "bf16", units, chunk_units, budget=budget, page_size=page,
                  n_recent_events=1)
    if draw_values:
        z_hist = np.exp(sigma * rng.standard_normal(len(units))).astype(np.float32)
        z_chunk = np.exp(sigma * rng.standard_normal(len(chunk_units))).astype(np.float32)
        head_scale = None
        if head_t_nu is not None:
            head_scale = np.abs(rng.standard_t(head_t_nu, size=h_kv)).astype(np.float32)
        (wl.q, wl.k_hist, wl.v_hist, wl.k_chunk, wl.v_chunk) = _draw_qkv(
            rng, wl.n_hist, wl.t, h_q, h_kv, d, "bf16",
            key_scale_hist=_per_token_scale(units, z_hist),
            key_scale_chunk=_per_token_scale(chunk_units, z_chunk),
            head_scale=head_scale)
    return wl


def layer_8b(seed: int = SEED_BASE + 2, n_hist: int = 16384, budget: int = 4096, page: int = 64,
             draw_values: bool = True) -> Workload:
    """Config 2: 640-token frames + 50-token audio segments, a 32-token text unit every 8 frames."""
    rng = np.random.Generator(np.random.PCG64(seed))
    spans = _av_stream_spans(rng, 640, 50, n_hist, text_every=8, text_len=32)
    return _layer_workload("layer_8b", rng, spans, [(640, MOD_VIDEO), (50, MOD_AUDIO)], budget, page,
                           draw_values=draw_values)


def long_stream(seed: int = SEED_BASE + 3, n_hist: int = 80000, budget: int = 8192, page: int = 64,
                draw_values: bool = True) -> Workload:
    """Config 3: 2,304-token frames every 2 s, 50 audio tokens per 2 s, Poisson text units."""
    rng = np.random.Generator(np.random.PCG64(seed))
    spans = _av_stream_spans(rng, 2304, 50, n_hist, text_poisson=2.0 / 30.0)
    return _layer_workload("long_stream", rng, spans, [(2304, MOD_VIDEO), (50, MOD_AUDIO)], budget, page,
                           draw_values=draw_values)


def sweep_cell(t: int, ratio: float, page: int, cell: int = 0, n_hist: int = 131072,
               seed: int = SEED_BASE + 5, draw_values: bool = True) -> Workload:
    """Config 5: heavy-tailed per-head key scales (Student-t, nu=3), no text, no prefix."""
    rng = np.random.Generator(np.random.PCG64(seed + cell))
    spans = _av_stream_spans(rng, 2304, 50, n_hist, prefix=0)
    budget = int(np.floor(ratio * n_hist))
    chunk = [(t - 50, MOD_VIDEO), (50, MOD_AUDIO)]
    wl = _layer_workload(f"sweep_T{t}_r{ratio}_P{page}", rng, spans, chunk, budget, page, head_t_nu=3.0,
                         draw_values=draw_values)
    return wl


# --------------------------------------------------------------------------
# config 4: the chunk schedule of the 36-layer stream loop (shapes only; the
# per-layer Q/K/V values are drawn by the caller, on device for the bench)
# --------------------------------------------------------------------------
def loop_schedule(n_chunks: int = 400, seed: int = SEED_BASE + 4):
    """Returns a list of per-chunk unit tables [(Uc, 6) int32] with event ids 1..n_chunks.
    Event 0 is the 16-token must-keep prefix unit the cache starts with."""
    rng = np.random.Generator(np.random.PCG64(seed))
    out = []
    for c in range(n_chunks):
        frame = int(rng.choice([640, 1280, 2304]))
        rate = float(rng.uniform(10.0, 25.0))
        audio = int(round(2.0 * rate))
        cu = make_units([(frame, MOD_VIDEO, c + 1), (audio, MOD_AUDIO, c + 1)], group_of_first=None)
        out.append(cu)
    return out


def loop_prefix_units() -> np.ndarray:
    return make_units([(16, MOD_TEXT, 0)])


def random_layer_inputs(rng, units, chunk_units, h_q=32, h_kv=8, d=128, dtype="bf16", sigma=0.5):
    """Q/K/V for an arbitrary (units, chunk_units) pair with the per-unit log-normal key scale."""
    n = int(units[:, 1].sum())
    t = int(chunk_units[:, 1].sum())
    z_hist = np.exp(sigma * rng.standard_normal(len(units))).astype(np.float32)
    z_chunk = np.exp(sigma * rng.standard_normal(len(chunk_units))).astype(np.float32)
    return _draw_qkv(rng, n, t, h_q, h_kv, d, dtype,
                     key_scale_hist=_per_token_scale(units, z_hist),
                     key_scale_chunk=_per_token_scale(chunk_units, z_chunk))


def small_mixed(seed: int, n_units: int = 9, h_q: int = 4, h_kv: int = 2, d: int = 64,
                dtype: str = "bf16", max_len: int = 300, t: int = 200, budget_frac: float = 0.4,
                page: int = 16) -> Workload:
    """A small ragged case with odd unit lengths for parity tests (several tiles, ragged tails)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    spans = [(int(rng.integers(3, 24)), MOD_TEXT, 0)]
    ev = 1
    while len(spans) < n_units:
        spans.append((int(rng.integers(1, max_len + 1)), MOD_VIDEO, ev))
        if len(spans) < n_units:
            spans.append((int(rng.integers(1, max(2, max_len // 4))), MOD_AUDIO, ev))
        if rng.random() < 0.3 and len(spans) < n_units:
            ev += 1
            spans.append((int(rng.integers(1, 40)), MOD_TEXT, ev))
        ev += 1
    units = make_units(spans)
    ta = max(1, t // 5)
    chunk_units = make_units([(t - ta, MOD_VIDEO, ev), (ta, MOD_AUDIO, ev)], group_of_first=None)
    n = int(units[:, 1].sum())
    wl = Workload(f"small_mixed_{seed}", h_q, h_kv, d, dtype, units, chunk_units,
                  budget=max(1, int(budget_frac * n)), page_size=page, n_recent_events=1)
    wl.q, wl.k_hist, wl.v_hist, wl.k_chunk, wl.v_chunk = random_layer_inputs(
        rng, units, chunk_units, h_q, h_kv, d, dtype)
    return wl
