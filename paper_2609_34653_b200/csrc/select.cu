// Budgeted unit selection: one CTA ranks the candidate units (bitonic sort of 64-bit keys in
// shared memory), one thread replays the first-fit walk over the ranked list, and the whole CTA
// then writes the unit codes, the re-indexed unit table and the per-token keep mask.
#include "common.cuh"

namespace {

constexpr int SEL_THREADS = 1024;
constexpr int SEL_MAX_UNITS = 4096;

// Order-preserving map of a non-NaN float to uint32 (larger float -> larger code, -0 == +0);
// NaN maps to 0, below every number.
__device__ __forceinline__ uint32_t score_code(float f) {
    if (f != f) return 0u;
    if (f == 0.0f) f = 0.0f;                       // -0 -> +0
    uint32_t b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

struct SelectArgs {
    const omni_unit* units; const int32_t* n_units_dev; int n_units_max;
    const float* scores; omni_select_params p;
    uint8_t* unit_keep; uint8_t* keep_mask; int n_hist_max;
    int32_t* n_kept_out; omni_unit* units_out; int32_t* n_units_out; int32_t* status;
    int p2;     // power of two >= n_units_max
};

__device__ int block_sum(int v, int* red) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if (lane == 0) red[wid] = v;
    __syncthreads();
    int t = 0;
    for (int w = 0; w < SEL_THREADS / 32; ++w) t += red[w];
    __syncthreads();
    return t;
}

// Exclusive scan over vals[0..n) (n <= 4 * SEL_THREADS) in shared memory; returns the total.
__device__ int block_excl_scan(int* vals, int n, int* red) {
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int ipt = (n + SEL_THREADS - 1) / SEL_THREADS;
    const int lo = min(tid * ipt, n), hi = min(lo + ipt, n);
    int sum = 0;
    for (int i = lo; i < hi; ++i) sum += vals[i];
    int incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
    }
    __syncthreads();
    if (lane == 31) red[wid] = incl;
    __syncthreads();
    if (wid == 0) {
        int v = red[lane];
        int inc2 = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int y = __shfl_up_sync(0xffffffffu, inc2, o);
            if (lane >= o) inc2 += y;
        }
        red[lane] = inc2 - v;
        if (lane == 31) red[32] = inc2;
    }
    __syncthreads();
    int run = red[wid] + incl - sum;
    for (int i = lo; i < hi; ++i) {
        int v = vals[i];
        vals[i] = run;
        run += v;
    }
    const int total = red[32];
    __syncthreads();
    return total;
}

__global__ void __launch_bounds__(SEL_THREADS, 1) select_units_kernel(const SelectArgs a) {
    extern __shared__ unsigned long long sm_keys[];                 // [p2]
    int* s_len = reinterpret_cast<int*>(sm_keys + a.p2);            // [p2] len in ranked order / scan values
    int* s_aux = s_len + a.p2;                                      // [p2] modality in ranked order / new starts
    int* s_start = s_aux + a.p2;                                    // [p2 + 1] unit starts
    uint8_t* s_keep = reinterpret_cast<uint8_t*>(s_start + a.p2 + 1);   // [p2]
    __shared__ int red[33];
    __shared__ int s_thr_event, s_all_recent, s_bad;
    const int tid = threadIdx.x;

    int U = a.n_units_dev ? *a.n_units_dev : a.n_units_max;
    if (U < 0 || U > a.n_units_max) {
        if (tid == 0) atomicOr(a.status, OMNI_DEV_BAD_COUNT);
        U = max(0, min(U, a.n_units_max));
    }
    if (tid == 0) { s_bad = 0; s_all_recent = 0; s_thr_event = 0; }
    __syncthreads();

    // ---- validate the table; find the oldest of the newest R events ----------------------------
    for (int u = tid; u < U; u += SEL_THREADS) {
        const omni_unit un = a.units[u];
        s_start[u] = un.start;
        bool bad = un.len <= 0 || un.modality < 0 || un.modality > 2;
        if (u == 0) bad |= un.start != 0;
        if (u + 1 < U) {
            const omni_unit nx = a.units[u + 1];
            bad |= (nx.start != un.start + un.len) || (nx.event < un.event);
        }
        if (bad) s_bad = 1;
    }
    if (tid == 0) {
        const int R = a.p.n_recent_events;
        if (R <= 0 || U == 0) {
            s_all_recent = -1;                       // no unit is recent
        } else {
            int distinct = 1, u = U - 1, ev = a.units[U - 1].event;
            while (u > 0) {
                const int e2 = a.units[u - 1].event;
                if (e2 != ev) {
                    if (distinct == R) break;
                    ++distinct;
                    ev = e2;
                }
                --u;
            }
            s_thr_event = ev;                        // events >= ev are the newest `distinct` (<= R) events
        }
    }
    __syncthreads();
    const int n_hist = U ? a.units[U - 1].start + a.units[U - 1].len : 0;
    if (s_bad || n_hist > a.n_hist_max) {
        if (tid == 0) atomicOr(a.status, s_bad ? OMNI_DEV_BAD_UNITS : OMNI_DEV_BAD_COUNT);
        if (tid == 0) { *a.n_kept_out = 0; *a.n_units_out = 0; }
        return;
    }
    if (tid == 0) s_start[U] = n_hist;
    const bool any_recent = s_all_recent == 0;
    const int thr = s_thr_event;

    // ---- protected set, keys ----------------------------------------------------------------------
    int prot_len = 0;
    for (int u = tid; u < a.p2; u += SEL_THREADS) {
        unsigned long long key = 0ull;
        if (u < U) {
            const omni_unit un = a.units[u];
            const bool prot = un.group == OMNI_GROUP_MUST_KEEP || (any_recent && un.event >= thr);
            s_keep[u] = prot ? OMNI_KEEP_WHOLE : OMNI_KEEP_DROPPED;
            if (prot) prot_len += un.len;
            else key = (1ull << 63) | ((unsigned long long)score_code(a.scores[u]) << 31) | (unsigned long long)u;
        }
        sm_keys[u] = key;
    }
    const int used0 = block_sum(prot_len, red);

    if (used0 < a.p.budget) {
        // ---- rank candidates: bitonic sort, descending ---------------------------------------------
        for (int k = 2; k <= a.p2; k <<= 1) {
            for (int j = k >> 1; j > 0; j >>= 1) {
                __syncthreads();
                for (int i = tid; i < a.p2; i += SEL_THREADS) {
                    const int ixj = i ^ j;
                    if (ixj > i) {
                        const unsigned long long x = sm_keys[i], y = sm_keys[ixj];
                        const bool desc = (i & k) == 0;
                        if (desc ? (x < y) : (x > y)) { sm_keys[i] = y; sm_keys[ixj] = x; }
                    }
                }
            }
        }
        __syncthreads();
        for (int i = tid; i < U; i += SEL_THREADS) {
            const unsigned long long key = sm_keys[i];
            if (key >> 63) {
                const int u = (int)(key & 0x7fffffffull);
                s_len[i] = a.units[u].len;
                s_aux[i] = a.units[u].modality;
            } else {
                s_len[i] = -1;                       // end of candidates
            }
        }
        __syncthreads();
        // ---- first-fit walk (sequential by definition) ---------------------------------------------
        if (tid == 0) {
            int rem = a.p.budget - used0;
            int cap[3] = {a.p.modality_cap[0], a.p.modality_cap[1], a.p.modality_cap[2]};
            for (int i = 0; i < U; ++i) {
                const int ln = s_len[i];
                if (ln < 0) break;
                const int m = s_aux[i];
                if (ln <= rem && (cap[m] < 0 || ln <= cap[m])) {
                    rem -= ln;
                    if (cap[m] >= 0) cap[m] -= ln;
                    s_keep[(int)(sm_keys[i] & 0x7fffffffull)] = OMNI_KEEP_WHOLE;
                }
            }
        }
        __syncthreads();
    }

    // ---- re-index survivors ------------------------------------------------------------------------
    for (int u = tid; u < U; u += SEL_THREADS) {
        const bool kp = s_keep[u] != 0;
        s_len[u] = kp ? a.units[u].len : 0;       // kept tokens per unit
        s_aux[u] = kp ? 1 : 0;                    // kept flag
    }
    __syncthreads();
    const int n_kept = block_excl_scan(s_len, U, red);        // s_len[u] = kept tokens before unit u
    const int n_units_kept = block_excl_scan(s_aux, U, red);  // s_aux[u] = kept units before unit u
    for (int u = tid; u < U; u += SEL_THREADS) {
        const uint8_t kp = s_keep[u];
        a.unit_keep[u] = kp;
        if (kp) {
            omni_unit un = a.units[u];
            un.group = un.group == OMNI_GROUP_MUST_KEEP ? OMNI_GROUP_MUST_KEEP
                       : ((any_recent && un.event >= thr) ? OMNI_GROUP_RECENT : OMNI_GROUP_SELECTED);
            un.start = s_len[u];
            a.units_out[s_aux[u]] = un;
        }
    }
    if (tid == 0) { *a.n_kept_out = n_kept; *a.n_units_out = n_units_kept; }

    // ---- per-token keep mask, 16 bytes per thread step -----------------------------------------------
    if (a.keep_mask) {
        const int n_vec = (n_hist + 15) >> 4;
        for (int vi = tid; vi < n_vec; vi += SEL_THREADS) {
            const int pos = vi << 4;
            int lo = 0, hi = U;                   // largest u with s_start[u] <= pos
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (s_start[mid] <= pos) lo = mid; else hi = mid;
            }
            int u = lo;
            uint32_t w[4] = {0, 0, 0, 0};
            for (int b = 0; b < 16; ++b) {
                const int p = pos + b;
                if (p >= n_hist) break;
                while (p >= s_start[u + 1]) ++u;
                if (s_keep[u]) w[b >> 2] |= 1u << ((b & 3) * 8);
            }
            if (pos + 16 <= a.n_hist_max) {
                *reinterpret_cast<uint4*>(a.keep_mask + pos) = make_uint4(w[0], w[1], w[2], w[3]);
            } else {
                for (int b = 0; b < 16 && pos + b < n_hist; ++b) a.keep_mask[pos + b] = (w[b >> 2] >> ((b & 3) * 8)) & 0xff;
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------------
// Structure-aware, score-free retention planning (Section 5.1): metadata only.  One CTA: the per-span rules
// run in parallel (the text budget is a prefix sum in time order), the event walk of the drop phase is
// sequential by definition and runs on one thread over the event runs of the table.
struct PlanArgs {
    const omni_unit* units; const int32_t* n_units_dev; int n_units_max;
    omni_structural_params p;
    uint8_t* unit_keep; int32_t* unit_kept_len; uint8_t* keep_mask; int n_hist_max;
    int32_t* n_kept_out; omni_unit* units_out; int32_t* n_units_out; int32_t* status;
};

__global__ void __launch_bounds__(SEL_THREADS, 1) plan_structural_kernel(const PlanArgs a) {
    extern __shared__ int sm_plan[];
    const int cap = a.n_units_max;
    int* s_start = sm_plan;                 // [cap + 1]
    int* s_len = s_start + cap + 1;         // [cap]
    int* s_meta = s_len + cap;              // [cap]  modality | must << 8 | boundary << 9 | recent << 10
    int* s_event = s_meta + cap;            // [cap]
    int* s_kept = s_event + cap;            // [cap]  kept tokens per span
    int* s_scan = s_kept + cap;             // [cap + 1] scan scratch (text prefix sums, new starts)
    int* s_idx = s_scan + cap + 1;          // [cap + 1] kept spans before a span
    int* s_drop = s_idx + cap + 1;          // [cap]  1: the span's event is dropped in the last phase
    __shared__ int red[33];
    __shared__ int s_thr_event, s_all_recent, s_bad;
    const int tid = threadIdx.x;

    int U = a.n_units_dev ? *a.n_units_dev : a.n_units_max;
    if (U < 0 || U > a.n_units_max) {
        if (tid == 0) atomicOr(a.status, OMNI_DEV_BAD_COUNT);
        U = max(0, min(U, a.n_units_max));
    }
    if (tid == 0) { s_bad = 0; s_all_recent = 0; s_thr_event = 0; }
    __syncthreads();
    for (int u = tid; u < U; u += SEL_THREADS) {
        const omni_unit un = a.units[u];
        s_start[u] = un.start; s_len[u] = un.len; s_event[u] = un.event;
        s_meta[u] = (un.modality & 0xff) | ((un.group == OMNI_GROUP_MUST_KEEP) << 8) | ((un.flags & OMNI_FLAG_BOUNDARY) ? (1 << 9) : 0);
        s_drop[u] = 0;
        bool bad = un.len <= 0 || un.modality < 0 || un.modality > 2;
        if (u == 0) bad |= un.start != 0;
        if (u + 1 < U) {
            const omni_unit nx = a.units[u + 1];
            bad |= (nx.start != un.start + un.len) || (nx.event < un.event);
        }
        if (bad) s_bad = 1;
    }
    __syncthreads();
    const int n_hist = U ? s_start[U - 1] + s_len[U - 1] : 0;
    if (s_bad || n_hist > a.n_hist_max) {
        if (tid == 0) {
            atomicOr(a.status, s_bad ? OMNI_DEV_BAD_UNITS : OMNI_DEV_BAD_COUNT);
            *a.n_kept_out = 0; *a.n_units_out = 0;
        }
        return;
    }
    if (tid == 0) {
        s_start[U] = n_hist;
        // the oldest of the newest R events
        const int R = a.p.n_recent_events;
        if (R <= 0 || U == 0) {
            s_all_recent = -1;
        } else {
            int distinct = 1, u = U - 1, ev = s_event[U - 1];
            while (u > 0) {
                const int e2 = s_event[u - 1];
                if (e2 != ev) {
                    if (distinct == R) break;
                    ++distinct;
                    ev = e2;
                }
                --u;
            }
            s_thr_event = ev;
        }
    }
    __syncthreads();
    const bool any_recent = s_all_recent == 0;
    const int thr = s_thr_event;
    const bool round = n_hist > a.p.high_watermark;          // retention starts above the high watermark only

    // ---- per-span rules -----------------------------------------------------------------------------
    for (int u = tid; u < U; u += SEL_THREADS) {
        const int meta = s_meta[u], mod = meta & 0xff, ln = s_len[u];
        const bool recent = any_recent && s_event[u] >= thr;
        if (recent) s_meta[u] = meta | (1 << 10);
        const bool whole = !round || (meta & (1 << 8)) || recent || (meta & (1 << 9));
        int kept = ln, text = 0;
        if (!whole) {
            if (mod == OMNI_MOD_TEXT) text = ln;             // decided by the shared budget below
            else kept = min(ln, max(0, mod == OMNI_MOD_VIDEO ? a.p.sink_prefix[0] : a.p.sink_prefix[1]));
        }
        s_kept[u] = kept;
        s_scan[u] = text;
    }
    __syncthreads();
    if (round) {
        // older text spans, oldest first, while the running total fits the budget: the first misfit ends it
        block_excl_scan(s_scan, U, red);
        for (int u = tid; u < U; u += SEL_THREADS) {
            const int meta = s_meta[u];
            const bool older_text = !(meta & ((1 << 8) | (1 << 9) | (1 << 10))) && (meta & 0xff) == OMNI_MOD_TEXT;
            if (older_text && s_scan[u] + s_len[u] > a.p.text_budget) s_kept[u] = 0;
        }
        __syncthreads();
    }
    int my = 0;
    for (int u = tid; u < U; u += SEL_THREADS) my += s_kept[u];
    const int total0 = block_sum(my, red);

    // ---- drop whole events, oldest first, partially retained ones before complete ones ------------------
    if (round && total0 > a.p.low_watermark && tid == 0) {
        int total = total0, n_alive = 0;
        // pass 1: classify the event runs (s_scan[first span of the run] = kept tokens outside the prefix,
        // s_idx[first span] = 1 if partially retained)
        for (int u0 = 0; u0 < U;) {
            int u1 = u0, ev_kept = 0, partial = 0;
            while (u1 < U && s_event[u1] == s_event[u0]) {
                if (!(s_meta[u1] & (1 << 8))) { ev_kept += s_kept[u1]; partial |= s_kept[u1] < s_len[u1]; }
                ++u1;
            }
            s_scan[u0] = ev_kept;
            s_idx[u0] = partial;
            n_alive += ev_kept > 0;
            u0 = u1;
        }
        for (int cls = 1; cls >= 0; --cls) {
            for (int u0 = 0; u0 < U;) {
                int u1 = u0;
                while (u1 < U && s_event[u1] == s_event[u0]) ++u1;
                if (s_scan[u0] > 0 && s_idx[u0] == cls) {
                    if (total <= a.p.low_watermark || n_alive <= 1) { cls = -1; break; }
                    total -= s_scan[u0];
                    --n_alive;
                    for (int u = u0; u < u1; ++u) s_drop[u] = 1;
                }
                u0 = u1;
            }
        }
    }
    __syncthreads();

    // ---- codes, re-indexed survivors ---------------------------------------------------------------------
    for (int u = tid; u < U; u += SEL_THREADS) {
        if (s_drop[u] && !(s_meta[u] & (1 << 8))) s_kept[u] = 0;
        s_scan[u] = s_kept[u];
        s_idx[u] = s_kept[u] > 0;
    }
    __syncthreads();
    const int n_kept = block_excl_scan(s_scan, U, red);       // s_scan[u] = kept tokens before span u
    const int n_units_kept = block_excl_scan(s_idx, U, red);  // s_idx[u] = kept spans before span u
    for (int u = tid; u < U; u += SEL_THREADS) {
        const int kept = s_kept[u], ln = s_len[u], meta = s_meta[u];
        a.unit_keep[u] = kept == 0 ? OMNI_KEEP_DROPPED : (kept == ln ? OMNI_KEEP_WHOLE : OMNI_KEEP_SINK_PREFIX);
        if (a.unit_kept_len) a.unit_kept_len[u] = kept;
        if (kept > 0) {
            omni_unit un = a.units[u];
            un.group = (meta & (1 << 8)) ? OMNI_GROUP_MUST_KEEP : ((meta & (1 << 10)) ? OMNI_GROUP_RECENT : OMNI_GROUP_SELECTED);
            un.start = s_scan[u];
            un.len = kept;
            a.units_out[s_idx[u]] = un;
        }
    }
    if (tid == 0) { *a.n_kept_out = n_kept; *a.n_units_out = n_units_kept; }

    // ---- per-token keep mask: the first kept tokens of every span ----------------------------------------
    if (a.keep_mask) {
        const int n_vec = (n_hist + 15) >> 4;
        for (int vi = tid; vi < n_vec; vi += SEL_THREADS) {
            const int pos = vi << 4;
            int lo = 0, hi = U;                   // largest u with s_start[u] <= pos
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (s_start[mid] <= pos) lo = mid; else hi = mid;
            }
            int u = lo;
            uint32_t w0 = 0, w1 = 0, w2 = 0, w3 = 0;
#pragma unroll
            for (int b = 0; b < 16; ++b) {
                const int p = pos + b;
                if (p < n_hist) {
                    while (p >= s_start[u + 1]) ++u;
                    if (p - s_start[u] < s_kept[u]) {
                        const uint32_t bit = 1u << ((b & 3) * 8);
                        if (b < 4) w0 |= bit; else if (b < 8) w1 |= bit; else if (b < 12) w2 |= bit; else w3 |= bit;
                    }
                }
            }
            if (pos + 16 <= a.n_hist_max) {
                *reinterpret_cast<uint4*>(a.keep_mask + pos) = make_uint4(w0, w1, w2, w3);
            } else {
#pragma unroll
                for (int b = 0; b < 16; ++b) {
                    const uint32_t w = b < 4 ? w0 : (b < 8 ? w1 : (b < 12 ? w2 : w3));
                    if (pos + b < n_hist) a.keep_mask[pos + b] = (w >> ((b & 3) * 8)) & 0xff;
                }
            }
        }
    }
}

}  // namespace

extern "C" omni_status omnitide_select_units(omnitide_ctx* ctx, void* stream, const omni_unit* units,
                                             const int32_t* n_units_dev, int32_t n_units_max, const float* scores,
                                             const omni_select_params* params, uint8_t* unit_keep_out,
                                             uint8_t* keep_mask_out, int32_t n_hist_max, int32_t* n_kept_out,
                                             omni_unit* units_out, int32_t* n_units_out) {
    if (!ctx) return OMNI_ERR_INVALID_ARG;
    if (!units || !scores || !params || !unit_keep_out || !n_kept_out || !units_out || !n_units_out)
        OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "select: null pointer");
    if (n_units_max <= 0 || n_units_max > ctx->g.u_cap) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "select: n_units_max %d outside (0, u_cap]", n_units_max);
    if (n_units_max > SEL_MAX_UNITS) OMNI_FAIL(ctx, OMNI_ERR_UNSUPPORTED, "select: more than %d units", SEL_MAX_UNITS);
    if (n_hist_max < 0 || n_hist_max > ctx->g.s_cap) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "select: n_hist_max outside [0, s_cap]");
    if (keep_mask_out && !omni_aligned16(keep_mask_out)) OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "select: keep_mask_out must be 16-byte aligned");
    if (units == units_out) OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "select: units_out must not alias units");
    SelectArgs a;
    a.units = units; a.n_units_dev = n_units_dev; a.n_units_max = n_units_max; a.scores = scores; a.p = *params;
    a.unit_keep = unit_keep_out; a.keep_mask = keep_mask_out; a.n_hist_max = n_hist_max; a.n_kept_out = n_kept_out;
    a.units_out = units_out; a.n_units_out = n_units_out; a.status = ctx->status_dev;
    a.p2 = 32;
    while (a.p2 < n_units_max) a.p2 <<= 1;
    const size_t smem = (size_t)a.p2 * (8 + 4 + 4 + 4 + 1) + 16;
    if (smem > 48 * 1024)
        OMNI_CUDA(ctx, cudaFuncSetAttribute(select_units_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    select_units_kernel<<<1, SEL_THREADS, smem, static_cast<cudaStream_t>(stream)>>>(a);
    OMNI_CHECK_LAUNCH(ctx, "select_units_kernel");
    return OMNI_OK;
}

extern "C" omni_status omnitide_plan_structural(omnitide_ctx* ctx, void* stream, const omni_unit* units,
                                                const int32_t* n_units_dev, int32_t n_units_max,
                                                const omni_structural_params* params, uint8_t* unit_keep_out,
                                                int32_t* unit_kept_len_out, uint8_t* keep_mask_out, int32_t n_hist_max,
                                                int32_t* n_kept_out, omni_unit* units_out, int32_t* n_units_out) {
    if (!ctx) return OMNI_ERR_INVALID_ARG;
    if (!units || !params || !unit_keep_out || !n_kept_out || !units_out || !n_units_out)
        OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "plan_structural: null pointer");
    if (n_units_max <= 0 || n_units_max > ctx->g.u_cap) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "plan_structural: n_units_max %d outside (0, u_cap]", n_units_max);
    if (n_units_max > SEL_MAX_UNITS) OMNI_FAIL(ctx, OMNI_ERR_UNSUPPORTED, "plan_structural: more than %d units", SEL_MAX_UNITS);
    if (n_hist_max < 0 || n_hist_max > ctx->g.s_cap) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "plan_structural: n_hist_max outside [0, s_cap]");
    if (keep_mask_out && !omni_aligned16(keep_mask_out)) OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "plan_structural: keep_mask_out must be 16-byte aligned");
    if (units == units_out) OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "plan_structural: units_out must not alias units");
    PlanArgs a;
    a.units = units; a.n_units_dev = n_units_dev; a.n_units_max = n_units_max; a.p = *params;
    a.unit_keep = unit_keep_out; a.unit_kept_len = unit_kept_len_out; a.keep_mask = keep_mask_out; a.n_hist_max = n_hist_max;
    a.n_kept_out = n_kept_out; a.units_out = units_out; a.n_units_out = n_units_out; a.status = ctx->status_dev;
    const size_t smem = ((size_t)8 * n_units_max + 4) * sizeof(int);
    if (smem > 48 * 1024)
        OMNI_CUDA(ctx, cudaFuncSetAttribute(plan_structural_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    plan_structural_kernel<<<1, SEL_THREADS, smem, static_cast<cudaStream_t>(stream)>>>(a);
    OMNI_CHECK_LAUNCH(ctx, "plan_structural_kernel");
    return OMNI_OK;
}
