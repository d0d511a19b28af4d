// Class-aware selective migration (Section 6.2 "Packing scattered entries" and "Checking layout
// improvement"; allocation classes and page promotion of Section 6.1).
//
// The plan is sequential by definition (every move changes which pages later candidates may use), so
// one CTA makes it: the layout lives in shared memory as one live bit per slot and one packed counter
// word per page; one warp walks the candidates, its lanes searching the pages before each one for the
// first admissible page, 32 at a time (block-wide barriers per candidate cost five times more).  The K/V rows then move in two
// grid-wide launches, sources to context staging and staging to destinations, because a destination
// may be the source of an earlier move of the same plan.
#include <algorithm>
#include <climits>

#include "common.cuh"

namespace {

constexpr int MC_THREADS = 1024;
constexpr int CAND_BIT = 0x80;

struct PlanArgs {
    uint8_t* mask;              // [S] in/out
    uint8_t* slot_class;        // [S] in/out
    const int32_t* s_span_dev;  // nullable
    int s_span_max;
    int page, sub, promote;
    int32_t* cand;              // [S] scratch: candidates in physical order, slot | class << 28
    int32_t* moves;             // [2 S] (src, dst) pairs
    uint8_t* moved_class;       // [S] scratch: class byte of every moved entry
    uint8_t* page_class_out;    // nullable
    omni_class_info* info;      // the move kernels read n_moves from it
    int32_t* status;
};

// counts of the three classes in a page, 16 bits each (bits 48-50: classes of its immovable entries)
__device__ __forceinline__ uint64_t field(int c) { return 1ull << (16 * c); }
__device__ __forceinline__ int total_of(uint64_t w) { return (int)((w & 0xffff) + ((w >> 16) & 0xffff) + ((w >> 32) & 0xffff)); }
__device__ __forceinline__ bool only_class(uint64_t w, int c) { return (w & 0xffffffffffffull & ~(0xffffull << (16 * c))) == 0; }

// first clear bit of the layout in [lo, hi), or -1
__device__ __forceinline__ int first_empty(const uint32_t* bits, int lo, int hi) {
    for (int w = lo >> 5; w <= (hi - 1) >> 5 && lo < hi; ++w) {
        uint32_t free_bits = ~bits[w];
        if (w == (lo >> 5)) free_bits &= 0xffffffffu << (lo & 31);
        if (w == ((hi - 1) >> 5) && (hi & 31)) free_bits &= (1u << (hi & 31)) - 1u;
        if (free_bits) return (w << 5) + __ffs(free_bits) - 1;
    }
    return -1;
}

// regions of `size` slots that hold a live bit, counted by the whole CTA (result in *out after the barrier)
__device__ __forceinline__ void count_active(const uint32_t* bits, int S, int size, int* out) {
    if (threadIdx.x == 0) *out = 0;
    __syncthreads();
    const int n = (S + size - 1) / size;
    int mine = 0;
    for (int r = threadIdx.x; r < n; r += MC_THREADS) {
        const int lo = r * size, hi = min(S, lo + size);
        bool any = false;
        for (int w = lo >> 5; w <= (hi - 1) >> 5 && !any; ++w) {
            uint32_t b = bits[w];
            if (w == (lo >> 5)) b &= 0xffffffffu << (lo & 31);
            if (w == ((hi - 1) >> 5) && (hi & 31)) b &= (1u << (hi & 31)) - 1u;
            any = b != 0;
        }
        mine += (int)any;
    }
    for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd(out, mine);
    __syncthreads();
}

// n-th (from 0) clear bit of the layout in [lo, hi), or -1
__device__ __forceinline__ int nth_empty(const uint32_t* bits, int lo, int hi, int n) {
    for (int w = lo >> 5; w <= (hi - 1) >> 5 && lo < hi; ++w) {
        uint32_t free_bits = ~bits[w];
        if (w == (lo >> 5)) free_bits &= 0xffffffffu << (lo & 31);
        if (w == ((hi - 1) >> 5) && (hi & 31)) free_bits &= (1u << (hi & 31)) - 1u;
        const int k = __popc(free_bits);
        if (n < k) {
            for (int j = 0; j < n; ++j) free_bits &= free_bits - 1;      // drop the n lowest empty slots
            return (w << 5) + __ffs(free_bits) - 1;
        }
        n -= k;
    }
    return -1;
}

__global__ void __launch_bounds__(MC_THREADS, 1) class_plan_kernel(const PlanArgs a) {
    extern __shared__ uint64_t mc_smem[];
    __shared__ int s_cnt[4];          // pages / subblocks before and after
    __shared__ int s_nmoves, s_bad, s_warp_tot[32];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    int S = a.s_span_dev ? *a.s_span_dev : a.s_span_max;
    if (S > a.s_span_max || S < 0) {
        if (tid == 0) {
            atomicOr(a.status, OMNI_DEV_BAD_COUNT);
            *a.info = omni_class_info{0, 0, 0, 0, 0, 0, 0, 0};
        }
        return;
    }
    const int P = a.page, n_pages = (S + P - 1) / P, n_words = (S + 31) / 32;
    const int p_shift = (P & (P - 1)) == 0 ? __ffs(P) - 1 : -1;
    auto page_of = [&](int s) { return p_shift >= 0 ? s >> p_shift : s / P; };
    unsigned long long* pw = reinterpret_cast<unsigned long long*>(mc_smem);   // [n_pages] class counts of the simulated layout
    uint32_t* bits = reinterpret_cast<uint32_t*>(mc_smem + n_pages);           // [n_words] its live bits
    if (tid == 0) { s_nmoves = 0; s_bad = 0; }
    // a warp owns a contiguous range of 32-slot words, so that the passes below need no block-wide step per word
    const int words_per_warp = (n_words + MC_THREADS / 32 - 1) / (MC_THREADS / 32);
    const int w_begin = min(n_words, wid * words_per_warp), w_end = min(n_words, w_begin + words_per_warp);

    // ---- the layout as stored: live bits and per-page class counts -------------------------------------------
    auto load_layout = [&]() {
        for (int q = tid; q < n_pages; q += MC_THREADS) pw[q] = 0;
        __syncthreads();
        constexpr int LB = 8;                          // words in flight per warp
        for (int w0 = w_begin; w0 < w_end; w0 += LB) {
            uint8_t mk[LB], cb[LB];
#pragma unroll
            for (int j = 0; j < LB; ++j) {
                const int s = (w0 + j) * 32 + lane;
                const bool in = w0 + j < w_end && s < S;
                mk[j] = in ? a.mask[s] : 0;
                cb[j] = in ? a.slot_class[s] : 0;
            }
#pragma unroll
            for (int j = 0; j < LB; ++j) {
                if (w0 + j >= w_end) break;
                const int s = (w0 + j) * 32 + lane;
                const bool live = mk[j] != 0;
                const int c = cb[j] & 3;
                const uint32_t bal = __ballot_sync(0xffffffffu, live);
                if (lane == 0) bits[w0 + j] = bal;
                if (live && c == 3) s_bad = 1;
                if ((P & 31) == 0) {
                    // the 32 slots of a word lie in one page: one shared-memory atomic per word
                    const uint32_t b0 = __ballot_sync(0xffffffffu, live && c == 0), b1 = __ballot_sync(0xffffffffu, live && c == 1),
                                   b2 = __ballot_sync(0xffffffffu, live && c == 2);
                    if (lane == 0 && (b0 | b1 | b2))
                        atomicAdd(&pw[page_of(s)], (unsigned long long)__popc(b0) | ((unsigned long long)__popc(b1) << 16) |
                                                       ((unsigned long long)__popc(b2) << 32));
                } else if (live && c < 3) {
                    atomicAdd(&pw[page_of(s)], (unsigned long long)field(c));
                }
            }
        }
        __syncthreads();
    };
    load_layout();
    if (s_bad) {
        if (tid == 0) {
            atomicOr(a.status, OMNI_DEV_BAD_UNITS);
            *a.info = omni_class_info{0, 0, 0, 0, 0, 0, 0, 0};
        }
        return;
    }
    count_active(bits, S, P, &s_cnt[0]);
    count_active(bits, S, a.sub, &s_cnt[1]);

    // ---- candidates in physical order: live, marked, and not in a page that is full.  Every other live entry is
    // immovable; the classes of a page's immovable entries go to bits 48-50 of its word (a page that holds an
    // immovable entry of another class can never take a candidate).  Two sweeps: count per warp, then write. ----
    int cand_base = 0;
    for (int sweep = 0; sweep < 2; ++sweep) {
        int n_mine = 0;
        for (int w = w_begin; w < w_end; ++w) {
            const int s = w * 32 + lane;
            const bool live = (bits[w] >> lane) & 1u;
            bool is_c = false;
            int c = 0;
            if (live) {
                const int cb = a.slot_class[s];
                const int q = page_of(s);
                c = cb & 3;
                is_c = (cb & CAND_BIT) && total_of(pw[q]) < min(P, S - q * P);
            }
            if (sweep == 0) {
                const bool fixed = live && !is_c;
                if ((P & 31) == 0) {
                    // one page per word: the lanes' classes are merged by ballots, one atomic per word
                    const uint32_t f0 = __ballot_sync(0xffffffffu, fixed && c == 0), f1 = __ballot_sync(0xffffffffu, fixed && c == 1),
                                   f2 = __ballot_sync(0xffffffffu, fixed && c == 2);
                    const unsigned long long m = (f0 ? 1ull : 0ull) | (f1 ? 2ull : 0ull) | (f2 ? 4ull : 0ull);
                    if (lane == 0 && m) atomicOr(&pw[page_of(w * 32)], m << 48);
                } else if (fixed) {
                    atomicOr(&pw[page_of(s)], 1ull << (48 + c));
                }
            }
            const uint32_t bal = __ballot_sync(0xffffffffu, is_c);
            if (sweep == 1 && is_c) a.cand[cand_base + n_mine + __popc(bal & ((1u << lane) - 1u))] = s | (c << 28);
            n_mine += __popc(bal);
        }
        if (sweep == 0) {
            if (lane == 0) s_warp_tot[wid] = n_mine;
            __syncthreads();
            for (int w = 0; w < wid; ++w) cand_base += s_warp_tot[w];
        }
    }
    __syncthreads();
    int n_cand = 0;
    for (int w = 0; w < MC_THREADS / 32; ++w) n_cand += s_warp_tot[w];

    // ---- the plan: one warp.  Consecutive candidates of one class in one source page are placed together: moving
    // one of them changes neither which page is the first admissible one nor the order of its empty slots. --------
    if (wid == 0) {
        int lo0 = 0, lo1 = 0, lo2 = 0, n_moves = 0;
        // the candidate list is read through two 32-entry register windows [i0, i0 + 32) and [i0 + 32, i0 + 64)
        int i0 = 0;
        int win0 = lane < n_cand ? a.cand[lane] : -1, win1 = 32 + lane < n_cand ? a.cand[32 + lane] : -1;
        for (int i = 0; i < n_cand;) {
            if (i >= i0 + 32) {
                i0 += 32;
                win0 = win1;
                win1 = i0 + 32 + lane < n_cand ? a.cand[i0 + 32 + lane] : -1;
            }
            const int idx = i - i0 + lane;                                       // < 64
            const int v0 = __shfl_sync(0xffffffffu, win0, idx & 31), v1 = __shfl_sync(0xffffffffu, win1, idx & 31);
            const int mine = idx < 32 ? v0 : v1;                                 // candidate i + lane, -1 past the end
            const int cur = __shfl_sync(0xffffffffu, mine, 0);
            const int s0 = cur & 0x0fffffff, c = cur >> 28, ps = page_of(s0);
            const int my_s = mine & 0x0fffffff;
            const bool same = mine >= 0 && (mine >> 28) == c && page_of(my_s) == ps;
            const uint32_t same_bal = __ballot_sync(0xffffffffu, same);
            const int run = same_bal == 0xffffffffu ? 32 : __ffs(~same_bal) - 1;   // leading lanes of the same page and class
            // skip for good the pages before this candidate that are full or hold an immovable entry of another class
            int lo = c == 0 ? lo0 : (c == 1 ? lo1 : lo2);
            const unsigned long long other_fixed = (7ull & ~(1ull << c)) << 48;
            while (lo < ps && (total_of(pw[lo]) == P || (pw[lo] & other_fixed))) ++lo;
            if (c == 0) lo0 = lo; else if (c == 1) lo1 = lo; else lo2 = lo;
            // first page before the candidate's own that has an empty slot and is empty or of class c
            int found = -1;
            for (int base = lo; base < ps && found < 0; base += 32) {
                const int q = base + lane;
                bool ok = false;
                if (q < ps) {
                    const uint64_t w = pw[q];
                    ok = only_class(w, c) && total_of(w) < P;
                }
                const uint32_t bal = __ballot_sync(0xffffffffu, ok);
                if (bal) found = base + __ffs(bal) - 1;
            }
            int n = 1, d = -1;
            if (found >= 0) {
                n = min(run, P - total_of(pw[found]));
                if (lane < n) d = nth_empty(bits, found * P, found * P + P, lane);
            } else if (lane == 0 && only_class(pw[ps], c)) {
                d = first_empty(bits, ps * P, s0);                                // inside its own page, one at a time
            }
            __syncwarp();                              // every lane has read the layout before it changes
            const uint32_t moved = __ballot_sync(0xffffffffu, d >= 0);
            if (moved) {
                // the destinations lie in one page and so do the sources: their bits are merged word by word across
                // the lanes (shared-memory atomics on one word would serialise the lanes)
                const int dp = found >= 0 ? found : ps;
                for (int w = (dp * P) >> 5; w <= (min(S, dp * P + P) - 1) >> 5; ++w) {
                    const uint32_t m = __reduce_or_sync(0xffffffffu, (d >= 0 && (d >> 5) == w) ? 1u << (d & 31) : 0u);
                    if (lane == 0 && m) bits[w] |= m;
                }
                __syncwarp();
                for (int w = (ps * P) >> 5; w <= (min(S, ps * P + P) - 1) >> 5; ++w) {
                    const uint32_t m = __reduce_or_sync(0xffffffffu, (d >= 0 && (my_s >> 5) == w) ? 1u << (my_s & 31) : 0u);
                    if (lane == 0 && m) bits[w] &= ~m;
                }
            }
            if (d >= 0) {
                a.moves[2 * (n_moves + lane)] = my_s;
                a.moves[2 * (n_moves + lane) + 1] = d;
            }
            const int n_moved = __popc(moved);
            if (lane == 0 && n_moved) {
                pw[found >= 0 ? found : ps] += (unsigned long long)n_moved * field(c);
                pw[ps] -= (unsigned long long)n_moved * field(c);
            }
            n_moves += n_moved;
            i += n;
            __syncwarp();
        }
        if (lane == 0) s_nmoves = n_moves;
    }
    __syncthreads();

    // ---- accept test ---------------------------------------------------------------------------------------
    count_active(bits, S, P, &s_cnt[2]);
    count_active(bits, S, a.sub, &s_cnt[3]);
    const int n_moves = s_nmoves;
    const bool accepted = n_moves > 0 && (s_cnt[2] < s_cnt[0] || s_cnt[3] < s_cnt[1]);
    if (tid == 0) {
        omni_class_info inf;
        inf.accepted = accepted;
        inf.n_moves = accepted ? n_moves : 0;
        inf.n_candidates = n_cand;
        inf.pages_before = s_cnt[0];
        inf.subblocks_before = s_cnt[1];
        inf.pages_after = accepted ? s_cnt[2] : s_cnt[0];
        inf.subblocks_after = accepted ? s_cnt[3] : s_cnt[1];
        inf.reserved = 0;
        *a.info = inf;
    }
    __syncthreads();

    // ---- the new mask and classes (a source is never the destination of an earlier move, so sources are read first) --
    if (accepted) {
        for (int i = tid; i < n_moves; i += MC_THREADS) a.moved_class[i] = a.slot_class[a.moves[2 * i]];
        __syncthreads();
        for (int i = tid; i < n_moves; i += MC_THREADS) {
            const int s = a.moves[2 * i];
            a.slot_class[s] = 0;
            a.mask[s] = 0;
        }
        __syncthreads();
        for (int i = tid; i < n_moves; i += MC_THREADS) {
            const int d = a.moves[2 * i + 1];
            a.slot_class[d] = a.moved_class[i];
            a.mask[d] = 1;
        }
        __syncthreads();
    } else if (n_moves > 0) {
        load_layout();                                 // the counts of the layout that stays
    }
    // ---- promotion of the pages packed full, page labels (from the per-page class counts) -------------------------
    auto promoted = [&](uint64_t w) {
        return accepted && a.promote && total_of(w) == P && (w & 0xffff) == 0;
    };
    if (accepted && a.promote) {
        for (int s = tid; s < S; s += MC_THREADS) {
            const uint64_t w = pw[page_of(s)];
            if (promoted(w) && ((w >> 32) & 0xffff)) a.slot_class[s] = (a.slot_class[s] & ~3) | 1;
        }
    }
    if (a.page_class_out) {
        for (int q = tid; q < n_pages; q += MC_THREADS) {
            const uint64_t w = pw[q];
            const int seen = ((w & 0xffff) ? 1 : 0) | (((w >> 16) & 0xffff) ? 2 : 0) | (((w >> 32) & 0xffff) ? 4 : 0);
            int label = seen == 0 ? 255 : (seen == 1 ? 0 : (seen == 2 ? 1 : (seen == 4 ? 2 : 254)));
            if (promoted(w)) label = 1;
            a.page_class_out[q] = (uint8_t)label;
        }
    }
}

// Copies the moved rows: phase 0 sources -> staging row i, phase 1 staging row i -> destinations.
__global__ void __launch_bounds__(256) class_move_kernel(char* k_cache, char* v_cache, char* k_stage, char* v_stage,
                                                         const int32_t* moves, const omni_class_info* info, int vpr,
                                                         size_t row_bytes, int phase) {
    const int n_moves = info->n_moves;
    const long long total = (long long)n_moves * 2 * vpr;             // (move, K or V, 16-byte vector)
    constexpr int BATCH = 4;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long base = (long long)blockIdx.x * blockDim.x + threadIdx.x; base < total; base += stride * BATCH) {
        uint4 buf[BATCH];
        const uint4* from[BATCH];
        uint4* to[BATCH];
#pragma unroll
        for (int u = 0; u < BATCH; ++u) {
            const long long idx = base + u * stride;
            from[u] = nullptr;
            if (idx < total) {
                const int v = (int)(idx % vpr);
                const long long rw = idx / vpr;
                const int i = (int)(rw >> 1);
                const bool is_v = rw & 1;
                const size_t cache_row = (size_t)moves[2 * i + phase];
                char* cache = (is_v ? v_cache : k_cache) + cache_row * row_bytes + (size_t)v * 16;
                char* stage = (is_v ? v_stage : k_stage) + (size_t)i * row_bytes + (size_t)v * 16;
                from[u] = reinterpret_cast<const uint4*>(phase == 0 ? cache : stage);
                to[u] = reinterpret_cast<uint4*>(phase == 0 ? stage : cache);
            }
        }
#pragma unroll
        for (int u = 0; u < BATCH; ++u)
            if (from[u]) buf[u] = *from[u];
#pragma unroll
        for (int u = 0; u < BATCH; ++u)
            if (from[u]) *to[u] = buf[u];
    }
}

}  // namespace

extern "C" omni_status omnipage_migrate_class(omnitide_ctx* ctx, void* stream, void* k_cache, void* v_cache,
                                              uint8_t* keep_mask, uint8_t* slot_class, const int32_t* s_span_dev,
                                              int32_t s_span_max, int32_t page_size, int32_t subblock, int32_t promote,
                                              int32_t* moves_out, uint8_t* page_class_out, omni_class_info* info_out) {
    if (!ctx) return OMNI_ERR_INVALID_ARG;
    if (!k_cache || !v_cache || !keep_mask || !slot_class || !info_out || s_span_max <= 0)
        OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "migrate_class: null pointer or empty span");
    if (page_size <= 0 || page_size > 32768 || subblock <= 0 || page_size % subblock)
        OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "migrate_class: the subblock size must divide the page size (<= 32768)");
    if (s_span_max > ctx->g.s_cap) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "migrate_class: s_span_max %d > s_cap %d", s_span_max, ctx->g.s_cap);
    if (s_span_max >= (1 << 28)) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "migrate_class: span above 2^28 slots");
    const size_t n_pages = ((size_t)s_span_max + page_size - 1) / page_size;
    const size_t smem = n_pages * sizeof(uint64_t) + (((size_t)s_span_max + 31) / 32) * sizeof(uint32_t) + 16;
    if (smem > 220 * 1024) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "migrate_class: the layout of %d slots does not fit one CTA", s_span_max);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!ctx->mc_moves) {
        OMNI_CUDA(ctx, cudaMalloc(&ctx->mc_moves, (size_t)ctx->g.s_cap * 2 * sizeof(int32_t)));
        OMNI_CUDA(ctx, cudaMalloc(&ctx->mc_class, (size_t)ctx->g.s_cap));
    }
    const omni_status ss = omni_inplace_staging(ctx);
    if (ss) return ss;
    PlanArgs a;
    a.mask = keep_mask; a.slot_class = slot_class; a.s_span_dev = s_span_dev; a.s_span_max = s_span_max;
    a.page = page_size; a.sub = subblock; a.promote = promote;
    a.cand = ctx->ws_slot_map; a.moves = moves_out ? moves_out : ctx->mc_moves; a.moved_class = ctx->mc_class;
    a.page_class_out = page_class_out; a.info = info_out; a.status = ctx->status_dev;
    if (smem > 48 * 1024)
        OMNI_CUDA(ctx, cudaFuncSetAttribute(class_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    class_plan_kernel<<<1, MC_THREADS, smem, st>>>(a);
    OMNI_CHECK_LAUNCH(ctx, "class_plan_kernel");
    const int vpr = (int)(ctx->row_bytes / 16);
    const int grid = 2 * ctx->sm_count;
    for (int phase = 0; phase < 2; ++phase) {
        class_move_kernel<<<grid, 256, 0, st>>>(static_cast<char*>(k_cache), static_cast<char*>(v_cache),
                                                static_cast<char*>(ctx->inplace_k), static_cast<char*>(ctx->inplace_v),
                                                a.moves, info_out, vpr, ctx->row_bytes, phase);
        OMNI_CHECK_LAUNCH(ctx, "class_move_kernel");
    }
    return OMNI_OK;
}
