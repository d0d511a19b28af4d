// Context life cycle, dispatch between the tensor-core and CUDA-core paths, and the whole-pass calls.
#include "common.cuh"

#include <new>

namespace {

bool tc_geometry(const omnitide_ctx* ctx) {
    return ctx->g.dtype == OMNI_DTYPE_BF16 && ctx->g.d == 128 && !ctx->force_cuda_cores;
}

template <typename T>
cudaError_t alloc(T** p, size_t n) {
    *p = nullptr;
    return cudaMalloc(reinterpret_cast<void**>(p), n ? n * sizeof(T) : sizeof(T));
}

void free_all(omnitide_ctx* c) {
    void* ptrs[] = {c->status_dev, c->score_part, c->score_tile_mass, c->score_mass64, c->inplace_k, c->inplace_v,
                    c->ws_scores, c->ws_unit_keep, c->ws_kept_len, c->ws_keep_mask, c->ws_slot_map, c->ws_counts, c->ws_info, c->st_q,
                    c->st_k, c->st_v, c->st_o, c->st_units, c->attn_part_o, c->attn_part_ml, c->cp_words, c->attn_live_idx, c->attn_live_mask,
                    c->attn_n_live, c->mig_plan, c->dec_counter, c->mc_moves, c->mc_class};
    for (void* p : ptrs)
        if (p) cudaFree(p);
    for (int b = 0; b < 2; ++b) {
        void* pl[] = {c->pl_q[b], c->pl_k[b], c->pl_v[b], c->pl_o[b], c->pl_units[b]};
        for (void* p : pl)
            if (p) cudaFree(p);
        cudaEvent_t evs[] = {c->pl_ev_q[b], c->pl_ev_kv[b], c->pl_ev_done[b], c->pl_ev_out[b]};
        for (cudaEvent_t e : evs)
            if (e) cudaEventDestroy(e);
    }
    if (c->pl_out) cudaStreamDestroy(c->pl_out);
    if (c->ev_fork) cudaEventDestroy(c->ev_fork);
    if (c->ev_kv) cudaEventDestroy(c->ev_kv);
    if (c->aux_stream) cudaStreamDestroy(c->aux_stream);
}

}  // namespace

extern "C" omni_status omnitide_create(omnitide_ctx** ctx_out, const omni_geometry* g) {
    if (!ctx_out) return OMNI_ERR_INVALID_ARG;
    *ctx_out = nullptr;
    if (!g) return OMNI_ERR_INVALID_ARG;
    if (g->h_q <= 0 || g->h_kv <= 0 || g->h_q % g->h_kv != 0 || g->d <= 0 || g->d % 8 != 0 || g->d > 256 ||
        (g->dtype != OMNI_DTYPE_BF16 && g->dtype != OMNI_DTYPE_FP32) || g->s_cap <= 0 || g->u_cap <= 0 || g->t_cap <= 0)
        return OMNI_ERR_UNSUPPORTED;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return OMNI_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return OMNI_ERR_CUDA;
    if (prop.major != 10) return OMNI_ERR_UNSUPPORTED;      // built for sm_100a only
    omnitide_ctx* c = new (std::nothrow) omnitide_ctx();
    if (!c) return OMNI_ERR_CUDA;
    memset(c, 0, sizeof(*c));
    c->g = *g;
    c->device = dev;
    c->sm_count = prop.multiProcessorCount;
    c->es = g->dtype == OMNI_DTYPE_BF16 ? 2 : 4;
    c->row_bytes = (size_t)g->h_kv * g->d * c->es;
    const size_t row_tiles = ((size_t)g->t_cap + 127) / 128 * g->h_q;
    const size_t q_elems = (size_t)g->t_cap * g->h_q * g->d;
    bool ok = true;
    ok &= alloc(&c->status_dev, 1) == cudaSuccess;
    ok &= alloc(&c->score_part, row_tiles * ((size_t)g->u_cap + 64) * 128) == cudaSuccess;   // + split boundaries
    ok &= alloc(&c->score_tile_mass, row_tiles * g->u_cap) == cudaSuccess;
    ok &= alloc(&c->score_mass64, (size_t)g->u_cap) == cudaSuccess;
    ok &= cudaStreamCreateWithFlags(&c->aux_stream, cudaStreamNonBlocking) == cudaSuccess;
    ok &= cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) == cudaSuccess;
    ok &= cudaEventCreateWithFlags(&c->ev_kv, cudaEventDisableTiming) == cudaSuccess;
    ok &= alloc(&c->attn_live_idx, (size_t)g->s_cap / 128 + 2) == cudaSuccess;
    ok &= alloc(&c->attn_live_mask, (size_t)g->s_cap / 128 + 2) == cudaSuccess;
    ok &= alloc(&c->attn_n_live, (size_t)1) == cudaSuccess;
    ok &= alloc(&c->dec_counter, (size_t)g->h_kv) == cudaSuccess;
    ok = ok && cudaMemset(c->dec_counter, 0, sizeof(int32_t) * (size_t)g->h_kv) == cudaSuccess;
    ok &= alloc(&c->cp_words, (size_t)c->sm_count + 1) == cudaSuccess;
    ok = ok && cudaMemset(c->cp_words, 0, ((size_t)c->sm_count + 1) * sizeof(unsigned long long)) == cudaSuccess;
    ok &= alloc(&c->ws_scores, (size_t)g->u_cap) == cudaSuccess;
    ok &= alloc(&c->ws_unit_keep, (size_t)g->u_cap + 16) == cudaSuccess;
    ok &= alloc(&c->ws_kept_len, (size_t)g->u_cap) == cudaSuccess;
    ok &= alloc(&c->ws_keep_mask, (size_t)g->s_cap + 16) == cudaSuccess;
    ok &= alloc(&c->ws_slot_map, (size_t)g->s_cap + 16) == cudaSuccess;
    ok &= alloc(&c->ws_counts, 4) == cudaSuccess;
    ok &= alloc(&c->ws_info, 1) == cudaSuccess;
    ok &= cudaMalloc(&c->st_q, q_elems * c->es) == cudaSuccess;
    ok &= cudaMalloc(&c->st_k, (size_t)g->t_cap * c->row_bytes) == cudaSuccess;
    ok &= cudaMalloc(&c->st_v, (size_t)g->t_cap * c->row_bytes) == cudaSuccess;
    ok &= cudaMalloc(&c->st_o, q_elems * 4) == cudaSuccess;
    ok &= alloc(&c->st_units, 64) == cudaSuccess;
    // split-item partials of the attention kernel: [SM][2 slots][2 tiles][128 rows] x (128 floats, (max, sum))
    ok &= alloc(&c->attn_part_o, (size_t)c->sm_count * 4 * 128 * 128) == cudaSuccess;
    ok &= alloc(&c->attn_part_ml, (size_t)c->sm_count * 4 * 128 * 2) == cudaSuccess;
    if (ok) ok = cudaMemset(c->status_dev, 0, sizeof(int32_t)) == cudaSuccess;
    if (ok) {
        cudaDriverEntryPointQueryResult qres;
        void* fn = nullptr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            c->encode_tiled = fn;
        else
            ok = false;
    }
    if (!ok) {
        cudaGetLastError();
        free_all(c);
        delete c;
        return OMNI_ERR_CUDA;
    }
    *ctx_out = c;
    return OMNI_OK;
}

extern "C" omni_status omnitide_destroy(omnitide_ctx* ctx) {
    if (!ctx) return OMNI_ERR_INVALID_ARG;
    cudaDeviceSynchronize();
    free_all(ctx);
    delete ctx;
    return OMNI_OK;
}

extern "C" omni_status omnitide_poll_status(omnitide_ctx* ctx, void* stream, int32_t* out) {
    if (!ctx || !out) return OMNI_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    OMNI_CUDA(ctx, cudaMemcpyAsync(out, ctx->status_dev, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    OMNI_CUDA(ctx, cudaMemsetAsync(ctx->status_dev, 0, sizeof(int32_t), st));
    OMNI_CUDA(ctx, cudaStreamSynchronize(st));
    return OMNI_OK;
}

extern "C" const char* omnitide_last_error(const omnitide_ctx* ctx) { return ctx ? ctx->err : "null context"; }
extern "C" int64_t omnitide_launch_count(const omnitide_ctx* ctx) { return ctx ? ctx->launches : 0; }

extern "C" omni_status omnitide_set_option(omnitide_ctx* ctx, int32_t option, int32_t value) {
    if (!ctx) return OMNI_ERR_INVALID_ARG;
    if (option == OMNI_OPT_FORCE_CUDA_CORES) { ctx->force_cuda_cores = value != 0; return OMNI_OK; }
    if (option == OMNI_OPT_SCORE_WINDOW) {
        if (value < 0) OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "score window must be >= 0");
        ctx->score_window = value;
        return OMNI_OK;
    }
    if (option == OMNI_OPT_HIGH_WATERMARK) {
        if (value < 0) OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "high watermark must be >= 0");
        ctx->high_watermark = value;
        return OMNI_OK;
    }
    OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "unknown option %d", option);
}

extern "C" omni_status omnitide_score_units(omnitide_ctx* ctx, void* stream, const void* q, int32_t t,
                                            const void* k_cache, const int32_t* n_hist_dev, int32_t n_hist_max,
                                            const omni_unit* units, const int32_t* n_units_dev, int32_t n_units_max,
                                            const float* w_modality, float scale, float* scores_out, float* mass_out) {
    if (!ctx) return OMNI_ERR_INVALID_ARG;
    if (!q || !k_cache || !units || !w_modality || !scores_out) OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "score: null pointer");
    if (t <= 0 || t > ctx->g.t_cap) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "score: t %d outside (0, t_cap]", t);
    if (n_hist_max <= 0 || n_hist_max > ctx->g.s_cap) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "score: n_hist_max outside (0, s_cap]");
    if (n_units_max <= 0 || n_units_max > ctx->g.u_cap) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "score: n_units_max outside (0, u_cap]");
    if (!omni_aligned16(q) || !omni_aligned16(k_cache)) OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "score: q/k_cache must be 16-byte aligned");
    if (scale <= 0.f) scale = 1.0f / sqrtf((float)ctx->g.d);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (tc_geometry(ctx))
        return omni_score_tc(ctx, st, q, t, k_cache, n_hist_dev, n_hist_max, units, n_units_dev, n_units_max, w_modality,
                             scale, scores_out, mass_out);
    return omni_score_simple(ctx, st, q, t, k_cache, n_hist_dev, n_hist_max, units, n_units_dev, n_units_max, w_modality,
                             scale, scores_out, mass_out);
}

static omni_status chunk_attention_impl(const uint8_t* hist_mask, omnitide_ctx* ctx, void* stream, const void* q, int32_t t,
                                                const void* k_hist, const void* v_hist, const int32_t* n_hist_dev,
                                                int32_t n_hist_max, const void* k_chunk, const void* v_chunk, float scale,
                                                void* o_out, int32_t out_dtype, float* lse_out) {
    if (!ctx) return OMNI_ERR_INVALID_ARG;
    if (!q || !k_chunk || !v_chunk || !o_out) OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "attention: null pointer");
    if (n_hist_max > 0 && (!k_hist || !v_hist)) OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "attention: history pointers are null");
    if (t <= 0 || t > ctx->g.t_cap) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "attention: t %d outside (0, t_cap]", t);
    if (n_hist_max < 0 || n_hist_max > ctx->g.s_cap) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "attention: n_hist_max outside [0, s_cap]");
    if (out_dtype != OMNI_DTYPE_BF16 && out_dtype != OMNI_DTYPE_FP32) OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "attention: bad out_dtype");
    if (!omni_aligned16(q) || !omni_aligned16(k_hist) || !omni_aligned16(v_hist) || !omni_aligned16(k_chunk) ||
        !omni_aligned16(v_chunk) || !omni_aligned16(o_out) || !omni_aligned16(hist_mask))
        OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "attention: pointers must be 16-byte aligned");
    if (scale <= 0.f) scale = 1.0f / sqrtf((float)ctx->g.d);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (tc_geometry(ctx)) {
        // one query and a dense history: the split-KV decode kernel (HBM-bound, no tensor-core work to do)
        if (t == 1 && !hist_mask) {
            const omni_status ds = omni_attention_decode(ctx, st, q, k_hist, v_hist, n_hist_dev, n_hist_max, k_chunk, v_chunk,
                                                         scale, o_out, out_dtype, lse_out);
            if (ds != OMNI_ERR_UNSUPPORTED) return ds;
        }
        return omni_attention_tc(ctx, st, q, t, k_hist, v_hist, n_hist_dev, n_hist_max, k_chunk, v_chunk, scale, o_out,
                                 out_dtype, lse_out, hist_mask);
    }
    return omni_attention_simple(ctx, st, q, t, k_hist, v_hist, n_hist_dev, n_hist_max, k_chunk, v_chunk, scale, o_out,
                                 out_dtype, lse_out, hist_mask);
}

extern "C" omni_status omnitide_chunk_attention(omnitide_ctx* ctx, void* stream, const void* q, int32_t t,
                                                const void* k_hist, const void* v_hist, const int32_t* n_hist_dev,
                                                int32_t n_hist_max, const void* k_chunk, const void* v_chunk, float scale,
                                                void* o_out, int32_t out_dtype, float* lse_out) {
    return chunk_attention_impl(nullptr, ctx, stream, q, t, k_hist, v_hist, n_hist_dev, n_hist_max, k_chunk, v_chunk, scale,
                                o_out, out_dtype, lse_out);
}

extern "C" omni_status omnitide_chunk_attention_masked(omnitide_ctx* ctx, void* stream, const void* q, int32_t t,
                                                       const void* k_hist, const void* v_hist, const uint8_t* hist_keep_mask,
                                                       const int32_t* s_span_dev, int32_t s_span_max, const void* k_chunk,
                                                       const void* v_chunk, float scale, void* o_out, int32_t out_dtype,
                                                       float* lse_out) {
    if (!ctx) return OMNI_ERR_INVALID_ARG;
    if (!hist_keep_mask && s_span_max > 0) OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "attention_masked: null keep mask");
    return chunk_attention_impl(hist_keep_mask, ctx, stream, q, t, k_hist, v_hist, s_span_dev, s_span_max, k_chunk, v_chunk,
                                scale, o_out, out_dtype, lse_out);
}

static omni_status chunk_step_impl(cudaEvent_t chunk_kv_ready, omnitide_ctx* ctx, void* stream, const void* q, const void* k_chunk,
                                           const void* v_chunk, int32_t t, const omni_unit* chunk_units,
                                           int32_t n_chunk_units, const void* k_cache, const void* v_cache,
                                           const int32_t* n_hist_dev, int32_t n_hist_max, const omni_unit* units,
                                           const int32_t* n_units_dev, int32_t n_units_max, const float* w_modality,
                                           const omni_select_params* params, int32_t page_size, float scale,
                                           void* k_cache_out, void* v_cache_out, omni_unit* units_out, int32_t* n_hist_out,
                                           int32_t* n_units_out, void* o_out, int32_t out_dtype,
                                           omni_compact_info* info_out) {
    if (!ctx) return OMNI_ERR_INVALID_ARG;
    if (!k_cache_out || !v_cache_out || k_cache_out == k_cache || v_cache_out == v_cache)
        OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "chunk_step: output caches must be distinct buffers");
    if (!units_out || !n_hist_out || !n_units_out || !params) OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "chunk_step: null pointer");
    int32_t* n_kept = ctx->ws_counts;
    int32_t* n_units_kept = ctx->ws_counts + 1;
    omni_compact_info* info = info_out ? info_out : ctx->ws_info;
    omni_status s;
    // observation window: only the last `score_window` queries of the chunk score the history (0: all of them)
    const void* q_score = q;
    int32_t t_score = t;
    if (ctx->score_window > 0 && ctx->score_window < t) {
        t_score = ctx->score_window;
        q_score = static_cast<const char*>(q) + (size_t)(t - t_score) * ctx->g.h_q * ctx->g.d * ctx->es;
    }
    // hysteresis (Section 5.1): a history that cannot exceed the high watermark has no retention round -- no scoring
    // pass, and the selection keeps every unit (an unbounded budget makes the stale scores irrelevant)
    omni_select_params keep_all;
    if (ctx->high_watermark > 0 && n_hist_max <= ctx->high_watermark) {
        keep_all = *params;
        keep_all.budget = INT32_MAX;
        keep_all.modality_cap[0] = keep_all.modality_cap[1] = keep_all.modality_cap[2] = -1;
        params = &keep_all;
    } else {
        s = omnitide_score_units(ctx, stream, q_score, t_score, k_cache, n_hist_dev, n_hist_max, units, n_units_dev, n_units_max,
                                 w_modality, scale, ctx->ws_scores, nullptr);
        if (s) return s;
    }
    // the keep decision stays per unit between the two steps: no token mask, no slot map inside the pass
    s = omnitide_select_units(ctx, stream, units, n_units_dev, n_units_max, ctx->ws_scores, params, ctx->ws_unit_keep,
                              nullptr, n_hist_max, n_kept, units_out, n_units_kept);
    if (s) return s;
    s = omnipage_compact_units(ctx, stream, k_cache, v_cache, k_cache_out, v_cache_out, units, n_units_dev, n_units_max,
                               ctx->ws_unit_keep, nullptr, n_hist_max, page_size, units_out, n_units_kept, nullptr, info,
                               nullptr);
    if (s) return s;
    // the chunk's K/V rows are first read here (scoring reads only Q and the cached keys)
    if (chunk_kv_ready) OMNI_CUDA(ctx, cudaStreamWaitEvent(static_cast<cudaStream_t>(stream), chunk_kv_ready, 0));
    s = omnitide_chunk_attention(ctx, stream, q, t, k_cache_out, v_cache_out, n_kept, n_hist_max, k_chunk, v_chunk, scale,
                                 o_out, out_dtype, nullptr);
    if (s) return s;
    return omnipage_append(ctx, stream, k_cache_out, v_cache_out, n_kept, k_chunk, v_chunk, t, units_out, n_units_kept,
                           chunk_units, n_chunk_units, n_hist_out, n_units_out);
}

extern "C" omni_status omnitide_chunk_step(omnitide_ctx* ctx, void* stream, const void* q, const void* k_chunk,
                                           const void* v_chunk, int32_t t, const omni_unit* chunk_units,
                                           int32_t n_chunk_units, const void* k_cache, const void* v_cache,
                                           const int32_t* n_hist_dev, int32_t n_hist_max, const omni_unit* units,
                                           const int32_t* n_units_dev, int32_t n_units_max, const float* w_modality,
                                           const omni_select_params* params, int32_t page_size, float scale,
                                           void* k_cache_out, void* v_cache_out, omni_unit* units_out, int32_t* n_hist_out,
                                           int32_t* n_units_out, void* o_out, int32_t out_dtype,
                                           omni_compact_info* info_out) {
    return chunk_step_impl(nullptr, ctx, stream, q, k_chunk, v_chunk, t, chunk_units, n_chunk_units, k_cache, v_cache,
                           n_hist_dev, n_hist_max, units, n_units_dev, n_units_max, w_modality, params, page_size, scale,
                           k_cache_out, v_cache_out, units_out, n_hist_out, n_units_out, o_out, out_dtype, info_out);
}

extern "C" omni_status omnitide_chunk_step_structural(omnitide_ctx* ctx, void* stream, const void* q, const void* k_chunk,
                                                      const void* v_chunk, int32_t t, const omni_unit* chunk_units,
                                                      int32_t n_chunk_units, const void* k_cache, const void* v_cache,
                                                      const int32_t* n_hist_dev, int32_t n_hist_max, const omni_unit* units,
                                                      const int32_t* n_units_dev, int32_t n_units_max,
                                                      const omni_structural_params* params, int32_t page_size, float scale,
                                                      void* k_cache_out, void* v_cache_out, omni_unit* units_out,
                                                      int32_t* n_hist_out, int32_t* n_units_out, void* o_out,
                                                      int32_t out_dtype, omni_compact_info* info_out) {
    if (!ctx) return OMNI_ERR_INVALID_ARG;
    if (!k_cache_out || !v_cache_out || k_cache_out == k_cache || v_cache_out == v_cache)
        OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "chunk_step_structural: output caches must be distinct buffers");
    if (!units_out || !n_hist_out || !n_units_out || !params)
        OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "chunk_step_structural: null pointer");
    int32_t* n_kept = ctx->ws_counts;
    int32_t* n_units_kept = ctx->ws_counts + 1;
    omni_compact_info* info = info_out ? info_out : ctx->ws_info;
    // plan from metadata alone (no scoring pass), pack the planned runs, attend, append
    omni_status s = omnitide_plan_structural(ctx, stream, units, n_units_dev, n_units_max, params, ctx->ws_unit_keep,
                                             ctx->ws_kept_len, nullptr, n_hist_max, n_kept, units_out, n_units_kept);
    if (s) return s;
    s = omnipage_compact_units(ctx, stream, k_cache, v_cache, k_cache_out, v_cache_out, units, n_units_dev, n_units_max,
                               ctx->ws_unit_keep, ctx->ws_kept_len, n_hist_max, page_size, units_out, n_units_kept, nullptr,
                               info, nullptr);
    if (s) return s;
    s = omnitide_chunk_attention(ctx, stream, q, t, k_cache_out, v_cache_out, n_kept, n_hist_max, k_chunk, v_chunk, scale,
                                 o_out, out_dtype, nullptr);
    if (s) return s;
    return omnipage_append(ctx, stream, k_cache_out, v_cache_out, n_kept, k_chunk, v_chunk, t, units_out, n_units_kept,
                           chunk_units, n_chunk_units, n_hist_out, n_units_out);
}

extern "C" omni_status omnitide_chunk_step_host(omnitide_ctx* ctx, void* stream, const void* q_host,
                                                const void* k_chunk_host, const void* v_chunk_host, int32_t t,
                                                const omni_unit* chunk_units_host, int32_t n_chunk_units,
                                                const void* k_cache, const void* v_cache, const int32_t* n_hist_dev,
                                                int32_t n_hist_max, const omni_unit* units, const int32_t* n_units_dev,
                                                int32_t n_units_max, const float* w_modality,
                                                const omni_select_params* params, int32_t page_size, float scale,
                                                void* k_cache_out, void* v_cache_out, omni_unit* units_out,
                                                int32_t* n_hist_out, int32_t* n_units_out, void* o_host, int32_t out_dtype,
                                                omni_compact_info* info_out) {
    if (!ctx) return OMNI_ERR_INVALID_ARG;
    if (!q_host || !k_chunk_host || !v_chunk_host || !o_host || (n_chunk_units > 0 && !chunk_units_host))
        OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "chunk_step_host: null pointer");
    if (t <= 0 || t > ctx->g.t_cap) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "chunk_step_host: t %d outside (0, t_cap]", t);
    if (n_chunk_units < 0 || n_chunk_units > 64) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "chunk_step_host: more than 64 chunk units");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t q_bytes = (size_t)t * ctx->g.h_q * ctx->g.d * ctx->es;
    const size_t kv_bytes = (size_t)t * ctx->row_bytes;
    // Q goes up on the caller's stream and scoring starts behind it; the chunk's K/V rows and unit records,
    // first needed by the attention step, go up on a second stream beside the scoring kernels.
    OMNI_CUDA(ctx, cudaEventRecord(ctx->ev_fork, st));       // orders the upload behind the previous call's readers of the staging
    OMNI_CUDA(ctx, cudaMemcpyAsync(ctx->st_q, q_host, q_bytes, cudaMemcpyHostToDevice, st));
    OMNI_CUDA(ctx, cudaStreamWaitEvent(ctx->aux_stream, ctx->ev_fork, 0));
    OMNI_CUDA(ctx, cudaMemcpyAsync(ctx->st_k, k_chunk_host, kv_bytes, cudaMemcpyHostToDevice, ctx->aux_stream));
    OMNI_CUDA(ctx, cudaMemcpyAsync(ctx->st_v, v_chunk_host, kv_bytes, cudaMemcpyHostToDevice, ctx->aux_stream));
    if (n_chunk_units)
        OMNI_CUDA(ctx, cudaMemcpyAsync(ctx->st_units, chunk_units_host, sizeof(omni_unit) * n_chunk_units,
                                       cudaMemcpyHostToDevice, ctx->aux_stream));
    OMNI_CUDA(ctx, cudaEventRecord(ctx->ev_kv, ctx->aux_stream));
    omni_status s = chunk_step_impl(ctx->ev_kv, ctx, stream, ctx->st_q, ctx->st_k, ctx->st_v, t, ctx->st_units, n_chunk_units,
                                    k_cache, v_cache, n_hist_dev, n_hist_max, units, n_units_dev, n_units_max,
                                    w_modality, params, page_size, scale, k_cache_out, v_cache_out, units_out,
                                    n_hist_out, n_units_out, ctx->st_o, out_dtype, info_out);
    if (s) return s;
    const size_t o_bytes = (size_t)t * ctx->g.h_q * ctx->g.d * (out_dtype == OMNI_DTYPE_FP32 ? 4 : 2);
    OMNI_CUDA(ctx, cudaMemcpyAsync(o_host, ctx->st_o, o_bytes, cudaMemcpyDeviceToHost, st));
    return OMNI_OK;
}

// Staging, stream and events of the pipelined host entry point (synchronous allocation on the first call).
static omni_status pipeline_init(omnitide_ctx* ctx) {
    if (ctx->pl_out) return OMNI_OK;
    const omni_geometry& g = ctx->g;
    const size_t q_elems = (size_t)g.t_cap * g.h_q * g.d;
    for (int b = 0; b < 2; ++b) {
        OMNI_CUDA(ctx, cudaMalloc(&ctx->pl_q[b], q_elems * ctx->es));
        OMNI_CUDA(ctx, cudaMalloc(&ctx->pl_k[b], (size_t)g.t_cap * ctx->row_bytes));
        OMNI_CUDA(ctx, cudaMalloc(&ctx->pl_v[b], (size_t)g.t_cap * ctx->row_bytes));
        OMNI_CUDA(ctx, cudaMalloc(&ctx->pl_o[b], q_elems * 4));
        OMNI_CUDA(ctx, cudaMalloc(reinterpret_cast<void**>(&ctx->pl_units[b]), 64 * sizeof(omni_unit)));
        OMNI_CUDA(ctx, cudaEventCreateWithFlags(&ctx->pl_ev_q[b], cudaEventDisableTiming));
        OMNI_CUDA(ctx, cudaEventCreateWithFlags(&ctx->pl_ev_kv[b], cudaEventDisableTiming));
        OMNI_CUDA(ctx, cudaEventCreateWithFlags(&ctx->pl_ev_done[b], cudaEventDisableTiming));
        OMNI_CUDA(ctx, cudaEventCreateWithFlags(&ctx->pl_ev_out[b], cudaEventDisableTiming));
    }
    OMNI_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->pl_out, cudaStreamNonBlocking));
    return OMNI_OK;
}

extern "C" omni_status omnitide_chunk_step_host_pipelined(omnitide_ctx* ctx, void* stream, const void* q_host,
                                                          const void* k_chunk_host, const void* v_chunk_host, int32_t t,
                                                          const omni_unit* chunk_units_host, int32_t n_chunk_units,
                                                          const void* k_cache, const void* v_cache, const int32_t* n_hist_dev,
                                                          int32_t n_hist_max, const omni_unit* units, const int32_t* n_units_dev,
                                                          int32_t n_units_max, const float* w_modality,
                                                          const omni_select_params* params, int32_t page_size, float scale,
                                                          void* k_cache_out, void* v_cache_out, omni_unit* units_out,
                                                          int32_t* n_hist_out, int32_t* n_units_out, void* o_host,
                                                          int32_t out_dtype, omni_compact_info* info_out) {
    if (!ctx) return OMNI_ERR_INVALID_ARG;
    if (!q_host || !k_chunk_host || !v_chunk_host || !o_host || (n_chunk_units > 0 && !chunk_units_host))
        OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "chunk_step_host_pipelined: null pointer");
    if (t <= 0 || t > ctx->g.t_cap) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "chunk_step_host_pipelined: t %d outside (0, t_cap]", t);
    if (n_chunk_units < 0 || n_chunk_units > 64) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "chunk_step_host_pipelined: more than 64 chunk units");
    const omni_status pi = pipeline_init(ctx);
    if (pi) return pi;
    cudaStream_t st = static_cast<cudaStream_t>(stream), in = ctx->aux_stream, out = ctx->pl_out;
    const int b = (int)(ctx->pl_calls & 1);
    const size_t q_bytes = (size_t)t * ctx->g.h_q * ctx->g.d * ctx->es;
    const size_t kv_bytes = (size_t)t * ctx->row_bytes;
    // uploads: behind the compute of the call before last, which read this buffer; ahead of everything else, so
    // that they run under the previous call's kernels
    OMNI_CUDA(ctx, cudaStreamWaitEvent(in, ctx->pl_ev_done[b], 0));
    OMNI_CUDA(ctx, cudaMemcpyAsync(ctx->pl_q[b], q_host, q_bytes, cudaMemcpyHostToDevice, in));
    OMNI_CUDA(ctx, cudaEventRecord(ctx->pl_ev_q[b], in));
    OMNI_CUDA(ctx, cudaMemcpyAsync(ctx->pl_k[b], k_chunk_host, kv_bytes, cudaMemcpyHostToDevice, in));
    OMNI_CUDA(ctx, cudaMemcpyAsync(ctx->pl_v[b], v_chunk_host, kv_bytes, cudaMemcpyHostToDevice, in));
    if (n_chunk_units)
        OMNI_CUDA(ctx, cudaMemcpyAsync(ctx->pl_units[b], chunk_units_host, sizeof(omni_unit) * n_chunk_units,
                                       cudaMemcpyHostToDevice, in));
    OMNI_CUDA(ctx, cudaEventRecord(ctx->pl_ev_kv[b], in));
    // compute: behind Q and behind the download of the call before last, which read this output buffer
    OMNI_CUDA(ctx, cudaStreamWaitEvent(st, ctx->pl_ev_q[b], 0));
    OMNI_CUDA(ctx, cudaStreamWaitEvent(st, ctx->pl_ev_out[b], 0));
    omni_status s = chunk_step_impl(ctx->pl_ev_kv[b], ctx, stream, ctx->pl_q[b], ctx->pl_k[b], ctx->pl_v[b], t, ctx->pl_units[b],
                                    n_chunk_units, k_cache, v_cache, n_hist_dev, n_hist_max, units, n_units_dev, n_units_max,
                                    w_modality, params, page_size, scale, k_cache_out, v_cache_out, units_out,
                                    n_hist_out, n_units_out, ctx->pl_o[b], out_dtype, info_out);
    if (s) return s;
    OMNI_CUDA(ctx, cudaEventRecord(ctx->pl_ev_done[b], st));
    // download on its own stream, under the next call's kernels
    const size_t o_bytes = (size_t)t * ctx->g.h_q * ctx->g.d * (out_dtype == OMNI_DTYPE_FP32 ? 4 : 2);
    OMNI_CUDA(ctx, cudaStreamWaitEvent(out, ctx->pl_ev_done[b], 0));
    OMNI_CUDA(ctx, cudaMemcpyAsync(o_host, ctx->pl_o[b], o_bytes, cudaMemcpyDeviceToHost, out));
    OMNI_CUDA(ctx, cudaEventRecord(ctx->pl_ev_out[b], out));
    ctx->pl_calls++;
    return OMNI_OK;
}

extern "C" omni_status omnitide_host_wait(omnitide_ctx* ctx) {
    if (!ctx) return OMNI_ERR_INVALID_ARG;
    OMNI_CUDA(ctx, cudaStreamSynchronize(ctx->aux_stream));
    if (ctx->pl_out) OMNI_CUDA(ctx, cudaStreamSynchronize(ctx->pl_out));
    return OMNI_OK;
}
