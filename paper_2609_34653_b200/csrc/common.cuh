// Shared host-side definitions of the library: the context, error helpers, launch accounting.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include "../../include/omnitide.h"

struct omnitide_ctx {
    omni_geometry g;
    int device;
    int sm_count;
    int es;                       // element size of the storage dtype
    size_t row_bytes;             // h_kv * d * es : one cache row
    int32_t* status_dev;          // device status word (OMNI_DEV_* bits)
    // ---- scratch owned by the context -------------------------------------------------
    float2* score_part;           // [row tiles][u_cap][128] per-(row, unit) (max, sum) partials
    float* score_tile_mass;       // [row tiles][u_cap] per-tile unit mass
    double* score_mass64;         // [u_cap] accumulator of the CUDA-core scoring path
    int32_t* score_seg;           // unit boundaries per key block (built per call)
    void* inplace_k;              // staging for in-place compaction, allocated on first use
    void* inplace_v;
    size_t inplace_rows;
    int32_t* mig_plan;            // [8] plan of the ordered-suffix migration, allocated on first use
    int32_t* mc_moves;            // [2 s_cap] (source, destination) pairs of the class-aware migration, allocated on first use
    uint8_t* mc_class;            // [s_cap] class bytes of its moved entries
    unsigned long long* cp_words; // [SMs] per-CTA count words of the compaction kernel, tagged with cp_epoch
    uint32_t cp_epoch;            // launches of the compaction kernel on this context so far
    // work buffers of omnitide_chunk_step
    float* ws_scores;             // [u_cap]
    uint8_t* ws_unit_keep;        // [u_cap]
    int32_t* ws_kept_len;         // [u_cap] tokens kept at the start of every unit (structural plan)
    uint8_t* ws_keep_mask;        // [s_cap]
    int32_t* ws_slot_map;         // [s_cap]
    int32_t* ws_counts;           // {n_kept, n_units_kept}
    omni_compact_info* ws_info;
    // staging of omnitide_chunk_step_host
    void* st_q; void* st_k; void* st_v; void* st_o; omni_unit* st_units;
    cudaStream_t aux_stream;      // carries the K/V chunk upload of chunk_step_host beside the scoring kernels
    cudaEvent_t ev_fork, ev_kv;
    // double-buffered staging of omnitide_chunk_step_host_pipelined, allocated on first use
    void* pl_q[2]; void* pl_k[2]; void* pl_v[2]; void* pl_o[2]; omni_unit* pl_units[2];
    cudaStream_t pl_out;          // carries the downloads; the uploads ride on aux_stream
    cudaEvent_t pl_ev_q[2], pl_ev_kv[2], pl_ev_done[2], pl_ev_out[2];
    int64_t pl_calls;             // pipelined calls so far: call n uses buffer n & 1
    // attention split-KV partials
    float* attn_part_o;           // allocated on first use
    float* attn_part_ml;
    size_t attn_part_cap;
    int32_t* attn_live_idx;       // [s_cap / 128 + 2] blocks of the history that hold a live slot (masked attention)
    uint4* attn_live_mask;        // [s_cap / 128 + 2] their 128 live bits
    int32_t* attn_n_live;
    int32_t* dec_counter;         // [h_kv] arrival counters of the decode kernel, zero between launches
    bool attn_attr_set;           // the attention kernel's shared-memory limit has been raised on this device
    // -----------------------------------------------------------------------------------
    void* encode_tiled;           // cuTensorMapEncodeTiled, resolved through the runtime
    int64_t launches;
    bool force_cuda_cores;        // OMNI_OPT_FORCE_CUDA_CORES
    int sc_split_items, sc_split_nkb, sc_split_best, sc_split_bps;   // the scoring kernel's last split decision (work items, key blocks -> splits)
    int score_window;             // OMNI_OPT_SCORE_WINDOW: trailing queries that score in omnitide_chunk_step (0: all)
    int high_watermark;           // OMNI_OPT_HIGH_WATERMARK: omnitide_chunk_step runs a retention round only above it (0: always)
    char err[256];
};

#define OMNI_FAIL(ctx, code, ...)                                   \
    do {                                                            \
        if (ctx) snprintf((ctx)->err, sizeof((ctx)->err), __VA_ARGS__); \
        return (code);                                              \
    } while (0)

#define OMNI_CUDA(ctx, expr)                                                          \
    do {                                                                              \
        cudaError_t e__ = (expr);                                                     \
        if (e__ != cudaSuccess)                                                       \
            OMNI_FAIL(ctx, OMNI_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e__)); \
    } while (0)

#define OMNI_CHECK_LAUNCH(ctx, name)                                                   \
    do {                                                                               \
        cudaError_t e__ = cudaGetLastError();                                          \
        if (e__ != cudaSuccess)                                                        \
            OMNI_FAIL(ctx, OMNI_ERR_CUDA, "launch %s: %s", name, cudaGetErrorString(e__)); \
        (ctx)->launches++;                                                             \
    } while (0)

static inline bool omni_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// internal entry points implemented per file
omni_status omni_inplace_staging(omnitide_ctx* ctx);   // allocates inplace_k / inplace_v (s_cap rows each) on first use
omni_status omni_attention_tc(omnitide_ctx* ctx, cudaStream_t st, const void* q, int t, const void* k_hist,
                              const void* v_hist, const int32_t* n_hist_dev, int n_hist_max, const void* k_chunk,
                              const void* v_chunk, float scale, void* o_out, int out_dtype, float* lse_out,
                              const uint8_t* hist_mask);
omni_status omni_attention_decode(omnitide_ctx* ctx, cudaStream_t st, const void* q, const void* k_hist, const void* v_hist,
                                  const int32_t* n_hist_dev, int n_hist_max, const void* k_chunk, const void* v_chunk,
                                  float scale, void* o_out, int out_dtype, float* lse_out);
omni_status omni_score_tc(omnitide_ctx* ctx, cudaStream_t st, const void* q, int t, const void* k_cache,
                          const int32_t* n_hist_dev, int n_hist_max, const omni_unit* units,
                          const int32_t* n_units_dev, int n_units_max, const float* w, float scale,
                          float* scores_out, float* mass_out);
omni_status omni_attention_simple(omnitide_ctx* ctx, cudaStream_t st, const void* q, int t, const void* k_hist,
                                  const void* v_hist, const int32_t* n_hist_dev, int n_hist_max, const void* k_chunk,
                                  const void* v_chunk, float scale, void* o_out, int out_dtype, float* lse_out,
                                  const uint8_t* hist_mask);
omni_status omni_score_simple(omnitide_ctx* ctx, cudaStream_t st, const void* q, int t, const void* k_cache,
                              const int32_t* n_hist_dev, int n_hist_max, const omni_unit* units,
                              const int32_t* n_units_dev, int n_units_max, const float* w, float scale,
                              float* scores_out, float* mass_out);
