// GQA chunk-prefill attention on tcgen05 tensor cores (bf16, head dim 128).
//
// One CTA owns a pair of 128-row query tiles of one head and walks the KV sequence (history blocks,
// then the causal chunk blocks) in 128-key blocks:
//   warp 9      TMA producer: Q tiles once, then K_j / V_j tiles through a 4-stage shared-memory ring
//   warp 8      one thread issues tcgen05.mma: S_t = Q_t K_j^T (operands in shared memory) and
//               O_t += P_t V_j (P read from tensor memory, V as an MN-major shared-memory operand)
//   warps 0-3   softmax of tile 0, one thread per query row: S from TMEM, running max with lazy
//   warps 4-7   rescale of O, exp2, P written back to TMEM as bf16 over the S columns; same for tile 1
// The two tiles alternate on the tensor pipe, so one tile's softmax overlaps the other's MMAs.
// TMEM map (512 columns): S0/P0 [0,128)  S1/P1 [128,256)  O0 [256,384)  O1 [384,512).
#include "common.cuh"
#include "tc_ptx.cuh"

namespace {

constexpr int BLK = 128;                 // rows per query tile and keys per KV block
constexpr int HD = 128;                  // head dim
constexpr int TILE_BYTES = BLK * HD * 2; // 32 KiB, stored as two 64-column halves of 16 KiB
constexpr int HALF_BYTES = TILE_BYTES / 2;
constexpr int NSTAGE = 4;
constexpr int ATT_THREADS = 320;
constexpr int SMEM_BYTES = 2 * TILE_BYTES + NSTAGE * TILE_BYTES + 1024 /*alignment*/ + 256 /*barriers*/;
constexpr float RESCALE_THRESHOLD = 8.0f;   // log2 units: P stays below 2^8

constexpr uint32_t IDESC_QK = tc::umma_idesc_bf16(128, 128, false, false);
constexpr uint32_t IDESC_PV = tc::umma_idesc_bf16(128, 128, false, true);

struct AttnParams {
    int t, h_q, h_kv;
    const int32_t* n_hist_dev; int n_hist_max;
    float scale_log2, scale;
    void* o_out; int out_dtype; float* lse_out;
    int32_t* status;
    int n_pairs;
};

struct Barriers {
    uint64_t q_full;
    uint64_t kv_full[NSTAGE];
    uint64_t kv_empty[NSTAGE];
    uint64_t s_full[2];
    uint64_t p_full[2];
    uint64_t o_done;
    uint32_t tmem_base;
    int abort_flag;
};

__global__ void __launch_bounds__(ATT_THREADS, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kh,
                    const __grid_constant__ CUtensorMap tm_vh, const __grid_constant__ CUtensorMap tm_kc,
                    const __grid_constant__ CUtensorMap tm_vc, const AttnParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - tc::smem_u32(smem_raw));
    const uint32_t q_smem = smem_base;                       // 2 tiles
    const uint32_t kv_smem = smem_base + 2 * TILE_BYTES;     // NSTAGE tiles
    Barriers* bars = reinterpret_cast<Barriers*>(smem_gen + 2 * TILE_BYTES + NSTAGE * TILE_BYTES);
    volatile int* abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // heavy work first: later row pairs see more causal blocks
    const int item = blockIdx.x;
    const int pair = p.n_pairs - 1 - item / p.h_q;
    const int head = item % p.h_q;
    const int kvh = head / (p.h_q / p.h_kv);

    int n_hist = p.n_hist_dev ? *p.n_hist_dev : p.n_hist_max;
    if (n_hist < 0 || n_hist > p.n_hist_max) {
        if (threadIdx.x == 0) atomicOr(p.status, OMNI_DEV_BAD_COUNT);
        n_hist = max(0, min(n_hist, p.n_hist_max));
    }
    const int nhb = (n_hist + BLK - 1) / BLK;
    const int hist_tail = n_hist - (nhb - 1) * BLK;          // valid keys in the last history block (if nhb > 0)
    const bool tail_partial = nhb > 0 && hist_tail < BLK;
    // tile tt covers chunk rows [(2*pair+tt)*128, +128); it needs chunk blocks 0 .. 2*pair+tt
    int nb[2];
#pragma unroll
    for (int tt = 0; tt < 2; ++tt) {
        const int row0 = (2 * pair + tt) * BLK;
        nb[tt] = row0 < p.t ? nhb + 2 * pair + tt + 1 : 0;
    }
    const int nb_max = max(nb[0], nb[1]);

    if (threadIdx.x == 0) {
        tc::mbar_init(tc::smem_u32(&bars->q_full), 1);
        for (int s = 0; s < NSTAGE; ++s) {
            tc::mbar_init(tc::smem_u32(&bars->kv_full[s]), 1);
            tc::mbar_init(tc::smem_u32(&bars->kv_empty[s]), 1);
        }
        for (int tt = 0; tt < 2; ++tt) {
            tc::mbar_init(tc::smem_u32(&bars->s_full[tt]), 1);
            tc::mbar_init(tc::smem_u32(&bars->p_full[tt]), 128);
        }
        tc::mbar_init(tc::smem_u32(&bars->o_done), 1);
        bars->abort_flag = 0;
        tc::fence_barrier_init();
    }
    if (warp == 8) tc::tmem_alloc<512>(tc::smem_u32(&bars->tmem_base));
    tc::tcgen05_fence_before();
    __syncthreads();
    tc::tcgen05_fence_after();
    const uint32_t tmem = bars->tmem_base;

    if (warp == 9) {
        // ================================ TMA producer ================================
        if (lane == 0) {
            tc::tma_prefetch_desc(&tm_q);
            tc::tma_prefetch_desc(&tm_kh);
            tc::tma_prefetch_desc(&tm_vh);
            tc::tma_prefetch_desc(&tm_kc);
            tc::tma_prefetch_desc(&tm_vc);
            const int n_active = (nb[0] > 0) + (nb[1] > 0);
            tc::mbar_expect_tx(tc::smem_u32(&bars->q_full), n_active * TILE_BYTES);
            for (int tt = 0; tt < 2; ++tt) {
                if (nb[tt] == 0) continue;
                const int row0 = (2 * pair + tt) * BLK;
                tc::tma_load_2d(q_smem + tt * TILE_BYTES, &tm_q, head * HD, row0, tc::smem_u32(&bars->q_full));
                tc::tma_load_2d(q_smem + tt * TILE_BYTES + HALF_BYTES, &tm_q, head * HD + 64, row0, tc::smem_u32(&bars->q_full));
            }
            const int n_loads = 2 * nb_max;
            int issued = 0;
            for (int idx = 0; idx < n_loads; ++idx) {
                const int j = idx >> 1, is_v = idx & 1;
                const int stage = idx % NSTAGE, use = idx / NSTAGE;
                if (!tc::mbar_wait(tc::smem_u32(&bars->kv_empty[stage]), (use & 1) ^ 1, abort_flag)) break;
                const uint32_t full = tc::smem_u32(&bars->kv_full[stage]);
                tc::mbar_expect_tx(full, TILE_BYTES);
                const bool hist = j < nhb;
                const CUtensorMap* map = hist ? (is_v ? &tm_vh : &tm_kh) : (is_v ? &tm_vc : &tm_kc);
                const int row = (hist ? j : j - nhb) * BLK;
                const uint32_t dst = kv_smem + stage * TILE_BYTES;
                tc::tma_load_2d(dst, map, kvh * HD, row, full);
                tc::tma_load_2d(dst + HALF_BYTES, map, kvh * HD + 64, row, full);
                issued = idx + 1;
            }
            if (*abort_flag) {
                // unwind: let copies still in flight land before the CTA exits (bounded by the abort flag)
                for (int idx = max(0, issued - NSTAGE); idx < issued; ++idx) {
                    const long long t0 = clock64();
                    while (!tc::mbar_try_wait(tc::smem_u32(&bars->kv_full[idx % NSTAGE]), (idx / NSTAGE) & 1) &&
                           clock64() - t0 < (1ll << 24)) {}
                }
            }
        }
    } else if (warp == 8) {
        // ================================ MMA issuer ================================
        if (lane == 0 && nb_max > 0) {
            bool ok = tc::mbar_wait(tc::smem_u32(&bars->q_full), 0, abort_flag);
            auto issue_qk = [&](int tt, int stage) {
                const uint32_t a0 = q_smem + tt * TILE_BYTES, b0 = kv_smem + stage * TILE_BYTES;
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {
                    const uint32_t off = (kk >> 2) * HALF_BYTES + (kk & 3) * 32;
                    tc::umma_ss(tmem + tt * 128, tc::umma_smem_desc(a0 + off, 16, 1024),
                                tc::umma_smem_desc(b0 + off, 16, 1024), IDESC_QK, kk > 0);
                }
            };
            auto issue_pv = [&](int tt, int stage, bool accumulate) {
                const uint32_t b0 = kv_smem + stage * TILE_BYTES;
#pragma unroll
                for (int kk = 0; kk < BLK / 16; ++kk) {
                    tc::umma_ts(tmem + 256 + tt * 128, tmem + tt * 128 + kk * 8,
                                tc::umma_smem_desc(b0 + kk * 2048, HALF_BYTES, 1024), IDESC_PV, accumulate || kk > 0);
                }
            };
            // S_t(0)
            if (ok) ok = tc::mbar_wait(tc::smem_u32(&bars->kv_full[0]), 0, abort_flag);
            tc::tcgen05_fence_after();
            for (int tt = 0; tt < 2; ++tt)
                if (nb[tt] > 0) {
                    issue_qk(tt, 0);
                    tc::umma_commit(tc::smem_u32(&bars->s_full[tt]));
                }
            tc::umma_commit(tc::smem_u32(&bars->kv_empty[0]));
            for (int j = 0; j < nb_max && ok; ++j) {
                const int v_idx = 2 * j + 1, v_stage = v_idx % NSTAGE;
                const int k_idx = 2 * j + 2, k_stage = k_idx % NSTAGE;
                const bool has_next = j + 1 < nb_max;
                ok = tc::mbar_wait(tc::smem_u32(&bars->kv_full[v_stage]), (v_idx / NSTAGE) & 1, abort_flag);
                if (ok && has_next) ok = tc::mbar_wait(tc::smem_u32(&bars->kv_full[k_stage]), (k_idx / NSTAGE) & 1, abort_flag);
                for (int tt = 0; tt < 2 && ok; ++tt) {
                    if (j < nb[tt]) {
                        ok = tc::mbar_wait(tc::smem_u32(&bars->p_full[tt]), j & 1, abort_flag);
                        tc::tcgen05_fence_after();
                        issue_pv(tt, v_stage, j > 0);
                    }
                    if (j + 1 < nb[tt]) {
                        issue_qk(tt, k_stage);
                        tc::umma_commit(tc::smem_u32(&bars->s_full[tt]));
                    }
                }
                tc::umma_commit(tc::smem_u32(&bars->kv_empty[v_stage]));
                if (has_next) tc::umma_commit(tc::smem_u32(&bars->kv_empty[k_stage]));
            }
            tc::umma_commit(tc::smem_u32(&bars->o_done));
        }
    } else {
        // ================================ softmax + epilogue ================================
        const int tt = warp >> 2;                          // tile of this warpgroup
        const int r = (warp & 3) * 32 + lane;              // row inside the tile == TMEM lane
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t s_tmem = tmem + tt * 128 + lane_addr;
        const uint32_t o_tmem = tmem + 256 + tt * 128 + lane_addr;
        const int row0 = (2 * pair + tt) * BLK;
        const int my_nb = nb[tt];
        const int diag_block = nhb + 2 * pair + tt;        // KV block index of the causal diagonal
        float m_ref = 0.f, l_sum = 0.f;
        bool ok = true;

        for (int j = 0; j < my_nb && ok; ++j) {
            ok = __all_sync(0xffffffffu, tc::mbar_wait(tc::smem_u32(&bars->s_full[tt]), j & 1, abort_flag));
            tc::tcgen05_fence_after();
            uint32_t sv[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) tc::tmem_ld32(s_tmem + c * 32, sv[c]);
            tc::tmem_wait_ld();

            // masking: ragged history tail, causal diagonal
            int n_valid = BLK;
            if (j == nhb - 1 && tail_partial) n_valid = hist_tail;
            if (j == diag_block) n_valid = r + 1;
            if (n_valid < BLK) {
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (c * 32 + i >= n_valid) sv[c][i] = 0xff800000u;   // -inf
            }
            float bm = -INFINITY;
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
                for (int i = 0; i < 32; ++i) bm = fmaxf(bm, __uint_as_float(sv[c][i]));
            if (bm == -INFINITY) bm = 0.f;

            float alpha = 1.f;
            bool need = false;
            if (j == 0) {
                m_ref = bm;
            } else if ((bm - m_ref) * p.scale_log2 > RESCALE_THRESHOLD) {
                alpha = tc::ex2_approx((m_ref - bm) * p.scale_log2);
                m_ref = bm;
                need = true;
            }
            if (__any_sync(0xffffffffu, need)) {
                // O_t of the previous blocks is complete: S_t(j) was committed after PV_t(j-1)
                l_sum *= alpha;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t ov[32];
                    tc::tmem_ld32(o_tmem + c * 32, ov);
                    tc::tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha);
                    tc::tmem_st32(o_tmem + c * 32, ov);
                }
            }
            const float neg_m = -m_ref * p.scale_log2;
            float rs = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float p0 = tc::ex2_approx(fmaf(__uint_as_float(sv[c][2 * i]), p.scale_log2, neg_m));
                    const float p1 = tc::ex2_approx(fmaf(__uint_as_float(sv[c][2 * i + 1]), p.scale_log2, neg_m));
                    pk[i] = tc::pack_bf16x2(p0, p1);
                    // the normaliser sums the ROUNDED weights the tensor core will use, so that the
                    // weights of a row sum to one exactly and the rounding of a dominant weight cancels
                    rs += __uint_as_float(pk[i] << 16) + __uint_as_float(pk[i] & 0xffff0000u);
                }
                tc::tmem_st16(s_tmem + c * 16, pk);
            }
            l_sum += rs;

            if (tt == 0 && tail_partial && j == nhb - 1) {
                // rows of the V tile past the end of the history may hold anything: zero them
                const int v_idx = 2 * j + 1, v_stage = v_idx % NSTAGE;
                ok = __all_sync(0xffffffffu, tc::mbar_wait(tc::smem_u32(&bars->kv_full[v_stage]), (v_idx / NSTAGE) & 1, abort_flag));
                if (r >= hist_tail) {
                    uint4* row_a = reinterpret_cast<uint4*>(smem_gen + 2 * TILE_BYTES + v_stage * TILE_BYTES + r * 128);
                    uint4* row_b = reinterpret_cast<uint4*>(smem_gen + 2 * TILE_BYTES + v_stage * TILE_BYTES + HALF_BYTES + r * 128);
#pragma unroll
                    for (int i = 0; i < 8; ++i) { row_a[i] = make_uint4(0, 0, 0, 0); row_b[i] = make_uint4(0, 0, 0, 0); }
                }
                tc::fence_proxy_async_smem();
            }
            tc::tmem_wait_st();
            tc::tcgen05_fence_before();
            tc::mbar_arrive(tc::smem_u32(&bars->p_full[tt]));
        }

        if (my_nb > 0) {
            ok = __all_sync(0xffffffffu, ok && tc::mbar_wait(tc::smem_u32(&bars->o_done), 0, abort_flag));
            tc::tcgen05_fence_after();
            const int row = row0 + r;
            const float inv = 1.f / l_sum;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t ov[32];
                tc::tmem_ld32(o_tmem + c * 32, ov);
                tc::tmem_wait_ld();
                if (row < p.t && ok) {
                    const size_t off = ((size_t)row * p.h_q + head) * HD + c * 32;
                    if (p.out_dtype == OMNI_DTYPE_FP32) {
                        float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.o_out) + off);
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            dst[i] = make_float4(__uint_as_float(ov[4 * i]) * inv, __uint_as_float(ov[4 * i + 1]) * inv,
                                                 __uint_as_float(ov[4 * i + 2]) * inv, __uint_as_float(ov[4 * i + 3]) * inv);
                    } else {
                        uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.o_out) + off);
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            uint4 v;
                            v.x = tc::pack_bf16x2(__uint_as_float(ov[8 * i]) * inv, __uint_as_float(ov[8 * i + 1]) * inv);
                            v.y = tc::pack_bf16x2(__uint_as_float(ov[8 * i + 2]) * inv, __uint_as_float(ov[8 * i + 3]) * inv);
                            v.z = tc::pack_bf16x2(__uint_as_float(ov[8 * i + 4]) * inv, __uint_as_float(ov[8 * i + 5]) * inv);
                            v.w = tc::pack_bf16x2(__uint_as_float(ov[8 * i + 6]) * inv, __uint_as_float(ov[8 * i + 7]) * inv);
                            dst[i] = v;
                        }
                    }
                }
            }
            if (p.lse_out && row < p.t && ok)
                p.lse_out[(size_t)row * p.h_q + head] = m_ref * p.scale + logf(l_sum);
        }
    }

    tc::tcgen05_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, OMNI_DEV_TIMEOUT);
    if (warp == 8) {
        tc::tcgen05_fence_after();
        tc::tmem_dealloc<512>(tmem);
    }
}

}  // namespace

omni_status omni_attention_tc(omnitide_ctx* ctx, cudaStream_t st, const void* q, int t, const void* k_hist,
                              const void* v_hist, const int32_t* n_hist_dev, int n_hist_max, const void* k_chunk,
                              const void* v_chunk, float scale, void* o_out, int out_dtype, float* lse_out) {
    const omni_geometry& g = ctx->g;
    CUtensorMap tm_q, tm_kh, tm_vh, tm_kc, tm_vc;
    const uint64_t q_inner = (uint64_t)g.h_q * HD, kv_inner = (uint64_t)g.h_kv * HD;
    bool ok = omni_make_map_bf16(ctx->encode_tiled, &tm_q, q, t, q_inner, BLK);
    ok &= omni_make_map_bf16(ctx->encode_tiled, &tm_kc, k_chunk, t, kv_inner, BLK);
    ok &= omni_make_map_bf16(ctx->encode_tiled, &tm_vc, v_chunk, t, kv_inner, BLK);
    // with an empty history the history maps are never used; point them at the chunk to stay valid
    ok &= omni_make_map_bf16(ctx->encode_tiled, &tm_kh, n_hist_max > 0 ? k_hist : k_chunk, n_hist_max > 0 ? n_hist_max : t, kv_inner, BLK);
    ok &= omni_make_map_bf16(ctx->encode_tiled, &tm_vh, n_hist_max > 0 ? v_hist : v_chunk, n_hist_max > 0 ? n_hist_max : t, kv_inner, BLK);
    if (!ok) OMNI_FAIL(ctx, OMNI_ERR_CUDA, "attention: cuTensorMapEncodeTiled failed");
    AttnParams p;
    p.t = t; p.h_q = g.h_q; p.h_kv = g.h_kv; p.n_hist_dev = n_hist_dev; p.n_hist_max = n_hist_max;
    p.scale = scale; p.scale_log2 = scale * 1.4426950408889634f;
    p.o_out = o_out; p.out_dtype = out_dtype; p.lse_out = lse_out; p.status = ctx->status_dev;
    p.n_pairs = (t + 2 * BLK - 1) / (2 * BLK);
    static bool attr_set = false;
    if (!attr_set) {
        OMNI_CUDA(ctx, cudaFuncSetAttribute(attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
        attr_set = true;
    }
    attention_tc_kernel<<<p.n_pairs * g.h_q, ATT_THREADS, SMEM_BYTES, st>>>(tm_q, tm_kh, tm_vh, tm_kc, tm_vc, p);
    OMNI_CHECK_LAUNCH(ctx, "attention_tc_kernel");
    return OMNI_OK;
}
