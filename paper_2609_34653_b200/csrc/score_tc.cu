// Unit scoring on tcgen05 tensor cores (bf16, head dim 128).
//
// score_u needs, for every query row, the softmax mass that falls on each history unit.  One pass
// over QK^T is enough: a CTA owns four 128-row query tiles of one head and one contiguous range
// of 128-key blocks ("split"); for every row a thread keeps a running max m and the sum of
// exp2(c*(s - m)) over the keys of the CURRENT unit, and when the unit (or the split) ends it
// writes the pair (m, sum) -- a flash-style partial -- to scratch.  A second kernel merges a row's
// partials into its normaliser and per-unit masses and reduces them over the 128 rows of a tile; a
// third sums the tiles in a fixed order.  Everything is deterministic (no floating-point atomics).
//
// The kernel is bound by the exponentials (16 per clock per SM on the special-function pipe), not by
// the contraction: a loop of this instruction mix reaches 52 / 72 / 84 / 86 % of that rate with
// 1 / 2 / 3 / 4 warps per scheduler, hence sixteen softmax warps (four per scheduler) and one S
// buffer per tile: while a warpgroup waits for its next S the other three keep the pipe busy.
//
//   warp 17     TMA producer: Q tiles once, then K blocks through a 2-stage shared-memory ring
//   warp 16     one thread issues tcgen05.mma S_t = Q_t K_j^T into TMEM, tile after tile
//   warps 4t..4t+3   row sums of tile t (one thread per row, S read from TMEM in 32-column chunks)
// TMEM map (512 columns): S of tile t at [128 t, 128 t + 128).
#include "common.cuh"

#include <algorithm>
#include <utility>
#include <vector>
#include "tc_ptx.cuh"

namespace {

constexpr int BLK = 128;
constexpr int HD = 128;
constexpr int TILE_BYTES = BLK * HD * 2;
constexpr int HALF_BYTES = TILE_BYTES / 2;
constexpr int NSTAGE = 2;
constexpr int NT = 4;                          // query tiles per CTA
constexpr int SC_THREADS = 32 * (4 * NT + 2);
constexpr int MAX_SPLITS = 64;
constexpr uint32_t IDESC_QK = tc::umma_idesc_bf16(128, 128, false, false);

struct ScoreParams {
    int t, h_q, h_kv;
    const int32_t* n_hist_dev; int n_hist_max;
    const omni_unit* units; const int32_t* n_units_dev; int n_units_max;
    float scale_log2;
    float2* part;             // [tile][seg_cap][128]
    int seg_cap;
    int ctas_per_kv, n_row_tiles, n_splits;                   // CTAs per KV head and split: ceil(n_row_tiles * G / NT)
    int bps;                                                  // key blocks per split (the last split of a history may be shorter)
    int32_t* status;
};

struct Barriers {
    uint64_t q_full;
    uint64_t k_full[NSTAGE];
    uint64_t k_empty[NSTAGE];
    uint64_t s_full[NT];
    uint64_t s_empty[NT];
    uint32_t tmem_base;
    int abort_flag;
};

constexpr int SMEM_FIXED = NT * TILE_BYTES + NSTAGE * TILE_BYTES + 1024 + 256;

using tc::pack2; using tc::unpack2; using tc::fma2; using tc::add2; using tc::max3;

#ifndef SC_POLY_EVERY
#define SC_POLY_EVERY 4        // every n-th pair of exponentials of a full chunk takes the polynomial path (0: none)
#endif
template <int PAIR>
__device__ __forceinline__ uint64_t exp2_pair(uint64_t x2) {
    if (SC_POLY_EVERY > 0 && (PAIR % SC_POLY_EVERY) == SC_POLY_EVERY - 1) return tc::exp2_poly2<4>(x2);
    float x0, x1;
    unpack2(x2, x0, x1);
    return pack2(tc::ex2_approx(x0), tc::ex2_approx(x1));
}

__host__ __device__ __forceinline__ int blocks_per_split(int nkb, int n_splits) { return (nkb + n_splits - 1) / n_splits; }

__global__ void __launch_bounds__(SC_THREADS, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k, const ScoreParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - tc::smem_u32(smem_raw));
    const uint32_t q_smem = smem_base;
    const uint32_t k_smem = smem_base + NT * TILE_BYTES;
    Barriers* bars = reinterpret_cast<Barriers*>(smem_gen + NT * TILE_BYTES + NSTAGE * TILE_BYTES);
    int* unit_end = reinterpret_cast<int*>(smem_gen + NT * TILE_BYTES + NSTAGE * TILE_BYTES + 256);   // [n_units_max]
    volatile int* abort_flag = &bars->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // The four tiles of a CTA share one KV head (hence one K stream): the (row tile, query head of the group)
    // pairs of a KV head are numbered row-tile-major and a CTA takes four consecutive ones, so no tile slot is
    // idle unless n_row_tiles * G is not a multiple of four (G = 4: one row tile, the four heads of the group).
    const int G = p.h_q / p.h_kv;
    const int per_split = p.ctas_per_kv * p.h_kv;
    const int split = blockIdx.x / per_split;
    const int rem = blockIdx.x % per_split;
    const int kvh = rem / p.ctas_per_kv;
    const int c_in_kv = rem % p.ctas_per_kv;
    auto row_of = [&](int tt) { return (c_in_kv * NT + tt) / G; };
    auto head_of = [&](int tt) { return kvh * G + (c_in_kv * NT + tt) % G; };

    int n_units = p.n_units_dev ? *p.n_units_dev : p.n_units_max;
    n_units = max(0, min(n_units, p.n_units_max));
    int n_hist = 0;
    if (n_units > 0) n_hist = p.units[n_units - 1].start + p.units[n_units - 1].len;
    if (n_hist > p.n_hist_max || (p.n_hist_dev && *p.n_hist_dev != n_hist)) {
        if (threadIdx.x == 0) atomicOr(p.status, OMNI_DEV_BAD_COUNT);
        return;
    }
    const int nkb = (n_hist + BLK - 1) / BLK;
    const int bps = p.bps;
    const int b0 = split * bps, b1 = min(nkb, b0 + bps);
    const int nb = b1 - b0;
    if (nb <= 0) return;
    uint32_t active_bits = 0;                  // bit tt: tile slot tt of this CTA holds a (row tile, head) pair
#pragma unroll
    for (int tt = 0; tt < NT; ++tt) active_bits |= (uint32_t)(row_of(tt) < p.n_row_tiles) << tt;
    auto is_active = [&](int tt) { return ((active_bits >> tt) & 1u) != 0; };

    for (int u = threadIdx.x; u < n_units; u += SC_THREADS) unit_end[u] = p.units[u].start + p.units[u].len;
    if (threadIdx.x == 0) {
        tc::mbar_init(tc::smem_u32(&bars->q_full), 1);
        for (int s = 0; s < NSTAGE; ++s) {
            tc::mbar_init(tc::smem_u32(&bars->k_full[s]), 1);
            tc::mbar_init(tc::smem_u32(&bars->k_empty[s]), 1);
        }
        for (int tt = 0; tt < NT; ++tt) {
            tc::mbar_init(tc::smem_u32(&bars->s_full[tt]), 1);
            tc::mbar_init(tc::smem_u32(&bars->s_empty[tt]), 128);
        }
        bars->abort_flag = 0;
        tc::fence_barrier_init();
    }
    if (warp == 4 * NT) tc::tmem_alloc<512>(tc::smem_u32(&bars->tmem_base));
    tc::tcgen05_fence_before();
    __syncthreads();
    tc::tcgen05_fence_after();
    const uint32_t tmem = bars->tmem_base;

    if (warp == 4 * NT + 1) {
        if (lane == 0) {
            tc::tma_prefetch_desc(&tm_q);
            tc::tma_prefetch_desc(&tm_k);
            int n_active = 0;
            for (int tt = 0; tt < NT; ++tt) n_active += (int)is_active(tt);
            tc::mbar_expect_tx(tc::smem_u32(&bars->q_full), n_active * TILE_BYTES);
            for (int tt = 0; tt < NT; ++tt) {
                if (!is_active(tt)) continue;
                const int row0 = row_of(tt) * BLK, head = head_of(tt);
                tc::tma_load_2d(q_smem + tt * TILE_BYTES, &tm_q, head * HD, row0, tc::smem_u32(&bars->q_full));
                tc::tma_load_2d(q_smem + tt * TILE_BYTES + HALF_BYTES, &tm_q, head * HD + 64, row0, tc::smem_u32(&bars->q_full));
            }
            int issued = 0;
            for (int j = 0; j < nb; ++j) {
                const int stage = j % NSTAGE, use = j / NSTAGE;
                if (!tc::mbar_wait(tc::smem_u32(&bars->k_empty[stage]), (use & 1) ^ 1, abort_flag)) break;
                const uint32_t full = tc::smem_u32(&bars->k_full[stage]);
                tc::mbar_expect_tx(full, TILE_BYTES);
                const uint32_t dst = k_smem + stage * TILE_BYTES;
                tc::tma_load_2d(dst, &tm_k, kvh * HD, (b0 + j) * BLK, full);
                tc::tma_load_2d(dst + HALF_BYTES, &tm_k, kvh * HD + 64, (b0 + j) * BLK, full);
                issued = j + 1;
            }
            if (*abort_flag) {
                for (int j = max(0, issued - NSTAGE); j < issued; ++j) {
                    const long long t0 = clock64();
                    while (!tc::mbar_try_wait(tc::smem_u32(&bars->k_full[j % NSTAGE]), (j / NSTAGE) & 1) &&
                           clock64() - t0 < (1ll << 24)) {}
                }
            }
        }
    } else if (warp == 4 * NT) {
        if (lane == 0) {
            const uint64_t q_desc0 = tc::umma_smem_desc(q_smem, 16, 1024), k_desc0 = tc::umma_smem_desc(k_smem, 16, 1024);
            bool ok = tc::mbar_wait(tc::smem_u32(&bars->q_full), 0, abort_flag);
            for (int j = 0; j < nb && ok; ++j) {
                const int stage = j % NSTAGE;
                ok = tc::mbar_wait(tc::smem_u32(&bars->k_full[stage]), (j / NSTAGE) & 1, abort_flag);
                for (int tt = 0; tt < NT && ok; ++tt) {
                    if (!is_active(tt)) continue;
                    ok = tc::mbar_wait(tc::smem_u32(&bars->s_empty[tt]), (j & 1) ^ 1, abort_flag);
                    tc::tcgen05_fence_after();
                    // descriptors differ from the tile's first one only in the address field (16-byte units; no carry out of it)
                    const uint64_t a_desc = q_desc0 + (uint64_t)((tt * TILE_BYTES) >> 4), b_desc = k_desc0 + (uint64_t)((stage * TILE_BYTES) >> 4);
#pragma unroll
                    for (int kk = 0; kk < HD / 16; ++kk) {
                        const uint32_t off = (kk >> 2) * HALF_BYTES + (kk & 3) * 32;
                        tc::umma_ss(tmem + tt * 128, a_desc + (off >> 4), b_desc + (off >> 4), IDESC_QK, kk > 0, 1u);
                    }
                    tc::umma_commit(tc::smem_u32(&bars->s_full[tt]));
                }
                tc::umma_commit(tc::smem_u32(&bars->k_empty[stage]));
            }
        }
    } else {
        const int tt = warp >> 2;
        if (is_active(tt)) {
            const int r = (warp & 3) * 32 + lane;
            const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
            const int tile = head_of(tt) * p.n_row_tiles + row_of(tt);
            float2* part = p.part + (size_t)tile * p.seg_cap * BLK + r;
            const float c = p.scale_log2;
            // unit that holds the first key of this split
            int key = b0 * BLK;
            int u = 0;
            {
                int lo = 0, hi = n_units - 1;          // smallest u with unit_end[u] > key
                while (lo < hi) {
                    const int mid = (lo + hi) >> 1;
                    if (unit_end[mid] > key) hi = mid; else lo = mid + 1;
                }
                u = lo;
            }
            int u_end = unit_end[u];
            float m = -INFINITY, acc = 0.f;
            bool ok = true;
            for (int j = 0; j < nb && ok; ++j) {
                ok = __all_sync(0xffffffffu, tc::mbar_wait(tc::smem_u32(&bars->s_full[tt]), j & 1, abort_flag));
                tc::tcgen05_fence_after();
                const uint32_t s_tmem = tmem + tt * 128 + lane_addr;
                // two register buffers: the TMEM load of chunk ch+1 is in flight while chunk ch is summed
                uint32_t sva[32], svb[32];
                auto process = [&](uint32_t (&sv)[32], const int ch) __attribute__((always_inline)) {
                    const int k0 = key + ch * 32;
                    const int n_valid = min(32, n_hist - k0);           // <= 0 past the end of the history
                    if (n_valid <= 0) return;
                    if (n_valid < 32) {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (i >= n_valid) sv[i] = 0xff800000u;
                    }
                    // row maximum of the chunk: a tree of three-input maxima (depth 4 instead of a chain of 31)
                    float t[11];
#pragma unroll
                    for (int i = 0; i < 10; ++i)
                        t[i] = max3(__uint_as_float(sv[3 * i]), __uint_as_float(sv[3 * i + 1]), __uint_as_float(sv[3 * i + 2]));
                    t[10] = fmaxf(__uint_as_float(sv[30]), __uint_as_float(sv[31]));
                    const float t0 = max3(t[0], t[1], t[2]), t1 = max3(t[3], t[4], t[5]), t2 = max3(t[6], t[7], t[8]);
                    const float cm = max3(max3(t0, t1, t2), t[9], t[10]);
                    const float m_new = fmaxf(m, cm);
                    acc *= tc::ex2_approx((m - m_new) * c);             // exp2(-inf) = 0 on the first chunk
                    m = m_new;
                    const float neg_m = -m * c;
                    if (k0 + 32 <= u_end) {
                        // the whole chunk lies inside the current unit
                        float s0, s1;
                        // pairs of columns: one packed FMA scales two logits, one packed add sums two weights
                        const uint64_t c2 = pack2(c, c), nm2 = pack2(neg_m, neg_m);
                        uint64_t a0 = 0ull, a1 = 0ull;
#define SC_PAIR(i, acc) \
    acc = add2(acc, exp2_pair<(i) / 2>(fma2(pack2(__uint_as_float(sv[i]), __uint_as_float(sv[i + 1])), c2, nm2)));
                        SC_PAIR(0, a0)  SC_PAIR(2, a1)  SC_PAIR(4, a0)  SC_PAIR(6, a1)
                        SC_PAIR(8, a0)  SC_PAIR(10, a1) SC_PAIR(12, a0) SC_PAIR(14, a1)
                        SC_PAIR(16, a0) SC_PAIR(18, a1) SC_PAIR(20, a0) SC_PAIR(22, a1)
                        SC_PAIR(24, a0) SC_PAIR(26, a1) SC_PAIR(28, a0) SC_PAIR(30, a1)
#undef SC_PAIR
                        unpack2(add2(a0, a1), s0, s1);
                        acc += s0 + s1;
                        if (k0 + 32 == u_end && k0 + 32 < n_hist) {
                            part[(size_t)(u + split) * BLK] = make_float2(m, acc);
                            acc = 0.f;
                            ++u;
                            u_end = unit_end[u];
                        }
                    } else {
                        // one or more unit boundaries inside the chunk (same columns for every row)
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            if (k0 + i == u_end && k0 + i < n_hist) {
                                part[(size_t)(u + split) * BLK] = make_float2(m, acc);
                                acc = 0.f;
                                ++u;
                                u_end = unit_end[u];
                            }
                            acc += tc::ex2_approx(fmaf(__uint_as_float(sv[i]), c, neg_m));
                        }
                    }
                };
                tc::tmem_ld32(s_tmem, sva);
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    tc::tmem_wait_ld();
                    tc::tmem_ld32(s_tmem + h * 64 + 32, svb);
                    process(sva, 2 * h);
                    tc::tmem_wait_ld();
                    if (h == 0) {
                        tc::tmem_ld32(s_tmem + 64, sva);
                    } else {
                        // S is in registers: the next block's MMA may overwrite it while the last chunk is summed
                        tc::tcgen05_fence_before();
                        tc::mbar_arrive(tc::smem_u32(&bars->s_empty[tt]));
                    }
                    process(svb, 2 * h + 1);
                }
                key += BLK;
            }
            // the split (or the history) ends inside unit u
            if (ok) part[(size_t)(u + split) * BLK] = make_float2(m, acc);
        }
    }

    tc::tcgen05_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, OMNI_DEV_TIMEOUT);
    if (warp == 4 * NT) {
        tc::tcgen05_fence_after();
        tc::tmem_dealloc<512>(tmem);
    }
}

// Merge the partials of each row, reduce over the 128 rows of a tile: tile_mass[tile][u].
// blockIdx.y cuts the units into COMBINE_Y ranges (every range recomputes the row normaliser, which is cheap).
constexpr int COMBINE_Y = 4;
__global__ void __launch_bounds__(128) score_combine_kernel(const ScoreParams p, float* tile_mass) {
    extern __shared__ int cmb_smem[];
    const int tile = blockIdx.x;
    const int row_tile = tile % p.n_row_tiles;
    const int r = threadIdx.x, lane = r & 31, wid = r >> 5;
    int n_units = p.n_units_dev ? *p.n_units_dev : p.n_units_max;
    n_units = max(0, min(n_units, p.n_units_max));
    if (n_units == 0) return;
    const int n_hist = p.units[n_units - 1].start + p.units[n_units - 1].len;
    if (n_hist > p.n_hist_max) return;
    const int nkb = (n_hist + BLK - 1) / BLK;
    const int bps = p.bps;
    // first and last split of every unit, once per CTA
    int* s_first = cmb_smem;                                  // [n_units]
    int* s_last = cmb_smem + p.n_units_max;                   // [n_units]
    float* red = reinterpret_cast<float*>(cmb_smem + 2 * p.n_units_max);   // [n_units][4]
    for (int u = r; u < n_units; u += 128) {
        const omni_unit un = p.units[u];
        s_first[u] = (un.start / BLK) / bps;
        s_last[u] = ((un.start + un.len - 1) / BLK) / bps;
    }
    __syncthreads();
    const bool valid = row_tile * BLK + r < p.t;
    const float2* part = p.part + (size_t)tile * p.seg_cap * BLK + r;
    const float c = p.scale_log2;
    // the row's partials are the consecutive slots [0, n_units + s_last[n_units-1]]: slot u + s holds (unit u, split s)
    const int n_slots = n_units + s_last[n_units - 1];
    float M = -INFINITY, Z = 0.f;
    if (valid) {
        for (int i0 = 0; i0 < n_slots; i0 += 8) {
            float2 ml[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) ml[k] = i0 + k < n_slots ? part[(size_t)(i0 + k) * BLK] : make_float2(-INFINITY, 0.f);
            float mx = M;
#pragma unroll
            for (int k = 0; k < 8; ++k) mx = fmaxf(mx, ml[k].x);
            float z = Z * tc::ex2_approx((M - mx) * c);
#pragma unroll
            for (int k = 0; k < 8; ++k) z += ml[k].y * tc::ex2_approx((ml[k].x - mx) * c);
            M = mx;
            Z = z;
        }
    }
    const float inv_z = valid ? 1.f / Z : 0.f;
    const int per_y = (n_units + COMBINE_Y - 1) / COMBINE_Y;
    const int u0 = blockIdx.y * per_y, u1 = min(n_units, u0 + per_y);
    for (int u = u0; u < u1; ++u) {
        float v = 0.f;
        if (valid) {
            for (int sp = s_first[u]; sp <= s_last[u]; ++sp) {
                const float2 ml = part[(size_t)(u + sp) * BLK];
                v += ml.y * tc::ex2_approx((ml.x - M) * c);
            }
            v *= inv_z;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) red[u * 4 + wid] = v;
    }
    __syncthreads();
    for (int u = u0 + r; u < u1; u += 128)
        tile_mass[(size_t)tile * p.n_units_max + u] = (red[u * 4] + red[u * 4 + 1]) + (red[u * 4 + 2] + red[u * 4 + 3]);
}

// mass_u = sum over tiles (fixed order) / rows;  score_u = w[modality] * mass_u * N / len_u
__global__ void __launch_bounds__(128) score_finalize_kernel(const float* tile_mass, int n_tiles, const omni_unit* units,
                                                             const int32_t* n_units_dev, int n_units_max, float w0, float w1,
                                                             float w2, float inv_rows, float* scores, float* mass) {
    __shared__ float red[128];
    int n_units = n_units_dev ? *n_units_dev : n_units_max;
    n_units = max(0, min(n_units, n_units_max));
    const int u = blockIdx.x;
    if (u >= n_units) return;
    float v = 0.f;
    for (int t = threadIdx.x; t < n_tiles; t += 128) v += tile_mass[(size_t)t * n_units_max + u];
    red[threadIdx.x] = v;
    __syncthreads();
    for (int s = 64; s > 0; s >>= 1) {
        if (threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const int n_hist = units[n_units - 1].start + units[n_units - 1].len;
        const omni_unit un = units[u];
        const float mu = red[0] * inv_rows;
        const int mod = min(max(un.modality, 0), 2);
        const float w = mod == 0 ? w0 : (mod == 1 ? w1 : w2);
        scores[u] = w * mu * (float)n_hist / (float)un.len;
        if (mass) mass[u] = mu;
    }
}

}  // namespace

omni_status omni_score_tc(omnitide_ctx* ctx, cudaStream_t st, const void* q, int t, const void* k_cache,
                          const int32_t* n_hist_dev, int n_hist_max, const omni_unit* units,
                          const int32_t* n_units_dev, int n_units_max, const float* w, float scale,
                          float* scores_out, float* mass_out) {
    const omni_geometry& g = ctx->g;
    CUtensorMap tm_q, tm_k;
    bool ok = omni_make_map_bf16(ctx->encode_tiled, &tm_q, q, t, (uint64_t)g.h_q * HD, BLK);
    ok &= omni_make_map_bf16(ctx->encode_tiled, &tm_k, k_cache, n_hist_max, (uint64_t)g.h_kv * HD, BLK);
    if (!ok) OMNI_FAIL(ctx, OMNI_ERR_CUDA, "score: cuTensorMapEncodeTiled failed");
    ScoreParams p;
    p.t = t; p.h_q = g.h_q; p.h_kv = g.h_kv; p.n_hist_dev = n_hist_dev; p.n_hist_max = n_hist_max;
    p.units = units; p.n_units_dev = n_units_dev; p.n_units_max = n_units_max;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.part = ctx->score_part; p.seg_cap = g.u_cap + MAX_SPLITS;
    p.n_row_tiles = (t + BLK - 1) / BLK;
    p.status = ctx->status_dev;
    // split the key range so that the grid fills whole waves of SMs and a split keeps >= 8 key blocks
    const int nkb_max = (n_hist_max + BLK - 1) / BLK;
    p.ctas_per_kv = (p.n_row_tiles * (g.h_q / g.h_kv) + NT - 1) / NT;
    const int base_items = p.ctas_per_kv * g.h_kv;
    // cost of a choice = the makespan when the hardware hands the CTAs out in block order to the SMs as they free up
    // (one CTA per SM; a CTA costs its key blocks plus a start-up allowance: Q load, pipeline fill, partial writes).
    // The CTAs of a split have equal length, so the simulation keeps (load, SM count) groups in ascending order.
    // Whole-wave counting misleads here: for a 625-block history it picks 11 even splits (11.3 waves), while 10 splits
    // of 66 blocks with a last one of 31 (10.3 waves, the short pieces filling the partial wave) are 4 % faster
    // (measured, and what this model says).
    if (ctx->sc_split_items != base_items || ctx->sc_split_nkb != nkb_max) {
        constexpr int STARTUP_BLOCKS = 3;
        int best = 1, best_bps = nkb_max;
        long long best_cost = -1;
        std::vector<std::pair<long long, int>> groups;
        for (int ks = 1; ks <= 32 && (ks == 1 || nkb_max / ks >= 8); ++ks) {
            // ks - 1 pieces of bps blocks and a shorter last one: a last piece of about half a piece fills the
            // partial last wave best, so sizes a little above the even one are tried too
            const int even = blocks_per_split(nkb_max, ks);
            for (int bps = even; bps < even + 12 && (ks == 1 ? bps == even : (long long)(ks - 1) * bps < nkb_max); ++bps) {
                groups.assign(1, std::make_pair(0ll, ctx->sm_count));
                long long makespan = 0;
                for (int sp = 0; sp < ks; ++sp) {
                    const int len = std::min(nkb_max, (sp + 1) * bps) - sp * bps;
                    const long long job = len + STARTUP_BLOCKS;
                    int left = base_items;
                    while (left > 0) {
                        const long long a = groups.front().first;
                        const int take = std::min(groups.front().second, left);
                        groups.front().second -= take;
                        if (groups.front().second == 0) groups.erase(groups.begin());
                        const long long b = a + job;
                        auto pos = groups.begin();
                        while (pos != groups.end() && pos->first < b) ++pos;
                        if (pos != groups.end() && pos->first == b) pos->second += take;
                        else groups.insert(pos, std::make_pair(b, take));
                        makespan = std::max(makespan, b);
                        left -= take;
                    }
                }
                if (best_cost < 0 || makespan < best_cost) { best_cost = makespan; best = ks; best_bps = bps; }
            }
        }
        ctx->sc_split_items = base_items;
        ctx->sc_split_nkb = nkb_max;
        ctx->sc_split_best = best;
        ctx->sc_split_bps = best_bps;
    }
    const int best = ctx->sc_split_best;
    p.n_splits = best;
    p.bps = ctx->sc_split_bps;
    const int smem = SMEM_FIXED + n_units_max * (int)sizeof(int);
    if (smem > 227 * 1024) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "score: too many units for one CTA's shared memory");
    OMNI_CUDA(ctx, cudaFuncSetAttribute(score_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    score_tc_kernel<<<base_items * p.n_splits, SC_THREADS, smem, st>>>(tm_q, tm_k, p);
    OMNI_CHECK_LAUNCH(ctx, "score_tc_kernel");
    const int n_tiles = p.n_row_tiles * g.h_q;
    score_combine_kernel<<<dim3(n_tiles, COMBINE_Y), 128, (size_t)n_units_max * 6 * sizeof(int), st>>>(p, ctx->score_tile_mass);
    OMNI_CHECK_LAUNCH(ctx, "score_combine_kernel");
    score_finalize_kernel<<<n_units_max, 128, 0, st>>>(ctx->score_tile_mass, n_tiles, units, n_units_dev, n_units_max,
                                                       w[0], w[1], w[2], 1.0f / ((float)t * g.h_q), scores_out, mass_out);
    OMNI_CHECK_LAUNCH(ctx, "score_finalize_kernel");
    return OMNI_OK;
}
