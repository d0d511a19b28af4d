// GQA chunk-prefill attention on tcgen05 tensor cores (bf16, head dim 128).
//
// Work unit: one 128-key KV block of one "item" = (pair of 128-row query tiles, head).  The KV sequence
// of an item is the history blocks followed by the causal chunk blocks.  The kernel is persistent, one
// CTA per SM: the units of all items are laid end to end and cut into equal contiguous shares, so every
// SM gets the same amount of tensor work whatever the number of items.  A share is a list of "parts"
// (item, block range).  A part that covers its whole item writes the output directly; an item cut
// between CTAs leaves un-normalised partial outputs with their (max, sum) in scratch and a small
// second kernel merges them.
//
// Inside a CTA:
//   warp 9      TMA producer: the part's Q tiles, then K_j / V_j tiles through a 4-stage shared-memory ring
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
    float* part_o;        // [cta][2 slots][2 tiles][128 rows][128] un-normalised partial outputs
    float2* part_ml;      // [cta][2 slots][2 tiles][128 rows] (running max, sum)
};

struct Barriers {
    uint64_t q_full;
    uint64_t kv_full[NSTAGE];
    uint64_t kv_empty[NSTAGE];
    uint64_t s_full[2];
    uint64_t p_full[2];
    uint64_t o_done;
    uint64_t o_free[2];
    uint32_t tmem_base;
    int abort_flag;
};

// ---- the work list: identical arithmetic in every role and in the merge kernel --------------------------
struct Sched {
    int nhb, n_pairs, h_q, t;
    __device__ int nb_pair(int pair) const {                 // KV blocks of an item = blocks of its last active tile
        return nhb + 2 * pair + (((2 * pair + 1) * BLK < t) ? 2 : 1);
    }
    __device__ long long total() const {
        long long w = 0;
        for (int pr = 0; pr < n_pairs; ++pr) w += (long long)h_q * nb_pair(pr);
        return w;
    }
    // items are ordered by descending pair, then head
    __device__ long long item_begin(int pair, int head) const {
        long long w = 0;
        for (int pr = n_pairs - 1; pr > pair; --pr) w += (long long)h_q * nb_pair(pr);
        return w + (long long)head * nb_pair(pair);
    }
    __device__ void locate(long long w, int& pair, int& head, int& j) const {
        long long base = 0;
        for (int pr = n_pairs - 1; pr >= 0; --pr) {
            const int nb = nb_pair(pr);
            const long long span = (long long)h_q * nb;
            if (w < base + span || pr == 0) {
                pair = pr;
                head = (int)((w - base) / nb);
                j = (int)((w - base) - (long long)head * nb);
                return;
            }
            base += span;
        }
    }
};
__device__ __forceinline__ long long share_begin(long long total, int cta, int n_cta) { return total * cta / n_cta; }

struct Part {
    int pair, head, j0, j1, nb_item;
    int cnt0, cnt1;       // blocks of this part tile 0 / tile 1 takes part in
    bool final_;          // the part covers the whole item
    int slot;             // partial slot of this CTA (when not final)
};

struct PartIter {
    Sched s;
    long long w, w_end;
    __device__ bool next(Part& p) {
        if (w >= w_end) return false;
        s.locate(w, p.pair, p.head, p.j0);
        p.nb_item = s.nb_pair(p.pair);
        const long long room = w_end - w;
        p.j1 = (int)min((long long)p.nb_item, (long long)p.j0 + room);
        w += p.j1 - p.j0;
        const int nb_t0 = (2 * p.pair) * BLK < s.t ? s.nhb + 2 * p.pair + 1 : 0;
        const int nb_t1 = (2 * p.pair + 1) * BLK < s.t ? s.nhb + 2 * p.pair + 2 : 0;
        p.cnt0 = max(0, min(p.j1, nb_t0) - p.j0);
        p.cnt1 = max(0, min(p.j1, nb_t1) - p.j0);
        p.final_ = p.j0 == 0 && p.j1 == p.nb_item;
        p.slot = p.j0 > 0 ? 0 : 1;
        return true;
    }
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

    int n_hist = p.n_hist_dev ? *p.n_hist_dev : p.n_hist_max;
    if (n_hist < 0 || n_hist > p.n_hist_max) {
        if (threadIdx.x == 0 && blockIdx.x == 0) atomicOr(p.status, OMNI_DEV_BAD_COUNT);
        n_hist = max(0, min(n_hist, p.n_hist_max));
    }
    const int nhb = (n_hist + BLK - 1) / BLK;
    const int hist_tail = n_hist - (nhb - 1) * BLK;          // valid keys in the last history block (if nhb > 0)
    const bool tail_partial = nhb > 0 && hist_tail < BLK;

    PartIter it;
    it.s.nhb = nhb; it.s.n_pairs = p.n_pairs; it.s.h_q = p.h_q; it.s.t = p.t;
    {
        const long long total = it.s.total();
        it.w = share_begin(total, blockIdx.x, gridDim.x);
        it.w_end = share_begin(total, blockIdx.x + 1, gridDim.x);
    }
    if (it.w >= it.w_end) return;                            // more CTAs than units

    if (threadIdx.x == 0) {
        tc::mbar_init(tc::smem_u32(&bars->q_full), 1);
        for (int s = 0; s < NSTAGE; ++s) {
            tc::mbar_init(tc::smem_u32(&bars->kv_full[s]), 1);
            tc::mbar_init(tc::smem_u32(&bars->kv_empty[s]), 1);
        }
        for (int tt = 0; tt < 2; ++tt) {
            tc::mbar_init(tc::smem_u32(&bars->s_full[tt]), 1);
            tc::mbar_init(tc::smem_u32(&bars->p_full[tt]), 128);
            tc::mbar_init(tc::smem_u32(&bars->o_free[tt]), 128);
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

    Part part;
    int part_idx = 0;
    int kv_base = 0;                                         // K/V tiles loaded by earlier parts of this CTA

    if (warp == 9) {
        // ================================ TMA producer ================================
        if (lane == 0) {
            tc::tma_prefetch_desc(&tm_q);
            tc::tma_prefetch_desc(&tm_kh);
            tc::tma_prefetch_desc(&tm_vh);
            tc::tma_prefetch_desc(&tm_kc);
            tc::tma_prefetch_desc(&tm_vc);
            int issued = 0;
            bool ok = true;
            while (ok && it.next(part)) {
                // the Q tiles are free once every MMA of the previous part has completed
                if (part_idx > 0) ok = tc::mbar_wait(tc::smem_u32(&bars->o_done), (part_idx - 1) & 1, abort_flag);
                if (!ok) break;
                const int kvh = part.head / (p.h_q / p.h_kv);
                const int n_active = (part.cnt0 > 0) + (part.cnt1 > 0);
                tc::mbar_expect_tx(tc::smem_u32(&bars->q_full), n_active * TILE_BYTES);
                for (int tt = 0; tt < 2; ++tt) {
                    if ((tt ? part.cnt1 : part.cnt0) == 0) continue;
                    const int row0 = (2 * part.pair + tt) * BLK;
                    tc::tma_load_2d(q_smem + tt * TILE_BYTES, &tm_q, part.head * HD, row0, tc::smem_u32(&bars->q_full));
                    tc::tma_load_2d(q_smem + tt * TILE_BYTES + HALF_BYTES, &tm_q, part.head * HD + 64, row0,
                                    tc::smem_u32(&bars->q_full));
                }
                const int n_loads = 2 * (part.j1 - part.j0);
                for (int i = 0; i < n_loads && ok; ++i) {
                    const int idx = kv_base + i;
                    const int j = part.j0 + (i >> 1), is_v = i & 1;
                    const int stage = idx % NSTAGE, use = idx / NSTAGE;
                    ok = tc::mbar_wait(tc::smem_u32(&bars->kv_empty[stage]), (use & 1) ^ 1, abort_flag);
                    if (!ok) break;
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
                kv_base += n_loads;
                ++part_idx;
            }
            if (*abort_flag) {
                // unwind: let copies still in flight land before the CTA exits (bounded)
                for (int idx = max(0, issued - NSTAGE); idx < issued; ++idx) {
                    const long long t0 = clock64();
                    while (!tc::mbar_try_wait(tc::smem_u32(&bars->kv_full[idx % NSTAGE]), (idx / NSTAGE) & 1) &&
                           clock64() - t0 < (1ll << 24)) {}
                }
            }
        }
    } else if (warp == 8) {
        // ================================ MMA issuer ================================
        if (lane == 0) {
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
            auto kv_wait = [&](int idx) {
                return tc::mbar_wait(tc::smem_u32(&bars->kv_full[idx % NSTAGE]), (idx / NSTAGE) & 1, abort_flag);
            };
            int sp0 = 0, sp1 = 0;                            // blocks handed to each tile's softmax so far
            bool ok = true;
            // one tile's share of a block step: O_t += P_t V_j, then S_t = Q_t K_{j+1}
            auto tile_step = [&](int tt, int cnt, int& sp, int jj, int v_stage, int k_stage) {
                if (jj < cnt) {
                    ok = tc::mbar_wait(tc::smem_u32(&bars->p_full[tt]), sp & 1, abort_flag);
                    ++sp;
                    // the first PV of a part overwrites O_t: the previous part's epilogue must have read it
                    if (ok && jj == 0 && part_idx > 0)
                        ok = tc::mbar_wait(tc::smem_u32(&bars->o_free[tt]), (part_idx - 1) & 1, abort_flag);
                    if (!ok) return;
                    tc::tcgen05_fence_after();
                    issue_pv(tt, v_stage, jj > 0);
                }
                if (jj + 1 < cnt) {
                    issue_qk(tt, k_stage);
                    tc::umma_commit(tc::smem_u32(&bars->s_full[tt]));
                }
            };
            while (ok && it.next(part)) {
                const int n = part.j1 - part.j0;
                ok = tc::mbar_wait(tc::smem_u32(&bars->q_full), part_idx & 1, abort_flag);
                if (ok) ok = kv_wait(kv_base);
                if (!ok) break;
                tc::tcgen05_fence_after();
                if (part.cnt0 > 0) {
                    issue_qk(0, kv_base % NSTAGE);
                    tc::umma_commit(tc::smem_u32(&bars->s_full[0]));
                }
                if (part.cnt1 > 0) {
                    issue_qk(1, kv_base % NSTAGE);
                    tc::umma_commit(tc::smem_u32(&bars->s_full[1]));
                }
                tc::umma_commit(tc::smem_u32(&bars->kv_empty[kv_base % NSTAGE]));
                for (int jj = 0; jj < n && ok; ++jj) {
                    const int v_idx = kv_base + 2 * jj + 1, k_idx = v_idx + 1;
                    const bool has_next = jj + 1 < n;
                    ok = kv_wait(v_idx);
                    if (ok && has_next) ok = kv_wait(k_idx);
                    if (ok) tile_step(0, part.cnt0, sp0, jj, v_idx % NSTAGE, k_idx % NSTAGE);
                    if (ok) tile_step(1, part.cnt1, sp1, jj, v_idx % NSTAGE, k_idx % NSTAGE);
                    if (!ok) break;
                    tc::umma_commit(tc::smem_u32(&bars->kv_empty[v_idx % NSTAGE]));
                    if (has_next) tc::umma_commit(tc::smem_u32(&bars->kv_empty[k_idx % NSTAGE]));
                }
                // every softmax warpgroup must have seen the previous part's o_done before this part's is
                // committed (a waiter may lag one mbarrier phase, never two)
                if (ok && part_idx > 0) ok = tc::mbar_wait(tc::smem_u32(&bars->o_free[0]), (part_idx - 1) & 1, abort_flag);
                if (ok && part_idx > 0) ok = tc::mbar_wait(tc::smem_u32(&bars->o_free[1]), (part_idx - 1) & 1, abort_flag);
                if (ok) tc::umma_commit(tc::smem_u32(&bars->o_done));
                kv_base += 2 * n;
                ++part_idx;
            }
        }
    } else {
        // ================================ softmax + epilogue ================================
        const int tt = warp >> 2;                          // tile of this warpgroup
        const int r = (warp & 3) * 32 + lane;              // row inside the tile == TMEM lane
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t s_tmem = tmem + tt * 128 + lane_addr;
        const uint32_t o_tmem = tmem + 256 + tt * 128 + lane_addr;
        int sp = 0;
        bool ok = true;
        while (it.next(part)) {
            const int row0 = (2 * part.pair + tt) * BLK;
            const int my_n = tt ? part.cnt1 : part.cnt0;
            const int diag_block = nhb + 2 * part.pair + tt;   // KV block index of the causal diagonal
            float m_ref = 0.f, l_sum = 0.f;

            for (int jj = 0; jj < my_n && ok; ++jj) {
                const int j = part.j0 + jj;
                ok = __all_sync(0xffffffffu, tc::mbar_wait(tc::smem_u32(&bars->s_full[tt]), sp & 1, abort_flag));
                ++sp;
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
                // eight independent running maxima (a single chain of 128 dependent max ops would stall)
                float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
                float mx4 = -INFINITY, mx5 = -INFINITY, mx6 = -INFINITY, mx7 = -INFINITY;
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        mx0 = fmaxf(mx0, __uint_as_float(sv[c][i]));
                        mx1 = fmaxf(mx1, __uint_as_float(sv[c][i + 1]));
                        mx2 = fmaxf(mx2, __uint_as_float(sv[c][i + 2]));
                        mx3 = fmaxf(mx3, __uint_as_float(sv[c][i + 3]));
                        mx4 = fmaxf(mx4, __uint_as_float(sv[c][i + 4]));
                        mx5 = fmaxf(mx5, __uint_as_float(sv[c][i + 5]));
                        mx6 = fmaxf(mx6, __uint_as_float(sv[c][i + 6]));
                        mx7 = fmaxf(mx7, __uint_as_float(sv[c][i + 7]));
                    }
                float bm = fmaxf(fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)), fmaxf(fmaxf(mx4, mx5), fmaxf(mx6, mx7)));
                if (bm == -INFINITY) bm = 0.f;

                float alpha = 1.f;
                bool need = false;
                if (jj == 0) {
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
                float rs0 = 0.f, rs1 = 0.f;
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
                        rs0 += __uint_as_float(pk[i] << 16);
                        rs1 += __uint_as_float(pk[i] & 0xffff0000u);
                    }
                    tc::tmem_st16(s_tmem + c * 16, pk);
                }
                l_sum += rs0 + rs1;

                if (tt == 0 && tail_partial && j == nhb - 1) {
                    // rows of the V tile past the end of the history may hold anything: zero them
                    const int v_idx = kv_base + 2 * jj + 1, v_stage = v_idx % NSTAGE;
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

            const int row = row0 + r;
            const size_t pslot = ((size_t)blockIdx.x * 2 + part.slot) * 2 + tt;
            if (my_n > 0) {
                ok = __all_sync(0xffffffffu, ok && tc::mbar_wait(tc::smem_u32(&bars->o_done), part_idx & 1, abort_flag));
                tc::tcgen05_fence_after();
                const float inv = part.final_ ? 1.f / l_sum : 1.f;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t ov[32];
                    tc::tmem_ld32(o_tmem + c * 32, ov);
                    tc::tmem_wait_ld();
                    if (!ok) continue;
                    if (!part.final_) {
                        float4* dst = reinterpret_cast<float4*>(p.part_o + (pslot * BLK + r) * HD + c * 32);
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            dst[i] = make_float4(__uint_as_float(ov[4 * i]), __uint_as_float(ov[4 * i + 1]),
                                                 __uint_as_float(ov[4 * i + 2]), __uint_as_float(ov[4 * i + 3]));
                    } else if (row < p.t) {
                        const size_t off = ((size_t)row * p.h_q + part.head) * HD + c * 32;
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
                if (ok && !part.final_) p.part_ml[pslot * BLK + r] = make_float2(m_ref, l_sum);
                if (ok && part.final_ && p.lse_out && row < p.t)
                    p.lse_out[(size_t)row * p.h_q + part.head] = m_ref * p.scale + logf(l_sum);
            } else {
                // no block of this tile in the part: still consume the part's o_done phase, in step with the others
                ok = __all_sync(0xffffffffu, ok && tc::mbar_wait(tc::smem_u32(&bars->o_done), part_idx & 1, abort_flag));
                if (!part.final_) p.part_ml[pslot * BLK + r] = make_float2(-INFINITY, 0.f);
            }
            // O_t (and the part's Q tile) may be reused
            tc::tcgen05_fence_before();
            tc::mbar_arrive(tc::smem_u32(&bars->o_free[tt]));
            kv_base += 2 * (part.j1 - part.j0);
            ++part_idx;
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

// Merge the partial outputs of every item that was cut between CTAs.  Grid (items, 8 groups of 32 rows);
// a warp owns 4 rows and a lane 4 of a row's 128 columns.
constexpr int MERGE_MAX_PARTS = 8;
__global__ void __launch_bounds__(256) attention_merge_kernel(const AttnParams p, int n_cta) {
    const int pair = p.n_pairs - 1 - blockIdx.x / p.h_q;
    const int head = blockIdx.x % p.h_q;
    int n_hist = p.n_hist_dev ? *p.n_hist_dev : p.n_hist_max;
    n_hist = max(0, min(n_hist, p.n_hist_max));
    Sched s;
    s.nhb = (n_hist + BLK - 1) / BLK; s.n_pairs = p.n_pairs; s.h_q = p.h_q; s.t = p.t;
    const long long total = s.total();
    const long long w0 = s.item_begin(pair, head);
    const int nb = s.nb_pair(pair);
    auto cta_of = [&](long long w) {
        int b = (int)(w * n_cta / total);
        b = max(0, min(b, n_cta - 1));
        while (b + 1 < n_cta && share_begin(total, b + 1, n_cta) <= w) ++b;
        while (b > 0 && share_begin(total, b, n_cta) > w) --b;
        return b;
    };
    const int b_first = cta_of(w0), b_last = cta_of(w0 + nb - 1);
    if (b_first == b_last) return;                           // the item was computed by one CTA
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int q4 = 0; q4 < 4; ++q4) {
        const int rr = blockIdx.y * 32 + warp * 4 + q4;      // 0..255: tile * 128 + row
        const int tt = rr / BLK, r = rr % BLK;
        const int row = (2 * pair + tt) * BLK + r;
        if (row >= p.t) continue;
        float M = -INFINITY;
        for (int b0 = b_first; b0 <= b_last; b0 += MERGE_MAX_PARTS) {      // (an item rarely has more than 3 parts)
            float2 ml[MERGE_MAX_PARTS];
#pragma unroll
            for (int i = 0; i < MERGE_MAX_PARTS; ++i) {
                const int b = b0 + i;
                ml[i] = make_float2(-INFINITY, 0.f);
                if (b <= b_last && share_begin(total, b, n_cta) != share_begin(total, b + 1, n_cta))
                    ml[i] = p.part_ml[(((size_t)b * 2 + (b == b_first ? 1 : 0)) * 2 + tt) * BLK + r];
            }
#pragma unroll
            for (int i = 0; i < MERGE_MAX_PARTS; ++i)
                if (ml[i].y > 0.f) M = fmaxf(M, ml[i].x);
        }
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float L = 0.f;
        for (int b0 = b_first; b0 <= b_last; b0 += MERGE_MAX_PARTS) {
            float2 ml[MERGE_MAX_PARTS];
            float4 o[MERGE_MAX_PARTS];
#pragma unroll
            for (int i = 0; i < MERGE_MAX_PARTS; ++i) {
                const int b = b0 + i;
                ml[i] = make_float2(-INFINITY, 0.f);
                o[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (b <= b_last && share_begin(total, b, n_cta) != share_begin(total, b + 1, n_cta)) {
                    const size_t pslot = ((size_t)b * 2 + (b == b_first ? 1 : 0)) * 2 + tt;
                    ml[i] = p.part_ml[pslot * BLK + r];
                    if (ml[i].y > 0.f) o[i] = *reinterpret_cast<const float4*>(p.part_o + (pslot * BLK + r) * HD + lane * 4);
                }
            }
#pragma unroll
            for (int i = 0; i < MERGE_MAX_PARTS; ++i) {
                if (!(ml[i].y > 0.f)) continue;
                const float wgt = exp2f((ml[i].x - M) * p.scale_log2);
                acc.x += wgt * o[i].x; acc.y += wgt * o[i].y; acc.z += wgt * o[i].z; acc.w += wgt * o[i].w;
                L += wgt * ml[i].y;
            }
        }
        const float inv = 1.f / L;
        const size_t off = ((size_t)row * p.h_q + head) * HD + lane * 4;
        if (p.out_dtype == OMNI_DTYPE_FP32) {
            *reinterpret_cast<float4*>(static_cast<float*>(p.o_out) + off) =
                make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
        } else {
            uint2 v;
            v.x = tc::pack_bf16x2(acc.x * inv, acc.y * inv);
            v.y = tc::pack_bf16x2(acc.z * inv, acc.w * inv);
            *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(p.o_out) + off) = v;
        }
        if (p.lse_out && lane == 0) p.lse_out[(size_t)row * p.h_q + head] = M * p.scale + logf(L);
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
    const int n_cta = ctx->sm_count;
    AttnParams p;
    p.t = t; p.h_q = g.h_q; p.h_kv = g.h_kv; p.n_hist_dev = n_hist_dev; p.n_hist_max = n_hist_max;
    p.scale = scale; p.scale_log2 = scale * 1.4426950408889634f;
    p.o_out = o_out; p.out_dtype = out_dtype; p.lse_out = lse_out; p.status = ctx->status_dev;
    p.n_pairs = (t + 2 * BLK - 1) / (2 * BLK);
    p.part_o = ctx->attn_part_o; p.part_ml = reinterpret_cast<float2*>(ctx->attn_part_ml);
    static bool attr_set = false;
    if (!attr_set) {
        OMNI_CUDA(ctx, cudaFuncSetAttribute(attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
        attr_set = true;
    }
    attention_tc_kernel<<<n_cta, ATT_THREADS, SMEM_BYTES, st>>>(tm_q, tm_kh, tm_vh, tm_kc, tm_vc, p);
    OMNI_CHECK_LAUNCH(ctx, "attention_tc_kernel");
    attention_merge_kernel<<<dim3(p.n_pairs * g.h_q, 8), 256, 0, st>>>(p, n_cta);
    OMNI_CHECK_LAUNCH(ctx, "attention_merge_kernel");
    return OMNI_OK;
}
