// GQA chunk-prefill attention on tcgen05 tensor cores (bf16, head dim 128).
//
// Work unit: one 128-key KV block of one "item" = (128-row query tile, head).  The KV sequence of an item
// is the history blocks followed by the causal chunk blocks.  The kernel is persistent, one CTA per SM:
// the units of all items are laid end to end and cut into equal contiguous shares, so every SM gets the
// same amount of tensor work whatever the number of items.  A share is a list of "parts" (item, block
// range).  A part that covers its whole item writes the output directly; an item cut between CTAs leaves
// un-normalised partial outputs with their (max, sum) in scratch and a small second kernel merges them.
//
// Inside a CTA:
//   warp 10     TMA producer: the part's Q tile, then K / V tiles (128 keys) through a 5-stage ring
//   warp 8      one thread issues S = Q K_j^T as one N = 128 instruction group (an M = 128 tcgen05.mma
//               occupies the tensor pipe for 64 clocks whatever N <= 128 is, so narrower blocks would waste
//               it); S is double-buffered and runs two blocks ahead of PV.
//   warp 9      one thread issues the PVs.  One thread cannot issue faster than one instruction per ~70-100
//               clocks, so QK and PV have an issuer each; they are ordered by the pv_done barriers.
//   warps 0-3   softmax warpgroup A: columns 0-63 of every S block (keys 0-63 of the block)
//   warps 4-7   softmax warpgroup B: columns 64-127.  One thread per query row and half block: logits
//               from tensor memory, running max with lazy rescale, exp2, P written back over the S columns
//               as bf16.  Each warpgroup is its own online-softmax stream with its own accumulator:
//               O_A += P_A V[keys 0-63], O_B += P_B V[keys 64-127]; the two are merged by their (max, sum)
//               when the part ends.  Two warpgroups keep the exp unit busy; splitting columns instead of
//               owning two query tiles leaves tensor memory for the second S buffer.
// TMEM map (512 columns): S buffer 0 [0,128)  S buffer 1 [128,256)  O_A [256,384)  O_B [384,512);
// P_A / P_B overwrite columns [0,32) / [64,96) of their S buffer.
#include "common.cuh"
#include "tc_ptx.cuh"

#include <algorithm>

namespace {

#ifndef ATT_POLY_EVERY
#define ATT_POLY_EVERY 4       // every n-th pair of exponentials takes the polynomial path (0: none); 4 measured best (+2 %)
#endif
template <int PAIR>
__device__ __forceinline__ uint64_t exp2_pair(uint64_t x2) {
    // degree 3 (relative error 7.5e-5) is far below the bf16 rounding of the weights
    if (ATT_POLY_EVERY > 0 && (PAIR % ATT_POLY_EVERY) == ATT_POLY_EVERY - 1) return tc::exp2_poly2<3>(x2);
    float x0, x1;
    tc::unpack2(x2, x0, x1);
    return tc::pack2(tc::ex2_approx(x0), tc::ex2_approx(x1));
}

constexpr int BQ = 128;                  // rows per query tile
constexpr int BK = 128;                  // keys per KV block
constexpr int HK = 64;                   // keys per softmax warpgroup and block
constexpr int HD = 128;                  // head dim
constexpr int TILE_BYTES = 128 * HD * 2; // 32 KiB (Q, K and V tiles), two 64-column halves of 16 KiB
constexpr int HALF_BYTES = TILE_BYTES / 2;
constexpr int NSTAGE = 5;
constexpr int ATT_THREADS = 352;
constexpr int XCH_BYTES = BQ * 2 * 8;    // (max, sum) of both warpgroups, exchanged when a part ends
constexpr int SMEM_BYTES = TILE_BYTES + NSTAGE * TILE_BYTES + 1024 /*alignment*/ + 512 /*barriers*/ + XCH_BYTES;
// O is rescaled only when the row max grows by more than this many log2 units (P stays below 2^8).
constexpr float RESCALE_THRESHOLD = 8.0f;

constexpr uint32_t IDESC_QK = tc::umma_idesc_bf16(128, BK, false, false);
constexpr uint32_t IDESC_PV = tc::umma_idesc_bf16(128, HD, false, true);

// Debug aid (-DATT_TRACE): CTA 0 records clock64() stamps of a few blocks and prints them at exit.
#ifdef ATT_TRACE
#define TRACE_N 40
#define TRACE(role, k) do { if (blockIdx.x == 0 && lane == 0 && trace_i < TRACE_N) trace_buf[((role) * TRACE_N + trace_i) * 6 + (k)] = clock64(); } while (0)
#define TRACE_NEXT() (++trace_i)
#else
#define TRACE(role, k)
#define TRACE_NEXT()
#endif

struct AttnParams {
    int t, h_q, h_kv;
    const int32_t* n_hist_dev; int n_hist_max;
    float scale_log2, scale;
    void* o_out; int out_dtype; float* lse_out;
    int32_t* status;
    int n_tiles;          // query tiles of 128 rows
    // history with holes (all three null: dense history): the 128-key blocks that hold a live slot, their live bits,
    // and how many there are; written by attn_block_scan_kernel before this launch
    const int32_t* live_idx; const uint4* live_mask; const int32_t* n_live;
    int pack_shift;       // >= 0: GQA-packed single tile, row r = (token r >> pack_shift, head of the group r & (G-1)); -1: off
    float* part_o;        // [cta][2 slots][128 rows][128] un-normalised partial outputs
    float2* part_ml;      // [cta][2 slots][128 rows] (running max, sum)
};

struct Barriers {
    uint64_t q_full;
    uint64_t q_free;            // every QK^T of the part has completed: the Q tile may be overwritten
    uint64_t kv_full[NSTAGE];
    uint64_t kv_empty[NSTAGE];
    uint64_t s_full;            // S of the next block is complete
    uint64_t s_free;            // both warpgroups hold S in registers: the next QK^T may overwrite it
    uint64_t p_full[2][2];      // [warpgroup][buffer]
    uint64_t pv_done[2];        // [buffer] both PVs of the block in that buffer have completed
    uint64_t o_done;
    uint64_t o_free;            // both warpgroups have read O of the part
    uint32_t tmem_base;
    int abort_flag;
};

// ---- the work list: identical arithmetic in every role and in the merge kernel --------------------------
struct Sched {
    int nhb, n_tiles, h_q;                                   // nhb: 128-key blocks of history
    __device__ int nb_item(int qt) const { return nhb + qt + 1; }      // history + chunk blocks 0 .. qt (the diagonal)
    __device__ long long total() const {
        return (long long)h_q * ((long long)n_tiles * (nhb + 1) + (long long)n_tiles * (n_tiles - 1) / 2);
    }
    // items are ordered by descending query tile, then head
    __device__ long long item_begin(int qt, int head) const {
        long long w = 0;
        for (int q = n_tiles - 1; q > qt; --q) w += (long long)h_q * nb_item(q);
        return w + (long long)head * nb_item(qt);
    }
    __device__ void locate(long long w, int& qt, int& head, int& j) const {
        long long base = 0;
        for (int q = n_tiles - 1; q >= 0; --q) {
            const int nb = nb_item(q);
            const long long span = (long long)h_q * nb;
            if (w < base + span || q == 0) {
                qt = q;
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
    int qt, head, j0, j1;
    bool final_;          // the part covers the whole item
    int slot;             // partial slot of this CTA (when not final)
};

struct PartIter {
    Sched s;
    long long w, w_end;
    __device__ bool next(Part& p) {
        if (w >= w_end) return false;
        s.locate(w, p.qt, p.head, p.j0);
        const int nb = s.nb_item(p.qt);
        p.j1 = (int)min((long long)nb, (long long)p.j0 + (w_end - w));
        w += p.j1 - p.j0;
        p.final_ = p.j0 == 0 && p.j1 == nb;
        p.slot = p.j0 > 0 ? 0 : 1;
        return true;
    }
};

// Position, in the part's load order  K0 K1 V0 K2 V1 K3 ... V_{n-2} V_{n-1},  of the V tile of local block jj.
__device__ __forceinline__ int pos_v(int jj, int n) { return n == 1 ? 1 : (jj == n - 1 ? 2 * n - 1 : 2 + 2 * jj); }

__device__ __forceinline__ void named_barrier_256(int id) { asm volatile("bar.sync %0, 256;" ::"r"(id) : "memory"); }

__global__ void __launch_bounds__(ATT_THREADS, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kh,
                    const __grid_constant__ CUtensorMap tm_vh, const __grid_constant__ CUtensorMap tm_kc,
                    const __grid_constant__ CUtensorMap tm_vc, const AttnParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - tc::smem_u32(smem_raw));
    const uint32_t q_smem = smem_base;                          // Q tile
    const uint32_t kv_smem = smem_base + TILE_BYTES;            // NSTAGE K/V tiles
    constexpr int KV_OFF = TILE_BYTES;
    Barriers* bars = reinterpret_cast<Barriers*>(smem_gen + KV_OFF + NSTAGE * TILE_BYTES);
    float2* xch = reinterpret_cast<float2*>(smem_gen + KV_OFF + NSTAGE * TILE_BYTES + 512);     // [2][128] (m, l)
    volatile int* abort_flag = &bars->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    int n_hist = p.n_hist_dev ? *p.n_hist_dev : p.n_hist_max;
    if (n_hist < 0 || n_hist > p.n_hist_max) {
        if (threadIdx.x == 0 && blockIdx.x == 0) atomicOr(p.status, OMNI_DEV_BAD_COUNT);
        n_hist = max(0, min(n_hist, p.n_hist_max));
    }
    // with holes only the live blocks are visited: block j of the history is block live_idx[j] of the cache
    const bool masked = p.live_idx != nullptr;
    const int nb_span = (n_hist + BK - 1) / BK;
    const int nhb = masked ? max(0, min(*p.n_live, nb_span)) : nb_span;
    const int hist_tail = n_hist - (nb_span - 1) * BK;       // slots of the span in its last block (if nb_span > 0)
    // rows of the last visited block beyond the span may hold anything: they are masked in S and zeroed in V
    const bool tail_partial = nhb > 0 && hist_tail < BK && (!masked || p.live_idx[nhb - 1] == nb_span - 1);

    PartIter it;
    // GQA-packed mode (few queries, e.g. decode): one tile holds all query heads of a KV group, items are KV heads
    const bool packed = p.pack_shift >= 0;
    it.s.nhb = nhb; it.s.n_tiles = p.n_tiles; it.s.h_q = packed ? p.h_kv : p.h_q;
    {
        const long long total = it.s.total();
        it.w = share_begin(total, blockIdx.x, gridDim.x);
        it.w_end = share_begin(total, blockIdx.x + 1, gridDim.x);
    }
    if (it.w >= it.w_end) return;                            // more CTAs than units

    if (threadIdx.x == 0) {
        tc::mbar_init(tc::smem_u32(&bars->q_full), 1);
        tc::mbar_init(tc::smem_u32(&bars->q_free), 1);
        for (int s = 0; s < NSTAGE; ++s) {
            tc::mbar_init(tc::smem_u32(&bars->kv_full[s]), 1);
            tc::mbar_init(tc::smem_u32(&bars->kv_empty[s]), 1);
        }
        tc::mbar_init(tc::smem_u32(&bars->s_full), 1);
        tc::mbar_init(tc::smem_u32(&bars->s_free), 256);
        for (int b = 0; b < 2; ++b) {
            tc::mbar_init(tc::smem_u32(&bars->p_full[0][b]), 128);
            tc::mbar_init(tc::smem_u32(&bars->p_full[1][b]), 128);
        }
        tc::mbar_init(tc::smem_u32(&bars->pv_done[0]), 1);
        tc::mbar_init(tc::smem_u32(&bars->pv_done[1]), 1);
        tc::mbar_init(tc::smem_u32(&bars->o_done), 2);                   // QK issuer and PV issuer
        tc::mbar_init(tc::smem_u32(&bars->o_free), 256);
        bars->abort_flag = 0;
        tc::fence_barrier_init();
    }
    if (warp == 8) tc::tmem_alloc<512>(tc::smem_u32(&bars->tmem_base));
    tc::tcgen05_fence_before();
    __syncthreads();
    tc::tcgen05_fence_after();
    const uint32_t tmem = bars->tmem_base;

#ifdef ATT_TRACE
    // the tail-part slot of the last CTA is never used by the kernel proper
    long long* trace_buf = reinterpret_cast<long long*>(p.part_o + ((size_t)(gridDim.x - 1) * 2 + 1) * BQ * HD);
    int trace_i = 0;
#endif
    Part part;
    int part_idx = 0;
    int kv_base = 0;                                         // K/V tiles loaded by earlier parts of this CTA

    if (warp == 10) {
        // ================================ TMA producer ================================
        if (lane == 0) {
            tc::tma_prefetch_desc(&tm_q);
            tc::tma_prefetch_desc(&tm_kh);
            tc::tma_prefetch_desc(&tm_vh);
            tc::tma_prefetch_desc(&tm_kc);
            tc::tma_prefetch_desc(&tm_vc);
            int issued = 0;
            bool ok = true;
            int kvh = 0;
            auto load_tile = [&](int j, bool is_v) {         // block j of the item, next ring slot
                const int idx = issued;
                const int stage = idx % NSTAGE, use = idx / NSTAGE;
                ok = tc::mbar_wait(tc::smem_u32(&bars->kv_empty[stage]), (use & 1) ^ 1, abort_flag);
                if (!ok) return;
                const uint32_t full = tc::smem_u32(&bars->kv_full[stage]);
                tc::mbar_expect_tx(full, TILE_BYTES);
                const bool hist = j < nhb;
                const CUtensorMap* map = hist ? (is_v ? &tm_vh : &tm_kh) : (is_v ? &tm_vc : &tm_kc);
                const int row = (hist ? (masked ? __ldg(p.live_idx + j) : j) : j - nhb) * BK;
                const uint32_t dst = kv_smem + stage * TILE_BYTES;
                tc::tma_load_2d(dst, map, kvh * HD, row, full);
                tc::tma_load_2d(dst + HALF_BYTES, map, kvh * HD + 64, row, full);
                issued = idx + 1;
            };
            while (ok && it.next(part)) {
                // the Q tile is free once every QK^T of the previous part has completed (its last softmax, its last PVs
                // and its epilogue still run: the next part's Q and first K tiles land under them)
                if (part_idx > 0) ok = tc::mbar_wait(tc::smem_u32(&bars->q_free), (part_idx - 1) & 1, abort_flag);
                if (!ok) break;
                kvh = packed ? part.head : part.head / (p.h_q / p.h_kv);
                tc::mbar_expect_tx(tc::smem_u32(&bars->q_full), TILE_BYTES);
                if (packed) {
                    const int h0 = kvh << p.pack_shift;      // first query head of the group
                    tc::tma_load_3d(q_smem, &tm_q, 0, h0, 0, tc::smem_u32(&bars->q_full));
                    tc::tma_load_3d(q_smem + HALF_BYTES, &tm_q, 64, h0, 0, tc::smem_u32(&bars->q_full));
                } else {
                    tc::tma_load_2d(q_smem, &tm_q, part.head * HD, part.qt * BQ, tc::smem_u32(&bars->q_full));
                    tc::tma_load_2d(q_smem + HALF_BYTES, &tm_q, part.head * HD + 64, part.qt * BQ, tc::smem_u32(&bars->q_full));
                }
                const int n = part.j1 - part.j0;
                load_tile(part.j0, false);
                if (ok && n > 1) load_tile(part.j0 + 1, false);
                for (int jj = 0; jj < n && ok; ++jj) {
                    load_tile(part.j0 + jj, true);
                    if (ok && jj + 2 < n) load_tile(part.j0 + jj + 2, false);
                }
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
        // ================================ QK issuer (one thread) ================================
        if (lane == 0) {
            auto wait = [&](uint64_t* bar, int parity) { return tc::mbar_wait(tc::smem_u32(bar), parity, abort_flag); };
            // S = Q K^T over the 128 keys of ring slot idx
            auto issue_qk = [&](int idx) {
                const uint32_t b0 = kv_smem + (idx % NSTAGE) * TILE_BYTES;
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {
                    const uint32_t off = (kk >> 2) * HALF_BYTES + (kk & 3) * 32;
                    tc::umma_ss(tmem, tc::umma_smem_desc(q_smem + off, 16, 1024), tc::umma_smem_desc(b0 + off, 16, 1024),
                                IDESC_QK, kk > 0, 1u);
                }
                tc::umma_commit(tc::smem_u32(&bars->s_full));
                tc::umma_commit(tc::smem_u32(&bars->kv_empty[idx % NSTAGE]));
            };
            int g = 0;                                       // blocks started so far
            bool ok = true;
            while (ok && it.next(part)) {
                const int n = part.j1 - part.j0;
                ok = wait(&bars->q_full, part_idx & 1);
                for (int jj = 0; jj < n && ok; ++jj) {
                    const int gb = g + jj;
                    const int idx = kv_base + (jj < 2 ? jj : 2 * jj - 1);      // K_jj in the part's load order
                    TRACE(2, 0);
                    ok = wait(&bars->kv_full[idx % NSTAGE], (idx / NSTAGE) & 1);
                    TRACE(2, 1);
                    // S is single-buffered: the softmax warps must hold the previous block in registers
                    if (ok && gb > 0) ok = wait(&bars->s_free, (gb - 1) & 1);
                    if (!ok) break;
                    tc::tcgen05_fence_after();
                    issue_qk(idx);
                    TRACE(2, 2); TRACE(2, 3); TRACE(2, 4);
                    TRACE_NEXT();
                }
                if (ok) tc::umma_commit(tc::smem_u32(&bars->q_free));
                // the softmax warpgroups must have seen the previous part's o_done before this part's is
                // committed (a waiter may lag one mbarrier phase, never two)
                if (ok && part_idx > 0) ok = wait(&bars->o_free, (part_idx - 1) & 1);
                if (ok) tc::umma_commit(tc::smem_u32(&bars->o_done));
                g += n;
                kv_base += 2 * n;
                ++part_idx;
            }
        }
    } else if (warp == 9) {
        // ================================ PV issuer (one thread) ================================
        if (lane == 0) {
            auto wait = [&](uint64_t* bar, int parity) { return tc::mbar_wait(tc::smem_u32(bar), parity, abort_flag); };
            // O_w += P_w[buf] V[keys 64w .. 64w+63] of ring stage `stage`
            auto issue_pv = [&](int w, int buf, int stage, bool accumulate) {
                const uint32_t b0 = kv_smem + stage * TILE_BYTES + w * (HK * 128);
#pragma unroll
                for (int kk = 0; kk < HK / 16; ++kk) {
                    tc::umma_ts(tmem + 256 + w * 128, tmem + 128 + buf * 64 + w * 32 + kk * 8,
                                tc::umma_smem_desc(b0 + kk * 2048, HALF_BYTES, 1024), IDESC_PV, accumulate || kk > 0, 1u);
                }
            };
            int g = 0;
            bool ok = true;
            while (ok && it.next(part)) {
                const int n = part.j1 - part.j0;
                for (int jj = 0; jj < n && ok; ++jj) {
                    const int v_idx = kv_base + pos_v(jj, n);
                    const int gb = g + jj, buf = gb & 1;
                    ok = wait(&bars->kv_full[v_idx % NSTAGE], (v_idx / NSTAGE) & 1);
                    if (ok) ok = wait(&bars->p_full[0][buf], (gb >> 1) & 1);
                    // the first PV of a part overwrites O: the previous part's epilogue must have read it
                    if (ok && jj == 0 && part_idx > 0) ok = wait(&bars->o_free, (part_idx - 1) & 1);
                    if (!ok) break;
                    tc::tcgen05_fence_after();
                    issue_pv(0, buf, v_idx % NSTAGE, jj > 0);
                    ok = wait(&bars->p_full[1][buf], (gb >> 1) & 1);
                    if (!ok) break;
                    tc::tcgen05_fence_after();
                    issue_pv(1, buf, v_idx % NSTAGE, jj > 0);
                    tc::umma_commit(tc::smem_u32(&bars->pv_done[buf]));
                    tc::umma_commit(tc::smem_u32(&bars->kv_empty[v_idx % NSTAGE]));
                }
                if (ok && part_idx > 0) ok = wait(&bars->o_free, (part_idx - 1) & 1);
                if (ok) tc::umma_commit(tc::smem_u32(&bars->o_done));
                g += n;
                kv_base += 2 * n;
                ++part_idx;
            }
        }
    } else {
        // ================================ softmax + epilogue ================================
        const int w = warp >> 2;                           // warpgroup: key half of every block
        const int r = (warp & 3) * 32 + lane;              // query row inside the tile == TMEM lane
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t o_own = tmem + 256 + w * 128 + lane_addr;
        int g = 0;                                         // blocks processed so far
        bool ok = true;
        while (it.next(part)) {
            const int n_part = part.j1 - part.j0;
            const int diag_block = nhb + part.qt;          // KV block index of the causal diagonal
            float m_ref = -INFINITY, l_sum = 0.f;

            for (int jj = 0; jj < n_part && ok; ++jj, ++g) {
                const int j = part.j0 + jj;
                const int buf = g & 1;                                     // P buffer of this block
                const uint32_t s_tmem = tmem + w * HK + lane_addr;
                const uint32_t p_tmem = tmem + 128 + buf * 64 + w * 32 + lane_addr;
                // live bits of this warpgroup's 64 keys (all ones for a dense history and for chunk blocks); the load is
                // issued before the wait for S so that its latency is hidden
                unsigned long long live = ~0ull;
                if (masked && j < nhb) live = __ldg(reinterpret_cast<const unsigned long long*>(p.live_mask + j) + w);
                ok = __all_sync(0xffffffffu, tc::mbar_wait(tc::smem_u32(&bars->s_full), g & 1, abort_flag));
                tc::tcgen05_fence_after();
                if ((warp & 3) == 0) TRACE(w, 0);
                uint32_t sa[32], sb[32];
                tc::tmem_ld32(s_tmem, sa);
                tc::tmem_ld32(s_tmem + 32, sb);
                tc::tmem_wait_ld();
                // the logits are in registers: S may be overwritten by the next block's QK^T
                tc::tcgen05_fence_before();
                tc::mbar_arrive(tc::smem_u32(&bars->s_free));

                // masking of this warpgroup's 64 keys: ragged history tail, causal diagonal
                int n_valid = HK;
                if (j == nhb - 1 && tail_partial) n_valid = hist_tail - w * HK;
                if (j == diag_block) n_valid = (packed ? (r >> p.pack_shift) : r) + 1 - w * HK;   // <= 0: the row sees nothing of this half
                if (n_valid < HK) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        if (i >= n_valid) sa[i] = 0xff800000u;           // -inf
                        if (32 + i >= n_valid) sb[i] = 0xff800000u;
                    }
                }
                if (live != ~0ull) {                         // holes inside the block (warp-uniform: one mask per block)
                    const uint32_t lo = (uint32_t)live, hi = (uint32_t)(live >> 32);
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        if (!((lo >> i) & 1u)) sa[i] = 0xff800000u;
                        if (!((hi >> i) & 1u)) sb[i] = 0xff800000u;
                    }
                }
                // row maximum of the 64 logits: three-input maxima, four independent chains
                float mx0 = tc::max3(__uint_as_float(sa[0]), __uint_as_float(sa[1]), __uint_as_float(sb[0]));
                float mx1 = tc::max3(__uint_as_float(sa[2]), __uint_as_float(sa[3]), __uint_as_float(sb[1]));
                float mx2 = tc::max3(__uint_as_float(sa[4]), __uint_as_float(sa[5]), __uint_as_float(sb[2]));
                float mx3 = tc::max3(__uint_as_float(sa[6]), __uint_as_float(sa[7]), __uint_as_float(sb[3]));
#pragma unroll
                for (int i = 8; i < 32; i += 8) {
                    mx0 = tc::max3(mx0, __uint_as_float(sa[i]), __uint_as_float(sa[i + 1]));
                    mx1 = tc::max3(mx1, __uint_as_float(sa[i + 2]), __uint_as_float(sa[i + 3]));
                    mx2 = tc::max3(mx2, __uint_as_float(sa[i + 4]), __uint_as_float(sa[i + 5]));
                    mx3 = tc::max3(mx3, __uint_as_float(sa[i + 6]), __uint_as_float(sa[i + 7]));
                }
#pragma unroll
                for (int i = 4; i < 28; i += 8) {
                    mx0 = tc::max3(mx0, __uint_as_float(sb[i]), __uint_as_float(sb[i + 1]));
                    mx1 = tc::max3(mx1, __uint_as_float(sb[i + 2]), __uint_as_float(sb[i + 3]));
                    mx2 = tc::max3(mx2, __uint_as_float(sb[i + 4]), __uint_as_float(sb[i + 5]));
                    mx3 = tc::max3(mx3, __uint_as_float(sb[i + 6]), __uint_as_float(sb[i + 7]));
                }
                mx0 = tc::max3(mx0, __uint_as_float(sb[28]), __uint_as_float(sb[29]));
                mx1 = tc::max3(mx1, __uint_as_float(sb[30]), __uint_as_float(sb[31]));
                const float bm = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
                if ((warp & 3) == 0) TRACE(w, 1);

                float alpha = 1.f;
                bool need = false;
                if (m_ref == -INFINITY) {
                    m_ref = bm;                              // first block with a visible key (may stay -inf)
                } else if ((bm - m_ref) * p.scale_log2 > RESCALE_THRESHOLD) {
                    alpha = tc::ex2_approx((m_ref - bm) * p.scale_log2);
                    m_ref = bm;
                    need = true;
                }
                // a row that has seen no key yet keeps m_ref = -inf; exponentiate against 0 so that P = 0, not NaN
                const float neg_m = m_ref == -INFINITY ? 0.f : -m_ref * p.scale_log2;
                // pairs of columns: a packed FMA scales two logits and a packed add sums two weights; every fourth
                // pair takes its exponentials from the polynomial on the FMA pipe
                const uint64_t c2 = tc::pack2(p.scale_log2, p.scale_log2), nm2 = tc::pack2(neg_m, neg_m);
                uint64_t rs0 = 0ull, rs1 = 0ull;
                uint32_t pk[32];
#define ATT_PAIR(src, i, dst, acc)                                                                            \
    {                                                                                                         \
        const uint64_t x2 = tc::fma2(tc::pack2(__uint_as_float(src[2 * (i)]), __uint_as_float(src[2 * (i) + 1])), c2, nm2); \
        float e0, e1;                                                                                         \
        tc::unpack2(exp2_pair<(dst)>(x2), e0, e1);                                                            \
        pk[dst] = tc::pack_bf16x2(e0, e1);                                                                    \
        /* the normaliser sums the ROUNDED weights the tensor core will use, so that the weights of a row */ \
        /* sum to one exactly and the rounding of a dominant weight cancels */                                \
        acc = tc::add2(acc, tc::pack2(__uint_as_float(pk[dst] << 16), __uint_as_float(pk[dst] & 0xffff0000u))); \
    }
#define ATT_PAIR4(i) ATT_PAIR(sa, i, i, rs0) ATT_PAIR(sb, i, 16 + (i), rs1)
                ATT_PAIR4(0)  ATT_PAIR4(1)  ATT_PAIR4(2)  ATT_PAIR4(3)  ATT_PAIR4(4)  ATT_PAIR4(5)  ATT_PAIR4(6)  ATT_PAIR4(7)
                ATT_PAIR4(8)  ATT_PAIR4(9)  ATT_PAIR4(10) ATT_PAIR4(11) ATT_PAIR4(12) ATT_PAIR4(13) ATT_PAIR4(14) ATT_PAIR4(15)
#undef ATT_PAIR4
#undef ATT_PAIR
                // the P buffer of block g was last read by the PVs of block g-2, which completed before the
                // wait of block g-1 below returned (or, for the first two blocks of a part, before the previous part ended)
                tc::tmem_st32(p_tmem, pk);
                if ((warp & 3) == 0) TRACE(w, 2);
                // O is touched only after the PVs of the previous block have completed (they have, by now, nearly always)
                if (jj > 0)
                    ok = __all_sync(0xffffffffu, tc::mbar_wait(tc::smem_u32(&bars->pv_done[(g - 1) & 1]), ((g - 1) >> 1) & 1, abort_flag));
                if (__any_sync(0xffffffffu, need)) {
                    tc::tcgen05_fence_after();
                    l_sum *= alpha;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t ov[32];
                        tc::tmem_ld32(o_own + c * 32, ov);
                        tc::tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha);
                        tc::tmem_st32(o_own + c * 32, ov);
                    }
                }
                {
                    float r0, r1;
                    tc::unpack2(tc::add2(rs0, rs1), r0, r1);
                    l_sum += r0 + r1;
                }
                if ((warp & 3) == 0) TRACE(w, 3);

                if (tail_partial && j == nhb - 1) {
                    // rows of the V tile past the end of the history may hold anything: this warpgroup zeroes
                    // the ones among its own 64 keys before it releases its PV
                    const int v_idx = kv_base + pos_v(jj, n_part), v_stage = v_idx % NSTAGE;
                    ok = __all_sync(0xffffffffu, tc::mbar_wait(tc::smem_u32(&bars->kv_full[v_stage]), (v_idx / NSTAGE) & 1, abort_flag));
                    const int key = w * HK + (r & (HK - 1));             // two threads per key row: each takes one 64-dim half
                    if (key >= hist_tail) {
                        uint4* row_v = reinterpret_cast<uint4*>(smem_gen + KV_OFF + v_stage * TILE_BYTES + (r >> 6) * HALF_BYTES + key * 128);
#pragma unroll
                        for (int i = 0; i < 8; ++i) row_v[i] = make_uint4(0, 0, 0, 0);
                    }
                    tc::fence_proxy_async_smem();
                }
                tc::tmem_wait_st();
                tc::tcgen05_fence_before();
                tc::mbar_arrive(tc::smem_u32(&bars->p_full[w][buf]));
                if ((warp & 3) == 0) { TRACE(w, 4); TRACE_NEXT(); }
            }

            // ---- end of the part: merge the two warpgroups' streams, write the output or the partial -------
            ok = __all_sync(0xffffffffu, ok && tc::mbar_wait(tc::smem_u32(&bars->o_done), part_idx & 1, abort_flag));
            tc::tcgen05_fence_after();
            xch[w * BQ + r] = make_float2(m_ref, l_sum);
            named_barrier_256(1);
            const float2 other = xch[(w ^ 1) * BQ + r];
            const float M = fmaxf(m_ref, other.x);
            const float w_own = l_sum > 0.f ? tc::ex2_approx((m_ref - M) * p.scale_log2) : 0.f;
            const float w_oth = other.y > 0.f ? tc::ex2_approx((other.x - M) * p.scale_log2) : 0.f;
            const float L = w_own * l_sum + w_oth * other.y;
            const float inv = part.final_ ? 1.f / L : 1.f;
            const uint32_t o_oth = tmem + 256 + (w ^ 1) * 128 + lane_addr;
            // output row and head of this TMEM lane
            const int row = packed ? (r >> p.pack_shift) : part.qt * BQ + r;
            const int out_head = packed ? (part.head << p.pack_shift) + (r & ((1 << p.pack_shift) - 1)) : part.head;
            const size_t pslot = (size_t)blockIdx.x * 2 + part.slot;
            // this warpgroup writes output columns [64 w, 64 w + 64)
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t oa[32], ob[32];
                tc::tmem_ld32(o_own + w * 64 + c * 32, oa);
                tc::tmem_ld32(o_oth + w * 64 + c * 32, ob);
                tc::tmem_wait_ld();
                if (!ok) continue;
                float v[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    // a stream that saw no key contributes nothing (its accumulator may hold anything)
                    const float va = w_own > 0.f ? w_own * __uint_as_float(oa[i]) : 0.f;
                    const float vb = w_oth > 0.f ? w_oth * __uint_as_float(ob[i]) : 0.f;
                    v[i] = (va + vb) * inv;
                }
                const int col = w * 64 + c * 32;
                if (row >= p.t) continue;                    // padding row of the tile: nothing reads it
                if (!part.final_) {
                    float4* dst = reinterpret_cast<float4*>(p.part_o + (pslot * BQ + r) * HD + col);
#pragma unroll
                    for (int i = 0; i < 8; ++i) dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                } else {
                    const size_t off = ((size_t)row * p.h_q + out_head) * HD + col;
                    if (p.out_dtype == OMNI_DTYPE_FP32) {
                        float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.o_out) + off);
#pragma unroll
                        for (int i = 0; i < 8; ++i) dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                    } else {
                        uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.o_out) + off);
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            dst[i] = make_uint4(tc::pack_bf16x2(v[8 * i], v[8 * i + 1]), tc::pack_bf16x2(v[8 * i + 2], v[8 * i + 3]),
                                                tc::pack_bf16x2(v[8 * i + 4], v[8 * i + 5]), tc::pack_bf16x2(v[8 * i + 6], v[8 * i + 7]));
                    }
                }
            }
            if (ok && w == 0) {
                if (!part.final_) { if (row < p.t) p.part_ml[pslot * BQ + r] = make_float2(M, L); }
                else if (p.lse_out && row < p.t) p.lse_out[(size_t)row * p.h_q + out_head] = M * p.scale + logf(L);
            }
            // O (and the part's Q tile) may be reused; the exchange buffer too, once both warpgroups are here
            tc::tcgen05_fence_before();
            tc::mbar_arrive(tc::smem_u32(&bars->o_free));
            named_barrier_256(2);
            kv_base += 2 * n_part;
            ++part_idx;
        }
    }

    tc::tcgen05_fence_before();
    __syncthreads();
#ifdef ATT_TRACE
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        const long long t0 = trace_buf[(2 * TRACE_N + 8) * 6];
        for (int role = 0; role < 3; ++role)
            for (int i = 8; i < TRACE_N; ++i) {
                const long long* e = trace_buf + (role * TRACE_N + i) * 6;
                printf("role %d blk %d : %lld %lld %lld %lld %lld\n", role, i, e[0] - t0, e[1] - t0, e[2] - t0, e[3] - t0, e[4] - t0);
            }
    }
#endif
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, OMNI_DEV_TIMEOUT);
    if (warp == 8) {
        tc::tcgen05_fence_after();
        tc::tmem_dealloc<512>(tmem);
    }
}

// History with holes: which 128-key blocks hold a live slot, and their live bits.  One CTA; thread b takes block b
// (and b + 1024, ...); the live blocks are numbered by a block-wide scan.  Slots at and beyond the span count as dead.
__global__ void __launch_bounds__(1024) attn_block_scan_kernel(const uint8_t* __restrict__ mask, const int32_t* n_hist_dev,
                                                               int n_hist_max, int32_t* live_idx, uint4* live_mask,
                                                               int32_t* n_live, int32_t* status) {
    __shared__ int warp_tot[32];
    __shared__ int s_base;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    int n_hist = n_hist_dev ? *n_hist_dev : n_hist_max;
    if (n_hist < 0 || n_hist > n_hist_max) {
        if (tid == 0) atomicOr(status, OMNI_DEV_BAD_COUNT);
        n_hist = max(0, min(n_hist, n_hist_max));
    }
    const int nb = (n_hist + BK - 1) / BK;
    if (tid == 0) s_base = 0;
    __syncthreads();
    for (int b0 = 0; b0 < nb; b0 += 1024) {
        const int b = b0 + tid;
        uint32_t bits[4] = {0u, 0u, 0u, 0u};
        if (b < nb) {
#pragma unroll
            for (int v = 0; v < 8; ++v) {
                const int pos = b * BK + v * 16;
                if (pos < n_hist) {
                    const uint4 m = __ldg(reinterpret_cast<const uint4*>(mask + pos));
                    const uint32_t w4[4] = {m.x, m.y, m.z, m.w};
                    uint32_t sixteen = 0u;
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint32_t nz = __vcmpne4(w4[k], 0u);        // 0xff per live byte
                        const uint32_t nib = ((nz >> 7) & 1u) | ((nz >> 14) & 2u) | ((nz >> 21) & 4u) | ((nz >> 28) & 8u);
                        sixteen |= nib << (4 * k);
                    }
                    const int valid = n_hist - pos;                      // < 16 only in the last vector of the span
                    if (valid < 16) sixteen &= (1u << valid) - 1u;
                    bits[v >> 1] |= sixteen << ((v & 1) * 16);
                }
            }
        }
        const bool live = (bits[0] | bits[1] | bits[2] | bits[3]) != 0u;
        const unsigned ballot = __ballot_sync(0xffffffffu, live);
        if (lane == 0) warp_tot[wid] = __popc(ballot);
        __syncthreads();
        int before = s_base + __popc(ballot & ((1u << lane) - 1u));
        for (int w = 0; w < wid; ++w) before += warp_tot[w];
        if (live) {
            live_idx[before] = b;
            live_mask[before] = make_uint4(bits[0], bits[1], bits[2], bits[3]);
        }
        __syncthreads();
        if (tid == 0) {
            int tot = 0;
            for (int w = 0; w < 32; ++w) tot += warp_tot[w];
            s_base += tot;
        }
        __syncthreads();
    }
    if (tid == 0) *n_live = s_base;
}

// Merge the partial outputs of every item that was cut between CTAs.  Grid (share boundaries, 4 groups of 32 rows);
// a warp owns 4 rows and a lane 4 of a row's 128 columns.  Shared memory: one int per CTA of the main kernel.
constexpr int MERGE_BATCH = 4;
__global__ void __launch_bounds__(256) attention_merge_kernel(const AttnParams p, int n_cta) {
    extern __shared__ __align__(16) int s_slot[];            // partial slot of every part of the item
    __shared__ int s_n, s_qt, s_head;
    // blockIdx.x + 1 = b: the boundary between the shares of CTA b-1 and CTA b of the main kernel.  An item is
    // cut only where a boundary falls strictly inside it, so the boundaries enumerate the cut items; an item
    // that holds several boundaries is merged by the first of them.
    // rows of this CTA's group of 32 that exist at all (a packed tile of a short chunk is mostly padding)
    {
        const int r_first = blockIdx.y * 32;
        const int row_first = p.pack_shift >= 0 ? (r_first >> p.pack_shift) : 0;
        if (p.pack_shift >= 0 && row_first >= p.t) return;
    }
    int n_hist = p.n_hist_dev ? *p.n_hist_dev : p.n_hist_max;
    n_hist = max(0, min(n_hist, p.n_hist_max));
    Sched s;
    s.nhb = (n_hist + BK - 1) / BK; s.n_tiles = p.n_tiles; s.h_q = p.pack_shift >= 0 ? p.h_kv : p.h_q;
    if (p.live_idx) s.nhb = max(0, min(*p.n_live, s.nhb));
    const long long total = s.total();
    // share boundaries, one per thread (the divisions run in parallel), kept behind the slot list
    long long* s_begin = reinterpret_cast<long long*>(s_slot + ((n_cta + 2) & ~1));         // [n_cta + 1]
    for (int bb = threadIdx.x; bb <= n_cta; bb += blockDim.x) s_begin[bb] = share_begin(total, bb, n_cta);
    __syncthreads();
    if (threadIdx.x == 0) {
        const int b = blockIdx.x + 1;
        const long long w = s_begin[b];
        int n = 0, qt = 0, head = 0, j = 0;
        if (w > 0 && w < total) {
            s.locate(w, qt, head, j);
            const long long w0 = w - j, w1 = w0 + s.nb_item(qt);            // the item is [w0, w1)
            if (j > 0 && s_begin[b - 1] <= w0) {
                // first part: the non-empty share that holds w0 (slot 1); then every non-empty share that
                // starts inside the item (slot 0)
                int bf = b - 1;
                while (bf > 0 && s_begin[bf] == s_begin[bf + 1]) --bf;
                s_slot[n++] = bf * 2 + 1;
                for (int bb = b; bb < n_cta; ++bb) {
                    if (s_begin[bb] >= w1) break;
                    if (s_begin[bb] != s_begin[bb + 1]) s_slot[n++] = bb * 2;
                }
            }
        }
        s_n = n; s_qt = qt; s_head = head;
    }
    __syncthreads();
    const int n_parts = s_n;
    if (n_parts == 0) return;                                // no item is cut at this boundary (or an earlier boundary owns it)
    // launched as a programmatic dependent of the main kernel: everything above ran beside it (it reads only what
    // earlier kernels wrote); the partials exist once the main grid has completed
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int qt = s_qt, head = s_head;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (n_parts <= 2) {
        // the usual case (an item cut once): the loads of the warp's four rows are issued together, one round trip
        const bool packed = p.pack_shift >= 0;
        float2 ml[4][2];
        float4 o[4][2];
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
            const int r = blockIdx.y * 32 + warp * 4 + q4;
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                ml[q4][i] = make_float2(-INFINITY, 0.f);
                o[q4][i] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (i < n_parts) {
                    const size_t pslot = (size_t)s_slot[i];
                    ml[q4][i] = p.part_ml[pslot * BQ + r];
                    o[q4][i] = *reinterpret_cast<const float4*>(p.part_o + (pslot * BQ + r) * HD + lane * 4);
                }
            }
        }
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
            const int r = blockIdx.y * 32 + warp * 4 + q4;
            const int row = packed ? (r >> p.pack_shift) : qt * BQ + r;
            const int out_head = packed ? (head << p.pack_shift) + (r & ((1 << p.pack_shift) - 1)) : head;
            if (row >= p.t) continue;
            float M = -INFINITY;
#pragma unroll
            for (int i = 0; i < 2; ++i)
                if (ml[q4][i].y > 0.f) M = fmaxf(M, ml[q4][i].x);
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            float L = 0.f;
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                if (!(ml[q4][i].y > 0.f)) continue;
                const float wgt = tc::ex2_approx((ml[q4][i].x - M) * p.scale_log2);
                acc.x += wgt * o[q4][i].x; acc.y += wgt * o[q4][i].y; acc.z += wgt * o[q4][i].z; acc.w += wgt * o[q4][i].w;
                L += wgt * ml[q4][i].y;
            }
            const float inv = 1.f / L;
            const size_t off = ((size_t)row * p.h_q + out_head) * HD + lane * 4;
            if (p.out_dtype == OMNI_DTYPE_FP32) {
                *reinterpret_cast<float4*>(static_cast<float*>(p.o_out) + off) =
                    make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
            } else {
                uint2 v;
                v.x = tc::pack_bf16x2(acc.x * inv, acc.y * inv);
                v.y = tc::pack_bf16x2(acc.z * inv, acc.w * inv);
                *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(p.o_out) + off) = v;
            }
            if (p.lse_out && lane == 0) p.lse_out[(size_t)row * p.h_q + out_head] = M * p.scale + logf(L);
        }
        return;
    }
    for (int q4 = 0; q4 < 4; ++q4) {
        const int r = blockIdx.y * 32 + warp * 4 + q4;       // row of the tile
        const bool packed = p.pack_shift >= 0;
        const int row = packed ? (r >> p.pack_shift) : qt * BQ + r;
        const int out_head = packed ? (head << p.pack_shift) + (r & ((1 << p.pack_shift) - 1)) : head;
        if (row >= p.t) continue;
        float M = -INFINITY;
        for (int i = 0; i < n_parts; ++i) {
            const float2 ml = p.part_ml[(size_t)s_slot[i] * BQ + r];
            if (ml.y > 0.f) M = fmaxf(M, ml.x);
        }
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float L = 0.f;
        for (int i0 = 0; i0 < n_parts; i0 += MERGE_BATCH) {
            float2 ml[MERGE_BATCH];
            float4 o[MERGE_BATCH];
#pragma unroll
            for (int i = 0; i < MERGE_BATCH; ++i) {
                ml[i] = make_float2(-INFINITY, 0.f);
                o[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (i0 + i < n_parts) {
                    const size_t pslot = (size_t)s_slot[i0 + i];
                    ml[i] = p.part_ml[pslot * BQ + r];
                    if (ml[i].y > 0.f) o[i] = *reinterpret_cast<const float4*>(p.part_o + (pslot * BQ + r) * HD + lane * 4);
                }
            }
#pragma unroll
            for (int i = 0; i < MERGE_BATCH; ++i) {
                if (!(ml[i].y > 0.f)) continue;
                const float wgt = tc::ex2_approx((ml[i].x - M) * p.scale_log2);
                acc.x += wgt * o[i].x; acc.y += wgt * o[i].y; acc.z += wgt * o[i].z; acc.w += wgt * o[i].w;
                L += wgt * ml[i].y;
            }
        }
        const float inv = 1.f / L;
        const size_t off = ((size_t)row * p.h_q + out_head) * HD + lane * 4;
        if (p.out_dtype == OMNI_DTYPE_FP32) {
            *reinterpret_cast<float4*>(static_cast<float*>(p.o_out) + off) =
                make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
        } else {
            uint2 v;
            v.x = tc::pack_bf16x2(acc.x * inv, acc.y * inv);
            v.y = tc::pack_bf16x2(acc.z * inv, acc.w * inv);
            *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(p.o_out) + off) = v;
        }
        if (p.lse_out && lane == 0) p.lse_out[(size_t)row * p.h_q + out_head] = M * p.scale + logf(L);
    }
}

}  // namespace

omni_status omni_attention_tc(omnitide_ctx* ctx, cudaStream_t st, const void* q, int t, const void* k_hist,
                              const void* v_hist, const int32_t* n_hist_dev, int n_hist_max, const void* k_chunk,
                              const void* v_chunk, float scale, void* o_out, int out_dtype, float* lse_out,
                              const uint8_t* hist_mask) {
    const omni_geometry& g = ctx->g;
    CUtensorMap tm_q, tm_kh, tm_vh, tm_kc, tm_vc;
    const uint64_t q_inner = (uint64_t)g.h_q * HD, kv_inner = (uint64_t)g.h_kv * HD;
    // few queries (decode, short chunks): all query heads of a KV group share one 128-row tile, so K and V are read
    // once per group and the tile is not 127/128 padding
    const int G = g.h_q / g.h_kv;
    int pack_shift = -1;
    if ((G & (G - 1)) == 0 && G <= BQ && (long long)t * G <= BQ)
        for (int sft = 0; sft < 8; ++sft) if ((1 << sft) == G) pack_shift = sft;
    bool ok = pack_shift >= 0 ? omni_make_map_q_packed(ctx->encode_tiled, &tm_q, q, t, g.h_q, G)
                              : omni_make_map_bf16(ctx->encode_tiled, &tm_q, q, t, q_inner, BQ);
    ok &= omni_make_map_bf16(ctx->encode_tiled, &tm_kc, k_chunk, t, kv_inner, BK);
    ok &= omni_make_map_bf16(ctx->encode_tiled, &tm_vc, v_chunk, t, kv_inner, BK);
    // with an empty history the history maps are never used; point them at the chunk to stay valid
    ok &= omni_make_map_bf16(ctx->encode_tiled, &tm_kh, n_hist_max > 0 ? k_hist : k_chunk, n_hist_max > 0 ? n_hist_max : t, kv_inner, BK);
    ok &= omni_make_map_bf16(ctx->encode_tiled, &tm_vh, n_hist_max > 0 ? v_hist : v_chunk, n_hist_max > 0 ? n_hist_max : t, kv_inner, BK);
    if (!ok) OMNI_FAIL(ctx, OMNI_ERR_CUDA, "attention: cuTensorMapEncodeTiled failed");
    AttnParams p;
    p.t = t; p.h_q = g.h_q; p.h_kv = g.h_kv; p.n_hist_dev = n_hist_dev; p.n_hist_max = n_hist_max;
    p.scale = scale; p.scale_log2 = scale * 1.4426950408889634f;
    p.o_out = o_out; p.out_dtype = out_dtype; p.lse_out = lse_out; p.status = ctx->status_dev;
    p.pack_shift = pack_shift;
    p.live_idx = nullptr; p.live_mask = nullptr; p.n_live = nullptr;
    if (hist_mask && n_hist_max > 0) {
        attn_block_scan_kernel<<<1, 1024, 0, st>>>(hist_mask, n_hist_dev, n_hist_max, ctx->attn_live_idx, ctx->attn_live_mask,
                                                   ctx->attn_n_live, ctx->status_dev);
        OMNI_CHECK_LAUNCH(ctx, "attn_block_scan_kernel");
        p.live_idx = ctx->attn_live_idx; p.live_mask = ctx->attn_live_mask; p.n_live = ctx->attn_n_live;
    }
    p.n_tiles = pack_shift >= 0 ? 1 : (t + BQ - 1) / BQ;
    const int n_items_heads = pack_shift >= 0 ? g.h_kv : g.h_q;
    // one CTA per SM, fewer when the whole job is small (at least 4 block steps per CTA)
    const long long nhb_max = (n_hist_max + BK - 1) / BK;
    const long long w_max = (long long)n_items_heads * ((long long)p.n_tiles * (nhb_max + 1) + (long long)p.n_tiles * (p.n_tiles - 1) / 2);
    const int n_cta = (int)std::max(1ll, std::min((long long)ctx->sm_count, w_max / 4));
    p.part_o = ctx->attn_part_o; p.part_ml = reinterpret_cast<float2*>(ctx->attn_part_ml);
    if (!ctx->attn_attr_set) {                               // per context, hence per device
        OMNI_CUDA(ctx, cudaFuncSetAttribute(attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
        ctx->attn_attr_set = true;
    }
    attention_tc_kernel<<<n_cta, ATT_THREADS, SMEM_BYTES, st>>>(tm_q, tm_kh, tm_vh, tm_kc, tm_vc, p);
    OMNI_CHECK_LAUNCH(ctx, "attention_tc_kernel");
    if (n_cta > 1) {
        // one CTA row per boundary between two shares: only an item cut there has partials to merge
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(n_cta - 1, 4);
        cfg.blockDim = dim3(256);
        cfg.dynamicSmemBytes = (n_cta + 2) * sizeof(int) + (n_cta + 1) * sizeof(long long);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;       // its prologue and its launch run under the main kernel
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        OMNI_CUDA(ctx, cudaLaunchKernelEx(&cfg, attention_merge_kernel, p, n_cta));
        ++ctx->launches;
    }
    return OMNI_OK;
}
