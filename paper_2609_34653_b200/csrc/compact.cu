// OmniPage eager compaction (mode PACK) and the append step.
//
// One kernel, one CTA per SM, does the whole compaction.  The keep mask is cut into one part per
// CTA; a CTA counts its own part (one 16-byte vector per lane, kept in registers), publishes the
// count in global memory and waits (bounded) until all CTAs have arrived: the launch is cooperative,
// so all CTAs are resident.  Each CTA then gathers the per-part counts, scans them, takes an equal
// share of the DESTINATION rows, rebuilds the source slots of that share from the mask parts that
// hold them and streams the rows HBM -> shared memory -> HBM with bulk asynchronous copies issued
// by one lane per warp (no per-vector instructions).  The slot map, the page classes and the integer
// summary come out of the same pass.  HBM traffic is one read and one write per retained row; the
// mask is read about once in total (every CTA reading all of it cost 4 us of L2 time).
#include "common.cuh"
#include "tc_ptx.cuh"

#include <algorithm>
#include <cmath>

namespace {


constexpr int CP_THREADS = 512;
constexpr int CP_WARPS = CP_THREADS / 32;

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::128B.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) {
    asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

__device__ __forceinline__ int nonzero_bytes(uint32_t w) { return __popc(__vcmpne4(w, 0u)) >> 3; }

__device__ __forceinline__ int warp_excl_scan(int x, int lane, int& total) {
    int incl = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
    }
    total = __shfl_sync(0xffffffffu, incl, 31);
    return incl - x;
}

// Exclusive scan of data[0..n) in shared memory by the whole block; data[n] receives the total.
__device__ int block_excl_scan(int* data, int n, int* warp_tot /*[CP_WARPS+1]*/) {
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int ipt = (n + CP_THREADS - 1) / CP_THREADS;
    const int lo = min(tid * ipt, n), hi = min(lo + ipt, n);
    int sum = 0;
    for (int i = lo; i < hi; ++i) sum += data[i];
    int wt;
    int excl = warp_excl_scan(sum, lane, wt);
    if (lane == 31) warp_tot[wid] = wt;
    __syncthreads();
    if (wid == 0) {
        int v = lane < CP_WARPS ? warp_tot[lane] : 0;
        int t2;
        int e = warp_excl_scan(v, lane, t2);
        if (lane < CP_WARPS) warp_tot[lane] = e;
        if (lane == 0) warp_tot[CP_WARPS] = t2;
    }
    __syncthreads();
    int run = warp_tot[wid] + excl;
    for (int i = lo; i < hi; ++i) {
        int v = data[i];
        data[i] = run;
        run += v;
    }
    const int total = warp_tot[CP_WARPS];
    if (tid == 0) data[n] = total;
    __syncthreads();
    return total;
}

struct CompactArgs {
    const char* k_src; const char* v_src; char* k_dst; char* v_dst;
    const uint8_t* mask; const int32_t* s_span_dev; int s_span_max;
    int page_size; int row_bytes; int vpr; int vpr_shift;
    const omni_unit* units_kept; const int32_t* n_units_kept_dev; int n_units_max;
    int32_t* slot_map; omni_compact_info* info; uint8_t* page_class; int32_t* status;
    int rows_cap;      // capacity of the per-CTA source list
    int max_chunks;    // capacity of the chunk-prefix array
    int n_slots;       // row buffers per warp for the bulk-copy path (0: move rows with vector loads/stores)
    int part_groups;   // 512-byte mask groups per CTA
    // ordered-suffix migration: the span that is packed starts at slot *span_off_dev (a multiple of 16; negative: nothing
    // to pack); mask, sources and slot map are taken from there and slot-map values count from there too
    const int32_t* span_off_dev;
    unsigned long long* words;   // [0]: arrival counter (low half, never reset); [1 + i]: (epoch << 32) | retained count of part i
    uint32_t epoch;
};

constexpr int CP_BATCH = 16;        // 16-byte vectors in flight per thread (vector path)
constexpr int CP_MAX_SLOTS = 4;     // more rows in flight per warp than this measured slower

// zeroes the bytes of v at and beyond `valid` (any int: <= 0 clears all, >= 16 keeps all)
__device__ __forceinline__ uint32_t clip_word(uint32_t w, int nv) {
    return nv >= 4 ? w : (nv <= 0 ? 0u : (w & ((1u << (8 * nv)) - 1u)));
}
__device__ __forceinline__ uint4 clip_vec(uint4 v, int valid) {
    v.x = clip_word(v.x, valid); v.y = clip_word(v.y, valid - 4);
    v.z = clip_word(v.z, valid - 8); v.w = clip_word(v.w, valid - 12);
    return v;
}
__device__ __forceinline__ uint32_t byte_at(const uint4& v, int b) {      // b is a compile-time constant after unrolling
    const uint32_t w = b < 4 ? v.x : (b < 8 ? v.y : (b < 12 ? v.z : v.w));
    return (w >> ((b & 3) * 8)) & 0xffu;
}
__device__ __forceinline__ int count_kept(const uint4& v) {
    return nonzero_bytes(v.x) + nonzero_bytes(v.y) + nonzero_bytes(v.z) + nonzero_bytes(v.w);
}
// index of the first zero byte of v, 16 if there is none
__device__ __forceinline__ int first_zero_byte(const uint4& v) {
    const uint32_t zx = __vcmpeq4(v.x, 0u), zy = __vcmpeq4(v.y, 0u), zz = __vcmpeq4(v.z, 0u), zw = __vcmpeq4(v.w, 0u);
    int z = 16;
    if (zw) z = 12 + ((__ffs(zw) - 1) >> 3);
    if (zz) z = 8 + ((__ffs(zz) - 1) >> 3);
    if (zy) z = 4 + ((__ffs(zy) - 1) >> 3);
    if (zx) z = (__ffs(zx) - 1) >> 3;
    return z;
}
__device__ __forceinline__ uint4 ld_mask(const uint8_t* mask, int vec) {
    return __ldg(reinterpret_cast<const uint4*>(mask) + vec);
}

// A warp holds the 512 mask bytes that start at `base` (16 per lane, v); `run` = retained slots before them.
// Writes the source slots of the destinations in [d0, d0 + n_rows) that fall in this group.
__device__ __forceinline__ void emit_sources(const uint4& v, int base, int run, int lane, int d0, int n_rows,
                                             int* src_list) {
    const int cnt = count_kept(v);
    int tot;
    int r = run + warp_excl_scan(cnt, lane, tot) - d0;
    if (cnt && r < n_rows && r + cnt > 0) {
        const int pos = base + lane * 16;
#pragma unroll
        for (int b = 0; b < 16; ++b)
            if (byte_at(v, b)) {
                if (r >= 0 && r < n_rows) src_list[r] = pos + b;
                ++r;
            }
    }
}
// Same group: writes slot_map for the slots below s.
__device__ __forceinline__ void emit_slot_map(const uint4& v, int base, int run, int lane, int s, int32_t* slot_map) {
    const int cnt = count_kept(v);
    int tot;
    int r = run + warp_excl_scan(cnt, lane, tot);
    const int pos = base + lane * 16;
    int o[16];
#pragma unroll
    for (int b = 0; b < 16; ++b) {
        const bool kept = byte_at(v, b) != 0;
        o[b] = kept ? r : -1;
        r += kept;
    }
    if (pos + 16 <= s) {
        int4* o4 = reinterpret_cast<int4*>(slot_map + pos);
        o4[0] = make_int4(o[0], o[1], o[2], o[3]);
        o4[1] = make_int4(o[4], o[5], o[6], o[7]);
        o4[2] = make_int4(o[8], o[9], o[10], o[11]);
        o4[3] = make_int4(o[12], o[13], o[14], o[15]);
    } else {
#pragma unroll
        for (int b = 0; b < 16; ++b)
            if (pos + b < s) slot_map[pos + b] = o[b];
    }
}

__device__ __forceinline__ void bulk_load(uint32_t smem_dst, const void* gsrc, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_dst), "l"(gsrc), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_store(void* gdst, uint32_t smem_src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_src), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}


__device__ __forceinline__ void st_relaxed_gpu(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long ld_relaxed_gpu(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

// element i of a device array of pointers, through the read-only path
template <class T, class P>
__device__ __forceinline__ T* ldg_ptr(P table, int i) {
    return reinterpret_cast<T*>(__ldg(reinterpret_cast<const unsigned long long*>(table) + i));
}

// One lane streams `mcp` row copies HBM -> shared memory -> HBM with cp.async.bulk, `n_slots` rows in flight:
// copy q reads src_of(q) and writes dst_of(q) (both called in increasing q).  Returns false after a timeout.
template <class SrcOf, class DstOf>
__device__ __forceinline__ bool bulk_copy_loop(const int mcp, SrcOf src_of, DstOf dst_of, const uint32_t row_bytes,
                                               const int n_slots, const uint32_t buf0, uint64_t* bars, int* abort_flag_p) {
    auto issue_load = [&](int q) {
        const int slot = q % n_slots;
        const uint32_t bar = tc::smem_u32(&bars[slot]);
        tc::mbar_expect_tx(bar, row_bytes);
        bulk_load(buf0 + slot * row_bytes, src_of(q), row_bytes, bar);
    };
    for (int q = 0; q < mcp && q < n_slots; ++q) issue_load(q);
    bool ok = true;
    for (int q = 0; q < mcp && ok; ++q) {
        const int slot = q % n_slots;
        ok = tc::mbar_wait(tc::smem_u32(&bars[slot]), (q / n_slots) & 1, abort_flag_p);
        if (!ok) break;
        bulk_store(dst_of(q), buf0 + slot * row_bytes, row_bytes);
        // the buffer of copy q-1 is free once its store has read it: refill it
        if (q >= 1 && q - 1 + n_slots < mcp) {
            asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
            issue_load(q - 1 + n_slots);
        }
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    return ok;
}

// Moves destination rows [d0, d0 + n_rows) of this CTA; src_list[r] is the source slot of row d0 + r.
template <class Args>
__device__ __forceinline__ void move_rows(const Args& a, const int* src_list, const int d0, const int n_rows, char* rowbuf,
                                          uint64_t (*cbar)[CP_MAX_SLOTS], int* abort_flag_p) {
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    if (a.n_slots > 0) {
        // bulk-copy path: lane 0 of every warp streams its rows HBM -> shared memory -> HBM with
        // cp.async.bulk, `n_slots` rows in flight per warp; no per-vector instructions at all.
        if (lane == 0) {
            const int n_copies = 2 * n_rows;                         // copy i: row i >> 1, K (even) or V (odd)
            const int mcp = n_copies > wid ? (n_copies - wid + CP_WARPS - 1) / CP_WARPS : 0;
            const uint32_t buf0 = tc::smem_u32(rowbuf) + (uint32_t)(wid * a.n_slots) * a.row_bytes;
            auto src_of = [&](int q) {
                const int i = wid + q * CP_WARPS;
                return ((i & 1) ? a.v_src : a.k_src) + (size_t)src_list[i >> 1] * a.row_bytes;
            };
            auto dst_of = [&](int q) {
                const int i = wid + q * CP_WARPS;
                return ((i & 1) ? a.v_dst : a.k_dst) + (size_t)(d0 + (i >> 1)) * a.row_bytes;
            };
            const bool ok = bulk_copy_loop(mcp, src_of, dst_of, a.row_bytes, a.n_slots, buf0, cbar[wid], abort_flag_p);
            if (!ok) atomicOr(a.status, OMNI_DEV_TIMEOUT);
        }
        return;
    }
    // vector path (rows too large for the buffers, or too small to be worth a bulk copy)
    const int total = n_rows * 2 * a.vpr;                    // (row, K or V, vector)
    for (int base = tid; base < total; base += CP_THREADS * CP_BATCH) {
        uint4 buf[CP_BATCH];
#pragma unroll
        for (int u = 0; u < CP_BATCH; ++u) {
            const int idx = base + u * CP_THREADS;
            if (idx < total) {
                int rw, v;
                if (a.vpr_shift >= 0) { rw = idx >> a.vpr_shift; v = idx & (a.vpr - 1); }
                else { rw = idx / a.vpr; v = idx - rw * a.vpr; }
                const size_t so = (size_t)src_list[rw >> 1] * a.row_bytes + (size_t)v * 16;
                buf[u] = ld_stream(reinterpret_cast<const uint4*>(((rw & 1) ? a.v_src : a.k_src) + so));
            }
        }
#pragma unroll
        for (int u = 0; u < CP_BATCH; ++u) {
            const int idx = base + u * CP_THREADS;
            if (idx < total) {
                int rw, v;
                if (a.vpr_shift >= 0) { rw = idx >> a.vpr_shift; v = idx & (a.vpr - 1); }
                else { rw = idx / a.vpr; v = idx - rw * a.vpr; }
                const size_t dof = (size_t)(d0 + (rw >> 1)) * a.row_bytes + (size_t)v * 16;
                st_stream(reinterpret_cast<uint4*>(((rw & 1) ? a.v_dst : a.k_dst) + dof), buf[u]);
            }
        }
    }
}

// 16 mask bytes at slot `pos` (a multiple of 16) with the bytes at and beyond s zeroed
__device__ __forceinline__ uint4 mask_at(const uint8_t* mask, int pos, int s) {
    uint4 v = make_uint4(0, 0, 0, 0);
    if (pos < s) v = clip_vec(ld_mask(mask, pos >> 4), s - pos);
    return v;
}

// The mask is cut into gridDim.x parts of `part_groups` groups of 512 bytes; CTA i counts part i alone and
// publishes the count in words[i] tagged with the epoch of this launch; every CTA then gathers all the
// counts (the only cross-CTA step: all CTAs are resident, one per SM, and the wait is bounded).
__global__ void __launch_bounds__(CP_THREADS, 1) compact_pack_kernel(const CompactArgs a_in) {
    CompactArgs a = a_in;
    int span_off = 0;
    bool empty_span = false;
    if (a_in.span_off_dev) {
        const int s_all = a_in.s_span_dev ? __ldg(a_in.s_span_dev) : a_in.s_span_max;
        span_off = __ldg(a_in.span_off_dev);
        if (span_off < 0 || span_off >= s_all) {
            // nothing to pack: an empty span at an offset that keeps the 16-byte mask loads and slot-map stores aligned
            empty_span = true;
            span_off = max(0, min(s_all, a_in.s_span_max)) & ~15;
        }
        a.mask += span_off;
        if (a.k_src) { a.k_src += (size_t)span_off * a.row_bytes; a.v_src += (size_t)span_off * a.row_bytes; }
        if (a.slot_map) a.slot_map += span_off;
        a.s_span_max -= span_off;
    }
    extern __shared__ __align__(128) int smem_i[];
    int* prefix = smem_i;                                   // [max_chunks]: part counts, then their exclusive scan
    int* src_list = smem_i + a.max_chunks;                  // [rows_cap]
    char* rowbuf = reinterpret_cast<char*>(smem_i + a.max_chunks + a.rows_cap);   // row buffers of the bulk-copy path
    __shared__ int warp_tot[CP_WARPS + 1];
    __shared__ int wcnt[CP_WARPS];
    __shared__ int s_misc[4];
    __shared__ uint64_t cbar[CP_WARPS][CP_MAX_SLOTS];
    __shared__ int abort_flag;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int G = gridDim.x;

    // ---- prologue: every load whose address needs no device-side count is issued before anything waits ----
    const int part_bytes = a.part_groups * 512;
    const int my_base = blockIdx.x * part_bytes;
    const int gpw = (a.part_groups + CP_WARPS - 1) / CP_WARPS;        // groups per warp (contiguous)
    const int wg0 = wid * gpw, wg1 = min(a.part_groups, wg0 + gpw);   // this warp's groups of the part
    uint4 mv = make_uint4(0, 0, 0, 0);                                // its first group stays in registers
    if (wg0 < wg1 && my_base + wg0 * 512 + lane * 16 < a.s_span_max) mv = ld_mask(a.mask, (my_base + wg0 * 512) / 16 + lane);
    int s = a.s_span_dev ? __ldg(a.s_span_dev) - span_off : a.s_span_max;
    if (empty_span) s = 0;
    int nu = 0, u_len = 0, u_group = -1;
    if (a.units_kept) {
        nu = a.n_units_kept_dev ? __ldg(a.n_units_kept_dev) : a.n_units_max;
        if (tid < a.n_units_max) { u_len = __ldg(&a.units_kept[tid].len); u_group = __ldg(&a.units_kept[tid].group); }
    }
    for (int c = tid; c < a.max_chunks; c += CP_THREADS) prefix[c] = 0;
    if (tid == 0) { s_misc[0] = 0; s_misc[1] = 0; s_misc[2] = G; abort_flag = 0; }
    if (lane == 0 && a.n_slots > 0) {
        for (int q = 0; q < a.n_slots; ++q) tc::mbar_init(tc::smem_u32(&cbar[wid][q]), 1);
        tc::fence_barrier_init();
    }
    if (s > a.s_span_max || s < 0) {
        if (tid == 0 && blockIdx.x == 0) atomicOr(a.status, OMNI_DEV_BAD_COUNT);
        s = max(0, min(s, a.s_span_max));
    }
    nu = max(0, min(nu, a.n_units_max));

    // ---- phase A: count the own part, publish, gather all parts ------------------------------------------
    mv = clip_vec(mv, s - (my_base + wg0 * 512 + lane * 16));
    {
        int cnt = count_kept(mv);
        for (int g = wg0 + 1; g < wg1; ++g) cnt += count_kept(mask_at(a.mask, my_base + g * 512 + lane * 16, s));
        cnt = __reduce_add_sync(0xffffffffu, cnt);
        if (lane == 0) wcnt[wid] = cnt;
    }
    // partitions from the compacted unit table
    int p0 = 0, p1 = 0;
    for (int u = tid; u < nu; u += CP_THREADS) {
        if (u >= CP_THREADS) { u_len = a.units_kept[u].len; u_group = a.units_kept[u].group; }
        if (u_group == OMNI_GROUP_MUST_KEEP) p0 += u_len;
        else if (u_group == OMNI_GROUP_SELECTED) p1 += u_len;
    }
    __syncthreads();
    if (a.units_kept) {
        p0 = __reduce_add_sync(0xffffffffu, p0);
        p1 = __reduce_add_sync(0xffffffffu, p1);
        if (lane == 0 && (p0 | p1)) { atomicAdd(&s_misc[0], p0); atomicAdd(&s_misc[1], p1); }
    }
    if (tid == 0) {
        int tot = 0;
#pragma unroll
        for (int w = 0; w < CP_WARPS; ++w) tot += wcnt[w];
        // publish the count tagged with the epoch, then arrive with release; the pollers acquire (measured
        // faster than relaxed accesses, which linger in the SM).  Readers check the tags as well.
        st_relaxed_gpu(a.words + 1 + blockIdx.x, ((unsigned long long)a.epoch << 32) | (unsigned)tot);
        asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(a.words) : "memory");
        const unsigned target = a.epoch * (unsigned)G;       // the counter never resets: epoch e ends at e * G
        const long long t0 = clock64();
        for (;;) {
            unsigned seen;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(a.words) : "memory");
            if ((int)(seen - target) >= 0) break;
            if (clock64() - t0 > (1ll << 31)) { abort_flag = 1; break; }
        }
    }
    __syncthreads();
    const bool want_lead = blockIdx.x == 0 && a.info != nullptr;   // only CTA 0 needs rows_moved
    int n_kept;
    if (G < CP_THREADS) {
        // thread t gathers the count of part t; the scan runs on the registers
        int cnt_t = 0;
        if (tid < G && !abort_flag) {
            const long long t0 = clock64();
            for (;;) {
                const unsigned long long w = ld_relaxed_gpu(a.words + 1 + tid);
                if ((uint32_t)(w >> 32) == a.epoch) { cnt_t = (int)(uint32_t)w; break; }
                if (clock64() - t0 > (1ll << 31)) { abort_flag = 1; break; }
            }
            // first part that is not retained completely
            if (want_lead && cnt_t < max(0, min(part_bytes, s - tid * part_bytes))) atomicMin(&s_misc[2], tid);
        }
        int tot;
        const int ex = warp_excl_scan(cnt_t, lane, tot);
        if (lane == 0) warp_tot[wid] = tot;
        __syncthreads();
        int base = 0;
        for (int w = 0; w < wid; ++w) base += warp_tot[w];
        if (tid <= G) prefix[tid] = base + ex;
        __syncthreads();
        n_kept = prefix[G];
    } else {
        if (!abort_flag) {
            for (int t = tid; t < G; t += CP_THREADS) {
                const long long t0 = clock64();
                for (;;) {
                    const unsigned long long w = ld_relaxed_gpu(a.words + 1 + t);
                    if ((uint32_t)(w >> 32) == a.epoch) { prefix[t] = (int)(uint32_t)w; break; }
                    if (clock64() - t0 > (1ll << 31)) { abort_flag = 1; break; }
                }
                if (want_lead && prefix[t] < max(0, min(part_bytes, s - t * part_bytes))) atomicMin(&s_misc[2], t);
            }
        }
        __syncthreads();
        n_kept = block_excl_scan(prefix, G, warp_tot);
    }
    if (abort_flag) {
        if (tid == 0) atomicOr(a.status, OMNI_DEV_TIMEOUT);
        return;
    }
    const int n0 = s_misc[0], n1 = s_misc[1];

    // ---- phase B: destination share of this CTA, slot map of its own part -------------------------------
    const int rows_per = (n_kept + G - 1) / G;
    const int d0 = min(n_kept, (int)blockIdx.x * rows_per);
    const int d1 = min(n_kept, d0 + rows_per);
    const int n_rows = min(d1 - d0, a.rows_cap);
    if (n_rows > 0) {
        // largest part c with prefix[c] <= d0: prefix is non-decreasing, so count the entries <= d0
        int n_le = 0;
        for (int c0 = 0; c0 < G; c0 += 32)
            n_le += __popc(__ballot_sync(0xffffffffu, c0 + lane < G && prefix[c0 + lane] <= d0));
        const int c_first = n_le - 1;
        // one warp per part that holds destinations of this CTA, taken from the last warp down (the first
        // warps write the slot map meanwhile); a part is walked four groups at a time, loads first
        for (int c = c_first + (CP_WARPS - 1 - wid); c < G; c += CP_WARPS) {
            const int pc = prefix[c];
            if (pc >= d1) break;
            if (prefix[c + 1] == pc) continue;
            int run = pc;
            for (int g0 = 0; g0 < a.part_groups && run < d1; g0 += 4) {
                uint4 v[4];
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    v[j] = g0 + j < a.part_groups ? mask_at(a.mask, c * part_bytes + (g0 + j) * 512 + lane * 16, s)
                                                  : make_uint4(0, 0, 0, 0);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (g0 + j < a.part_groups && run < d1) {
                        emit_sources(v[j], c * part_bytes + (g0 + j) * 512, run, lane, d0, n_rows, src_list);
                        run += __reduce_add_sync(0xffffffffu, count_kept(v[j]));
                    }
                }
            }
        }
    }
    if (a.slot_map && wg0 < wg1) {
        int run = prefix[blockIdx.x];
        for (int w = 0; w < wid; ++w) run += wcnt[w];
        for (int g = wg0; g < wg1; ++g) {
            const int base = my_base + g * 512;
            if (base >= s) break;
            const uint4 v = g == wg0 ? mv : mask_at(a.mask, base + lane * 16, s);
            emit_slot_map(v, base, run + span_off, lane, s, a.slot_map);
            run += __reduce_add_sync(0xffffffffu, count_kept(v));
        }
    }
    // ---- integer summary and page classes ------------------------------------------------------------
    if (want_lead && wid == CP_WARPS - 1) {
        // a retained row keeps its slot exactly when every slot before it is retained: rows_moved counts the
        // retained rows behind the first slot that is dropped
        const int c_open = s_misc[2];
        int lead = s;
        if (c_open < G) {
            for (int g = 0; g < a.part_groups; ++g) {
                const int base = c_open * part_bytes + g * 512;
                if (base >= s) break;
                const uint4 v = mask_at(a.mask, base + lane * 16, s);
                const int z = first_zero_byte(v);
                const int cand = __reduce_min_sync(0xffffffffu, z < 16 ? base + lane * 16 + z : 0x7fffffff);
                if (cand != 0x7fffffff) { lead = min(cand, s); break; }
            }
        }
        if (lane == 0) {
            a.info->n_kept = n_kept;
            a.info->span_pages = (n_kept + a.page_size - 1) / a.page_size;
            a.info->rows_moved = n_kept - min(lead, n_kept);
            a.info->part_begin[0] = 0;
            a.info->part_begin[1] = a.units_kept ? n0 : 0;
            a.info->part_begin[2] = a.units_kept ? n0 + n1 : 0;
            a.info->part_begin[3] = n_kept;
            a.info->reserved = 0;
        }
    }
    if (a.page_class) {
        const int n_pages = (a.s_span_max + a.page_size - 1) / a.page_size;
        for (int p = blockIdx.x * CP_THREADS + tid; p < n_pages; p += G * CP_THREADS) {
            const long long lo = (long long)p * a.page_size;
            const long long hi = min(lo + a.page_size, (long long)n_kept);
            uint8_t cls = OMNI_PAGE_EMPTY;
            if (hi > lo) {
                if (lo < n0) cls = OMNI_GROUP_MUST_KEEP;
                else if (hi - lo == a.page_size) cls = OMNI_GROUP_SELECTED;
                else cls = OMNI_GROUP_RECENT;
            }
            a.page_class[p] = cls;
        }
    }
    if (a.k_dst == nullptr) return;
    __syncthreads();                                        // the source list is complete

    move_rows(a, src_list, d0, n_rows, rowbuf, cbar, &abort_flag);
}

// ---------------------------------------------------------------------------------------------------
// Unit-granular compaction: the keep decision is one code per unit, so the gather is a list of at most
// n_units contiguous runs and no mask is read.  No CTA needs anything from another: every CTA loads the
// unit table (one round trip), scans the kept lengths, takes its share of the destination rows and
// starts copying.
struct CompactUnitsArgs {
    const char* k_src; const char* v_src; char* k_dst; char* v_dst;
    const omni_unit* units; const int32_t* n_units_dev; int n_units_max; const uint8_t* unit_keep;
    const int32_t* unit_kept_len;   // nullable: tokens kept at the start of every unit (sink prefixes); else whole units
    int s_span_max; int page_size; int row_bytes; int vpr; int vpr_shift;
    const omni_unit* units_kept; const int32_t* n_units_kept_dev;
    int32_t* slot_map; omni_compact_info* info; uint8_t* page_class; int32_t* status;
    int rows_cap; int n_slots;
    // RoPE re-index of the moved keys (rope_dims == 0: off): bf16 rows of heads of rope_head_dim elements
    int rope_dims; int rope_head_dim; double rope_log2_base;
    // batched form: n_layers caches share the one source -> destination map (device arrays of n_layers pointers)
    int n_layers;
    const char* const* k_src_l; const char* const* v_src_l; char* const* k_dst_l; char* const* v_dst_l;
};

// The same row mover with the keys re-rotated to their new positions (Section 5.2: a kept token's position drops by
// the number of deleted tokens before it and the runtime applies the matching RoPE adjustment to its cached key).
// Positions are slot indices, so the shift of row r is (d0 + r) - src_list[r].  The whole warp takes part: lane 0
// drives the bulk copies, and once a K row has landed in shared memory every lane rotates the pairs
// (i, i + rope_dims / 2) of its dimensions i = lane, lane + 32, ... in all heads, in place, before the row is stored.
// A warp takes the K and the V row of the same destination rows (every warp rotates as much as any other) and keeps
// the sines and cosines of the last shift: the rows of a kept run share theirs.
// Angles are formed and reduced to one turn in double (a shift of 1e5 positions times a float frequency would lose
// the phase), the rotation itself runs in fp32 and the result is rounded to bf16 (nearest even).
__device__ __forceinline__ void move_rows_rope(const CompactUnitsArgs& a, const int* src_list, const int d0, const int n_rows,
                                               char* rowbuf, uint64_t (*cbar)[CP_MAX_SLOTS], int* abort_flag_p) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    // copy q of this warp: row wid + (q / 2) * CP_WARPS, its K row for even q and its V row for odd q, so that every
    // warp has the same share of rotations
    const int my_rows = n_rows > wid ? (n_rows - wid + CP_WARPS - 1) / CP_WARPS : 0;
    const int mcp = 2 * my_rows;
    char* gbuf0 = rowbuf + (size_t)(wid * a.n_slots) * a.row_bytes;
    const uint32_t buf0 = tc::smem_u32(gbuf0);
    const int half = a.rope_dims >> 1, n_heads = (a.row_bytes >> 1) / a.rope_head_dim;
    auto row_of = [&](int q) { return wid + (q >> 1) * CP_WARPS; };
    auto src_of = [&](int q) { return ((q & 1) ? a.v_src : a.k_src) + (size_t)src_list[row_of(q)] * a.row_bytes; };
    auto issue_load = [&](int q) {
        const int slot = q % a.n_slots;
        const uint32_t bar = tc::smem_u32(&cbar[wid][slot]);
        tc::mbar_expect_tx(bar, a.row_bytes);
        bulk_load(buf0 + slot * a.row_bytes, src_of(q), a.row_bytes, bar);
    };
    if (lane == 0)
        for (int q = 0; q < mcp && q < a.n_slots; ++q) issue_load(q);
    // the frequencies (double: a shift of 1e5 positions times a float frequency would lose the phase) are formed
    // while the first rows are in flight; rope_dims <= 256: at most four per lane
    double inv_freq[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int i = lane + 32 * j;
        inv_freq[j] = 0.0;
        if (32 * j < half) inv_freq[j] = i < half ? exp2(-(2.0 * i / a.rope_dims) * a.rope_log2_base) : 0.0;
    }
    bool ok = true;
    int delta_of_trig = 0;                                   // the shift cs[] / sn[] were computed for (0: none yet)
    float cs[4], sn[4];
    for (int q = 0; q < mcp && ok; ++q) {
        const int slot = q % a.n_slots;
        ok = __all_sync(0xffffffffu, tc::mbar_wait(tc::smem_u32(&cbar[wid][slot]), (q / a.n_slots) & 1, abort_flag_p));
        if (!ok) break;
        const int row = row_of(q);
        const int delta = (d0 + row) - src_list[row];
        if (!(q & 1) && delta != 0) {
            if (delta != delta_of_trig) {                    // the rows of a kept run share their shift
                delta_of_trig = delta;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    // the phase is reduced to one turn in double (three operations), then the fast fp32 sine and
                    // cosine (absolute error about 2^-21, far below the bf16 step of the result) do the rest
                    const double turns = (double)delta * inv_freq[j] * 0.15915494309189535;
                    __sincosf((float)((turns - rint(turns)) * 6.283185307179586), &sn[j], &cs[j]);
                }
            }
            __nv_bfloat16* r = reinterpret_cast<__nv_bfloat16*>(gbuf0 + (size_t)slot * a.row_bytes);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int i = lane + 32 * j;
                if (i < half) {
                    const float c = cs[j], s_ = sn[j];
                    int h = 0;
                    for (; h + 4 <= n_heads; h += 4) {       // four heads at a time: eight independent loads in flight
                        __nv_bfloat16* px = r + h * a.rope_head_dim + i;
                        float x[4], y[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            x[k] = __bfloat162float(px[k * a.rope_head_dim]);
                            y[k] = __bfloat162float(px[k * a.rope_head_dim + half]);
                        }
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            px[k * a.rope_head_dim] = __float2bfloat16_rn(x[k] * c - y[k] * s_);
                            px[k * a.rope_head_dim + half] = __float2bfloat16_rn(x[k] * s_ + y[k] * c);
                        }
                    }
                    for (; h < n_heads; ++h) {
                        __nv_bfloat16* px = r + h * a.rope_head_dim + i;
                        const float x = __bfloat162float(px[0]), y = __bfloat162float(px[half]);
                        px[0] = __float2bfloat16_rn(x * c - y * s_);
                        px[half] = __float2bfloat16_rn(x * s_ + y * c);
                    }
                }
            }
            tc::fence_proxy_async_smem();                    // the bulk store reads what the lanes just wrote
        }
        __syncwarp();
        if (lane == 0) {
            const char* dst_base = (q & 1) ? a.v_dst : a.k_dst;
            bulk_store(const_cast<char*>(dst_base) + (size_t)(d0 + row) * a.row_bytes, buf0 + slot * a.row_bytes, a.row_bytes);
            if (q >= 1 && q - 1 + a.n_slots < mcp) {
                asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                issue_load(q - 1 + a.n_slots);
            }
        }
        __syncwarp();
    }
    if (lane == 0) {
        asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        if (!ok) atomicOr(a.status, OMNI_DEV_TIMEOUT);
    }
}

template <bool BATCHED>
__global__ void __launch_bounds__(CP_THREADS, 1) compact_units_kernel(const CompactUnitsArgs a) {
    extern __shared__ __align__(128) int smem_i[];
    int* ustart = smem_i;                                   // [n_units_max]
    int* ulen = smem_i + a.n_units_max;                     // [n_units_max]: 0 for a unit outside the span
    int* prefix = smem_i + 2 * a.n_units_max;               // [n_units_max + 1]: kept lengths, then their exclusive scan
    int* src_list = prefix + a.n_units_max + 8;             // [rows_cap]
    char* rowbuf = reinterpret_cast<char*>(smem_i) + ((((size_t)3 * a.n_units_max + 8 + a.rows_cap) * sizeof(int) + 127) & ~(size_t)127);
    __shared__ int warp_tot[CP_WARPS + 1];
    __shared__ int s_misc[4];
    __shared__ uint64_t cbar[CP_WARPS][CP_MAX_SLOTS];
    __shared__ int abort_flag;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int G = gridDim.x;

    // ---- prologue: all loads that need no device-side count first ------------------------------------------
    int nu = a.n_units_dev ? __ldg(a.n_units_dev) : a.n_units_max;
    int u_start = 0, u_len = 0, u_keep = 0, u_klen = -1, k_len = 0, k_group = -1;
    if (tid < a.n_units_max) {
        u_start = __ldg(&a.units[tid].start);
        u_len = __ldg(&a.units[tid].len);
        u_keep = __ldg(a.unit_keep + tid);
        if (a.unit_kept_len) u_klen = __ldg(a.unit_kept_len + tid);
    }
    int nuk = 0;
    if (a.units_kept) {
        nuk = a.n_units_kept_dev ? __ldg(a.n_units_kept_dev) : a.n_units_max;
        if (tid < a.n_units_max) { k_len = __ldg(&a.units_kept[tid].len); k_group = __ldg(&a.units_kept[tid].group); }
    }
    if (tid == 0) { s_misc[0] = 0; s_misc[1] = 0; s_misc[2] = 0x7fffffff; s_misc[3] = 0; abort_flag = 0; }
    if (lane == 0 && a.n_slots > 0) {
        for (int q = 0; q < a.n_slots; ++q) tc::mbar_init(tc::smem_u32(&cbar[wid][q]), 1);
        tc::fence_barrier_init();
    }
    __syncthreads();
    if (nu < 0 || nu > a.n_units_max) {
        if (tid == 0 && blockIdx.x == 0) atomicOr(a.status, OMNI_DEV_BAD_COUNT);
        nu = max(0, min(nu, a.n_units_max));
    }
    nuk = max(0, min(nuk, a.n_units_max));
    // kept length per unit; a unit outside [0, s_span_max) is an error and counts as dropped
    bool bad = false;
    for (int u = tid; u < nu; u += CP_THREADS) {
        if (u >= CP_THREADS) {
            u_start = a.units[u].start; u_len = a.units[u].len; u_keep = a.unit_keep[u];
            u_klen = a.unit_kept_len ? a.unit_kept_len[u] : -1;
        }
        const bool inside = u_start >= 0 && u_len > 0 && (long long)u_start + u_len <= a.s_span_max;
        bad |= !inside;
        const bool keep = inside && u_keep != OMNI_KEEP_DROPPED;
        // tokens kept at the start of the unit: all of it, or the given prefix length
        const int klen = !keep ? 0 : (a.unit_kept_len ? max(0, min(u_klen, u_len)) : u_len);
        ustart[u] = u_start;
        ulen[u] = inside ? u_len : 0;
        prefix[u] = klen;
        if (klen < u_len) atomicMin(&s_misc[2], u);          // first unit with a dropped slot (for rows_moved)
        if (u == nu - 1) s_misc[3] = inside ? u_start + u_len : 0;   // end of the history
    }
    if (bad) atomicOr(a.status, OMNI_DEV_BAD_UNITS);
    {
        int p0 = 0, p1 = 0;
        for (int u = tid; u < nuk; u += CP_THREADS) {
            if (u >= CP_THREADS) { k_len = a.units_kept[u].len; k_group = a.units_kept[u].group; }
            if (k_group == OMNI_GROUP_MUST_KEEP) p0 += k_len;
            else if (k_group == OMNI_GROUP_SELECTED) p1 += k_len;
        }
        p0 = __reduce_add_sync(0xffffffffu, p0);
        p1 = __reduce_add_sync(0xffffffffu, p1);
        if (lane == 0 && (p0 | p1)) { atomicAdd(&s_misc[0], p0); atomicAdd(&s_misc[1], p1); }
    }
    int n_kept;
    if (nu < CP_THREADS) {
        // one unit per thread: the scan runs on the registers (one barrier for the warp totals, one for the result)
        const int mine = tid < nu ? prefix[tid] : 0;        // written by this thread above
        int tot;
        const int ex = warp_excl_scan(mine, lane, tot);
        if (lane == 0) warp_tot[wid] = tot;
        __syncthreads();
        int base = 0;
        for (int w = 0; w < wid; ++w) base += warp_tot[w];
        if (tid <= nu) prefix[tid] = base + ex;
        __syncthreads();
        n_kept = prefix[nu];
    } else {
        if (tid == 0) prefix[nu] = 0;
        __syncthreads();
        n_kept = block_excl_scan(prefix, nu, warp_tot);
    }
    const int n0 = s_misc[0], n1 = s_misc[1], u_open = s_misc[2], n_hist = s_misc[3];

    // ---- destination share: the source slot of every row by a search over the scanned lengths --------------
    int d0 = 0, n_rows = 0;
    if (!BATCHED) {
        const int rows_per = (n_kept + G - 1) / G;
        d0 = min(n_kept, (int)blockIdx.x * rows_per);
        const int d1 = min(n_kept, d0 + rows_per);
        n_rows = min(d1 - d0, a.rows_cap);
        for (int r = tid; r < n_rows; r += CP_THREADS) {
            const int dd = d0 + r;
            int lo = 0, hi = nu;                             // largest u with prefix[u] <= dd (its kept length is > 0)
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (prefix[mid] <= dd) lo = mid; else hi = mid;
            }
            src_list[r] = ustart[lo] + (dd - prefix[lo]);
        }
    }
    // ---- slot map (optional): unit u belongs to CTA u % G -----------------------------------------------------
    if (a.slot_map) {
        for (int u = blockIdx.x; u < nu; u += G) {
            const int st = ustart[u], ln = ulen[u];
            const int base = prefix[u], klen = prefix[u + 1] - prefix[u];
            for (int i = tid; i < ln; i += CP_THREADS) a.slot_map[st + i] = i < klen ? base + i : -1;
        }
    }
    // ---- integer summary and page classes ------------------------------------------------------------------
    if (a.info && blockIdx.x == 0 && tid == 0) {
        // retained rows before the first dropped slot: the units before the first shortened one, plus its kept prefix
        const int lead = u_open < nu ? ustart[u_open] + (prefix[u_open + 1] - prefix[u_open]) : n_hist;
        a.info->n_kept = n_kept;
        a.info->span_pages = (n_kept + a.page_size - 1) / a.page_size;
        a.info->rows_moved = n_kept - min(lead, n_kept);
        a.info->part_begin[0] = 0;
        a.info->part_begin[1] = a.units_kept ? n0 : 0;
        a.info->part_begin[2] = a.units_kept ? n0 + n1 : 0;
        a.info->part_begin[3] = n_kept;
        a.info->reserved = 0;
    }
    if (a.page_class) {
        const int n_pages = (a.s_span_max + a.page_size - 1) / a.page_size;
        for (int p = blockIdx.x * CP_THREADS + tid; p < n_pages; p += G * CP_THREADS) {
            const long long lo = (long long)p * a.page_size;
            const long long hi = min(lo + a.page_size, (long long)n_kept);
            uint8_t cls = OMNI_PAGE_EMPTY;
            if (hi > lo) {
                if (lo < n0) cls = OMNI_GROUP_MUST_KEEP;
                else if (hi - lo == a.page_size) cls = OMNI_GROUP_SELECTED;
                else cls = OMNI_GROUP_RECENT;
            }
            a.page_class[p] = cls;
        }
    }
    if (!BATCHED) {
        if (a.k_dst == nullptr) return;
        __syncthreads();                                    // the source list is complete
        if (a.rope_dims > 0) move_rows_rope(a, src_list, d0, n_rows, rowbuf, cbar, &abort_flag);
        else move_rows(a, src_list, d0, n_rows, rowbuf, cbar, &abort_flag);
        return;
    }
    // ---- batched form: copies are numbered layer-major, (layer, destination row, K or V), and every CTA takes an
    // equal contiguous range of them; a lane walks its copies in increasing order, so the unit that holds a
    // destination row is found by stepping forward (a binary search only when the layer changes)
    __syncthreads();
    if (lane == 0 && n_kept > 0) {
        const int total = 2 * n_kept * a.n_layers;           // the host bounds this below 2^31
        const int per = (total + G - 1) / G;
        const int c0 = min(total, (int)blockIdx.x * per), c1 = min(total, c0 + per);
        const int mine = c1 - c0;
        const int mcp = mine > wid ? (mine - wid + CP_WARPS - 1) / CP_WARPS : 0;
        const uint32_t buf0 = tc::smem_u32(rowbuf) + (uint32_t)(wid * a.n_slots) * a.row_bytes;
        int u_cur = 0, layer_cur = -1;
        auto src_of = [&](int q) {
            const int c = c0 + wid + q * CP_WARPS;
            const int f = c >> 1, layer = f / n_kept, dd = f - layer * n_kept;
            if (layer != layer_cur) {
                int lo = 0, hi = nu;
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (prefix[mid] <= dd) lo = mid; else hi = mid;
                }
                u_cur = lo;
                layer_cur = layer;
            } else {
                while (dd >= prefix[u_cur + 1]) ++u_cur;     // also steps over dropped units (equal prefixes)
            }
            const char* base = ldg_ptr<const char>((c & 1) ? a.v_src_l : a.k_src_l, layer);
            return base + (size_t)(ustart[u_cur] + (dd - prefix[u_cur])) * a.row_bytes;
        };
        auto dst_of = [&](int q) {
            const int c = c0 + wid + q * CP_WARPS;
            const int f = c >> 1, layer = f / n_kept, dd = f - layer * n_kept;
            char* base = ldg_ptr<char>((c & 1) ? a.v_dst_l : a.k_dst_l, layer);
            return base + (size_t)dd * a.row_bytes;
        };
        if (!bulk_copy_loop(mcp, src_of, dst_of, a.row_bytes, a.n_slots, buf0, cbar[wid], &abort_flag))
            atomicOr(a.status, OMNI_DEV_TIMEOUT);
    }
}

// Dense copy of `n_rows` rows (device count) from staging back to the cache (in-place mode), and
// the chunk append.  n_rows = *n_dev clamped to n_max; destination starts at row *dst_row_dev.
__global__ void __launch_bounds__(256) copy_rows_kernel(const char* __restrict__ k_from, const char* __restrict__ v_from,
                                                        char* __restrict__ k_to, char* __restrict__ v_to,
                                                        const int32_t* n_dev, int n_max, const int32_t* dst_row_dev,
                                                        int dst_row_cap, int row_bytes, int32_t* status) {
    int n = n_dev ? *n_dev : n_max;
    n = max(0, min(n, n_max));
    const int dst_row = dst_row_dev ? *dst_row_dev : 0;
    if (dst_row < 0 || dst_row + n > dst_row_cap) {
        if (threadIdx.x == 0 && blockIdx.x == 0) atomicOr(status, OMNI_DEV_BAD_COUNT);
        return;
    }
    const long long vecs = (long long)n * (row_bytes >> 4);
    const uint4* kf = reinterpret_cast<const uint4*>(k_from);
    const uint4* vf = reinterpret_cast<const uint4*>(v_from);
    uint4* kt = reinterpret_cast<uint4*>(k_to + (size_t)dst_row * row_bytes);
    uint4* vt = reinterpret_cast<uint4*>(v_to + (size_t)dst_row * row_bytes);
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < vecs; i += stride * 4) {
        uint4 a[4], b[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const long long j = i + u * stride;
            if (j < vecs) { a[u] = ld_stream(kf + j); b[u] = ld_stream(vf + j); }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const long long j = i + u * stride;
            if (j < vecs) { st_stream(kt + j, a[u]); st_stream(vt + j, b[u]); }
        }
    }
}

__global__ void append_units_kernel(omni_unit* units, const int32_t* n_units_dev, const omni_unit* chunk_units,
                                    int n_chunk_units, int u_cap, const int32_t* n_kept_dev, int t, int s_cap,
                                    int32_t* n_hist_out, int32_t* n_units_out, int32_t* status) {
    const int nu = *n_units_dev;
    const int nk = *n_kept_dev;
    __syncthreads();     // every thread has read the counts before thread 0 may overwrite aliases
    if (nu < 0 || nu + n_chunk_units > u_cap || nk < 0 || nk + t > s_cap) {
        if (threadIdx.x == 0) atomicOr(status, OMNI_DEV_BAD_COUNT);
        return;
    }
    for (int i = threadIdx.x; i < n_chunk_units; i += blockDim.x) {
        omni_unit u = chunk_units[i];
        u.start += nk;
        u.group = OMNI_GROUP_RECENT;
        units[nu + i] = u;
    }
    if (threadIdx.x == 0) {
        *n_hist_out = nk + t;
        *n_units_out = nu + n_chunk_units;
    }
}

}  // namespace

// ---------------------------------------------------------------------------------------------------
// Ordered-suffix migration (Section 6.2): plan on one CTA, pack the chosen suffix with the mask kernel above
// (through staging: a move may land on a source row of another move), then rewrite the mask of the suffix.
// plan[0] = first slot of the suffix the pack kernel works on (the span itself when nothing qualifies: an empty
// suffix), plan[1] = suffix start or -1, plan[2] = span after the move, plan[3] = span before, plan[4] = live slots.
__global__ void __launch_bounds__(CP_THREADS, 1) suffix_plan_kernel(const uint8_t* __restrict__ mask, const int32_t* s_span_dev,
                                                                    int s_span_max, int page, int theta, int32_t* plan,
                                                                    int32_t* status) {
    extern __shared__ int pg_cnt[];                          // [pages + 1]: live slots per page, reversed, then their scan
    __shared__ int warp_tot[CP_WARPS + 1];
    __shared__ int s_best;
    const int tid = threadIdx.x;
    int S = s_span_dev ? *s_span_dev : s_span_max;
    if (S < 0 || S > s_span_max) {
        if (tid == 0) atomicOr(status, OMNI_DEV_BAD_COUNT);
        S = max(0, min(S, s_span_max));
    }
    const int n_pages = (S + page - 1) / page;
    if (tid == 0) s_best = -1;
    for (int pg = tid; pg < n_pages; pg += CP_THREADS) {
        int cnt = 0;
        const int hi = min(S, (pg + 1) * page);
        for (int pos = pg * page; pos < hi; pos += 16) {
            const uint4 v = clip_vec(ld_mask(mask, pos >> 4), hi - pos);
            cnt += count_kept(v);
        }
        pg_cnt[n_pages - 1 - pg] = cnt;                      // reversed: a prefix sum becomes a suffix sum
    }
    __syncthreads();
    const int total_live = block_excl_scan(pg_cnt, n_pages, warp_tot);   // pg_cnt[j] = live slots in the last j pages
    // suffix that starts at page i holds pg_cnt[n_pages - i] live slots
    for (int i = tid; i < n_pages; i += CP_THREADS) {
        const int live = pg_cnt[n_pages - i];
        const int new_span = i * page + live;
        if (n_pages - (new_span + page - 1) / page >= theta) atomicMax(&s_best, i);
    }
    __syncthreads();
    if (tid == 0) {
        const int i = s_best;
        plan[0] = i >= 0 ? i * page : S;
        plan[1] = i >= 0 ? i * page : -1;
        plan[2] = i >= 0 ? i * page + pg_cnt[n_pages - i] : S;
        plan[3] = S;
        plan[4] = total_live;
    }
}

__global__ void __launch_bounds__(256) suffix_finish_kernel(uint8_t* mask, int32_t* s_span_dev, int page, const int32_t* plan,
                                                            const omni_compact_info* pack_info, int32_t* slot_map,
                                                            omni_compact_info* info) {
    const int start = plan[1], new_span = plan[2], S = plan[3];
    const int gtid = blockIdx.x * blockDim.x + threadIdx.x, gsz = gridDim.x * blockDim.x;
    const int keep_from = start >= 0 ? start : S;            // slots before it keep their place and their holes
    if (slot_map)
        for (int sl = gtid; sl < keep_from; sl += gsz) slot_map[sl] = mask[sl] ? sl : -1;
    if (start >= 0)
        for (int sl = start + gtid; sl < S; sl += gsz) mask[sl] = sl < new_span ? 1 : 0;
    if (gtid == 0) {
        if (start >= 0 && s_span_dev) *s_span_dev = new_span;
        if (info) {
            info->n_kept = plan[4];
            info->span_pages = (new_span + page - 1) / page;
            info->rows_moved = start >= 0 ? pack_info->rows_moved : 0;
            info->part_begin[0] = start;
            info->part_begin[1] = new_span;
            info->part_begin[2] = (S + page - 1) / page - (new_span + page - 1) / page;
            info->part_begin[3] = S;
            info->reserved = 0;
        }
    }
}

// Staging rows of the in-place mode, allocated on the first in-place call on a context (synchronous).
omni_status omni_inplace_staging(omnitide_ctx* ctx) {
    if (ctx->inplace_rows >= (size_t)ctx->g.s_cap) return OMNI_OK;
    if (ctx->inplace_k) cudaFree(ctx->inplace_k);
    if (ctx->inplace_v) cudaFree(ctx->inplace_v);
    ctx->inplace_k = ctx->inplace_v = nullptr;
    ctx->inplace_rows = 0;
    OMNI_CUDA(ctx, cudaMalloc(&ctx->inplace_k, (size_t)ctx->g.s_cap * ctx->row_bytes));
    OMNI_CUDA(ctx, cudaMalloc(&ctx->inplace_v, (size_t)ctx->g.s_cap * ctx->row_bytes));
    ctx->inplace_rows = ctx->g.s_cap;
    return OMNI_OK;
}

static omni_status compact_pack_impl(const int32_t* span_off_dev, omnitide_ctx* ctx, void* stream, const void* k_src, const void* v_src,
                                        void* k_dst, void* v_dst, const uint8_t* keep_mask,
                                        const int32_t* s_span_dev, int32_t s_span_max, int32_t page_size, int32_t mode,
                                        const omni_unit* units_kept, const int32_t* n_units_kept_dev,
                                        int32_t n_units_max, int32_t* slot_map_out, omni_compact_info* info_out,
                                        uint8_t* page_class_out) {
    if (!ctx) return OMNI_ERR_INVALID_ARG;
    if (mode != OMNI_COMPACT_PACK) OMNI_FAIL(ctx, OMNI_ERR_UNSUPPORTED, "compact: only mode PACK is built");
    if (!keep_mask || s_span_max < 0 || page_size <= 0) OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "compact: bad mask/span/page");
    if (s_span_max > ctx->g.s_cap) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "compact: s_span_max %d > s_cap %d", s_span_max, ctx->g.s_cap);
    if ((k_src == nullptr) != (k_dst == nullptr) || (k_src == nullptr) != (v_src == nullptr) ||
        (v_src == nullptr) != (v_dst == nullptr))
        OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "compact: K/V source and destination must be given together");
    if (!omni_aligned16(keep_mask) || !omni_aligned16(k_src) || !omni_aligned16(v_src) || !omni_aligned16(k_dst) ||
        !omni_aligned16(v_dst) || !omni_aligned16(slot_map_out))
        OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "compact: pointers must be 16-byte aligned");
    if (units_kept && n_units_max > ctx->g.u_cap) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "compact: n_units_max > u_cap");
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    const bool in_place = k_src && (k_src == k_dst || v_src == v_dst);
    void* kd = k_dst;
    void* vd = v_dst;
    if (in_place) {
        const omni_status ss = omni_inplace_staging(ctx);
        if (ss) return ss;
        kd = ctx->inplace_k;
        vd = ctx->inplace_v;
    }

    CompactArgs a;
    a.k_src = static_cast<const char*>(k_src); a.v_src = static_cast<const char*>(v_src);
    a.k_dst = static_cast<char*>(kd); a.v_dst = static_cast<char*>(vd);
    a.mask = keep_mask; a.s_span_dev = s_span_dev; a.s_span_max = s_span_max;
    a.page_size = page_size; a.row_bytes = (int)ctx->row_bytes; a.vpr = (int)(ctx->row_bytes >> 4);
    a.vpr_shift = -1;
    for (int sft = 0; sft < 20; ++sft) if ((1 << sft) == a.vpr) a.vpr_shift = sft;
    a.units_kept = units_kept; a.n_units_kept_dev = n_units_kept_dev; a.n_units_max = n_units_max;
    a.slot_map = slot_map_out; a.info = info_out; a.page_class = page_class_out; a.status = ctx->status_dev;
    const int grid = ctx->sm_count;
    a.rows_cap = (s_span_max + grid - 1) / grid + 1;
    a.max_chunks = std::max(256, (grid + 2 + 3) & ~3);       // the one-warp scan touches 256 entries
    a.rows_cap = (a.rows_cap + 3) & ~3;                      // keep what follows 16-byte aligned
    const int n_grp = (s_span_max + 511) / 512;
    a.part_groups = std::max(1, (n_grp + grid - 1) / grid);
    ++ctx->cp_epoch;                                         // wraps together with the 32-bit arrival counter
    a.words = ctx->cp_words;
    a.span_off_dev = span_off_dev;
    a.epoch = ctx->cp_epoch;
    const size_t smem_lists = (size_t)(a.max_chunks + a.rows_cap) * sizeof(int);
    const size_t budget = 200 * 1024;
    a.n_slots = 0;
    if (k_src && ctx->row_bytes >= 512 && smem_lists < budget) {
        const size_t per_warp = (budget - smem_lists) / CP_WARPS;
        a.n_slots = (int)std::min<size_t>(CP_MAX_SLOTS, per_warp / ctx->row_bytes);
        if (a.n_slots < 2) a.n_slots = 0;
    }
    const size_t smem = smem_lists + (size_t)a.n_slots * CP_WARPS * ctx->row_bytes;
    if (smem > 200 * 1024) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "compact: span too large for one launch");
    if (smem > 48 * 1024)
        OMNI_CUDA(ctx, cudaFuncSetAttribute(compact_pack_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    {
        // cooperative: the CTAs wait for one another's counts, so all of them must be resident
        void* kargs[] = {&a};
        const cudaError_t le = cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(compact_pack_kernel), dim3(grid),
                                                           dim3(CP_THREADS), kargs, smem, st);
        if (le != cudaSuccess) {
            --ctx->cp_epoch;                                 // nothing arrived: keep the counter in step
            OMNI_FAIL(ctx, OMNI_ERR_CUDA, "launch compact_pack_kernel: %s", cudaGetErrorString(le));
        }
        ctx->launches++;
    }
    if (in_place) {
        if (!info_out) OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "compact: in-place mode needs info_out");
        copy_rows_kernel<<<ctx->sm_count * 4, 256, 0, st>>>(
            static_cast<const char*>(kd), static_cast<const char*>(vd), static_cast<char*>(k_dst),
            static_cast<char*>(v_dst), &info_out->n_kept, s_span_max, span_off_dev, ctx->g.s_cap, (int)ctx->row_bytes,
            ctx->status_dev);
        OMNI_CHECK_LAUNCH(ctx, "copy_rows_kernel");
    }
    return OMNI_OK;
}

static omni_status compact_units_impl(const omni_rope_params* rope, omnitide_ctx* ctx, void* stream, const void* k_src, const void* v_src,
                                              void* k_dst, void* v_dst, const omni_unit* units,
                                              const int32_t* n_units_dev, int32_t n_units_max, const uint8_t* unit_keep,
                                              const int32_t* unit_kept_len, int32_t s_span_max, int32_t page_size,
                                              const omni_unit* units_kept,
                                              const int32_t* n_units_kept_dev, int32_t* slot_map_out,
                                              omni_compact_info* info_out, uint8_t* page_class_out) {
    if (!ctx) return OMNI_ERR_INVALID_ARG;
    if (!units || !unit_keep || n_units_max <= 0 || s_span_max < 0 || page_size <= 0)
        OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "compact_units: bad unit table/span/page");
    if (s_span_max > ctx->g.s_cap) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "compact_units: s_span_max %d > s_cap %d", s_span_max, ctx->g.s_cap);
    if (n_units_max > ctx->g.u_cap) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "compact_units: n_units_max > u_cap");
    if ((k_src == nullptr) != (k_dst == nullptr) || (k_src == nullptr) != (v_src == nullptr) ||
        (v_src == nullptr) != (v_dst == nullptr))
        OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "compact_units: K/V source and destination must be given together");
    if (!omni_aligned16(k_src) || !omni_aligned16(v_src) || !omni_aligned16(k_dst) || !omni_aligned16(v_dst))
        OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "compact_units: pointers must be 16-byte aligned");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool in_place = k_src && (k_src == k_dst || v_src == v_dst);
    void* kd = k_dst;
    void* vd = v_dst;
    if (in_place) {
        if (!info_out) OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "compact_units: in-place mode needs info_out");
        const omni_status ss = omni_inplace_staging(ctx);
        if (ss) return ss;
        kd = ctx->inplace_k;
        vd = ctx->inplace_v;
    }
    CompactUnitsArgs a;
    a.k_src = static_cast<const char*>(k_src); a.v_src = static_cast<const char*>(v_src);
    a.k_dst = static_cast<char*>(kd); a.v_dst = static_cast<char*>(vd);
    a.units = units; a.n_units_dev = n_units_dev; a.n_units_max = n_units_max; a.unit_keep = unit_keep;
    a.unit_kept_len = unit_kept_len;
    a.s_span_max = s_span_max; a.page_size = page_size; a.row_bytes = (int)ctx->row_bytes;
    a.vpr = (int)(ctx->row_bytes >> 4); a.vpr_shift = -1;
    for (int sft = 0; sft < 20; ++sft) if ((1 << sft) == a.vpr) a.vpr_shift = sft;
    a.units_kept = units_kept; a.n_units_kept_dev = n_units_kept_dev;
    a.slot_map = slot_map_out; a.info = info_out; a.page_class = page_class_out; a.status = ctx->status_dev;
    const int grid = ctx->sm_count;
    a.n_layers = 1; a.k_src_l = a.v_src_l = nullptr; a.k_dst_l = a.v_dst_l = nullptr;
    a.rope_dims = 0; a.rope_head_dim = ctx->g.d; a.rope_log2_base = 0.0;
    if (rope) {
        if (ctx->g.dtype != OMNI_DTYPE_BF16) OMNI_FAIL(ctx, OMNI_ERR_UNSUPPORTED, "compact_units_rope: bf16 caches only");
        if (rope->n_dims <= 0 || (rope->n_dims & 1) || rope->n_dims > ctx->g.d || rope->n_dims > 256 || !(rope->theta_base > 1.0f))
            OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "compact_units_rope: n_dims must be even, in (0, min(d, 256)], theta_base > 1");
        a.rope_dims = rope->n_dims;
        a.rope_log2_base = std::log2((double)rope->theta_base);
    }
    a.rows_cap = (((s_span_max + grid - 1) / grid + 1) + 3) & ~3;
    const size_t smem_lists = ((size_t)3 * n_units_max + 8 + a.rows_cap) * sizeof(int);
    const size_t smem_lists_al = (smem_lists + 127) & ~(size_t)127;
    const size_t budget = 200 * 1024;
    if (smem_lists_al > budget) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "compact_units: unit table too large for one launch");
    a.n_slots = 0;
    if (k_src && ctx->row_bytes >= 512) {
        const size_t per_warp = (budget - smem_lists_al) / CP_WARPS;
        a.n_slots = (int)std::min<size_t>(CP_MAX_SLOTS, per_warp / ctx->row_bytes);
        if (a.n_slots < 2) a.n_slots = 0;
    }
    if (rope && a.n_slots == 0 && k_src) OMNI_FAIL(ctx, OMNI_ERR_UNSUPPORTED, "compact_units_rope: rows of 512 bytes to 12 KB only");
    const size_t smem = smem_lists_al + (size_t)a.n_slots * CP_WARPS * ctx->row_bytes;
    if (smem > 48 * 1024)
        OMNI_CUDA(ctx, cudaFuncSetAttribute(compact_units_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    compact_units_kernel<false><<<grid, CP_THREADS, smem, st>>>(a);
    OMNI_CHECK_LAUNCH(ctx, "compact_units_kernel");
    if (in_place) {
        copy_rows_kernel<<<ctx->sm_count * 4, 256, 0, st>>>(
            static_cast<const char*>(kd), static_cast<const char*>(vd), static_cast<char*>(k_dst),
            static_cast<char*>(v_dst), &info_out->n_kept, s_span_max, nullptr, ctx->g.s_cap, (int)ctx->row_bytes,
            ctx->status_dev);
        OMNI_CHECK_LAUNCH(ctx, "copy_rows_kernel");
    }
    return OMNI_OK;
}

extern "C" omni_status omnipage_compact(omnitide_ctx* ctx, void* stream, const void* k_src, const void* v_src,
                                        void* k_dst, void* v_dst, const uint8_t* keep_mask,
                                        const int32_t* s_span_dev, int32_t s_span_max, int32_t page_size, int32_t mode,
                                        const omni_unit* units_kept, const int32_t* n_units_kept_dev,
                                        int32_t n_units_max, int32_t* slot_map_out, omni_compact_info* info_out,
                                        uint8_t* page_class_out) {
    return compact_pack_impl(nullptr, ctx, stream, k_src, v_src, k_dst, v_dst, keep_mask, s_span_dev, s_span_max, page_size,
                             mode, units_kept, n_units_kept_dev, n_units_max, slot_map_out, info_out, page_class_out);
}

extern "C" omni_status omnipage_migrate_suffix(omnitide_ctx* ctx, void* stream, void* k_cache, void* v_cache,
                                               uint8_t* keep_mask, int32_t* s_span_dev, int32_t s_span_max,
                                               int32_t page_size, int32_t min_pages_saved, int32_t* slot_map_out,
                                               omni_compact_info* info_out) {
    if (!ctx) return OMNI_ERR_INVALID_ARG;
    if (!k_cache || !v_cache || !keep_mask || !s_span_dev || s_span_max <= 0)
        OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "migrate_suffix: null pointer or empty span");
    if (page_size <= 0 || (page_size & 15)) OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "migrate_suffix: page size must be a multiple of 16");
    if (min_pages_saved < 1) OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "migrate_suffix: the threshold is at least one page");
    if (s_span_max > ctx->g.s_cap) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "migrate_suffix: s_span_max %d > s_cap %d", s_span_max, ctx->g.s_cap);
    if (!omni_aligned16(keep_mask)) OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "migrate_suffix: the mask must be 16-byte aligned");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!ctx->mig_plan) OMNI_CUDA(ctx, cudaMalloc(&ctx->mig_plan, 8 * sizeof(int32_t)));
    const size_t plan_smem = ((size_t)(s_span_max + page_size - 1) / page_size + 2) * sizeof(int);
    if (plan_smem > 200 * 1024) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "migrate_suffix: too many pages for one launch");
    if (plan_smem > 48 * 1024)
        OMNI_CUDA(ctx, cudaFuncSetAttribute(suffix_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan_smem));
    suffix_plan_kernel<<<1, CP_THREADS, plan_smem, st>>>(keep_mask, s_span_dev, s_span_max, page_size, min_pages_saved,
                                                         ctx->mig_plan, ctx->status_dev);
    OMNI_CHECK_LAUNCH(ctx, "suffix_plan_kernel");
    // the pack of the suffix, in place through staging; its slot map counts from the start of the suffix on
    const omni_status ps = compact_pack_impl(ctx->mig_plan, ctx, stream, k_cache, v_cache, k_cache, v_cache, keep_mask,
                                             s_span_dev, s_span_max, page_size, OMNI_COMPACT_PACK, nullptr, nullptr, 1,
                                             slot_map_out, ctx->ws_info, nullptr);
    if (ps) return ps;
    suffix_finish_kernel<<<std::min(ctx->sm_count, 64), 256, 0, st>>>(keep_mask, s_span_dev, page_size, ctx->mig_plan,
                                                                       ctx->ws_info, slot_map_out, info_out);
    OMNI_CHECK_LAUNCH(ctx, "suffix_finish_kernel");
    return OMNI_OK;
}

extern "C" omni_status omnipage_compact_units(omnitide_ctx* ctx, void* stream, const void* k_src, const void* v_src,
                                              void* k_dst, void* v_dst, const omni_unit* units,
                                              const int32_t* n_units_dev, int32_t n_units_max, const uint8_t* unit_keep,
                                              const int32_t* unit_kept_len, int32_t s_span_max, int32_t page_size,
                                              const omni_unit* units_kept,
                                              const int32_t* n_units_kept_dev, int32_t* slot_map_out,
                                              omni_compact_info* info_out, uint8_t* page_class_out) {
    return compact_units_impl(nullptr, ctx, stream, k_src, v_src, k_dst, v_dst, units, n_units_dev, n_units_max, unit_keep,
                              unit_kept_len, s_span_max, page_size, units_kept, n_units_kept_dev, slot_map_out, info_out,
                              page_class_out);
}

extern "C" omni_status omnipage_compact_units_rope(omnitide_ctx* ctx, void* stream, const void* k_src, const void* v_src,
                                                   void* k_dst, void* v_dst, const omni_unit* units,
                                                   const int32_t* n_units_dev, int32_t n_units_max,
                                                   const uint8_t* unit_keep, const int32_t* unit_kept_len,
                                                   int32_t s_span_max, int32_t page_size, const omni_unit* units_kept,
                                                   const int32_t* n_units_kept_dev, int32_t* slot_map_out,
                                                   omni_compact_info* info_out, uint8_t* page_class_out,
                                                   const omni_rope_params* rope) {
    if (!ctx) return OMNI_ERR_INVALID_ARG;
    if (!rope) OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "compact_units_rope: null rope parameters");
    return compact_units_impl(rope, ctx, stream, k_src, v_src, k_dst, v_dst, units, n_units_dev, n_units_max, unit_keep,
                              unit_kept_len, s_span_max, page_size, units_kept, n_units_kept_dev, slot_map_out, info_out,
                              page_class_out);
}

extern "C" omni_status omnipage_compact_units_batched(omnitide_ctx* ctx, void* stream, const void* const* k_src,
                                                      const void* const* v_src, void* const* k_dst, void* const* v_dst,
                                                      int32_t n_layers, const omni_unit* units, const int32_t* n_units_dev,
                                                      int32_t n_units_max, const uint8_t* unit_keep,
                                                      const int32_t* unit_kept_len, int32_t s_span_max,
                                                      int32_t page_size, const omni_unit* units_kept,
                                                      const int32_t* n_units_kept_dev, int32_t* slot_map_out,
                                                      omni_compact_info* info_out, uint8_t* page_class_out) {
    if (!ctx) return OMNI_ERR_INVALID_ARG;
    if (!units || !unit_keep || n_units_max <= 0 || s_span_max < 0 || page_size <= 0 || n_layers <= 0 || !k_src || !v_src ||
        !k_dst || !v_dst)
        OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "compact_units_batched: bad unit table/span/page/layers");
    if (s_span_max > ctx->g.s_cap) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "compact_units_batched: s_span_max %d > s_cap %d", s_span_max, ctx->g.s_cap);
    if (n_units_max > ctx->g.u_cap) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "compact_units_batched: n_units_max > u_cap");
    if (2ll * s_span_max * n_layers >= (1ll << 31))
        OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "compact_units_batched: 2 * s_span_max * n_layers must stay below 2^31");
    if (ctx->row_bytes < 512 || (ctx->row_bytes & 15))
        OMNI_FAIL(ctx, OMNI_ERR_UNSUPPORTED, "compact_units_batched: rows of at least 512 bytes (a multiple of 16) only");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CompactUnitsArgs a;
    a.k_src = a.v_src = nullptr; a.k_dst = a.v_dst = nullptr;
    a.units = units; a.n_units_dev = n_units_dev; a.n_units_max = n_units_max; a.unit_keep = unit_keep;
    a.unit_kept_len = unit_kept_len;
    a.s_span_max = s_span_max; a.page_size = page_size; a.row_bytes = (int)ctx->row_bytes;
    a.vpr = (int)(ctx->row_bytes >> 4); a.vpr_shift = -1;
    a.units_kept = units_kept; a.n_units_kept_dev = n_units_kept_dev;
    a.slot_map = slot_map_out; a.info = info_out; a.page_class = page_class_out; a.status = ctx->status_dev;
    a.n_layers = n_layers;
    a.rope_dims = 0; a.rope_head_dim = ctx->g.d; a.rope_log2_base = 0.0;
    a.k_src_l = reinterpret_cast<const char* const*>(k_src); a.v_src_l = reinterpret_cast<const char* const*>(v_src);
    a.k_dst_l = reinterpret_cast<char* const*>(k_dst); a.v_dst_l = reinterpret_cast<char* const*>(v_dst);
    const int grid = ctx->sm_count;
    a.rows_cap = 4;                                          // no per-row source list in the batched form
    const size_t smem_lists_al = ((((size_t)3 * n_units_max + 8 + a.rows_cap) * sizeof(int)) + 127) & ~(size_t)127;
    const size_t budget = 200 * 1024;
    if (smem_lists_al + 2 * CP_WARPS * ctx->row_bytes > budget)
        OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "compact_units_batched: unit table or rows too large for one launch");
    const size_t per_warp = (budget - smem_lists_al) / CP_WARPS;
    a.n_slots = (int)std::min<size_t>(CP_MAX_SLOTS, per_warp / ctx->row_bytes);
    const size_t smem = smem_lists_al + (size_t)a.n_slots * CP_WARPS * ctx->row_bytes;
    if (smem > 48 * 1024)
        OMNI_CUDA(ctx, cudaFuncSetAttribute(compact_units_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    compact_units_kernel<true><<<grid, CP_THREADS, smem, st>>>(a);
    OMNI_CHECK_LAUNCH(ctx, "compact_units_kernel(batched)");
    return OMNI_OK;
}

extern "C" omni_status omnipage_append(omnitide_ctx* ctx, void* stream, void* k_cache, void* v_cache,
                                       const int32_t* n_kept_dev, const void* k_chunk, const void* v_chunk, int32_t t,
                                       omni_unit* units, const int32_t* n_units_dev, const omni_unit* chunk_units,
                                       int32_t n_chunk_units, int32_t* n_hist_out, int32_t* n_units_out) {
    if (!ctx) return OMNI_ERR_INVALID_ARG;
    if (!k_cache || !v_cache || !n_kept_dev || !k_chunk || !v_chunk || t < 0 || !units || !n_units_dev ||
        (!chunk_units && n_chunk_units > 0) || n_chunk_units < 0 || !n_hist_out || !n_units_out)
        OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "append: null pointer or negative count");
    if (t > ctx->g.t_cap) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "append: t %d > t_cap %d", t, ctx->g.t_cap);
    if (!omni_aligned16(k_cache) || !omni_aligned16(v_cache) || !omni_aligned16(k_chunk) || !omni_aligned16(v_chunk))
        OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "append: pointers must be 16-byte aligned");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (t > 0) {
        const long long vecs = (long long)t * (ctx->row_bytes >> 4);
        int grid = (int)((vecs + 256 * 4 - 1) / (256 * 4));
        grid = grid < 1 ? 1 : (grid > ctx->sm_count * 8 ? ctx->sm_count * 8 : grid);
        copy_rows_kernel<<<grid, 256, 0, st>>>(static_cast<const char*>(k_chunk), static_cast<const char*>(v_chunk),
                                               static_cast<char*>(k_cache), static_cast<char*>(v_cache), nullptr, t,
                                               n_kept_dev, ctx->g.s_cap, (int)ctx->row_bytes, ctx->status_dev);
        OMNI_CHECK_LAUNCH(ctx, "copy_rows_kernel(append)");
    }
    append_units_kernel<<<1, 64, 0, st>>>(units, n_units_dev, chunk_units, n_chunk_units, ctx->g.u_cap, n_kept_dev, t,
                                          ctx->g.s_cap, n_hist_out, n_units_out, ctx->status_dev);
    OMNI_CHECK_LAUNCH(ctx, "append_units_kernel");
    return OMNI_OK;
}
