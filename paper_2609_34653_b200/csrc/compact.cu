// OmniPage eager compaction (mode PACK) and the append step.
//
// One persistent kernel does the whole compaction: every CTA scans the keep mask (a few tens of
// KB, served from L2) into per-chunk prefix counts held in shared memory, so no CTA waits on
// another; the retained rows are then split evenly by DESTINATION slot across the CTAs, each
// of which rebuilds the source slots of its share from the mask and moves the rows with 16-byte
// vector loads/stores, eight in flight per thread.  The slot map, page classes and the integer
// summary come out of the same scan.  HBM traffic is one read and one write per retained row.
#include "common.cuh"

namespace {

constexpr int CP_THREADS = 512;
constexpr int CP_WARPS = CP_THREADS / 32;
constexpr int CP_UNROLL = 8;
constexpr int CP_MAX_CHUNKS = 2048;

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

// Loads the 16 mask bytes at [pos, pos+16) with positions >= s read as zero.
__device__ __forceinline__ uint4 load_mask16(const uint8_t* mask, int pos, int s) {
    uint4 v = make_uint4(0, 0, 0, 0);
    if (pos + 16 <= s) {
        v = *reinterpret_cast<const uint4*>(mask + pos);
    } else if (pos < s) {
        uint32_t w[4] = {0, 0, 0, 0};
        for (int b = 0; b < s - pos; ++b) w[b >> 2] |= (mask[pos + b] ? 1u : 0u) << ((b & 3) * 8);
        v = make_uint4(w[0], w[1], w[2], w[3]);
    }
    return v;
}

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
    int page_size; int row_bytes; int vpr; int vpr_shift; int chunk_shift;
    const omni_unit* units_kept; const int32_t* n_units_kept_dev; int n_units_max;
    int32_t* slot_map; omni_compact_info* info; uint8_t* page_class; int32_t* status;
    int rows_cap;      // capacity of the per-CTA source list
};

__global__ void __launch_bounds__(CP_THREADS, 1) compact_pack_kernel(const CompactArgs a) {
    extern __shared__ int smem_i[];
    int* prefix = smem_i;                                   // [n_chunks + 1]
    __shared__ int warp_tot[CP_WARPS + 1];
    __shared__ int s_misc[4];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;

    int s = a.s_span_dev ? *a.s_span_dev : a.s_span_max;
    if (s > a.s_span_max || s < 0) {
        if (tid == 0 && blockIdx.x == 0) atomicOr(a.status, OMNI_DEV_BAD_COUNT);
        s = max(0, min(s, a.s_span_max));
    }
    const int chunk_bytes = 1 << a.chunk_shift;
    const int n_chunks = (s + chunk_bytes - 1) >> a.chunk_shift;
    int* src_list = smem_i + (((a.s_span_max + chunk_bytes - 1) >> a.chunk_shift) + 2);
    const int vec_per_lane = chunk_bytes >> 9;              // 16-byte vectors per lane per chunk

    // ---- phase A: every CTA counts every chunk -------------------------------------------
    for (int c = wid; c < n_chunks; c += CP_WARPS) {
        int cnt = 0;
        const int base = c << a.chunk_shift;
        for (int k = 0; k < vec_per_lane; ++k) {
            uint4 v = load_mask16(a.mask, base + k * 512 + lane * 16, s);
            cnt += nonzero_bytes(v.x) + nonzero_bytes(v.y) + nonzero_bytes(v.z) + nonzero_bytes(v.w);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
        if (lane == 0) prefix[c] = cnt;
    }
    __syncthreads();
    const int n_kept = block_excl_scan(prefix, n_chunks, warp_tot);

    // ---- partitions from the compacted unit table -----------------------------------------
    int n0 = 0, n1 = 0;
    if (a.units_kept) {
        int nu = a.n_units_kept_dev ? *a.n_units_kept_dev : a.n_units_max;
        nu = max(0, min(nu, a.n_units_max));
        int p0 = 0, p1 = 0;
        for (int u = tid; u < nu; u += CP_THREADS) {
            const omni_unit un = a.units_kept[u];
            if (un.group == OMNI_GROUP_MUST_KEEP) p0 += un.len;
            else if (un.group == OMNI_GROUP_SELECTED) p1 += un.len;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            p0 += __shfl_xor_sync(0xffffffffu, p0, o);
            p1 += __shfl_xor_sync(0xffffffffu, p1, o);
        }
        if (tid == 0) { s_misc[0] = 0; s_misc[1] = 0; }
        __syncthreads();
        if (lane == 0) { atomicAdd(&s_misc[0], p0); atomicAdd(&s_misc[1], p1); }
        __syncthreads();
        n0 = s_misc[0];
        n1 = s_misc[1];
    }

    // ---- phase B: destination share of this CTA, slot map of its source chunks ---------------
    const int G = gridDim.x;
    const int rows_per = (n_kept + G - 1) / G;
    const int d0 = min(n_kept, (int)blockIdx.x * rows_per);
    const int d1 = min(n_kept, d0 + rows_per);
    const int n_rows = min(d1 - d0, a.rows_cap);

    // first chunk that holds destination d0: largest c with prefix[c] <= d0
    int c_first = 0;
    {
        int lo = 0, hi = n_chunks;       // prefix[lo] <= d0 invariant (prefix[0] = 0)
        while (hi - lo > 1) {
            int mid = (lo + hi) >> 1;
            if (prefix[mid] <= d0) lo = mid; else hi = mid;
        }
        c_first = lo;
    }
    int moved_local = 0;
    // chunks needed for the gather list [c_first, ...) and chunks owned for the slot map (c % G == b)
    for (int pass = 0; pass < 2; ++pass) {
        int c_begin, c_step;
        if (pass == 0) { c_begin = c_first + wid; c_step = CP_WARPS; }
        else { c_begin = blockIdx.x + wid * G; c_step = CP_WARPS * G; }
        for (int c = c_begin; c < n_chunks; c += c_step) {
            if (pass == 0 && (n_rows <= 0 || prefix[c] >= d1)) break;
            if (pass == 1 && !a.slot_map && !a.info) break;
            int run = prefix[c];
            const int base = c << a.chunk_shift;
            for (int k = 0; k < vec_per_lane; ++k) {
                const int pos = base + k * 512 + lane * 16;
                uint4 v = load_mask16(a.mask, pos, s);
                const uint32_t w[4] = {v.x, v.y, v.z, v.w};
                int cnt = nonzero_bytes(w[0]) + nonzero_bytes(w[1]) + nonzero_bytes(w[2]) + nonzero_bytes(w[3]);
                int tot;
                int r = run + warp_excl_scan(cnt, lane, tot);
                run += tot;
                int32_t out[16];
#pragma unroll
                for (int b = 0; b < 16; ++b) {
                    const bool kept = (w[b >> 2] >> ((b & 3) * 8)) & 0xffu;
                    out[b] = kept ? r : -1;
                    if (kept) {
                        if (pass == 0) {
                            if (r >= d0 && r - d0 < n_rows) src_list[r - d0] = pos + b;
                        } else if (r != pos + b) {
                            ++moved_local;
                        }
                        ++r;
                    }
                }
                if (pass == 1 && a.slot_map) {
                    if (pos + 16 <= s) {
                        int4* o4 = reinterpret_cast<int4*>(a.slot_map + pos);
                        o4[0] = make_int4(out[0], out[1], out[2], out[3]);
                        o4[1] = make_int4(out[4], out[5], out[6], out[7]);
                        o4[2] = make_int4(out[8], out[9], out[10], out[11]);
                        o4[3] = make_int4(out[12], out[13], out[14], out[15]);
                    } else {
                        for (int b = 0; b < 16 && pos + b < s; ++b) a.slot_map[pos + b] = out[b];
                    }
                }
            }
        }
    }
    // ---- integer summary and page classes ------------------------------------------------------
    if (a.info) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) moved_local += __shfl_xor_sync(0xffffffffu, moved_local, o);
        if (lane == 0 && moved_local) atomicAdd(&a.info->rows_moved, moved_local);
        if (blockIdx.x == 0 && tid == 0) {
            a.info->n_kept = n_kept;
            a.info->span_pages = (n_kept + a.page_size - 1) / a.page_size;
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
    __syncthreads();

    // ---- phase C: move the rows ----------------------------------------------------------------
    if (a.k_dst == nullptr) return;
    const long long total = (long long)n_rows * 2 * a.vpr;
    for (long long base = tid; base < total; base += (long long)CP_THREADS * CP_UNROLL) {
        uint4 buf[CP_UNROLL];
        uint4* dst[CP_UNROLL];
#pragma unroll
        for (int u = 0; u < CP_UNROLL; ++u) {
            const long long idx = base + (long long)u * CP_THREADS;
            dst[u] = nullptr;
            if (idx < total) {
                int rw, v;
                if (a.vpr_shift >= 0) { rw = (int)(idx >> a.vpr_shift); v = (int)(idx & (a.vpr - 1)); }
                else { rw = (int)(idx / a.vpr); v = (int)(idx - (long long)rw * a.vpr); }
                const int r = rw >> 1;
                const bool is_v = rw & 1;
                const size_t so = (size_t)src_list[r] * a.row_bytes + (size_t)v * 16;
                const size_t dof = (size_t)(d0 + r) * a.row_bytes + (size_t)v * 16;
                buf[u] = ld_stream(reinterpret_cast<const uint4*>((is_v ? a.v_src : a.k_src) + so));
                dst[u] = reinterpret_cast<uint4*>((is_v ? a.v_dst : a.k_dst) + dof);
            }
        }
#pragma unroll
        for (int u = 0; u < CP_UNROLL; ++u)
            if (dst[u]) st_stream(dst[u], buf[u]);
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

extern "C" omni_status omnipage_compact(omnitide_ctx* ctx, void* stream, const void* k_src, const void* v_src,
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
        if (ctx->inplace_rows < (size_t)ctx->g.s_cap) {
            // first in-place call on this context: allocate the staging rows (synchronous)
            if (ctx->inplace_k) cudaFree(ctx->inplace_k);
            if (ctx->inplace_v) cudaFree(ctx->inplace_v);
            ctx->inplace_k = ctx->inplace_v = nullptr;
            ctx->inplace_rows = 0;
            OMNI_CUDA(ctx, cudaMalloc(&ctx->inplace_k, (size_t)ctx->g.s_cap * ctx->row_bytes));
            OMNI_CUDA(ctx, cudaMalloc(&ctx->inplace_v, (size_t)ctx->g.s_cap * ctx->row_bytes));
            ctx->inplace_rows = ctx->g.s_cap;
        }
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
    a.chunk_shift = 9;
    while (((s_span_max + (1 << a.chunk_shift) - 1) >> a.chunk_shift) > CP_MAX_CHUNKS) ++a.chunk_shift;
    a.units_kept = units_kept; a.n_units_kept_dev = n_units_kept_dev; a.n_units_max = n_units_max;
    a.slot_map = slot_map_out; a.info = info_out; a.page_class = page_class_out; a.status = ctx->status_dev;
    const int grid = ctx->sm_count;
    a.rows_cap = (s_span_max + grid - 1) / grid + 1;
    const int max_chunks = ((s_span_max + (1 << a.chunk_shift) - 1) >> a.chunk_shift) + 2;
    const size_t smem = (size_t)(max_chunks + a.rows_cap) * sizeof(int);
    if (smem > 200 * 1024) OMNI_FAIL(ctx, OMNI_ERR_CAPACITY, "compact: span too large for one launch");
    if (info_out) OMNI_CUDA(ctx, cudaMemsetAsync(&info_out->rows_moved, 0, sizeof(int32_t), st));
    if (smem > 48 * 1024)
        OMNI_CUDA(ctx, cudaFuncSetAttribute(compact_pack_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    compact_pack_kernel<<<grid, CP_THREADS, smem, st>>>(a);
    OMNI_CHECK_LAUNCH(ctx, "compact_pack_kernel");
    if (in_place) {
        if (!info_out) OMNI_FAIL(ctx, OMNI_ERR_INVALID_ARG, "compact: in-place mode needs info_out");
        copy_rows_kernel<<<ctx->sm_count * 4, 256, 0, st>>>(
            static_cast<const char*>(kd), static_cast<const char*>(vd), static_cast<char*>(k_dst),
            static_cast<char*>(v_dst), &info_out->n_kept, s_span_max, nullptr, ctx->g.s_cap, (int)ctx->row_bytes,
            ctx->status_dev);
        OMNI_CHECK_LAUNCH(ctx, "copy_rows_kernel");
    }
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
