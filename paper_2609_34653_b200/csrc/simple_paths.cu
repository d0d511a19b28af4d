// CUDA-core fp32 paths for geometries the tensor-core kernels do not cover (fp32 storage, head
// dims other than 128).  One warp owns one (query row, head); lanes split the head dimension.
#include "common.cuh"

namespace {

constexpr int SP_WARPS = 4;
constexpr int SP_MAX_EPL = 8;      // elements per lane: d <= 256

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// ------------------------------------------------------------------------------------------------
// attention: online softmax over history rows then chunk rows 0..i
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(SP_WARPS * 32) attention_rows_kernel(
    const T* __restrict__ q, int t, int h_q, int h_kv, int d, const T* __restrict__ k_hist,
    const T* __restrict__ v_hist, const int32_t* n_hist_dev, int n_hist_max, const T* __restrict__ k_chunk,
    const T* __restrict__ v_chunk, float scale, void* o_out, int out_dtype, float* lse_out, int32_t* status,
    const uint8_t* __restrict__ hist_mask) {
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * SP_WARPS + (threadIdx.x >> 5);
    if (row >= (long long)t * h_q) return;
    const int i = (int)(row / h_q), h = (int)(row % h_q);
    const int g = h / (h_q / h_kv);
    int n_hist = n_hist_dev ? *n_hist_dev : n_hist_max;
    if (n_hist > n_hist_max || n_hist < 0) {
        if (lane == 0) atomicOr(status, OMNI_DEV_BAD_COUNT);
        n_hist = max(0, min(n_hist, n_hist_max));
    }
    float qr[SP_MAX_EPL], acc[SP_MAX_EPL];
#pragma unroll
    for (int e = 0; e < SP_MAX_EPL; ++e) {
        const int c = lane + 32 * e;
        qr[e] = c < d ? to_f32(q[((size_t)i * h_q + h) * d + c]) * scale : 0.f;
        acc[e] = 0.f;
    }
    float m = -INFINITY, l = 0.f;
    const size_t kv_stride = (size_t)h_kv * d;
    const int n_keys = n_hist + i + 1;
    for (int j = 0; j < n_keys; ++j) {
        if (hist_mask && j < n_hist && hist_mask[j] == 0) continue;      // a hole of the history: not visible
        const T* kr = j < n_hist ? k_hist + (size_t)j * kv_stride + (size_t)g * d
                                 : k_chunk + (size_t)(j - n_hist) * kv_stride + (size_t)g * d;
        const T* vr = j < n_hist ? v_hist + (size_t)j * kv_stride + (size_t)g * d
                                 : v_chunk + (size_t)(j - n_hist) * kv_stride + (size_t)g * d;
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < SP_MAX_EPL; ++e) {
            const int c = lane + 32 * e;
            if (c < d) s += qr[e] * to_f32(kr[c]);
        }
        s = warp_sum(s);
        const float m_new = fmaxf(m, s);
        const float alpha = __expf(m - m_new);      // exp(-inf) = 0 on the first key
        const float p = __expf(s - m_new);
        l = l * alpha + p;
#pragma unroll
        for (int e = 0; e < SP_MAX_EPL; ++e) {
            const int c = lane + 32 * e;
            if (c < d) acc[e] = acc[e] * alpha + p * to_f32(vr[c]);
        }
        m = m_new;
    }
    const float inv = 1.f / l;
#pragma unroll
    for (int e = 0; e < SP_MAX_EPL; ++e) {
        const int c = lane + 32 * e;
        if (c < d) {
            const size_t o = ((size_t)i * h_q + h) * d + c;
            if (out_dtype == OMNI_DTYPE_FP32) static_cast<float*>(o_out)[o] = acc[e] * inv;
            else static_cast<__nv_bfloat16*>(o_out)[o] = __float2bfloat16_rn(acc[e] * inv);
        }
    }
    if (lse_out && lane == 0) lse_out[(size_t)i * h_q + h] = m + logf(l);
}

// ------------------------------------------------------------------------------------------------
// scoring: pass 1 row max and normaliser over the history keys, pass 2 per-unit sums
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(SP_WARPS * 32) score_rows_kernel(
    const T* __restrict__ q, int t, int h_q, int h_kv, int d, const T* __restrict__ k_cache,
    const int32_t* n_hist_dev, int n_hist_max, const omni_unit* __restrict__ units, const int32_t* n_units_dev,
    int n_units_max, float scale, double* mass64, int32_t* status) {
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * SP_WARPS + (threadIdx.x >> 5);
    if (row >= (long long)t * h_q) return;
    const int i = (int)(row / h_q), h = (int)(row % h_q);
    const int g = h / (h_q / h_kv);
    int n_units = n_units_dev ? *n_units_dev : n_units_max;
    n_units = max(0, min(n_units, n_units_max));
    if (n_units == 0) return;
    int n_hist = units[n_units - 1].start + units[n_units - 1].len;
    if (n_hist > n_hist_max || (n_hist_dev && *n_hist_dev != n_hist)) {
        if (lane == 0) atomicOr(status, OMNI_DEV_BAD_COUNT);
        return;
    }
    float qr[SP_MAX_EPL];
#pragma unroll
    for (int e = 0; e < SP_MAX_EPL; ++e) {
        const int c = lane + 32 * e;
        qr[e] = c < d ? to_f32(q[((size_t)i * h_q + h) * d + c]) * scale : 0.f;
    }
    const size_t kv_stride = (size_t)h_kv * d;
    float m = -INFINITY, l = 0.f;
    for (int j = 0; j < n_hist; ++j) {
        const T* kr = k_cache + (size_t)j * kv_stride + (size_t)g * d;
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < SP_MAX_EPL; ++e) {
            const int c = lane + 32 * e;
            if (c < d) s += qr[e] * to_f32(kr[c]);
        }
        s = warp_sum(s);
        const float m_new = fmaxf(m, s);
        l = l * __expf(m - m_new) + __expf(s - m_new);
        m = m_new;
    }
    const float inv = 1.f / l;
    int u = 0;
    int u_end = units[0].start + units[0].len;
    float acc = 0.f;
    for (int j = 0; j < n_hist; ++j) {
        if (j >= u_end) {
            if (lane == 0) atomicAdd(&mass64[u], (double)acc);
            acc = 0.f;
            ++u;
            u_end = units[u].start + units[u].len;
        }
        const T* kr = k_cache + (size_t)j * kv_stride + (size_t)g * d;
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < SP_MAX_EPL; ++e) {
            const int c = lane + 32 * e;
            if (c < d) s += qr[e] * to_f32(kr[c]);
        }
        s = warp_sum(s);
        acc += __expf(s - m) * inv;
    }
    if (lane == 0) atomicAdd(&mass64[u], (double)acc);
}

}  // namespace

// score_u = w[modality] * mass_u * N / len_u from a double mass accumulator (sum over rows)
__global__ void score_finalize64_kernel(const double* mass64, const omni_unit* units, const int32_t* n_units_dev,
                                        int n_units_max, float w0, float w1, float w2, float inv_rows, float* scores, float* mass) {
    int n_units = n_units_dev ? *n_units_dev : n_units_max;
    n_units = max(0, min(n_units, n_units_max));
    if (n_units == 0) return;
    const int n_hist = units[n_units - 1].start + units[n_units - 1].len;
    for (int u = blockIdx.x * blockDim.x + threadIdx.x; u < n_units; u += gridDim.x * blockDim.x) {
        const omni_unit un = units[u];
        const float mu = (float)(mass64[u] * (double)inv_rows);
        const int mod = min(max(un.modality, 0), 2);
        const float w = mod == 0 ? w0 : (mod == 1 ? w1 : w2);
        scores[u] = w * mu * (float)n_hist / (float)un.len;
        if (mass) mass[u] = mu;
    }
}

omni_status omni_attention_simple(omnitide_ctx* ctx, cudaStream_t st, const void* q, int t, const void* k_hist,
                                  const void* v_hist, const int32_t* n_hist_dev, int n_hist_max, const void* k_chunk,
                                  const void* v_chunk, float scale, void* o_out, int out_dtype, float* lse_out,
                                  const uint8_t* hist_mask) {
    const omni_geometry& g = ctx->g;
    const long long rows = (long long)t * g.h_q;
    const int grid = (int)((rows + SP_WARPS - 1) / SP_WARPS);
    if (g.dtype == OMNI_DTYPE_FP32)
        attention_rows_kernel<float><<<grid, SP_WARPS * 32, 0, st>>>(
            (const float*)q, t, g.h_q, g.h_kv, g.d, (const float*)k_hist, (const float*)v_hist, n_hist_dev, n_hist_max,
            (const float*)k_chunk, (const float*)v_chunk, scale, o_out, out_dtype, lse_out, ctx->status_dev, hist_mask);
    else
        attention_rows_kernel<__nv_bfloat16><<<grid, SP_WARPS * 32, 0, st>>>(
            (const __nv_bfloat16*)q, t, g.h_q, g.h_kv, g.d, (const __nv_bfloat16*)k_hist, (const __nv_bfloat16*)v_hist,
            n_hist_dev, n_hist_max, (const __nv_bfloat16*)k_chunk, (const __nv_bfloat16*)v_chunk, scale, o_out,
            out_dtype, lse_out, ctx->status_dev, hist_mask);
    OMNI_CHECK_LAUNCH(ctx, "attention_rows_kernel");
    return OMNI_OK;
}

omni_status omni_score_simple(omnitide_ctx* ctx, cudaStream_t st, const void* q, int t, const void* k_cache,
                              const int32_t* n_hist_dev, int n_hist_max, const omni_unit* units,
                              const int32_t* n_units_dev, int n_units_max, const float* w, float scale,
                              float* scores_out, float* mass_out) {
    const omni_geometry& g = ctx->g;
    OMNI_CUDA(ctx, cudaMemsetAsync(ctx->score_mass64, 0, sizeof(double) * (size_t)g.u_cap, st));
    const long long rows = (long long)t * g.h_q;
    const int grid = (int)((rows + SP_WARPS - 1) / SP_WARPS);
    if (g.dtype == OMNI_DTYPE_FP32)
        score_rows_kernel<float><<<grid, SP_WARPS * 32, 0, st>>>((const float*)q, t, g.h_q, g.h_kv, g.d,
                                                                 (const float*)k_cache, n_hist_dev, n_hist_max, units,
                                                                 n_units_dev, n_units_max, scale, ctx->score_mass64,
                                                                 ctx->status_dev);
    else
        score_rows_kernel<__nv_bfloat16><<<grid, SP_WARPS * 32, 0, st>>>(
            (const __nv_bfloat16*)q, t, g.h_q, g.h_kv, g.d, (const __nv_bfloat16*)k_cache, n_hist_dev, n_hist_max,
            units, n_units_dev, n_units_max, scale, ctx->score_mass64, ctx->status_dev);
    OMNI_CHECK_LAUNCH(ctx, "score_rows_kernel");
    score_finalize64_kernel<<<(n_units_max + 255) / 256, 256, 0, st>>>(ctx->score_mass64, units, n_units_dev, n_units_max,
                                                                       w[0], w[1], w[2], 1.0f / (float)rows, scores_out, mass_out);
    OMNI_CHECK_LAUNCH(ctx, "score_finalize64_kernel");
    return OMNI_OK;
}

// ------------------------------------------------------------------------------------------------
// Scoring without any allocation, for callers that have no context and may not call cudaMalloc.
// The per-unit accumulator that the CUDA-core scoring kernel adds into lives in a fixed array in
// device global memory that is part of the library image (every device that loads the library
// carries these few KB until the process exits).
// ------------------------------------------------------------------------------------------------
namespace {

constexpr int NOALLOC_MAX_UNITS = OMNITIDE_NOALLOC_MAX_UNITS;
constexpr int NOALLOC_MAX_DEVICES = 64;

static __device__ __align__(256) double g_noalloc_mass[NOALLOC_MAX_UNITS];
static __device__ __align__(256) int32_t g_noalloc_status[64];

// Device addresses of the two arrays, looked up once per device.  The array names above are only
// host-side handles here: a kernel must be given the address that cudaGetSymbolAddress returns
// while that device is current.
struct NoallocDevice {
    double* mass;
    int32_t* status;
    bool ready;
};
NoallocDevice g_noalloc_dev[NOALLOC_MAX_DEVICES];

omni_status noalloc_setup(int dev, NoallocDevice** out) {
    if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return OMNI_ERR_UNSUPPORTED;
    NoallocDevice& d = g_noalloc_dev[dev];
    if (!d.ready) {
        void* p_mass = nullptr;
        void* p_status = nullptr;
        if (cudaGetSymbolAddress(&p_mass, g_noalloc_mass) != cudaSuccess) return OMNI_ERR_CUDA;
        if (cudaGetSymbolAddress(&p_status, g_noalloc_status) != cudaSuccess) return OMNI_ERR_CUDA;
        d.mass = static_cast<double*>(p_mass);
        d.status = static_cast<int32_t*>(p_status);
        d.ready = true;
    }
    *out = &d;
    return OMNI_OK;
}

}  // namespace

extern "C" omni_status omnitide_score_units_noalloc(void* stream, int32_t h_q, int32_t h_kv, int32_t d, int32_t dtype,
                                                    const void* q, int32_t t, const void* k_cache, int32_t n_hist,
                                                    const omni_unit* units, int32_t n_units, const float* w_modality,
                                                    float scale, float* scores_out, float* mass_out) {
    if (!q || !k_cache || !units || !w_modality || !scores_out) return OMNI_ERR_INVALID_ARG;
    if (h_q <= 0 || h_kv <= 0 || h_q % h_kv != 0 || d <= 0 || d % 8 != 0 || d > 256 ||
        (dtype != OMNI_DTYPE_BF16 && dtype != OMNI_DTYPE_FP32))
        return OMNI_ERR_UNSUPPORTED;
    if (t <= 0 || n_hist <= 0 || n_units <= 0) return OMNI_ERR_INVALID_ARG;
    if (n_units > NOALLOC_MAX_UNITS) return OMNI_ERR_CAPACITY;       // the fixed accumulator array is full
    if (!omni_aligned16(q) || !omni_aligned16(k_cache)) return OMNI_ERR_INVALID_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return OMNI_ERR_CUDA;
    NoallocDevice* nd = nullptr;
    omni_status s = noalloc_setup(dev, &nd);
    if (s != OMNI_OK) return s;
    if (scale <= 0.f) scale = 1.0f / sqrtf((float)d);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the array still holds the sums of the previous call: the accumulators must start at zero
    if (cudaMemsetAsync(nd->mass, 0, sizeof(double) * (size_t)n_units, st) != cudaSuccess) return OMNI_ERR_CUDA;
    const long long rows = (long long)t * h_q;
    const int grid = (int)((rows + SP_WARPS - 1) / SP_WARPS);
    if (dtype == OMNI_DTYPE_FP32)
        score_rows_kernel<float><<<grid, SP_WARPS * 32, 0, st>>>((const float*)q, t, h_q, h_kv, d, (const float*)k_cache,
                                                                 nullptr, n_hist, units, nullptr, n_units, scale, nd->mass,
                                                                 nd->status);
    else
        score_rows_kernel<__nv_bfloat16><<<grid, SP_WARPS * 32, 0, st>>>(
            (const __nv_bfloat16*)q, t, h_q, h_kv, d, (const __nv_bfloat16*)k_cache, nullptr, n_hist, units, nullptr,
            n_units, scale, nd->mass, nd->status);
    if (cudaGetLastError() != cudaSuccess) return OMNI_ERR_CUDA;
    score_finalize64_kernel<<<(n_units + 255) / 256, 256, 0, st>>>(nd->mass, units, nullptr, n_units, w_modality[0],
                                                                   w_modality[1], w_modality[2], 1.0f / (float)rows,
                                                                   scores_out, mass_out);
    if (cudaGetLastError() != cudaSuccess) return OMNI_ERR_CUDA;
    return OMNI_OK;
}
