// Decode-phase attention: ONE new token against the retained history (bf16, head dim 128, GQA).
//
// The work is a single pass over K and V (2 x N x 256 bytes per KV head): bound by HBM, with nothing for the
// tensor cores to do (G <= 8 query rows per KV head).  Split-KV on CUDA cores: grid (splits, KV heads); a warp
// takes two keys per step (one per half-warp, a lane holds 8 of the 128 dimensions as one 16-byte load), keeps
// the G query heads of the group in registers and an online softmax per head; halves, warps and finally the
// splits are merged by log-sum-exp.  The last CTA of a KV head to finish (a counter, no waiting) merges the
// splits and writes the output, so the whole step is one launch.
#include "common.cuh"

#include <algorithm>

namespace {

constexpr int DEC_THREADS = 256;
constexpr int DEC_WARPS = DEC_THREADS / 32;
constexpr int DEC_D = 128;
constexpr int DEC_BATCH = 2;              // key pairs per batch per warp; the next batch is loaded under the arithmetic of this one
constexpr int DEC_CTAS_PER_SM = 2;        // splits are sized for about two CTAs per SM in all
constexpr int DEC_MAX_SPLIT = 64;         // the weights of the final merge live in shared memory (2 * G * 64 floats)

struct DecodeParams {
    const __nv_bfloat16* q;               // [1][h_q][128]
    const __nv_bfloat16* k_hist; const __nv_bfloat16* v_hist; const int32_t* n_hist_dev; int n_hist_max;
    const __nv_bfloat16* k_chunk; const __nv_bfloat16* v_chunk;       // [1][h_kv][128]: the token's own key and value
    int h_q, h_kv; float scale_log2, scale;
    void* o_out; int out_dtype; float* lse_out;
    float* part_o; float2* part_ml;       // [split][h_q][128], [split][h_q]
    int32_t* counter;                     // [h_kv], zero between launches
    int32_t* status;
};

__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

__device__ __forceinline__ float fast_ex2(float x) {          // ex2.approx: exp2(-inf) = 0
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int G>
__global__ void __launch_bounds__(DEC_THREADS, (G <= 4 ? 2 : 1)) decode_attention_kernel(const DecodeParams p) {
    __shared__ float s_o[DEC_WARPS][G][DEC_D];
    __shared__ float2 s_ml[DEC_WARPS][G];
    __shared__ int s_last;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, half = lane >> 4, sub = lane & 15;
    const int kvh = blockIdx.y, split = blockIdx.x, n_split = gridDim.x;
    int n_hist = p.n_hist_dev ? *p.n_hist_dev : p.n_hist_max;
    if (n_hist < 0 || n_hist > p.n_hist_max) {
        if (tid == 0 && split == 0 && kvh == 0) atomicOr(p.status, OMNI_DEV_BAD_COUNT);
        n_hist = max(0, min(n_hist, p.n_hist_max));
    }
    const int total = n_hist + 1;                            // the history and the token itself
    const int per = (total + n_split - 1) / n_split;
    const int k0 = split * per, k1 = min(total, k0 + per);
    const size_t row = (size_t)p.h_kv * DEC_D;

    float qf[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        float t8[8];
        unpack8(__ldg(reinterpret_cast<const uint4*>(p.q + (size_t)(kvh * G + g) * DEC_D + sub * 8)), t8);
#pragma unroll
        for (int i = 0; i < 8; ++i) qf[g][i] = t8[i] * p.scale_log2;
    }
    float m[G], l[G], o[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        m[g] = -INFINITY; l[g] = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) o[g][i] = 0.f;
    }
    auto k_ptr = [&](int key) {
        return key < n_hist ? p.k_hist + (size_t)key * row + (size_t)kvh * DEC_D + sub * 8 : p.k_chunk + (size_t)kvh * DEC_D + sub * 8;
    };
    auto v_ptr = [&](int key) {
        return key < n_hist ? p.v_hist + (size_t)key * row + (size_t)kvh * DEC_D + sub * 8 : p.v_chunk + (size_t)kvh * DEC_D + sub * 8;
    };
    // the trip count depends on the warp only: both half-warps take part in every full-mask shuffle below.
    // The loads of batch n + 1 are issued before the arithmetic of batch n (a warp has only three or four batches:
    // without this every one of them pays a full memory round trip).
    uint4 kk_next[DEC_BATCH], vv_next[DEC_BATCH];
    auto load_batch = [&](int base) {
#pragma unroll
        for (int b = 0; b < DEC_BATCH; ++b) {
            const int key = base + half + b * DEC_WARPS * 2;
            kk_next[b] = make_uint4(0, 0, 0, 0);
            vv_next[b] = make_uint4(0, 0, 0, 0);
            if (key < k1) {
                kk_next[b] = __ldg(reinterpret_cast<const uint4*>(k_ptr(key)));
                vv_next[b] = __ldg(reinterpret_cast<const uint4*>(v_ptr(key)));
            }
        }
    };
    if (k0 + warp * 2 < k1) load_batch(k0 + warp * 2);
    for (int base = k0 + warp * 2; base < k1; base += DEC_WARPS * 2 * DEC_BATCH) {
        const int key0 = base + half;
        uint4 kk[DEC_BATCH], vv[DEC_BATCH];
#pragma unroll
        for (int b = 0; b < DEC_BATCH; ++b) { kk[b] = kk_next[b]; vv[b] = vv_next[b]; }
        if (base + DEC_WARPS * 2 * DEC_BATCH < k1) load_batch(base + DEC_WARPS * 2 * DEC_BATCH);
        // scores of the batch first (an invalid key scores -inf), then ONE rescale per head for the whole batch
        float kf[DEC_BATCH][8];
#pragma unroll
        for (int b = 0; b < DEC_BATCH; ++b) unpack8(kk[b], kf[b]);
        float sc[G][DEC_BATCH];
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int b = 0; b < DEC_BATCH; ++b) {
                float s = 0.f;
#pragma unroll
                for (int i = 0; i < 8; ++i) s = fmaf(qf[g][i], kf[b][i], s);
                sc[g][b] = s;
            }
#pragma unroll
        for (int d = 8; d > 0; d >>= 1)
#pragma unroll
            for (int g = 0; g < G; ++g)
#pragma unroll
                for (int b = 0; b < DEC_BATCH; ++b) sc[g][b] += __shfl_xor_sync(0xffffffffu, sc[g][b], d);   // over the 16 lanes of the key
        float vf[DEC_BATCH][8];
#pragma unroll
        for (int b = 0; b < DEC_BATCH; ++b) unpack8(vv[b], vf[b]);
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float m_new = m[g];
#pragma unroll
            for (int b = 0; b < DEC_BATCH; ++b) {
                if (key0 + b * DEC_WARPS * 2 >= k1) sc[g][b] = -INFINITY;
                m_new = fmaxf(m_new, sc[g][b]);
            }
            if (m_new == -INFINITY) continue;                // nothing seen yet
            const float alpha = fast_ex2(m[g] - m_new);
            float pw[DEC_BATCH], ps = 0.f;
#pragma unroll
            for (int b = 0; b < DEC_BATCH; ++b) { pw[b] = fast_ex2(sc[g][b] - m_new); ps += pw[b]; }
            l[g] = fmaf(l[g], alpha, ps);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float acc = o[g][i] * alpha;
#pragma unroll
                for (int b = 0; b < DEC_BATCH; ++b) acc = fmaf(pw[b], vf[b][i], acc);
                o[g][i] = acc;
            }
            m[g] = m_new;
        }
    }
    // ---- merge the two half-warps, then the warps of the CTA ------------------------------------------------
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const float m_o = __shfl_xor_sync(0xffffffffu, m[g], 16), l_o = __shfl_xor_sync(0xffffffffu, l[g], 16);
        const float M = fmaxf(m[g], m_o);
        const float wa = m[g] == -INFINITY ? 0.f : exp2f(m[g] - M), wb = m_o == -INFINITY ? 0.f : exp2f(m_o - M);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float oo = __shfl_xor_sync(0xffffffffu, o[g][i], 16);
            o[g][i] = o[g][i] * wa + oo * wb;
        }
        l[g] = l[g] * wa + l_o * wb;
        m[g] = M;
        if (half == 0) {
#pragma unroll
            for (int i = 0; i < 8; ++i) s_o[warp][g][sub * 8 + i] = o[g][i];
            if (sub == 0) s_ml[warp][g] = make_float2(M, l[g]);
        }
    }
    __syncthreads();
    for (int e = tid; e < G * DEC_D; e += DEC_THREADS) {
        const int g = e / DEC_D, dim = e % DEC_D;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < DEC_WARPS; ++w) M = fmaxf(M, s_ml[w][g].x);
        float acc = 0.f, L = 0.f;
#pragma unroll
        for (int w = 0; w < DEC_WARPS; ++w) {
            const float2 ml = s_ml[w][g];
            const float wgt = ml.x == -INFINITY ? 0.f : exp2f(ml.x - M);
            acc += wgt * s_o[w][g][dim];
            L += wgt * ml.y;
        }
        const int head = kvh * G + g;
        p.part_o[((size_t)split * p.h_q + head) * DEC_D + dim] = acc;
        if (dim == 0) p.part_ml[(size_t)split * p.h_q + head] = make_float2(M, L);
    }
    // ---- the last CTA of this KV head to arrive merges the splits (no CTA waits for another) ------------------
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = atomicAdd(p.counter + kvh, 1) == n_split - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // weights of the splits first (all loads in parallel), then the weighted sums with the loads unrolled
    float (*s_w)[DEC_MAX_SPLIT] = reinterpret_cast<float (*)[DEC_MAX_SPLIT]>(&s_o[0][0][0]);      // [G][splits], reuses s_o
    float* s_l = &s_o[0][0][0] + G * DEC_MAX_SPLIT;                                                  // [G][splits]
    __shared__ float s_M[G], s_L[G];
    for (int idx = tid; idx < G * n_split; idx += DEC_THREADS) {
        const int g = idx / n_split, sp = idx - g * n_split;
        const float2 ml = __ldcg(&p.part_ml[(size_t)sp * p.h_q + kvh * G + g]);
        s_w[g][sp] = ml.x;
        s_l[g * DEC_MAX_SPLIT + sp] = ml.y;
    }
    __syncthreads();
    if (tid < G) {
        float M = -INFINITY, L = 0.f;
        for (int sp = 0; sp < n_split; ++sp) M = fmaxf(M, s_w[tid][sp]);
        for (int sp = 0; sp < n_split; ++sp) {
            const float wgt = s_w[tid][sp] == -INFINITY ? 0.f : exp2f(s_w[tid][sp] - M);
            L += wgt * s_l[tid * DEC_MAX_SPLIT + sp];
            s_w[tid][sp] = wgt;
        }
        s_M[tid] = M;
        s_L[tid] = L;
    }
    __syncthreads();
    for (int e = tid; e < G * DEC_D; e += DEC_THREADS) {
        const int g = e / DEC_D, dim = e % DEC_D, head = kvh * G + g;
        float acc = 0.f;
#pragma unroll 8
        for (int sp = 0; sp < n_split; ++sp)
            acc += s_w[g][sp] * __ldcg(&p.part_o[((size_t)sp * p.h_q + head) * DEC_D + dim]);
        const float r = acc / s_L[g];
        const size_t off = (size_t)head * DEC_D + dim;
        if (p.out_dtype == OMNI_DTYPE_FP32) static_cast<float*>(p.o_out)[off] = r;
        else static_cast<__nv_bfloat16*>(p.o_out)[off] = __float2bfloat16_rn(r);
        if (p.lse_out && dim == 0) p.lse_out[head] = (s_M[g] + log2f(s_L[g])) * 0.6931471805599453f;
    }
    if (tid == 0) p.counter[kvh] = 0;                        // ready for the next launch on this context
}

}  // namespace

// t == 1, bf16, d == 128, G in {1, 2, 4, 8}, dense history.  Returns OMNI_ERR_UNSUPPORTED otherwise (the caller falls back).
omni_status omni_attention_decode(omnitide_ctx* ctx, cudaStream_t st, const void* q, const void* k_hist, const void* v_hist,
                                  const int32_t* n_hist_dev, int n_hist_max, const void* k_chunk, const void* v_chunk,
                                  float scale, void* o_out, int out_dtype, float* lse_out) {
    const omni_geometry& g = ctx->g;
    const int G = g.h_q / g.h_kv;
    if (g.d != DEC_D || g.dtype != OMNI_DTYPE_BF16 || (G != 1 && G != 2 && G != 4 && G != 8)) return OMNI_ERR_UNSUPPORTED;
    DecodeParams p;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.k_hist = static_cast<const __nv_bfloat16*>(k_hist); p.v_hist = static_cast<const __nv_bfloat16*>(v_hist);
    p.n_hist_dev = n_hist_dev; p.n_hist_max = n_hist_max;
    p.k_chunk = static_cast<const __nv_bfloat16*>(k_chunk); p.v_chunk = static_cast<const __nv_bfloat16*>(v_chunk);
    p.h_q = g.h_q; p.h_kv = g.h_kv; p.scale = scale; p.scale_log2 = scale * 1.4426950408889634f;
    p.o_out = o_out; p.out_dtype = out_dtype; p.lse_out = lse_out;
    p.part_o = ctx->attn_part_o; p.part_ml = reinterpret_cast<float2*>(ctx->attn_part_ml);
    p.counter = ctx->dec_counter; p.status = ctx->status_dev;
    // about two CTAs per SM in all, at least 64 keys per split, and no more splits than the partial buffers hold
    int n_split = std::max(1, (DEC_CTAS_PER_SM * ctx->sm_count) / g.h_kv);
    n_split = std::min(n_split, std::max(1, (n_hist_max + 1 + 63) / 64));
    n_split = std::min(n_split, DEC_MAX_SPLIT);
    n_split = std::min<long long>(n_split, (long long)ctx->sm_count * 4 * 128 * 128 / ((long long)g.h_q * DEC_D));
    const dim3 grid(n_split, g.h_kv);
    switch (G) {
        case 1: decode_attention_kernel<1><<<grid, DEC_THREADS, 0, st>>>(p); break;
        case 2: decode_attention_kernel<2><<<grid, DEC_THREADS, 0, st>>>(p); break;
        case 4: decode_attention_kernel<4><<<grid, DEC_THREADS, 0, st>>>(p); break;
        default: decode_attention_kernel<8><<<grid, DEC_THREADS, 0, st>>>(p); break;
    }
    OMNI_CHECK_LAUNCH(ctx, "decode_attention_kernel");
    return OMNI_OK;
}
