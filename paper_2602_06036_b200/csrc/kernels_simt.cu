// Generic CUDA-core kernels, templated on the storage type. They are the whole fp32 path (the
// tiny configuration) and the small element-wise steps of the bf16 path; the bf16 contractions
// and attention have tensor-core kernels of their own.
#include "dflash_internal.h"
#include "ptx_sm100.cuh"

#include <math_constants.h>

#include <algorithm>

namespace dflash {

long long g_launches = 0;

#define DFLASH_CHECK_LAUNCH()                                     \
    do {                                                          \
        ++g_launches;                                             \
        if (cudaPeekAtLastError() != cudaSuccess) return DFLASH_ERR_CUDA; \
    } while (0)

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Block-wide sum / max for blockDim.x <= 1024 (multiple of 32). `red` holds 32 floats.
__device__ __forceinline__ float block_sum(float v, float* red) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) red[w] = v;
    __syncthreads();
    float t = (lane < nw) ? red[lane] : 0.f;
    return warp_sum(t);
}
__device__ __forceinline__ float block_max(float v, float* red) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
    v = warp_max(v);
    __syncthreads();
    if (lane == 0) red[w] = v;
    __syncthreads();
    float t = (lane < nw) ? red[lane] : -CUDART_INF_F;
    return warp_max(t);
}

// ------------------------------------------------------------------------------------------
// embedding gather: row 0 of each block = anchor, rows 1.. = mask token (Sec. 4.2)
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void embed_kernel(const T* __restrict__ E, const int32_t* __restrict__ anchor,
                             const int32_t* __restrict__ token_ids, float* __restrict__ x, int B, int D, int V,
                             int mask_id, int32_t* status) {
    const int row = blockIdx.x, b = row / B, r = row % B;
    int id = token_ids ? token_ids[row] : ((r == 0) ? anchor[b] : mask_id);
    if (id < 0 || id >= V) {
        if (threadIdx.x == 0 && status) atomicOr(status, DFLASH_DEV_BAD_TOKEN);
        id = 0;
    }
    const T* src = E + (size_t)id * D;
    float* dst = x + (size_t)row * D;
    for (int d = threadIdx.x; d < D; d += blockDim.x) dst[d] = to_f(src[d]);
}

int launch_embed(const Launch& L, const int32_t* anchor, const int32_t* token_ids, float* x, int batch, int block_rows) {
    const dflash_config& c = L.h->cfg;
    const int rows = batch * block_rows;
    if (c.dtype == DFLASH_F32)
        embed_kernel<float><<<rows, 256, 0, L.st>>>((const float*)L.h->w.embed, anchor, token_ids, x, block_rows,
                                                    c.d_model, c.vocab, c.mask_token_id, L.status);
    else
        embed_kernel<__nv_bfloat16><<<rows, 256, 0, L.st>>>((const __nv_bfloat16*)L.h->w.embed, anchor, token_ids, x,
                                                            block_rows, c.d_model, c.vocab,
                                                            c.mask_token_id, L.status);
    DFLASH_CHECK_LAUNCH();
    return DFLASH_OK;
}

// ------------------------------------------------------------------------------------------
// RMSNorm (App. A.3): out = g * y * rsqrt(mean(y^2) + eps); statistics in fp32
// ------------------------------------------------------------------------------------------
template <typename Tin, typename Tg, typename Tout>
__global__ void rmsnorm_kernel(const Tin* __restrict__ in, const Tg* __restrict__ g, Tout* __restrict__ out,
                               int dim, float eps, int apply) {
    __shared__ float red[32];
    const Tin* src = in + (size_t)blockIdx.x * dim;
    Tout* dst = out + (size_t)blockIdx.x * dim;
    float scale = 1.f;
    if (apply) {
        float ss = 0.f;
        for (int d = threadIdx.x; d < dim; d += blockDim.x) { float v = to_f(src[d]); ss += v * v; }
        ss = block_sum(ss, red);
        scale = rsqrtf(ss / (float)dim + eps);
    }
    for (int d = threadIdx.x; d < dim; d += blockDim.x) {
        float v = to_f(src[d]);
        dst[d] = from_f<Tout>(apply ? v * scale * to_f(g[d]) : v);
    }
}

int launch_rmsnorm(const Launch& L, const void* in, bool in_is_f32, const void* g, bool apply, void* out,
                   int rows, int dim) {
    const dflash_config& c = L.h->cfg;
    if (rows == 0) return DFLASH_OK;
    const int ap = apply ? 1 : 0;
    if (c.dtype == DFLASH_F32) {
        rmsnorm_kernel<float, float, float><<<rows, 256, 0, L.st>>>((const float*)in, (const float*)g,
                                                                    (float*)out, dim, c.rms_eps, ap);
    } else if (in_is_f32) {
        rmsnorm_kernel<float, __nv_bfloat16, __nv_bfloat16><<<rows, 256, 0, L.st>>>(
            (const float*)in, (const __nv_bfloat16*)g, (__nv_bfloat16*)out, dim, c.rms_eps, ap);
    } else {
        rmsnorm_kernel<__nv_bfloat16, __nv_bfloat16, __nv_bfloat16><<<rows, 256, 0, L.st>>>(
            (const __nv_bfloat16*)in, (const __nv_bfloat16*)g, (__nv_bfloat16*)out, dim, c.rms_eps, ap);
    }
    DFLASH_CHECK_LAUNCH();
    return DFLASH_OK;
}

// ------------------------------------------------------------------------------------------
// Y[M,N] (+)= X[M,K] * W[N,K]^T on CUDA cores, fp32 accumulate. 64x64 tile, 4x4 per thread.
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const T* __restrict__ X, const T* __restrict__ W,
                                                        float* __restrict__ Y, int M, int N, int K,
                                                        int accumulate) {
    constexpr int BM = 64, BN = 64, BK = 16;
    __shared__ float sx[BK][BM + 1];
    __shared__ float sw[BK][BN + 1];
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;   // tx -> n, ty -> m
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    for (int k0 = 0; k0 < K; k0 += BK) {
        // 64 rows x 16 k = 1024 elements per operand, 4 per thread
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int e = threadIdx.x + i * 256;
            const int r = e / BK, kk = e % BK;
            const int k = k0 + kk;
            sx[kk][r] = (m0 + r < M && k < K) ? to_f(X[(size_t)(m0 + r) * K + k]) : 0.f;
            sw[kk][r] = (n0 + r < N && k < K) ? to_f(W[(size_t)(n0 + r) * K + k]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = sx[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = sw[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty * 4 + i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n >= N) continue;
            float* y = Y + (size_t)m * N + n;
            *y = accumulate ? (*y + acc[i][j]) : acc[i][j];
        }
    }
}

int launch_gemm_simt(const Launch& L, const void* X, const void* W, float* Y, int M, int N, int K,
                     bool accumulate) {
    if (M == 0 || N == 0) return DFLASH_OK;
    dim3 grid((N + 63) / 64, (M + 63) / 64);
    if (L.h->cfg.dtype == DFLASH_F32)
        gemm_simt_kernel<float><<<grid, 256, 0, L.st>>>((const float*)X, (const float*)W, Y, M, N, K,
                                                        accumulate ? 1 : 0);
    else
        gemm_simt_kernel<__nv_bfloat16><<<grid, 256, 0, L.st>>>((const __nv_bfloat16*)X,
                                                                (const __nv_bfloat16*)W, Y, M, N, K,
                                                                accumulate ? 1 : 0);
    DFLASH_CHECK_LAUNCH();
    return DFLASH_OK;
}

// ------------------------------------------------------------------------------------------
// split the fused projection into q, k, v and rotate q and k (rotate-half pairing)
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void rope_split_kernel(const float* __restrict__ qkv, const int32_t* __restrict__ ctx_len,
                                  int rows_per_seq, T* __restrict__ q, T* __restrict__ k,
                                  T* __restrict__ v, int Hq, int Hkv, int hd, int use_rope,
                                  const float* __restrict__ cs, const float* __restrict__ sn, int max_pos,
                                  int32_t* status, const T* __restrict__ gq, const T* __restrict__ gk, float eps) {
    __shared__ float rnorm[128];          // per (q or k) head: rsqrt(mean square + eps), 1 without the head norm
    const int row = blockIdx.x, b = row / rows_per_seq, r = row % rows_per_seq;
    const int half = hd / 2;
    int pos = ctx_len[b] + r;
    if (use_rope && (pos < 0 || pos >= max_pos)) {
        if (threadIdx.x == 0 && status) atomicOr(status, DFLASH_DEV_CTX_OVERFLOW);
        pos = pos < 0 ? 0 : max_pos - 1;
    }
    const int qdim = Hq * hd, kdim = Hkv * hd;
    const float* src = qkv + (size_t)row * (qdim + 2 * kdim);
    for (int head = threadIdx.x >> 5; head < Hq + Hkv; head += blockDim.x >> 5) {     // one warp per head
        float s = 0.f;
        if (gq)
            for (int i = threadIdx.x & 31; i < hd; i += 32) s += src[head * hd + i] * src[head * hd + i];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if ((threadIdx.x & 31) == 0 && head < 128) rnorm[head] = gq ? rsqrtf(s / (float)hd + eps) : 1.f;
    }
    __syncthreads();
    // rotated part: q heads then k heads
    for (int e = threadIdx.x; e < (Hq + Hkv) * half; e += blockDim.x) {
        const int head = e / half, i = e % half;
        float a = src[head * hd + i], bb = src[head * hd + i + half];
        if (gq) {
            const T* g = head < Hq ? gq : gk;
            a *= rnorm[head] * to_f(g[i]);
            bb *= rnorm[head] * to_f(g[i + half]);
        }
        float c = 1.f, s = 0.f;
        if (use_rope) { c = cs[(size_t)pos * half + i]; s = sn[(size_t)pos * half + i]; }
        const float o1 = a * c - bb * s, o2 = bb * c + a * s;
        if (head < Hq) {
            q[(size_t)row * qdim + head * hd + i] = from_f<T>(o1);
            q[(size_t)row * qdim + head * hd + i + half] = from_f<T>(o2);
        } else {
            const int kh = head - Hq;
            k[(size_t)row * kdim + kh * hd + i] = from_f<T>(o1);
            k[(size_t)row * kdim + kh * hd + i + half] = from_f<T>(o2);
        }
    }
    for (int e = threadIdx.x; e < kdim; e += blockDim.x)
        v[(size_t)row * kdim + e] = from_f<T>(src[qdim + kdim + e]);
}

int launch_rope_split(const Launch& L, const float* qkv, const int32_t* ctx_len, int rows_per_seq, int rows,
                      void* q, void* k, void* v, const void* g_q, const void* g_k) {
    const dflash_config& c = L.h->cfg;
    if (rows == 0) return DFLASH_OK;
    if (g_q && c.n_q_heads + c.n_kv_heads > 128) return DFLASH_ERR_UNSUPPORTED;
    if (c.dtype == DFLASH_F32)
        rope_split_kernel<float><<<rows, 256, 0, L.st>>>(qkv, ctx_len, rows_per_seq, (float*)q, (float*)k,
                                                         (float*)v, c.n_q_heads, c.n_kv_heads, c.head_dim,
                                                         c.use_rope, L.h->w.rope_cos, L.h->w.rope_sin,
                                                         L.h->w.rope_max_pos, L.status, (const float*)g_q, (const float*)g_k,
                                                         c.rms_eps);
    else
        rope_split_kernel<__nv_bfloat16><<<rows, 256, 0, L.st>>>(
            qkv, ctx_len, rows_per_seq, (__nv_bfloat16*)q, (__nv_bfloat16*)k, (__nv_bfloat16*)v, c.n_q_heads,
            c.n_kv_heads, c.head_dim, c.use_rope, L.h->w.rope_cos, L.h->w.rope_sin, L.h->w.rope_max_pos,
            L.status, (const __nv_bfloat16*)g_q, (const __nv_bfloat16*)g_k, c.rms_eps);
    DFLASH_CHECK_LAUNCH();
    return DFLASH_OK;
}

// ------------------------------------------------------------------------------------------
// SwiGLU on the interleaved gate/up projection: h_j = silu(gu[2j]) * gu[2j+1]
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void swiglu_kernel(const float* __restrict__ gu, T* __restrict__ h, int64_t n) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const float g = gu[2 * i], u = gu[2 * i + 1];
    h[i] = from_f<T>(g / (1.f + __expf(-g)) * u);
}

int launch_swiglu(const Launch& L, const float* gu, void* h, int rows) {
    const dflash_config& c = L.h->cfg;
    const int64_t n = (int64_t)rows * c.d_ffn;
    if (n == 0) return DFLASH_OK;
    const int grid = (int)((n + 255) / 256);
    if (c.dtype == DFLASH_F32) swiglu_kernel<float><<<grid, 256, 0, L.st>>>(gu, (float*)h, n);
    else swiglu_kernel<__nv_bfloat16><<<grid, 256, 0, L.st>>>(gu, (__nv_bfloat16*)h, n);
    DFLASH_CHECK_LAUNCH();
    return DFLASH_OK;
}

// ------------------------------------------------------------------------------------------
// attention over [paged context ; block] on CUDA cores: one CTA per (row, q head, sequence),
// keys in chunks of 128 with a running (max, sum) softmax.
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(128) attention_simt_kernel(
    const T* __restrict__ q, const T* __restrict__ k_blk, const T* __restrict__ v_blk,
    const T* __restrict__ pool, const int32_t* __restrict__ page_table, const int32_t* __restrict__ ctx_len,
    T* __restrict__ out, int R, int Hq, int Hkv, int hd, int PG, int max_pages, int n_pages, int layer,
    float scale, int causal, int32_t* status, float* __restrict__ lse) {
    __shared__ float sq[128];
    __shared__ float sp[128];
    __shared__ float red[32];
    const int r = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int kvh = h / (Hq / Hkv);
    const int tid = threadIdx.x;
    const int L = ctx_len[b];
    const int n_keys = L + R;
    const size_t row = (size_t)b * R + r;
    if (tid < hd) sq[tid] = to_f(q[(row * Hq + h) * hd + tid]) * scale;
    __syncthreads();

    float m = -CUDART_INF_F, l = 0.f, acc = 0.f;
    for (int j0 = 0; j0 < n_keys; j0 += 128) {
        const int j = j0 + tid;
        const T* kp = nullptr;
        const T* vp = nullptr;
        if (j < L) {
            const int pidx = j / PG;
            const int page = pidx < max_pages ? page_table[(size_t)b * max_pages + pidx] : -1;
            if (page >= 0 && page < n_pages) {
                const size_t base = ((((size_t)layer * n_pages + page) * 2) * Hkv + kvh) * PG * hd;
                kp = pool + base + (size_t)(j % PG) * hd;
                vp = kp + (size_t)Hkv * PG * hd;
            } else if (status) {
                atomicOr(status, DFLASH_DEV_BAD_PAGE);
            }
        } else if (j < n_keys) {
            const int rr = j - L;
            if (!causal || rr <= r) {
                kp = k_blk + (((size_t)b * R + rr) * Hkv + kvh) * hd;
                vp = v_blk + (((size_t)b * R + rr) * Hkv + kvh) * hd;
            }
        }
        float s = -CUDART_INF_F;
        if (kp) {
            float d = 0.f;
            for (int e = 0; e < hd; ++e) d = fmaf(sq[e], to_f(kp[e]), d);
            s = d;
        }
        const float cmax = block_max(s, red);
        const float m_new = fmaxf(m, cmax);          // finite: every chunk holds >= 1 visible key or m stays
        float p = 0.f, corr = 1.f;
        if (m_new > -CUDART_INF_F) {
            p = kp ? __expf(s - m_new) : 0.f;
            corr = (m > -CUDART_INF_F) ? __expf(m - m_new) : 0.f;
        }
        sp[tid] = p;
        const float psum = block_sum(p, red);         // contains __syncthreads: sp is visible after it
        l = l * corr + psum;
        m = m_new;
        // thread d accumulates output component d over the chunk's keys
        if (tid < hd) {
            float a = acc * corr;
            const int lim = min(128, n_keys - j0);
            for (int jj = 0; jj < lim; ++jj) {
                const float pj = sp[jj];
                if (pj == 0.f) continue;
                const int jg = j0 + jj;
                const T* vv;
                if (jg < L) {
                    const int page = page_table[(size_t)b * max_pages + jg / PG];
                    vv = pool + (((((size_t)layer * n_pages + page) * 2 + 1) * Hkv + kvh) * PG + (jg % PG)) * hd;
                } else {
                    vv = v_blk + (((size_t)b * R + (jg - L)) * Hkv + kvh) * hd;
                }
                a = fmaf(pj, to_f(vv[tid]), a);
            }
            acc = a;
        }
        __syncthreads();
    }
    if (tid < hd) out[(row * Hq + h) * hd + tid] = from_f<T>(l > 0.f ? acc / l : 0.f);
    if (lse && tid == 0) lse[row * Hq + h] = l > 0.f ? m + logf(l) : -CUDART_INF_F;
}

int launch_attention_simt(const Launch& L, const dflash_attn_args& a) {
    const dflash_config& c = L.h->cfg;
    if (a.batch == 0 || a.rows == 0) return DFLASH_OK;
    dim3 grid(a.rows, c.n_q_heads, a.batch);
    const int causal = a.mode == DFLASH_ATTN_CAUSAL ? 1 : 0;
    if (c.dtype == DFLASH_F32)
        attention_simt_kernel<float><<<grid, 128, 0, L.st>>>(
            (const float*)a.q, (const float*)a.k_blk, (const float*)a.v_blk, (const float*)a.kv_pool,
            a.page_table, a.ctx_len, (float*)a.out, a.rows, c.n_q_heads, c.n_kv_heads, c.head_dim, c.page_size,
            a.max_pages, a.n_pool_pages, a.layer, c.softmax_scale, causal, L.status, a.lse_out);
    else
        attention_simt_kernel<__nv_bfloat16><<<grid, 128, 0, L.st>>>(
            (const __nv_bfloat16*)a.q, (const __nv_bfloat16*)a.k_blk, (const __nv_bfloat16*)a.v_blk,
            (const __nv_bfloat16*)a.kv_pool, a.page_table, a.ctx_len, (__nv_bfloat16*)a.out, a.rows,
            c.n_q_heads, c.n_kv_heads, c.head_dim, c.page_size, a.max_pages, a.n_pool_pages, a.layer,
            c.softmax_scale, causal, L.status, a.lse_out);
    DFLASH_CHECK_LAUNCH();
    return DFLASH_OK;
}

// ------------------------------------------------------------------------------------------
// context K/V of one layer: rotate K, scatter K and V into the paged pool
// kv: [rows, 2*Hkv*hd] fp32 (K heads then V heads)
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void ctx_scatter_kernel(const float* __restrict__ kv, const int32_t* __restrict__ n_new,
                                   const int32_t* __restrict__ ctx_len, const int32_t* __restrict__ page_table,
                                   T* __restrict__ pool, int max_new, int Hkv, int hd, int PG, int max_pages,
                                   int n_pages, int layer, int use_rope, const float* __restrict__ cs,
                                   const float* __restrict__ sn, int max_pos, int32_t* status,
                                   const T* __restrict__ gk, float eps) {
    __shared__ float rnorm[128];
    const int row = blockIdx.x, b = row / max_new, r = row % max_new;
    const int nn = n_new ? n_new[b] : max_new;
    if (r >= nn) return;
    const int pos = ctx_len[b] + r;
    const int pidx = pos / PG;
    if (pos < 0 || pidx >= max_pages || (use_rope && pos >= max_pos)) {
        if (threadIdx.x == 0 && status) atomicOr(status, DFLASH_DEV_CTX_OVERFLOW);
        return;
    }
    const int page = page_table[(size_t)b * max_pages + pidx];
    if (page < 0 || page >= n_pages) {
        if (threadIdx.x == 0 && status) atomicOr(status, DFLASH_DEV_BAD_PAGE);
        return;
    }
    const int half = hd / 2, kdim = Hkv * hd;
    const float* src = kv + (size_t)row * 2 * kdim;
    T* kdst = pool + ((((size_t)layer * n_pages + page) * 2) * Hkv) * PG * hd + (size_t)(pos % PG) * hd;
    T* vdst = kdst + (size_t)Hkv * PG * hd;
    for (int head = threadIdx.x >> 5; head < Hkv; head += blockDim.x >> 5) {          // one warp per key head
        float s = 0.f;
        if (gk)
            for (int i = threadIdx.x & 31; i < hd; i += 32) s += src[head * hd + i] * src[head * hd + i];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if ((threadIdx.x & 31) == 0 && head < 128) rnorm[head] = gk ? rsqrtf(s / (float)hd + eps) : 1.f;
    }
    __syncthreads();
    for (int e = threadIdx.x; e < Hkv * half; e += blockDim.x) {
        const int head = e / half, i = e % half;
        float a = src[head * hd + i], bb = src[head * hd + i + half];
        if (gk) {
            a *= rnorm[head] * to_f(gk[i]);
            bb *= rnorm[head] * to_f(gk[i + half]);
        }
        float c = 1.f, s = 0.f;
        if (use_rope) { c = cs[(size_t)pos * half + i]; s = sn[(size_t)pos * half + i]; }
        kdst[(size_t)head * PG * hd + i] = from_f<T>(a * c - bb * s);
        kdst[(size_t)head * PG * hd + i + half] = from_f<T>(bb * c + a * s);
    }
    for (int e = threadIdx.x; e < kdim; e += blockDim.x) {
        const int head = e / hd, i = e % hd;
        vdst[(size_t)head * PG * hd + i] = from_f<T>(src[kdim + e]);
    }
}

int launch_ctx_scatter(const Launch& L, const float* kv, const dflash_ctx_args& a, int layer, const void* g_k) {
    const dflash_config& c = L.h->cfg;
    const int rows = a.batch * a.max_new;
    if (rows == 0) return DFLASH_OK;
    if (c.dtype == DFLASH_F32)
        ctx_scatter_kernel<float><<<rows, 128, 0, L.st>>>(
            kv, a.n_new, a.ctx_len, a.page_table, (float*)a.kv_pool, a.max_new, c.n_kv_heads, c.head_dim,
            c.page_size, a.max_pages, a.n_pool_pages, layer, c.use_rope, L.h->w.rope_cos, L.h->w.rope_sin,
            L.h->w.rope_max_pos, L.status, (const float*)g_k, c.rms_eps);
    else
        ctx_scatter_kernel<__nv_bfloat16><<<rows, 128, 0, L.st>>>(
            kv, a.n_new, a.ctx_len, a.page_table, (__nv_bfloat16*)a.kv_pool, a.max_new, c.n_kv_heads,
            c.head_dim, c.page_size, a.max_pages, a.n_pool_pages, layer, c.use_rope, L.h->w.rope_cos,
            L.h->w.rope_sin, L.h->w.rope_max_pos, L.status, (const __nv_bfloat16*)g_k, c.rms_eps);
    DFLASH_CHECK_LAUNCH();
    return DFLASH_OK;
}

// ------------------------------------------------------------------------------------------
// row-wise argmax with runner-up: lowest index among equal maxima, NaN never wins
// ------------------------------------------------------------------------------------------
struct Top2 {
    float v1; int i1; float v2;
};
__device__ __forceinline__ void top2_push(Top2& t, float v, int i) {
    if (v > t.v1 || (v == t.v1 && i < t.i1)) { t.v2 = t.v1; t.v1 = v; t.i1 = i; }
    else if (v > t.v2) t.v2 = v;
}
__device__ __forceinline__ Top2 top2_merge(const Top2& a, const Top2& b) {
    Top2 r;
    if (b.v1 > a.v1 || (b.v1 == a.v1 && b.i1 < a.i1)) { r.v1 = b.v1; r.i1 = b.i1; r.v2 = fmaxf(a.v1, b.v2); }
    else { r.v1 = a.v1; r.i1 = a.i1; r.v2 = fmaxf(a.v2, b.v1); }
    return r;
}

// Stage 1: grid (segments, rows). Each CTA scans one contiguous segment of one row with 16-byte
// loads (scalar at a misaligned head/tail) and writes that segment's (max, index, runner-up).
// V2: also track the runner-up value (for the margin). Without it (the accept step only needs the winner) the scan
// is one compare and two selects per entry, which keeps the kernel memory-bound: the compare-and-shift chain of the
// top-2 update was measured at 82 % instruction-issue utilisation and 31 % of DRAM bandwidth.
// Scans entries [lo, hi) of a row with 16-byte loads (scalar at a misaligned head / tail), all 256 threads of the
// CTA; the CTA's result is returned by thread 0 (sh: 8 entries of shared memory).
template <typename T, bool V2>
__device__ __forceinline__ Top2 scan_segment(const T* __restrict__ src, int lo, int hi, Top2* sh) {
    constexpr int VEC = 16 / (int)sizeof(T);
    Top2 t{-CUDART_INF_F, 0x7fffffff, -CUDART_INF_F};
    if (lo < hi) {
        // first index at or after lo whose address is 16-byte aligned
        const uintptr_t addr = reinterpret_cast<uintptr_t>(src + lo);
        int head = (int)(((16 - (addr & 15)) & 15) / sizeof(T));
        head = min(head, hi - lo);
        const int body = (hi - lo - head) / VEC;
        for (int i = threadIdx.x; i < head; i += blockDim.x) top2_push(t, to_f(src[lo + i]), lo + i);
        const uint4* v = reinterpret_cast<const uint4*>(src + lo + head);
        // four 16-byte loads in flight per thread: a long segment (few segments per row when there are many rows) is
        // otherwise one dependent load after the other
        constexpr int INFL = 4;
        int i = threadIdx.x;
        for (; i + (INFL - 1) * (int)blockDim.x < body; i += INFL * blockDim.x) {
            uint4 w[INFL];
#pragma unroll
            for (int u = 0; u < INFL; ++u) w[u] = __ldg(v + i + u * blockDim.x);
#pragma unroll
            for (int u = 0; u < INFL; ++u) {
                const T* e = reinterpret_cast<const T*>(&w[u]);
                const int base = lo + head + (i + u * (int)blockDim.x) * VEC;
                if constexpr (V2) {
#pragma unroll
                    for (int k = 0; k < VEC; ++k) top2_push(t, to_f(e[k]), base + k);
                } else {      // rising index order inside a thread: strictly greater keeps the lowest index; NaN never wins
#pragma unroll
                    for (int k = 0; k < VEC; ++k) {
                        const float x = to_f(e[k]);
                        const bool up = x > t.v1;
                        t.v1 = up ? x : t.v1;
                        t.i1 = up ? base + k : t.i1;
                    }
                }
            }
        }
        for (; i < body; i += blockDim.x) {
            const uint4 w = __ldg(v + i);
            const T* e = reinterpret_cast<const T*>(&w);
            const int base = lo + head + i * VEC;
#pragma unroll
            for (int k = 0; k < VEC; ++k) top2_push(t, to_f(e[k]), base + k);
        }
        for (int i = lo + head + body * VEC + threadIdx.x; i < hi; i += blockDim.x) top2_push(t, to_f(src[i]), i);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Top2 u;
        u.v1 = __shfl_xor_sync(0xffffffffu, t.v1, o);
        u.i1 = __shfl_xor_sync(0xffffffffu, t.i1, o);
        u.v2 = __shfl_xor_sync(0xffffffffu, t.v2, o);
        t = top2_merge(t, u);
    }
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (lane == 0) sh[w] = t;
    __syncthreads();
    Top2 r = sh[0];
    if (threadIdx.x == 0)
        for (int i = 1; i < (int)(blockDim.x >> 5); ++i) r = top2_merge(r, sh[i]);
    return r;
}

template <typename T, bool V2>
__global__ void __launch_bounds__(256) row_argmax_seg_kernel(const T* __restrict__ logits, int64_t row_stride,
                                                             int vocab, int seg_len, float4* __restrict__ out) {
    __shared__ Top2 sh[8];
    ptx::pdl_trigger();
    ptx::pdl_wait();      // the scratch written below may alias what the previous kernel still uses
    const int seg = blockIdx.x, nseg = gridDim.x, row = blockIdx.y;
    const int lo = seg * seg_len, hi = min(vocab, lo + seg_len);
    const Top2 r = scan_segment<T, V2>(logits + (size_t)row * row_stride, lo, hi, sh);
    if (threadIdx.x == 0) out[(size_t)row * nseg + seg] = make_float4(r.v1, __int_as_float(r.i1), r.v2, 0.f);
}

// Stage 2: one warp per row merges the segments.
__global__ void __launch_bounds__(256) row_argmax_merge_kernel(const float4* __restrict__ seg, int nseg, int rows,
                                                               int32_t* __restrict__ ids, float* __restrict__ top1,
                                                               float* __restrict__ margin) {
    ptx::pdl_trigger();
    ptx::pdl_wait();
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= rows) return;
    const int lane = threadIdx.x & 31;
    Top2 t{-CUDART_INF_F, 0x7fffffff, -CUDART_INF_F};
    for (int i = lane; i < nseg; i += 32) {
        const float4 e = seg[(size_t)row * nseg + i];
        t = top2_merge(t, Top2{e.x, __float_as_int(e.y), e.z});
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Top2 u;
        u.v1 = __shfl_xor_sync(0xffffffffu, t.v1, o);
        u.i1 = __shfl_xor_sync(0xffffffffu, t.i1, o);
        u.v2 = __shfl_xor_sync(0xffffffffu, t.v2, o);
        t = top2_merge(t, u);
    }
    if (lane == 0) {
        ids[row] = (t.i1 == 0x7fffffff) ? 0 : t.i1;      // nothing compared greater than -inf
        if (top1) top1[row] = t.v1;
        if (margin) margin[row] = t.v1 - t.v2;
    }
}

int row_argmax_segments(int rows, int vocab, int sm_count) {
    int nseg = (4 * sm_count + rows - 1) / std::max(rows, 1);
    nseg = std::max(1, std::min(nseg, 64));
    nseg = std::min(nseg, std::max(1, vocab / 2048));
    return std::max(nseg, 1);
}

int launch_row_argmax(const Launch& L, const void* logits, int dtype, int64_t row_stride, int rows, int vocab,
                      float4* seg_scratch, int32_t* ids, float* top1, float* margin) {
    if (rows == 0) return DFLASH_OK;
    const int nseg = row_argmax_segments(rows, vocab, L.h->sm_count);
    const int seg_len = ((vocab + nseg - 1) / nseg + 7) / 8 * 8;
    dim3 grid(nseg, rows);
    // programmatic dependent launch: each kernel's blocks become resident while its predecessor drains
    cudaError_t e;
    if (dtype == DFLASH_F32)
        e = launch_pdl(row_argmax_seg_kernel<float, true>, grid, dim3(256), 0, L.st, (const float*)logits, row_stride, vocab, seg_len,
                       seg_scratch);
    else
        e = launch_pdl(row_argmax_seg_kernel<__nv_bfloat16, true>, grid, dim3(256), 0, L.st, (const __nv_bfloat16*)logits, row_stride,
                       vocab, seg_len, seg_scratch);
    ++g_launches;
    if (e != cudaSuccess) return DFLASH_ERR_CUDA;
    e = launch_pdl(row_argmax_merge_kernel, dim3((rows + 7) / 8), dim3(256), 0, L.st, (const float4*)seg_scratch, nseg, rows, ids,
                   top1, margin);
    ++g_launches;
    if (e != cudaSuccess) return DFLASH_ERR_CUDA;
    return DFLASH_OK;
}

// ------------------------------------------------------------------------------------------
// accept rule (Sec. 3.1): longest agreeing prefix + bonus token, one thread per sequence
// ------------------------------------------------------------------------------------------
__global__ void accept_kernel(const int32_t* __restrict__ target_ids, const int32_t* __restrict__ draft_ids,
                              int draft_stride, int batch, int gamma, const int32_t* ctx_len,
                              int32_t* __restrict__ accept_len, int32_t* __restrict__ out_tokens,
                              int32_t* __restrict__ bonus, int32_t* new_ctx_len,
                              int32_t* __restrict__ target_ids_out) {      // new_ctx_len may alias ctx_len: neither is restrict
    ptx::pdl_trigger();
    ptx::pdl_wait();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= batch) return;
    const int32_t* p = target_ids + (size_t)b * (gamma + 1);
    const int32_t* d = draft_ids + (size_t)b * draft_stride;
    int a = 0;
    while (a < gamma && d[a] == p[a]) ++a;
    int32_t* o = out_tokens + (size_t)b * (gamma + 1);
    for (int i = 0; i <= gamma; ++i) o[i] = i < a ? d[i] : (i == a ? p[a] : -1);
    const int32_t len = ctx_len[b];
    accept_len[b] = a + 1;
    bonus[b] = p[a];
    new_ctx_len[b] = len + a + 1;
    if (target_ids_out && target_ids_out != target_ids)
        for (int i = 0; i <= gamma; ++i) target_ids_out[(size_t)b * (gamma + 1) + i] = p[i];
}

int launch_accept(const Launch& L, const dflash_verify_args& a, const int32_t* target_ids) {
    if (a.batch == 0) return DFLASH_OK;
    const cudaError_t e = launch_pdl(accept_kernel, dim3((a.batch + 127) / 128), dim3(128), 0, L.st, target_ids, a.draft_ids,
                                     a.draft_stride, a.batch, a.gamma, a.ctx_len, a.accept_len, a.out_tokens, a.bonus,
                                     a.new_ctx_len, a.target_ids_out);
    ++g_launches;
    if (e != cudaSuccess) return DFLASH_ERR_CUDA;
    return DFLASH_OK;
}

// Merges the segments of the gamma + 1 rows of sequence b (a warp per row) and applies the accept rule (one thread).
__device__ __forceinline__ void merge_and_accept(const float4* seg, int nseg, int b, const int32_t* __restrict__ draft_ids, int draft_stride,
                                                 int gamma, const int32_t* ctx_len, int32_t* __restrict__ accept_len,
                                                 int32_t* __restrict__ out_tokens, int32_t* __restrict__ bonus, int32_t* new_ctx_len,
                                                 int32_t* __restrict__ target_ids_out, int32_t* s_p) {
    const int lane = threadIdx.x & 31;
    const int n_warps = blockDim.x >> 5;
    // A warp takes rows w, w + n_warps, ...: the entries of up to RB of its rows are requested together (one round
    // trip through L2 instead of one per row; up to 64 segments per row = two entries per lane).
    constexpr int RB = 3;
    for (int j0 = threadIdx.x >> 5; j0 <= gamma; j0 += RB * n_warps) {
        float4 e0[RB], e1[RB];
#pragma unroll
        for (int u = 0; u < RB; ++u) {
            const int j = j0 + u * n_warps;
            const size_t row = (size_t)b * (gamma + 1) + j;
            const float4 none = make_float4(-CUDART_INF_F, __int_as_float(0x7fffffff), -CUDART_INF_F, 0.f);
            e0[u] = (j <= gamma && lane < nseg) ? __ldcg(seg + row * nseg + lane) : none;
            e1[u] = (j <= gamma && lane + 32 < nseg) ? __ldcg(seg + row * nseg + lane + 32) : none;
        }
#pragma unroll
        for (int u = 0; u < RB; ++u) {
        const int j = j0 + u * n_warps;
        if (j > gamma) break;
        const size_t row = (size_t)b * (gamma + 1) + j;
        Top2 t{e0[u].x, __float_as_int(e0[u].y), e0[u].z};
        t = top2_merge(t, Top2{e1[u].x, __float_as_int(e1[u].y), e1[u].z});
        for (int i = lane + 64; i < nseg; i += 32) {      // (never with the segment counts the launches choose)
            const float4 e = __ldcg(seg + row * nseg + i);
            t = top2_merge(t, Top2{e.x, __float_as_int(e.y), e.z});
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            Top2 u;
            u.v1 = __shfl_xor_sync(0xffffffffu, t.v1, o);
            u.i1 = __shfl_xor_sync(0xffffffffu, t.i1, o);
            u.v2 = __shfl_xor_sync(0xffffffffu, t.v2, o);
            t = top2_merge(t, u);
        }
        if (lane == 0) {
            const int32_t id = (t.i1 == 0x7fffffff) ? 0 : t.i1;      // nothing compared greater than -inf
            s_p[j] = id;
            if (target_ids_out) target_ids_out[row] = id;
        }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const int32_t* d = draft_ids + (size_t)b * draft_stride;
        const int32_t len = ctx_len[b];      // new_ctx_len may alias ctx_len: read before anything is written
        int a = 0;
        while (a < gamma && d[a] == s_p[a]) ++a;
        int32_t* o = out_tokens + (size_t)b * (gamma + 1);
        for (int i = 0; i <= gamma; ++i) o[i] = i < a ? d[i] : (i == a ? s_p[a] : -1);
        accept_len[b] = a + 1;
        bonus[b] = s_p[a];
        new_ctx_len[b] = len + a + 1;
    }
}

// Second launch of the two-launch form (more sequences than tickets): one CTA per sequence.
__global__ void __launch_bounds__(256) argmax_accept_kernel(const float4* __restrict__ seg, int nseg,
                                                            const int32_t* __restrict__ draft_ids, int draft_stride, int gamma,
                                                            const int32_t* ctx_len, int32_t* __restrict__ accept_len,
                                                            int32_t* __restrict__ out_tokens, int32_t* __restrict__ bonus,
                                                            int32_t* new_ctx_len, int32_t* __restrict__ target_ids_out) {
    __shared__ int32_t s_p[65];
    ptx::pdl_trigger();
    ptx::pdl_wait();
    merge_and_accept(seg, nseg, blockIdx.x, draft_ids, draft_stride, gamma, ctx_len, accept_len, out_tokens, bonus, new_ctx_len,
                     target_ids_out, s_p);
}

// Greedy verification from logits in ONE launch: every CTA scans one segment of one row; the CTA that takes the last
// ticket of its sequence merges the sequence's segments and applies the accept rule. The tickets live in the library
// image (zero at load); atomicInc wraps the last ticket back to zero, so a call leaves them as it found them. Calls
// that overlap on one GPU would mix their tickets: like every call of the library, verify calls run one after the other.
constexpr int VERIFY_TICKETS = 4096;      // sequences per call on this path (more take the two-launch path)
__device__ unsigned int g_verify_tickets[VERIFY_TICKETS];

template <typename T>
__global__ void __launch_bounds__(256) verify_fused_kernel(const T* __restrict__ logits, int64_t row_stride, int vocab, int seg_len,
                                                           float4* seg_out, const int32_t* __restrict__ draft_ids, int draft_stride,
                                                           int gamma, const int32_t* ctx_len, int32_t* __restrict__ accept_len,
                                                           int32_t* __restrict__ out_tokens, int32_t* __restrict__ bonus,
                                                           int32_t* new_ctx_len, int32_t* __restrict__ target_ids_out,
                                                           unsigned long long* trace) {
    __shared__ Top2 sh[8];
    __shared__ int32_t s_p[65];
    __shared__ int s_last;
    if (threadIdx.x == 0) ptx::trace_min(trace, 0);
    ptx::pdl_trigger();
    ptx::pdl_wait();
    if (threadIdx.x == 0) ptx::trace_min(trace, 1);
    const int seg = blockIdx.x, nseg = gridDim.x, row = blockIdx.y;
    const int b = row / (gamma + 1);
    const int lo = seg * seg_len, hi = min(vocab, lo + seg_len);
    const Top2 r = scan_segment<T, false>(logits + (size_t)row * row_stride, lo, hi, sh);
    if (threadIdx.x == 0) {
        seg_out[(size_t)row * nseg + seg] = make_float4(r.v1, __int_as_float(r.i1), r.v2, 0.f);
        // one ticket with release (this CTA's result) and acquire (the results of the CTAs before it) semantics; the
        // barrier below hands what thread 0 acquired to the rest of the CTA
        const unsigned int n = (unsigned int)nseg * (unsigned int)(gamma + 1);
        unsigned int old;
        asm volatile("atom.acq_rel.gpu.global.inc.u32 %0, [%1], %2;" : "=r"(old) : "l"(&g_verify_tickets[b]), "r"(n - 1) : "memory");
        s_last = old == n - 1 ? 1 : 0;
    }
    __syncthreads();
    if (!s_last) {
        if (threadIdx.x == 0) ptx::trace_max(trace, 3);
        return;
    }
    merge_and_accept(seg_out, nseg, b, draft_ids, draft_stride, gamma, ctx_len, accept_len, out_tokens, bonus, new_ctx_len,
                     target_ids_out, s_p);
    __syncthreads();
    if (threadIdx.x == 0) ptx::trace_max(trace, 3);
}

int launch_verify_logits(const Launch& L, const dflash_verify_args& a, int64_t row_stride, float4* seg_scratch) {
    if (a.batch == 0) return DFLASH_OK;
    if (a.gamma > 64) return DFLASH_ERR_INVALID_ARG;
    const int rows = a.batch * (a.gamma + 1);
    const int nseg = row_argmax_segments(rows, a.vocab, L.h->sm_count);
    const int seg_len = ((a.vocab + nseg - 1) / nseg + 7) / 8 * 8;
    dim3 grid(nseg, rows);
    cudaError_t e;
    if (a.batch <= VERIFY_TICKETS) {
        if (a.logits_dtype == DFLASH_F32)
            e = launch_pdl(verify_fused_kernel<float>, grid, dim3(256), 0, L.st, (const float*)a.logits, row_stride, a.vocab, seg_len,
                           seg_scratch, a.draft_ids, a.draft_stride, a.gamma, a.ctx_len, a.accept_len, a.out_tokens, a.bonus,
                           a.new_ctx_len, a.target_ids_out, L.trace);
        else
            e = launch_pdl(verify_fused_kernel<__nv_bfloat16>, grid, dim3(256), 0, L.st, (const __nv_bfloat16*)a.logits, row_stride,
                           a.vocab, seg_len, seg_scratch, a.draft_ids, a.draft_stride, a.gamma, a.ctx_len, a.accept_len, a.out_tokens,
                           a.bonus, a.new_ctx_len, a.target_ids_out, L.trace);
        ++g_launches;
        return e == cudaSuccess ? DFLASH_OK : DFLASH_ERR_CUDA;
    }
    if (a.logits_dtype == DFLASH_F32)
        e = launch_pdl(row_argmax_seg_kernel<float, false>, grid, dim3(256), 0, L.st, (const float*)a.logits, row_stride, a.vocab, seg_len,
                       seg_scratch);
    else
        e = launch_pdl(row_argmax_seg_kernel<__nv_bfloat16, false>, grid, dim3(256), 0, L.st, (const __nv_bfloat16*)a.logits, row_stride,
                       a.vocab, seg_len, seg_scratch);
    ++g_launches;
    if (e != cudaSuccess) return DFLASH_ERR_CUDA;
    e = launch_pdl(argmax_accept_kernel, dim3(a.batch), dim3(256), 0, L.st, (const float4*)seg_scratch, nseg, a.draft_ids,
                   a.draft_stride, a.gamma, a.ctx_len, a.accept_len, a.out_tokens, a.bonus, a.new_ctx_len, a.target_ids_out);
    ++g_launches;
    return e == cudaSuccess ? DFLASH_OK : DFLASH_ERR_CUDA;
}

// Zeroing as a kernel (not a memset) so that it takes part in programmatic dependent launch: its
// blocks are resident while the previous call's last kernel drains, and the kernel after it chains on.
// It releases its dependents only after its own wait: every kernel of this call therefore starts after
// all work queued before the call has ended, which is what lets later kernels of the call read data of
// earlier calls (the cached context) ahead of their own grid dependency.
__global__ void __launch_bounds__(256) zero_kernel(uint4* __restrict__ dst, int64_t n16) {
    ptx::pdl_wait();          // the tickets may still be read by the previous kernel
    ptx::pdl_trigger();
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += (int64_t)gridDim.x * blockDim.x)
        dst[i] = make_uint4(0, 0, 0, 0);
}
int launch_zero(const Launch& L, void* dst, int64_t bytes) {      // dst 16-byte aligned, bytes a multiple of 16
    if (bytes <= 0) return DFLASH_OK;
    const int64_t n16 = bytes / 16;
    const int grid = (int)std::min<int64_t>((n16 + 255) / 256, 64);
    const cudaError_t e = launch_pdl(zero_kernel, dim3(grid), dim3(256), 0, L.st, reinterpret_cast<uint4*>(dst), n16);
    ++g_launches;
    return e == cudaSuccess ? DFLASH_OK : DFLASH_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------
// the target's verify pass: block K/V into its cache, tapped hidden rows into the drafter's operand
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(128) kv_commit_kernel(const T* __restrict__ k_blk, const T* __restrict__ v_blk, int rows_per_seq,
                                                        const int32_t* __restrict__ ctx_len, const int32_t* __restrict__ page_table,
                                                        int max_pages, T* __restrict__ pool, int n_pages, int layer, int Hkv, int hd,
                                                        int PG, int32_t* status) {
    ptx::pdl_trigger();
    ptx::pdl_wait();
    const int row = blockIdx.x, b = row / rows_per_seq, r = row % rows_per_seq;
    const int pos = ctx_len[b] + r, pidx = pos / PG;
    if (pos < 0 || pidx >= max_pages) {
        if (threadIdx.x == 0 && status) atomicOr(status, DFLASH_DEV_CTX_OVERFLOW);
        return;
    }
    const int page = page_table[(size_t)b * max_pages + pidx];
    if (page < 0 || page >= n_pages) {
        if (threadIdx.x == 0 && status) atomicOr(status, DFLASH_DEV_BAD_PAGE);
        return;
    }
    const int kdim = Hkv * hd;
    T* kdst = pool + ((((size_t)layer * n_pages + page) * 2) * Hkv) * PG * hd + (size_t)(pos % PG) * hd;
    T* vdst = kdst + (size_t)Hkv * PG * hd;
    for (int e = threadIdx.x; e < kdim; e += blockDim.x) {
        const int head = e / hd, i = e % hd;
        kdst[(size_t)head * PG * hd + i] = k_blk[(size_t)row * kdim + e];
        vdst[(size_t)head * PG * hd + i] = v_blk[(size_t)row * kdim + e];
    }
}
int launch_kv_commit(const Launch& L, const void* k_blk, const void* v_blk, int batch, int rows_per_seq, const int32_t* ctx_len,
                     const int32_t* page_table, int max_pages, void* pool, int n_pages, int layer) {
    const dflash_config& c = L.h->cfg;
    const int rows = batch * rows_per_seq;
    if (rows == 0) return DFLASH_OK;
    cudaError_t e;
    if (c.dtype == DFLASH_F32)
        e = launch_pdl(kv_commit_kernel<float>, dim3(rows), dim3(128), 0, L.st, (const float*)k_blk, (const float*)v_blk, rows_per_seq,
                       ctx_len, page_table, max_pages, (float*)pool, n_pages, layer, c.n_kv_heads, c.head_dim, c.page_size, L.status);
    else
        e = launch_pdl(kv_commit_kernel<__nv_bfloat16>, dim3(rows), dim3(128), 0, L.st, (const __nv_bfloat16*)k_blk,
                       (const __nv_bfloat16*)v_blk, rows_per_seq, ctx_len, page_table, max_pages, (__nv_bfloat16*)pool, n_pages,
                       layer, c.n_kv_heads, c.head_dim, c.page_size, L.status);
    ++g_launches;
    return e == cudaSuccess ? DFLASH_OK : DFLASH_ERR_CUDA;
}

template <typename T>
__global__ void __launch_bounds__(256) tap_copy_kernel(const float* __restrict__ x, T* __restrict__ feats, int D, int ld_out, int off) {
    ptx::pdl_trigger();
    ptx::pdl_wait();
    const float* src = x + (size_t)blockIdx.x * D;
    T* dst = feats + (size_t)blockIdx.x * ld_out + off;
    for (int d = threadIdx.x; d < D; d += blockDim.x) dst[d] = from_f<T>(src[d]);
}
int launch_tap_copy(const Launch& L, const float* x, void* feats, int rows, int D, int ld_out, int off) {
    if (rows == 0) return DFLASH_OK;
    cudaError_t e;
    if (L.h->cfg.dtype == DFLASH_F32)
        e = launch_pdl(tap_copy_kernel<float>, dim3(rows), dim3(256), 0, L.st, x, (float*)feats, D, ld_out, off);
    else
        e = launch_pdl(tap_copy_kernel<__nv_bfloat16>, dim3(rows), dim3(256), 0, L.st, x, (__nv_bfloat16*)feats, D, ld_out, off);
    ++g_launches;
    return e == cudaSuccess ? DFLASH_OK : DFLASH_ERR_CUDA;
}

__global__ void copy_f32_kernel(const float* __restrict__ src, float* __restrict__ dst, int64_t n) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) dst[i] = src[i];
}
int launch_copy_f32(const Launch& L, const float* src, float* dst, int64_t n) {
    if (n == 0) return DFLASH_OK;
    copy_f32_kernel<<<(int)((n + 255) / 256), 256, 0, L.st>>>(src, dst, n);
    DFLASH_CHECK_LAUNCH();
    return DFLASH_OK;
}

}  // namespace dflash
