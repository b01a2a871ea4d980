// Row-wise softmax statistics over logits that sit in HBM, shared by the sampling calls and the
// training loss of a block: per (row, segment) the maximum and the sum of exponentials in one pass,
// and the merge of a row's segments by a group of lanes.
#pragma once

#include "dflash_internal.h"
#include "ptx_sm100.cuh"

#include <math_constants.h>

#include <algorithm>

namespace dflash {
namespace {

constexpr int MAX_STAT_SEG = 16;   // segments of a row's softmax statistics
constexpr float LOG2E = 1.4426950408889634f;

// 2^x by the special-function unit alone (2 ulp, results below 2^-126 flush to zero): for sums of many
// exponentials, where the library routine's extra range handling is most of a term's cost
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float as_f(float v) { return v; }
__device__ __forceinline__ float as_f(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float ld_logit(const void* row, int bf16, int i) {
    return bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(row)[i]) : reinterpret_cast<const float*>(row)[i];
}

// One set of rows: row r is row (r / group_rows) * group_pitch + r % group_rows of `logits`
// (the drafts of a sequence may be the first gamma of B stored rows).
struct StatsJob {
    const void* logits;
    int64_t row_stride;
    int32_t bf16, rows, group_rows, group_pitch;
};

// (max, sum of exp2((z - max) c)) of two partial results
__device__ __forceinline__ float2 stat_merge(float2 a, float2 b, float c) {
    const float m = fmaxf(a.x, b.x);
    if (m == -CUDART_INF_F) return make_float2(m, 0.f);
    return make_float2(m, a.y * exp2f((a.x - m) * c) + b.y * exp2f((b.x - m) * c));
}
// one more value into a running (max, sum)
__device__ __forceinline__ void stat_raise(float2& t, float m_new, float c) {      // the maximum grows to m_new
    if (m_new > t.x) {
        t.y = t.x > -CUDART_INF_F ? t.y * exp2f((t.x - m_new) * c) : 0.f;
        t.x = m_new;
    }
}

__device__ __forceinline__ void unpack16(const uint4& v, float (&f)[4], float) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
}
__device__ __forceinline__ void unpack16(const uint4& v, float (&f)[8], __nv_bfloat16) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        f[2 * k] = __uint_as_float(w[k] << 16);
        f[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
    }
}

// (max, sum) of entries [lo, hi) of one row by the CTA, in one pass: 16-byte loads (several per thread in
// flight) where the row allows it, a running (max, sum) per thread, one merge over the CTA at the end.
template <typename T>
__device__ __forceinline__ float2 segment_stats(const T* __restrict__ src, int lo, int hi, float c, float2* sh) {
    constexpr int VE = 16 / (int)sizeof(T), CH = 4;
    float2 t = make_float2(-CUDART_INF_F, 0.f);
    const bool vec = (reinterpret_cast<uintptr_t>(src + lo) & 15) == 0;
    const int n_vec = vec ? (hi - lo) / VE : 0;
    const uint4* vsrc = reinterpret_cast<const uint4*>(src + lo);
    for (int v0 = threadIdx.x; v0 < n_vec; v0 += blockDim.x * CH) {
        uint4 raw[CH];
#pragma unroll
        for (int k = 0; k < CH; ++k) {
            const int v = v0 + k * blockDim.x;
            raw[k] = v < n_vec ? vsrc[v] : make_uint4(0, 0, 0, 0);
        }
        float f[CH][VE];
        float m = -CUDART_INF_F;
#pragma unroll
        for (int k = 0; k < CH; ++k) {
            unpack16(raw[k], f[k], T());
            if (v0 + k * (int)blockDim.x < n_vec) {
#pragma unroll
                for (int e = 0; e < VE; ++e) m = fmaxf(m, f[k][e]);
            }
        }
        stat_raise(t, m, c);
        if (t.x > -CUDART_INF_F) {
#pragma unroll
            for (int k = 0; k < CH; ++k) {
                if (v0 + k * (int)blockDim.x < n_vec) {
#pragma unroll
                    for (int e = 0; e < VE; ++e) t.y += fast_exp2((f[k][e] - t.x) * c);
                }
            }
        }
    }
    for (int i = lo + n_vec * VE + threadIdx.x; i < hi; i += blockDim.x) {      // what 16-byte loads do not cover
        const float x = as_f(src[i]);
        stat_raise(t, x, c);
        if (t.x > -CUDART_INF_F) t.y += exp2f((x - t.x) * c);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        float2 u;
        u.x = __shfl_xor_sync(0xffffffffu, t.x, o);
        u.y = __shfl_xor_sync(0xffffffffu, t.y, o);
        t = stat_merge(t, u, c);
    }
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = t;
    __syncthreads();
    // every thread merges the warps' results: the maximum first, then one rescaled term per warp
    const int n_warps = (int)(blockDim.x >> 5);
    float m = sh[0].x;
    for (int w = 1; w < n_warps; ++w) m = fmaxf(m, sh[w].x);
    float z = 0.f;
    if (m > -CUDART_INF_F)
        for (int w = 0; w < n_warps; ++w) z += sh[w].y > 0.f ? sh[w].y * fast_exp2((sh[w].x - m) * c) : 0.f;
    return make_float2(m, z);
}

// grid (stat segments, rows of job 0 + rows of job 1): out[row][seg] = (max, sum of exp2((z - max) c)) of the segment
__global__ void __launch_bounds__(256) softmax_stats_kernel(StatsJob j0, StatsJob j1, int vocab, int seg_len, float c,
                                                            float2* __restrict__ out, int32_t* __restrict__ tickets, int n_tickets) {
    __shared__ float2 sh[8];
    ptx::pdl_trigger();
    ptx::pdl_wait();
    if (blockIdx.x == 0 && blockIdx.y == 0)
        for (int i = threadIdx.x; i < n_tickets; i += blockDim.x) tickets[i] = 0;
    const int seg = blockIdx.x, nseg = gridDim.x;
    int row = blockIdx.y;
    const bool second = row >= j0.rows;
    const StatsJob& j = second ? j1 : j0;
    if (second) row -= j0.rows;
    const size_t src_row = (size_t)(row / j.group_rows) * j.group_pitch + row % j.group_rows;
    const int lo = seg * seg_len, hi = min(vocab, lo + seg_len);
    float2 r;
    if (j.bf16) r = segment_stats(reinterpret_cast<const __nv_bfloat16*>(j.logits) + src_row * j.row_stride, lo, hi, c, sh);
    else r = segment_stats(reinterpret_cast<const float*>(j.logits) + src_row * j.row_stride, lo, hi, c, sh);
    if (threadIdx.x == 0) out[(size_t)blockIdx.y * nseg + seg] = r;
}

// whole-row (max, sum) from the segment results, by a group of LANES adjacent lanes of a warp (all 32
// lanes of the warp call it; `sub` = lane % LANES): the maximum first, then one rescaled term per segment
template <int LANES>
__device__ __forceinline__ float2 row_stat(const float2* seg, int nseg, float c, int sub) {
    constexpr int MAX_PER = (MAX_STAT_SEG + LANES - 1) / LANES;
    float2 v[MAX_PER];
    float m = -CUDART_INF_F;
#pragma unroll
    for (int k = 0; k < MAX_PER; ++k) {
        const int i = sub + k * LANES;
        v[k] = i < nseg ? seg[i] : make_float2(-CUDART_INF_F, 0.f);
        m = fmaxf(m, v[k].x);
    }
#pragma unroll
    for (int o = LANES / 2; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float z = 0.f;
    if (m > -CUDART_INF_F) {
#pragma unroll
        for (int k = 0; k < MAX_PER; ++k)
            if (v[k].y > 0.f) z += v[k].y * exp2f((v[k].x - m) * c);
    }
#pragma unroll
    for (int o = LANES / 2; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    return make_float2(m, z);
}

int n_stat_segments(int vocab) { return std::max(1, std::min(MAX_STAT_SEG, vocab / 8192)); }
int segment_len(int vocab, int nseg) { return ((vocab + nseg - 1) / nseg + 7) / 8 * 8; }

StatsJob stats_job(const void* logits, int dtype, int64_t ld, int rows, int group_rows, int group_pitch) {
    StatsJob j;
    j.logits = logits; j.row_stride = ld; j.bf16 = dtype == DFLASH_BF16; j.rows = rows;
    j.group_rows = std::max(group_rows, 1); j.group_pitch = std::max(group_pitch, 1);
    return j;
}
// out [rows of both jobs][n_stat]; `tickets` (may be nullptr with n_tickets = 0) are zeroed by the launch
int launch_softmax_stats(cudaStream_t st, const StatsJob& j0, const StatsJob& j1, int vocab, int n_stat, float c, float2* out,
                         int32_t* tickets, int n_tickets) {
    if (j0.rows + j1.rows == 0) return DFLASH_OK;
    const cudaError_t e = launch_pdl(softmax_stats_kernel, dim3(n_stat, j0.rows + j1.rows), dim3(256), 0, st, j0, j1, vocab,
                                     segment_len(vocab, n_stat), c, out, tickets, n_tickets);
    g_launches += 1;
    return e == cudaSuccess ? DFLASH_OK : DFLASH_ERR_CUDA;
}

}  // namespace
}  // namespace dflash
