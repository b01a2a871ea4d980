// Sampling (temperature > 0) drafting and verification: the paper's T = 1 setting (Sec. 5.1).
// The rule is standard speculative sampling, which the paper relies on without restating it:
//   p_j = softmax(target_logits[j] / T),  q_j = softmax(draft_logits[j] / T);
//   draft j is kept while u_j * q_j(d_j) < p_j(d_j); at the first rejection a, one token is drawn from
//   max(p_a - q_a, 0) (from p_a if that is all zero); with every draft kept, one token from p_gamma.
// Every draw maps a uniform u in [0, 1) (an INPUT: the library draws no random numbers) to the first
// vocabulary index whose running sum of weights reaches u * total.
//
// All of it is row-wise streaming over logits that already sit in HBM (bytes: each logits row once
// for the softmax statistics, the one row pair per sequence that emits a token twice more):
//   1. softmax_stats_seg_kernel   per (row, segment): running maximum and sum of exponentials
//   2. verify_plan_kernel / rows_plan_kernel   merge the segments, take the accept decisions
//      (a few gathered logits per sequence), describe the one draw each sequence / row needs
//   3. weights_seg_kernel          per (draw, segment): sum of the weights, in double
//   4. select_kernel               per draw: the segment, then the index inside it
// Sums that decide an index are accumulated in double in a fixed order, so a result is reproducible
// and differs from exact arithmetic only when u * total lies within ~1e-6 (relative) of an interval edge.
#include "dflash_internal.h"
#include "ptx_sm100.cuh"

#include <math_constants.h>

#include <algorithm>

namespace dflash {
namespace {

#define SAMPLE_TRY(expr)                  \
    do {                                  \
        const int rc__ = (expr);          \
        if (rc__ != DFLASH_OK) return rc__; \
    } while (0)

constexpr int MAX_SEG = 64;
constexpr float LOG2E = 1.4426950408889634f;

struct Draw {                 // one inverse-CDF draw
    const void* p_row;        // weights p_i = exp2((z_i - m_p) c) * inv_zp
    const void* q_row;        // nullptr: w = p;  else w = max(p - q, 0), falling back to p when that sums to 0
    float m_p, inv_zp, m_q, inv_zq;
    float u;
    int32_t p_bf16, q_bf16;   // element types of the two rows
    int32_t* out;             // where the drawn index goes
    int32_t* out2;            // second copy (bonus), may be nullptr
    float* prob;              // probability p(index), may be nullptr
};

__device__ __forceinline__ float as_f(float v) { return v; }
__device__ __forceinline__ float as_f(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float ld_logit(const void* row, int bf16, int i) {
    return bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(row)[i]) : reinterpret_cast<const float*>(row)[i];
}

// (max, sum of exp2((z - max) c)) of two partial results
__device__ __forceinline__ float2 stat_merge(float2 a, float2 b, float c) {
    const float m = fmaxf(a.x, b.x);
    if (m == -CUDART_INF_F) return make_float2(m, 0.f);
    return make_float2(m, a.y * exp2f((a.x - m) * c) + b.y * exp2f((b.x - m) * c));
}

// grid (nseg, rows). Row r is row (r / group_rows) * group_pitch + r % group_rows of `logits`
// (the drafts of a sequence may be the first gamma of B stored rows).
template <typename T>
__global__ void __launch_bounds__(256) softmax_stats_seg_kernel(const T* __restrict__ logits, int64_t row_stride, int group_rows,
                                                                int group_pitch, int vocab, int seg_len, float c,
                                                                float2* __restrict__ out) {
    __shared__ float2 sh[8];
    ptx::pdl_trigger();
    ptx::pdl_wait();
    const int seg = blockIdx.x, nseg = gridDim.x, row = blockIdx.y;
    const T* src = logits + ((size_t)(row / group_rows) * group_pitch + row % group_rows) * row_stride;
    const int lo = seg * seg_len, hi = min(vocab, lo + seg_len);
    float m = -CUDART_INF_F;
    for (int i = lo + threadIdx.x; i < hi; i += blockDim.x) m = fmaxf(m, as_f(src[i]));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5].x = m;
    __syncthreads();
    m = sh[0].x;
    for (int w = 1; w < 8; ++w) m = fmaxf(m, sh[w].x);
    __syncthreads();
    float s = 0.f;
    if (m > -CUDART_INF_F)
        for (int i = lo + threadIdx.x; i < hi; i += blockDim.x) s += exp2f((as_f(src[i]) - m) * c);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5].y = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int w = 0; w < 8; ++w) t += sh[w].y;
        out[(size_t)row * nseg + seg] = make_float2(m, t);
    }
}

// whole-row (max, sum) from the segment results, by one warp
__device__ __forceinline__ float2 row_stat(const float2* seg, int nseg, float c, int lane) {
    float2 t = make_float2(-CUDART_INF_F, 0.f);
    for (int i = lane; i < nseg; i += 32) t = stat_merge(t, seg[i], c);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        float2 u;
        u.x = __shfl_xor_sync(0xffffffffu, t.x, o);
        u.y = __shfl_xor_sync(0xffffffffu, t.y, o);
        t = stat_merge(t, u, c);
    }
    return t;
}

// one warp per row: the draw of plain sampling
__global__ void __launch_bounds__(32) rows_plan_kernel(const void* logits, int bf16, int64_t row_stride, int es, int n_rows,
                                                       int nseg, float c, const float2* __restrict__ stats,
                                                       const float* __restrict__ u, int32_t* ids, float* prob, Draw* draws) {
    ptx::pdl_trigger();
    ptx::pdl_wait();
    const int row = blockIdx.x, lane = threadIdx.x;
    const float2 st = row_stat(stats + (size_t)row * nseg, nseg, c, lane);
    if (lane == 0) {
        Draw d{};
        d.p_row = reinterpret_cast<const char*>(logits) + (size_t)row * row_stride * es;
        d.q_row = nullptr;
        d.m_p = st.x; d.inv_zp = st.y > 0.f ? 1.f / st.y : 0.f;
        d.u = u[row];
        d.p_bf16 = bf16;
        d.out = ids + row; d.out2 = nullptr; d.prob = prob ? prob + row : nullptr;
        draws[row] = d;
    }
}

// one warp per sequence: accept decisions in order, then the draw that ends the cycle
__global__ void __launch_bounds__(32) verify_plan_kernel(dflash_verify_sample_args a, int nseg, float c,
                                                         const float2* __restrict__ t_stats, const float2* __restrict__ d_stats,
                                                         Draw* draws) {
    ptx::pdl_trigger();
    ptx::pdl_wait();
    const int b = blockIdx.x, lane = threadIdx.x;
    const int g = a.gamma, V = a.vocab;
    const int t_es = a.target_dtype == DFLASH_BF16 ? 2 : 4, d_es = a.draft_dtype == DFLASH_BF16 ? 2 : 4;
    const int64_t t_ld = a.target_row_stride ? a.target_row_stride : V, d_ld = a.draft_row_stride ? a.draft_row_stride : V;
    const int32_t* ids = a.draft_ids + (size_t)b * a.draft_stride;
    int32_t* out = a.out_tokens + (size_t)b * (g + 1);
    int acc = 0;
    float2 ts = make_float2(0.f, 0.f), ds = make_float2(0.f, 0.f);
    const char* t_row = nullptr;
    const char* d_row = nullptr;
    for (; acc <= g; ++acc) {
        t_row = reinterpret_cast<const char*>(a.target_logits) + ((size_t)b * (g + 1) + acc) * t_ld * t_es;
        ts = row_stat(t_stats + ((size_t)b * (g + 1) + acc) * nseg, nseg, c, lane);
        if (acc == g) break;
        d_row = reinterpret_cast<const char*>(a.draft_logits) + ((size_t)b * a.draft_rows_per_seq + acc) * d_ld * d_es;
        ds = row_stat(d_stats + ((size_t)b * g + acc) * nseg, nseg, c, lane);
        int tok = ids[acc];
        bool keep = false;
        if (tok >= 0 && tok < V) {
            const float p = ts.y > 0.f ? exp2f((ld_logit(t_row, t_es == 2, tok) - ts.x) * c) / ts.y : 0.f;
            const float q = ds.y > 0.f ? exp2f((ld_logit(d_row, d_es == 2, tok) - ds.x) * c) / ds.y : 0.f;
            keep = a.u_accept[(size_t)b * g + acc] * q < p;
        } else if (lane == 0 && a.dev_status) {
            atomicOr(a.dev_status, DFLASH_DEV_BAD_TOKEN);
        }
        if (!keep) break;
    }
    if (lane == 0) {
        for (int i = 0; i <= g; ++i) out[i] = i < acc ? ids[i] : -1;
        a.accept_len[b] = acc + 1;
        a.new_ctx_len[b] = a.ctx_len[b] + acc + 1;
        Draw d{};
        d.p_row = t_row; d.p_bf16 = t_es == 2;
        d.m_p = ts.x; d.inv_zp = ts.y > 0.f ? 1.f / ts.y : 0.f;
        if (acc < g) {
            d.q_row = d_row; d.q_bf16 = d_es == 2;
            d.m_q = ds.x; d.inv_zq = ds.y > 0.f ? 1.f / ds.y : 0.f;
        }
        d.u = a.u_final[b];
        d.out = out + acc; d.out2 = a.bonus + b; d.prob = nullptr;
        draws[b] = d;
    }
}

__device__ __forceinline__ void draw_weights(const Draw& d, float c, int i, float& w_res, float& w_p) {
    w_p = exp2f((ld_logit(d.p_row, d.p_bf16, i) - d.m_p) * c) * d.inv_zp;
    w_res = w_p;
    if (d.q_row) {
        const float q = exp2f((ld_logit(d.q_row, d.q_bf16, i) - d.m_q) * c) * d.inv_zq;
        w_res = fmaxf(w_p - q, 0.f);
    }
}

// block-wide sum of two doubles per thread (fixed order); result valid in thread 0
__device__ __forceinline__ void block_sum2(double& a, double& b, double* sh) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        a += __shfl_xor_sync(0xffffffffu, a, o);
        b += __shfl_xor_sync(0xffffffffu, b, o);
    }
    const int w = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0) { sh[2 * w] = a; sh[2 * w + 1] = b; }
    __syncthreads();
    if (threadIdx.x == 0) {
        a = 0.0; b = 0.0;
        for (int i = 0; i < (int)(blockDim.x >> 5); ++i) { a += sh[2 * i]; b += sh[2 * i + 1]; }
    }
    __syncthreads();
}

// grid (nseg, draws): seg_w[draw][seg] = (sum of residual weights, sum of p)
__global__ void __launch_bounds__(256) weights_seg_kernel(const Draw* __restrict__ draws, int vocab, int seg_len, float c,
                                                          double2* __restrict__ seg_w) {
    __shared__ double sh[16];
    ptx::pdl_trigger();
    ptx::pdl_wait();
    const Draw d = draws[blockIdx.y];
    const int seg = blockIdx.x, nseg = gridDim.x;
    const int lo = seg * seg_len, hi = min(vocab, lo + seg_len);
    // a thread owns a contiguous run of the segment, so select_kernel can redo exactly the same sums
    const int per = (seg_len + blockDim.x - 1) / blockDim.x;
    double sr = 0.0, sp = 0.0;
    for (int i = lo + threadIdx.x * per, e = min(hi, i + per); i < e; ++i) {
        float wr, wp;
        draw_weights(d, c, i, wr, wp);
        sr += (double)wr;
        sp += (double)wp;
    }
    block_sum2(sr, sp, sh);
    if (threadIdx.x == 0) seg_w[(size_t)blockIdx.y * nseg + seg] = make_double2(sr, sp);
}

// grid (draws): find the segment, then the thread run, then the index
__global__ void __launch_bounds__(256) select_kernel(const Draw* __restrict__ draws, int vocab, int seg_len, int nseg, float c,
                                                     const double2* __restrict__ seg_w) {
    __shared__ double s_run[256];
    ptx::pdl_trigger();
    ptx::pdl_wait();
    __shared__ double s_x;
    __shared__ int s_seg, s_use_p, s_owner;
    const Draw d = draws[blockIdx.x];
    if (threadIdx.x == 0) {
        double tot_r = 0.0, tot_p = 0.0;
        for (int s = 0; s < nseg; ++s) { tot_r += seg_w[(size_t)blockIdx.x * nseg + s].x; tot_p += seg_w[(size_t)blockIdx.x * nseg + s].y; }
        const int use_p = (d.q_row == nullptr || !(tot_r > 0.0)) ? 1 : 0;
        const double total = use_p ? tot_p : tot_r;
        double x = (double)d.u * total, before = 0.0;
        int pick = -1, last = -1;
        for (int s = 0; s < nseg; ++s) {
            const double w = use_p ? seg_w[(size_t)blockIdx.x * nseg + s].y : seg_w[(size_t)blockIdx.x * nseg + s].x;
            if (w > 0.0) {
                last = s;
                if (before + w >= x) { pick = s; break; }
                before += w;
            }
        }
        if (pick < 0) {            // u * total beyond the last edge by rounding: the last non-empty segment
            pick = last;
            before = 0.0;
            for (int s = 0; s < last; ++s) before += use_p ? seg_w[(size_t)blockIdx.x * nseg + s].y : seg_w[(size_t)blockIdx.x * nseg + s].x;
        }
        s_seg = pick; s_use_p = use_p; s_x = x - before;
    }
    __syncthreads();
    const int seg = s_seg, use_p = s_use_p;
    if (seg < 0) {                // no weight anywhere (all logits -inf): emit token 0
        if (threadIdx.x == 0) {
            *d.out = 0;
            if (d.out2) *d.out2 = 0;
            if (d.prob) *d.prob = 0.f;
        }
        return;
    }
    const int lo = seg * seg_len, hi = min(vocab, lo + seg_len);
    const int per = (seg_len + blockDim.x - 1) / blockDim.x;
    const int my_lo = lo + threadIdx.x * per, my_hi = min(hi, my_lo + per);
    double run = 0.0;
    for (int i = my_lo; i < my_hi; ++i) {
        float wr, wp;
        draw_weights(d, c, i, wr, wp);
        run += (double)(use_p ? wp : wr);
    }
    s_run[threadIdx.x] = run;
    __syncthreads();
    if (threadIdx.x == 0) {
        const double x = s_x;
        double before = 0.0;
        int pick = -1, last = -1;
        for (int t = 0; t < (int)blockDim.x; ++t) {
            const double w = s_run[t];
            if (w > 0.0) {
                last = t;
                if (before + w >= x) { pick = t; break; }
                before += w;
            }
        }
        if (pick < 0) {
            pick = last;
            before = 0.0;
            for (int t = 0; t < last; ++t) before += s_run[t];
        }
        s_owner = pick;
        s_x = x - before;
    }
    __syncthreads();
    if ((int)threadIdx.x == s_owner) {
        const double x = s_x;
        double cum = 0.0;
        int pick = -1, last = -1;
        float p_pick = 0.f, p_last = 0.f;
        for (int i = my_lo; i < my_hi; ++i) {
            float wr, wp;
            draw_weights(d, c, i, wr, wp);
            const float w = use_p ? wp : wr;
            if (w > 0.f) {
                last = i; p_last = wp;
                cum += (double)w;
                if (cum >= x) { pick = i; p_pick = wp; break; }
            }
        }
        if (pick < 0) { pick = last; p_pick = p_last; }
        *d.out = pick;
        if (d.out2) *d.out2 = pick;
        if (d.prob) *d.prob = p_pick;
    }
}

int n_segments(int vocab) { return std::max(1, std::min(MAX_SEG, vocab / 2048)); }
int segment_len(int vocab, int nseg) { return ((vocab + nseg - 1) / nseg + 7) / 8 * 8; }

struct Scratch {
    float2* stats;     // [n_rows][nseg]
    Draw* draws;       // [n_draws]
    double2* seg_w;    // [n_draws][nseg]
    int64_t bytes;
};
Scratch carve_scratch(void* base, int64_t n_rows, int64_t n_draws, int nseg) {
    Scratch s;
    char* p = reinterpret_cast<char*>(base);
    int64_t off = 0;
    auto take = [&](int64_t bytes) { char* r = p ? p + off : nullptr; off += (bytes + 255) / 256 * 256; return r; };
    s.stats = reinterpret_cast<float2*>(take(n_rows * nseg * (int64_t)sizeof(float2)));
    s.draws = reinterpret_cast<Draw*>(take(n_draws * (int64_t)sizeof(Draw)));
    s.seg_w = reinterpret_cast<double2*>(take(n_draws * nseg * (int64_t)sizeof(double2)));
    s.bytes = off;
    return s;
}

int launch_stats(cudaStream_t st, const void* logits, int dtype, int64_t ld, int rows, int group_rows, int group_pitch, int vocab,
                 int nseg, int seg_len, float c, float2* out) {
    if (rows == 0) return DFLASH_OK;
    dim3 grid(nseg, rows);
    cudaError_t e;
    if (dtype == DFLASH_BF16)
        e = launch_pdl(softmax_stats_seg_kernel<__nv_bfloat16>, grid, dim3(256), 0, st, (const __nv_bfloat16*)logits, ld, group_rows,
                       group_pitch, vocab, seg_len, c, out);
    else
        e = launch_pdl(softmax_stats_seg_kernel<float>, grid, dim3(256), 0, st, (const float*)logits, ld, group_rows, group_pitch,
                       vocab, seg_len, c, out);
    g_launches += 1;
    return e == cudaSuccess ? DFLASH_OK : DFLASH_ERR_CUDA;
}

int launch_draws(cudaStream_t st, const Scratch& s, int n_draws, int vocab, int nseg, int seg_len, float c) {
    if (n_draws == 0) return DFLASH_OK;
    const cudaError_t e1 = launch_pdl(weights_seg_kernel, dim3(nseg, n_draws), dim3(256), 0, st, (const Draw*)s.draws, vocab, seg_len, c,
                                      s.seg_w);
    const cudaError_t e2 = launch_pdl(select_kernel, dim3(n_draws), dim3(256), 0, st, (const Draw*)s.draws, vocab, seg_len, nseg, c,
                                      (const double2*)s.seg_w);
    g_launches += 2;
    return (e1 == cudaSuccess && e2 == cudaSuccess) ? DFLASH_OK : DFLASH_ERR_CUDA;
}

bool dtype_ok(int d) { return d == DFLASH_F32 || d == DFLASH_BF16; }

}  // namespace
}  // namespace dflash

using namespace dflash;

extern "C" {

int64_t dflash_sample_workspace_bytes(int32_t n_rows, int32_t vocab) {
    if (n_rows < 0 || vocab < 1) return -1;
    return carve_scratch(nullptr, n_rows, n_rows, n_segments(vocab)).bytes;
}

int32_t dflash_sample_rows(dflash_handle* h, const dflash_sample_args* a, void* stream) {
    if (!h || !a) return DFLASH_ERR_INVALID_ARG;
    if (a->n_rows < 0 || a->vocab < 1 || !(a->temperature > 0.f) || !dtype_ok(a->logits_dtype)) return DFLASH_ERR_INVALID_ARG;
    if (a->n_rows == 0) return DFLASH_OK;
    if (!a->logits || !a->u || !a->ids) return DFLASH_ERR_INVALID_ARG;
    if (!a->workspace || (reinterpret_cast<uintptr_t>(a->workspace) & 255)) return DFLASH_ERR_WORKSPACE;
    const int nseg = n_segments(a->vocab), seg_len = segment_len(a->vocab, nseg);
    const Scratch s = carve_scratch(a->workspace, a->n_rows, a->n_rows, nseg);
    if (s.bytes > a->workspace_bytes) return DFLASH_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const float c = LOG2E / a->temperature;
    const int64_t ld = a->row_stride ? a->row_stride : a->vocab;
    SAMPLE_TRY(launch_stats(st, a->logits, a->logits_dtype, ld, a->n_rows, a->n_rows, a->n_rows, a->vocab, nseg, seg_len, c, s.stats));
    const cudaError_t e = launch_pdl(rows_plan_kernel, dim3(a->n_rows), dim3(32), 0, st, a->logits, (int)(a->logits_dtype == DFLASH_BF16),
                                     ld, a->logits_dtype == DFLASH_BF16 ? 2 : 4, a->n_rows, nseg, c, (const float2*)s.stats, a->u,
                                     a->ids, a->prob, s.draws);
    g_launches += 1;
    if (e != cudaSuccess) return DFLASH_ERR_CUDA;
    return launch_draws(st, s, a->n_rows, a->vocab, nseg, seg_len, c);
}

int32_t dflash_verify_accept_sample(dflash_handle* h, const dflash_verify_sample_args* a, void* stream) {
    if (!h || !a) return DFLASH_ERR_INVALID_ARG;
    if (a->batch < 0 || a->gamma < 0 || a->vocab < 1 || !(a->temperature > 0.f)) return DFLASH_ERR_INVALID_ARG;
    if (!dtype_ok(a->target_dtype) || (a->gamma > 0 && !dtype_ok(a->draft_dtype))) return DFLASH_ERR_INVALID_ARG;
    if (a->batch == 0) return DFLASH_OK;
    if (!a->target_logits || !a->u_final || !a->ctx_len || !a->accept_len || !a->out_tokens || !a->bonus || !a->new_ctx_len)
        return DFLASH_ERR_INVALID_ARG;
    if (a->gamma > 0 && (!a->draft_logits || !a->draft_ids || !a->u_accept || a->draft_rows_per_seq < a->gamma ||
                         a->draft_stride < a->gamma))
        return DFLASH_ERR_INVALID_ARG;
    if ((int64_t)a->batch * (2 * a->gamma + 1) > (1 << 22)) return DFLASH_ERR_UNSUPPORTED;
    if (!a->workspace || (reinterpret_cast<uintptr_t>(a->workspace) & 255)) return DFLASH_ERR_WORKSPACE;
    const int nseg = n_segments(a->vocab), seg_len = segment_len(a->vocab, nseg);
    const int64_t t_rows = (int64_t)a->batch * (a->gamma + 1), d_rows = (int64_t)a->batch * a->gamma;
    const Scratch s = carve_scratch(a->workspace, t_rows + d_rows, a->batch, nseg);
    if (s.bytes > a->workspace_bytes) return DFLASH_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const float c = LOG2E / a->temperature;
    const int64_t t_ld = a->target_row_stride ? a->target_row_stride : a->vocab;
    const int64_t d_ld = a->draft_row_stride ? a->draft_row_stride : a->vocab;
    SAMPLE_TRY(launch_stats(st, a->target_logits, a->target_dtype, t_ld, (int)t_rows, (int)t_rows, (int)t_rows, a->vocab, nseg, seg_len, c,
                            s.stats));
    float2* d_stats = s.stats + t_rows * nseg;
    if (a->gamma > 0)      // the gamma draft rows of sequence b start at stored row b * draft_rows_per_seq
        SAMPLE_TRY(launch_stats(st, a->draft_logits, a->draft_dtype, d_ld, (int)d_rows, a->gamma, a->draft_rows_per_seq, a->vocab, nseg,
                                seg_len, c, d_stats));
    const cudaError_t e = launch_pdl(verify_plan_kernel, dim3(a->batch), dim3(32), 0, st, *a, nseg, c, (const float2*)s.stats,
                                     (const float2*)d_stats, s.draws);
    g_launches += 1;
    if (e != cudaSuccess) return DFLASH_ERR_CUDA;
    return launch_draws(st, s, a->batch, a->vocab, nseg, seg_len, c);
}

}  // extern "C"
