// Sampling (temperature > 0) drafting and verification: the paper's T = 1 setting (Sec. 5.1).
// The rule is standard speculative sampling, which the paper relies on without restating it:
//   p_j = softmax(target_logits[j] / T),  q_j = softmax(draft_logits[j] / T);
//   draft j is kept while u_j * q_j(d_j) < p_j(d_j); at the first rejection a, one token is drawn from
//   max(p_a - q_a, 0) (from p_a if that is all zero); with every draft kept, one token from p_gamma.
// Every draw maps a uniform u in [0, 1) (an INPUT: the library draws no random numbers) to the first
// vocabulary index whose running sum of weights reaches u * total.
//
// All of it is row-wise streaming over logits that already sit in HBM (bytes: each logits row once
// for the softmax statistics, the one row pair per sequence that emits a token twice more), in two
// launches per call:
//   1. softmax_stats_kernel   per (row, segment): running maximum and sum of exponentials (target and
//      draft rows of a verification in the same launch); it also zeroes the tickets of launch 2
//   2. rows_draw_kernel / verify_draw_kernel   per (draw, segment): every CTA merges the segment
//      statistics it needs and describes its draw itself (for a verification: the accept decisions, from
//      a few gathered logits per sequence; the CTA of segment 0 writes them out), sums the weights of its
//      segment in double, and the CTA that arrives last at the draw's ticket picks the segment, then the
//      index inside it
// Sums that decide an index are accumulated in double in a fixed order, so a result is reproducible
// and differs from exact arithmetic only when u * total lies within ~1e-6 (relative) of an interval edge.
#include "softmax_rows.cuh"

namespace dflash {
namespace {

#define SAMPLE_TRY(expr)                  \
    do {                                  \
        const int rc__ = (expr);          \
        if (rc__ != DFLASH_OK) return rc__; \
    } while (0)

constexpr int MAX_SEG = 64;        // segments of a draw

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

constexpr int DRAW_WARPS = 8;
constexpr int PLAN_MAX_GAMMA = 64;

// Accept decisions of sequence b, by the whole CTA: every row's statistics and accept test by its own
// warp, then the decisions in order (the first failed test ends the cycle). Thread 0 returns the draw
// that ends the cycle in *draw and, if `write`, stores the kept drafts and the lengths.
__device__ __forceinline__ void verify_plan(const dflash_verify_sample_args& a, int b, int nseg, float c, const float2* t_stats,
                                            const float2* d_stats, bool write, Draw* draw) {
    __shared__ float2 s_ts[PLAN_MAX_GAMMA + 1], s_ds[PLAN_MAX_GAMMA];
    __shared__ int s_keep[PLAN_MAX_GAMMA], s_bad[PLAN_MAX_GAMMA];
    const int g = a.gamma, V = a.vocab;
    const int t_es = a.target_dtype == DFLASH_BF16 ? 2 : 4, d_es = a.draft_dtype == DFLASH_BF16 ? 2 : 4;
    const int64_t t_ld = a.target_row_stride ? a.target_row_stride : V, d_ld = a.draft_row_stride ? a.draft_row_stride : V;
    const int32_t* ids = a.draft_ids + (size_t)b * a.draft_stride;
    const char* t_base = reinterpret_cast<const char*>(a.target_logits) + (size_t)b * (g + 1) * t_ld * t_es;
    const char* d_base = reinterpret_cast<const char*>(a.draft_logits) + (size_t)b * a.draft_rows_per_seq * d_ld * d_es;
    // 4 lanes per row pair (target row r, draft row r): 64 pairs per round of the CTA
    constexpr int GL = 4;
    const int sub = threadIdx.x % GL;
    for (int r0 = 0; r0 <= g; r0 += DRAW_WARPS * 32 / GL) {
        const int r = r0 + threadIdx.x / GL;
        const bool t_on = r <= g, d_on = r < g;
        const float2 ts = row_stat<GL>(t_stats + ((size_t)b * (g + 1) + (t_on ? r : 0)) * nseg, t_on ? nseg : 0, c, sub);
        const float2 ds = row_stat<GL>(d_stats + ((size_t)b * g + (d_on ? r : 0)) * nseg, d_on ? nseg : 0, c, sub);
        if (sub == 0 && t_on) s_ts[r] = ts;
        if (sub == 0 && d_on) {
            const char* t_row = t_base + (size_t)r * t_ld * t_es;
            const char* d_row = d_base + (size_t)r * d_ld * d_es;
            const int tok = ids[r];
            bool keep = false;
            const bool ok = tok >= 0 && tok < V;
            if (ok) {
                const float p = ts.y > 0.f ? exp2f((ld_logit(t_row, t_es == 2, tok) - ts.x) * c) / ts.y : 0.f;
                const float q = ds.y > 0.f ? exp2f((ld_logit(d_row, d_es == 2, tok) - ds.x) * c) / ds.y : 0.f;
                keep = a.u_accept[(size_t)b * g + r] * q < p;
            }
            s_ds[r] = ds; s_keep[r] = keep ? 1 : 0; s_bad[r] = ok ? 0 : 1;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int acc = 0;
        while (acc < g && s_keep[acc]) ++acc;
        int32_t* out = a.out_tokens + (size_t)b * (g + 1);
        if (write) {
            if (acc < g && s_bad[acc] && a.dev_status) atomicOr(a.dev_status, DFLASH_DEV_BAD_TOKEN);
            for (int i = 0; i <= g; ++i)
                if (i != acc) out[i] = i < acc ? ids[i] : -1;       // out[acc] is the drawn token's place
            a.accept_len[b] = acc + 1;
            a.new_ctx_len[b] = a.ctx_len[b] + acc + 1;
        }
        const float2 ts = s_ts[acc];
        Draw d{};
        d.p_row = t_base + (size_t)acc * t_ld * t_es; d.p_bf16 = t_es == 2;
        d.m_p = ts.x; d.inv_zp = ts.y > 0.f ? 1.f / ts.y : 0.f;
        if (acc < g) {
            const float2 ds = s_ds[acc];
            d.q_row = d_base + (size_t)acc * d_ld * d_es; d.q_bf16 = d_es == 2;
            d.m_q = ds.x; d.inv_zq = ds.y > 0.f ? 1.f / ds.y : 0.f;
        }
        d.u = a.u_final[b];
        d.out = out + acc; d.out2 = a.bonus + b; d.prob = nullptr;
        *draw = d;
    }
}

__device__ __forceinline__ void weights_of(const Draw& d, float c, float zp, float zq, float& w_res, float& w_p) {
    w_p = exp2f((zp - d.m_p) * c) * d.inv_zp;
    w_res = w_p;
    if (d.q_row) {
        const float q = exp2f((zq - d.m_q) * c) * d.inv_zq;
        w_res = fmaxf(w_p - q, 0.f);
    }
}
__device__ __forceinline__ void draw_weights(const Draw& d, float c, int i, float& w_res, float& w_p) {
    weights_of(d, c, ld_logit(d.p_row, d.p_bf16, i), d.q_row ? ld_logit(d.q_row, d.q_bf16, i) : 0.f, w_res, w_p);
}

// Sums of the weights of entries [lo, hi) in index order, in double. The logits are fetched RUN_BATCH at a
// time (independent loads in flight) and added one by one, so the result does not depend on the batching.
constexpr int RUN_BATCH = 8;
__device__ __forceinline__ void run_sums(const Draw& d, float c, int lo, int hi, double& sum_res, double& sum_p) {
    for (int i0 = lo; i0 < hi; i0 += RUN_BATCH) {
        float zp[RUN_BATCH], zq[RUN_BATCH];
#pragma unroll
        for (int j = 0; j < RUN_BATCH; ++j) {
            const int i = min(i0 + j, hi - 1);
            zp[j] = ld_logit(d.p_row, d.p_bf16, i);
            zq[j] = d.q_row ? ld_logit(d.q_row, d.q_bf16, i) : 0.f;
        }
#pragma unroll
        for (int j = 0; j < RUN_BATCH; ++j) {
            if (i0 + j < hi) {
                float wr, wp;
                weights_of(d, c, zp[j], zq[j], wr, wp);
                sum_res += (double)wr;
                sum_p += (double)wp;
            }
        }
    }
}

// A thread's run held in registers (runs of at most RUN_MAX entries: vocabularies up to 64 x 256 x 16):
// fetched once, summed and, by the one thread that owns the drawn index, walked again without a reload.
constexpr int RUN_MAX = 16;
struct RunCache {
    float zp[RUN_MAX], zq[RUN_MAX];
};
__device__ __forceinline__ void run_load(const void* p_row, int p_bf16, const void* q_row, int q_bf16, int lo, int hi, RunCache& rc) {
#pragma unroll
    for (int j = 0; j < RUN_MAX; ++j) {
        const bool on = lo + j < hi;
        rc.zp[j] = on ? ld_logit(p_row, p_bf16, lo + j) : 0.f;
        rc.zq[j] = on && q_row ? ld_logit(q_row, q_bf16, lo + j) : 0.f;
    }
}
__device__ __forceinline__ void run_sums_cached(const Draw& d, float c, const RunCache& rc, int n, double& sum_res, double& sum_p) {
#pragma unroll
    for (int j = 0; j < RUN_MAX; ++j) {
        if (j < n) {
            float wr, wp;
            weights_of(d, c, rc.zp[j], rc.zq[j], wr, wp);
            sum_res += (double)wr;
            sum_p += (double)wp;
        }
    }
}

// Inclusive prefix sums of one (a, b) pair per thread over the CTA, in a fixed order (inside a warp by
// doubling, then the warps in order); `tot` = the last thread's inclusive sums. sh: 2 * warps doubles.
__device__ __forceinline__ void block_scan2(double& a, double& b, double& excl_a, double& excl_b, double& tot_a, double& tot_b,
                                            double* sh) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double va = __shfl_up_sync(0xffffffffu, a, o), vb = __shfl_up_sync(0xffffffffu, b, o);
        if (lane >= o) { a += va; b += vb; }
    }
    __syncthreads();                  // sh may still be read from an earlier use
    if (lane == 31) { sh[2 * warp] = a; sh[2 * warp + 1] = b; }
    __syncthreads();
    double off_a = 0.0, off_b = 0.0;
    tot_a = 0.0; tot_b = 0.0;
    for (int w = 0; w < n_warps; ++w) {
        if (w == warp) { off_a = tot_a; off_b = tot_b; }
        tot_a += sh[2 * w]; tot_b += sh[2 * w + 1];
    }
    a += off_a; b += off_b;
    excl_a = __shfl_up_sync(0xffffffffu, a, 1);
    excl_b = __shfl_up_sync(0xffffffffu, b, 1);
    if (lane == 0) { excl_a = off_a; excl_b = off_b; }
}

// The first thread whose weight is positive and whose inclusive sum reaches x; if rounding left x beyond
// the last edge, the last thread with a positive weight; -1 if no thread has weight. Same value in all threads.
__device__ __forceinline__ int first_reaching(double w, double incl, double x, int* s_hit, int* s_last, int* s_owner) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const unsigned hit = __ballot_sync(0xffffffffu, w > 0.0 && incl >= x);
    const unsigned pos = __ballot_sync(0xffffffffu, w > 0.0);
    if (lane == 0) {
        s_hit[warp] = hit ? warp * 32 + __ffs(hit) - 1 : -1;
        s_last[warp] = pos ? warp * 32 + 31 - __clz(pos) : -1;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int owner = -1, last = -1;
        for (int i = 0; i < n_warps; ++i) {
            if (owner < 0 && s_hit[i] >= 0) owner = s_hit[i];
            if (s_last[i] >= 0) last = s_last[i];
        }
        *s_owner = owner >= 0 ? owner : last;
    }
    __syncthreads();
    return *s_owner;
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

// The draw itself, by the whole CTA, once every segment's weights are known: the segment, then the
// thread run, then the index.
__device__ __forceinline__ void select_index(const Draw& d, int vocab, int seg_len, int nseg, float c, const double2* seg_w) {
    __shared__ double s_scan[2 * DRAW_WARPS];
    __shared__ int s_hit[DRAW_WARPS], s_last[DRAW_WARPS], s_owner;
    __shared__ double s_x;
    // ---- the segment (thread s holds segment s)
    double2 w = make_double2(0.0, 0.0);
    if ((int)threadIdx.x < nseg) w = __ldcg(seg_w + threadIdx.x);       // written by other CTAs of this launch
    double in_r = w.x, in_p = w.y, ex_r, ex_p, tot_r, tot_p;
    block_scan2(in_r, in_p, ex_r, ex_p, tot_r, tot_p, s_scan);
    const int use_p = (d.q_row == nullptr || !(tot_r > 0.0)) ? 1 : 0;
    double x = (double)d.u * (use_p ? tot_p : tot_r);
    const int seg = first_reaching(use_p ? w.y : w.x, use_p ? in_p : in_r, x, s_hit, s_last, &s_owner);
    if (seg < 0) {                // no weight anywhere (all logits -inf): emit token 0
        if (threadIdx.x == 0) {
            *d.out = 0;
            if (d.out2) *d.out2 = 0;
            if (d.prob) *d.prob = 0.f;
        }
        return;
    }
    if ((int)threadIdx.x == seg) s_x = x - (use_p ? ex_p : ex_r);
    // ---- the thread run inside it
    const int lo = seg * seg_len, hi = min(vocab, lo + seg_len);
    const int per = (seg_len + blockDim.x - 1) / blockDim.x;
    const int my_lo = lo + threadIdx.x * per, my_hi = min(hi, my_lo + per);
    const bool cached = per <= RUN_MAX;
    RunCache rc;
    double run_r = 0.0, run_p = 0.0;
    if (cached) {
        run_load(d.p_row, d.p_bf16, d.q_row, d.q_bf16, my_lo, my_hi, rc);
        run_sums_cached(d, c, rc, my_hi - my_lo, run_r, run_p);
    } else {
        run_sums(d, c, my_lo, my_hi, run_r, run_p);
    }
    const double run = use_p ? run_p : run_r;
    double ir = run_r, ip = run_p;
    block_scan2(ir, ip, ex_r, ex_p, tot_r, tot_p, s_scan);      // (its first barrier also publishes s_x)
    x = s_x;
    const int owner = first_reaching(run, use_p ? ip : ir, x, s_hit, s_last, &s_owner);
    if (owner < 0) {              // cannot happen for a segment chosen by its weight; defined anyway
        if (threadIdx.x == 0) {
            *d.out = lo;
            if (d.out2) *d.out2 = lo;
            if (d.prob) *d.prob = 0.f;
        }
        return;
    }
    // ---- the index inside the run
    if ((int)threadIdx.x == owner) {
        const double xr = x - (use_p ? ex_p : ex_r);
        double cum = 0.0;
        int pick = -1, last = -1;
        float p_pick = 0.f, p_last = 0.f;
        if (cached) {
#pragma unroll
            for (int j = 0; j < RUN_MAX; ++j) {
                if (my_lo + j < my_hi && pick < 0) {
                    float wr, wp;
                    weights_of(d, c, rc.zp[j], rc.zq[j], wr, wp);
                    const float wt = use_p ? wp : wr;
                    if (wt > 0.f) {
                        last = my_lo + j; p_last = wp;
                        cum += (double)wt;
                        if (cum >= xr) { pick = my_lo + j; p_pick = wp; }
                    }
                }
            }
        } else {
            for (int i = my_lo; i < my_hi; ++i) {
                float wr, wp;
                draw_weights(d, c, i, wr, wp);
                const float wt = use_p ? wp : wr;
                if (wt > 0.f) {
                    last = i; p_last = wp;
                    cum += (double)wt;
                    if (cum >= xr) { pick = i; p_pick = wp; break; }
                }
            }
        }
        if (pick < 0) { pick = last; p_pick = p_last; }
        *d.out = pick;
        if (d.out2) *d.out2 = pick;
        if (d.prob) *d.prob = p_pick;
    }
}

// CTA (segment, draw): the weights of the segment, summed in double with a thread owning a contiguous run
// (select_index redoes exactly the same sums); the CTA that arrives last at the draw's ticket draws.
// `pre`: the thread's run is already in `rc` (fetched before the draw was known in full).
__device__ __forceinline__ void segment_weights_then_draw(const Draw& d, int draw, int vocab, int seg_len, float c, double2* seg_w,
                                                          int32_t* tickets, bool pre, RunCache& rc) {
    __shared__ double sh[2 * DRAW_WARPS];
    __shared__ int s_is_last;
    const int seg = blockIdx.x, nseg = gridDim.x;
    const int lo = seg * seg_len, hi = min(vocab, lo + seg_len);
    const int per = (seg_len + blockDim.x - 1) / blockDim.x;
    double sr = 0.0, sp = 0.0;
    const int my_lo = lo + threadIdx.x * per, my_hi = min(hi, my_lo + per);
    if (per <= RUN_MAX) {
        if (!pre) run_load(d.p_row, d.p_bf16, d.q_row, d.q_bf16, my_lo, my_hi, rc);
        run_sums_cached(d, c, rc, my_hi - my_lo, sr, sp);
    } else {
        run_sums(d, c, my_lo, my_hi, sr, sp);
    }
    block_sum2(sr, sp, sh);
    if (threadIdx.x == 0) {
        seg_w[(size_t)draw * nseg + seg] = make_double2(sr, sp);
        __threadfence();
        const int t = atomicAdd(tickets + draw, 1);
        s_is_last = t == nseg - 1;
    }
    __syncthreads();
    if (!s_is_last) return;
    __threadfence();
    select_index(d, vocab, seg_len, nseg, c, seg_w + (size_t)draw * nseg);
}

// grid (nseg, rows): plain sampling, one draw per row
__global__ void __launch_bounds__(DRAW_WARPS * 32) rows_draw_kernel(const void* logits, int bf16, int64_t row_stride, int es, int vocab,
                                                                    int seg_len, float c, const float2* __restrict__ stats,
                                                                    int n_stat, const float* __restrict__ u, int32_t* ids,
                                                                    float* prob, double2* seg_w, int32_t* tickets) {
    __shared__ float2 s_st;
    ptx::pdl_trigger();
    ptx::pdl_wait();
    const int row = blockIdx.y;
    const char* p_row = reinterpret_cast<const char*>(logits) + (size_t)row * row_stride * es;
    // the thread's logits travel while warp 0 merges the row's statistics
    RunCache rc;
    const int per = (seg_len + blockDim.x - 1) / blockDim.x;
    const bool pre = per <= RUN_MAX;
    if (pre) {
        const int lo = blockIdx.x * seg_len, hi = min(vocab, lo + seg_len);
        const int my_lo = lo + threadIdx.x * per;
        run_load(p_row, bf16, nullptr, 0, my_lo, min(hi, my_lo + per), rc);
    }
    if (threadIdx.x < 32) {
        const float2 st = row_stat<32>(stats + (size_t)row * n_stat, n_stat, c, threadIdx.x);
        if (threadIdx.x == 0) s_st = st;
    }
    __syncthreads();
    Draw d{};
    d.p_row = p_row;
    d.q_row = nullptr;
    d.m_p = s_st.x; d.inv_zp = s_st.y > 0.f ? 1.f / s_st.y : 0.f;
    d.u = u[row];
    d.p_bf16 = bf16;
    d.out = ids + row; d.out2 = nullptr; d.prob = prob ? prob + row : nullptr;
    segment_weights_then_draw(d, row, vocab, seg_len, c, seg_w, tickets, pre, rc);
}

// grid (nseg, batch): speculative-sampling verification, one draw per sequence
__global__ void __launch_bounds__(DRAW_WARPS * 32) verify_draw_kernel(dflash_verify_sample_args a, int seg_len, float c,
                                                                      const float2* __restrict__ t_stats,
                                                                      const float2* __restrict__ d_stats, int n_stat,
                                                                      double2* seg_w, int32_t* tickets) {
    __shared__ Draw s_draw;
    ptx::pdl_trigger();
    ptx::pdl_wait();
    const int b = blockIdx.y;
    verify_plan(a, b, n_stat, c, t_stats, d_stats, blockIdx.x == 0, &s_draw);
    __syncthreads();
    const Draw d = s_draw;
    RunCache rc;
    segment_weights_then_draw(d, b, a.vocab, seg_len, c, seg_w, tickets, false, rc);
}

int n_segments(int vocab) { return std::max(1, std::min(MAX_SEG, vocab / 2048)); }

struct Scratch {
    float2* stats;     // [n_rows][stat segments]
    double2* seg_w;    // [n_draws][nseg]
    int32_t* tickets;  // [n_draws] segments of a draw that have delivered their weights
    int64_t bytes;
};
Scratch carve_scratch(void* base, int64_t n_rows, int64_t n_draws, int nseg, int n_stat) {
    Scratch s;
    char* p = reinterpret_cast<char*>(base);
    int64_t off = 0;
    auto take = [&](int64_t bytes) { char* r = p ? p + off : nullptr; off += (bytes + 255) / 256 * 256; return r; };
    s.stats = reinterpret_cast<float2*>(take(n_rows * n_stat * (int64_t)sizeof(float2)));
    s.seg_w = reinterpret_cast<double2*>(take(n_draws * nseg * (int64_t)sizeof(double2)));
    s.tickets = reinterpret_cast<int32_t*>(take(n_draws * (int64_t)sizeof(int32_t)));
    s.bytes = off;
    return s;
}

int launch_stats(cudaStream_t st, const StatsJob& j0, const StatsJob& j1, int vocab, int n_stat, float c, const Scratch& s,
                 int n_tickets) {
    return launch_softmax_stats(st, j0, j1, vocab, n_stat, c, s.stats, s.tickets, n_tickets);
}

bool dtype_ok(int d) { return d == DFLASH_F32 || d == DFLASH_BF16; }

}  // namespace
}  // namespace dflash

using namespace dflash;

extern "C" {

int64_t dflash_sample_workspace_bytes(int32_t n_rows, int32_t vocab) {
    if (n_rows < 0 || vocab < 1) return -1;
    return carve_scratch(nullptr, n_rows, n_rows, n_segments(vocab), n_stat_segments(vocab)).bytes;
}

int32_t dflash_sample_rows(dflash_handle* h, const dflash_sample_args* a, void* stream) {
    if (!h || !a) return DFLASH_ERR_INVALID_ARG;
    if (a->n_rows < 0 || a->vocab < 1 || !(a->temperature > 0.f) || !dtype_ok(a->logits_dtype)) return DFLASH_ERR_INVALID_ARG;
    if (a->n_rows == 0) return DFLASH_OK;
    if (a->n_rows > 65535) return DFLASH_ERR_UNSUPPORTED;      // rows are the grid's second dimension
    if (!a->logits || !a->u || !a->ids) return DFLASH_ERR_INVALID_ARG;
    if (!a->workspace || (reinterpret_cast<uintptr_t>(a->workspace) & 255)) return DFLASH_ERR_WORKSPACE;
    const int nseg = n_segments(a->vocab), seg_len = segment_len(a->vocab, nseg);
    const int n_stat = n_stat_segments(a->vocab);
    const Scratch s = carve_scratch(a->workspace, a->n_rows, a->n_rows, nseg, n_stat);
    if (s.bytes > a->workspace_bytes) return DFLASH_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const float c = LOG2E / a->temperature;
    const int64_t ld = a->row_stride ? a->row_stride : a->vocab;
    const StatsJob none = stats_job(nullptr, DFLASH_F32, 0, 0, 1, 1);
    SAMPLE_TRY(launch_stats(st, stats_job(a->logits, a->logits_dtype, ld, a->n_rows, a->n_rows, a->n_rows), none, a->vocab, n_stat, c, s,
                            a->n_rows));
    const cudaError_t e = launch_pdl(rows_draw_kernel, dim3(nseg, a->n_rows), dim3(DRAW_WARPS * 32), 0, st, a->logits,
                                     (int)(a->logits_dtype == DFLASH_BF16), ld, a->logits_dtype == DFLASH_BF16 ? 2 : 4, a->vocab, seg_len,
                                     c, (const float2*)s.stats, n_stat, a->u, a->ids, a->prob, s.seg_w, s.tickets);
    g_launches += 1;
    return e == cudaSuccess ? DFLASH_OK : DFLASH_ERR_CUDA;
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
    if (a->gamma > PLAN_MAX_GAMMA || (int64_t)a->batch * (2 * a->gamma + 1) > 65535) return DFLASH_ERR_UNSUPPORTED;
    if (!a->workspace || (reinterpret_cast<uintptr_t>(a->workspace) & 255)) return DFLASH_ERR_WORKSPACE;
    const int nseg = n_segments(a->vocab), seg_len = segment_len(a->vocab, nseg);
    const int64_t t_rows = (int64_t)a->batch * (a->gamma + 1), d_rows = (int64_t)a->batch * a->gamma;
    const int n_stat = n_stat_segments(a->vocab);
    const Scratch s = carve_scratch(a->workspace, t_rows + d_rows, a->batch, nseg, n_stat);
    if (s.bytes > a->workspace_bytes) return DFLASH_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const float c = LOG2E / a->temperature;
    const int64_t t_ld = a->target_row_stride ? a->target_row_stride : a->vocab;
    const int64_t d_ld = a->draft_row_stride ? a->draft_row_stride : a->vocab;
    // the gamma draft rows of sequence b start at stored row b * draft_rows_per_seq
    SAMPLE_TRY(launch_stats(st, stats_job(a->target_logits, a->target_dtype, t_ld, (int)t_rows, (int)t_rows, (int)t_rows),
                            stats_job(a->draft_logits, a->draft_dtype, d_ld, (int)d_rows, a->gamma, a->draft_rows_per_seq), a->vocab, n_stat,
                            c, s, a->batch));
    const float2* d_stats = s.stats + t_rows * n_stat;
    const cudaError_t e = launch_pdl(verify_draw_kernel, dim3(nseg, a->batch), dim3(DRAW_WARPS * 32), 0, st, *a, seg_len, c,
                                     (const float2*)s.stats, d_stats, n_stat, s.seg_w, s.tickets);
    g_launches += 1;
    return e == cudaSuccess ? DFLASH_OK : DFLASH_ERR_CUDA;
}

}  // extern "C"
