// Training side: position-weighted cross entropy of draft blocks (Sec. 4.2 "Loss weighting", Eq. 4):
//   w_k = exp(-(k - 1) / gamma) for block position k >= 1 (position 0 is the clean anchor, no loss),
//   row_loss = w_k (logsumexp(z) - z[target]),  dlogits = grad_scale w_k (softmax(z) - onehot(target)).
// HBM-bound streaming over the logits in one launch: persistent CTAs take whole rows; a CTA reads its row
// once for the maximum and the sum of exponentials and a second time, from L2 (the row was just read and
// a few hundred rows in flight fit the cache), to write the gradient. A last launch adds the rows up in a
// fixed order.
#include "softmax_rows.cuh"

namespace dflash {
namespace {

constexpr int LOSS_THREADS = 512, LOSS_CTAS_PER_SM = 2;      // the rows in flight (one per CTA, read twice) must fit L2

struct LossParams {
    const void* logits;
    const int32_t* targets;
    void* dlogits;
    float* row_loss;
    int32_t* status;
    int64_t ld, d_ld;
    int32_t in_bf16, out_bf16, vocab, B, n_rows;
    float inv_gamma, grad_scale;
};

// i a multiple of 8, row 16-byte aligned
__device__ __forceinline__ void load8(const void* row, int bf16, int i, float (&z)[8]) {
    if (bf16) {
        const uint4 v = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(row) + i);
        unpack16(v, z, __nv_bfloat16());
    } else {
        float a[4], b[4];
        unpack16(*reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(row) + i), a, 0.f);
        unpack16(*reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(row) + i + 4), b, 0.f);
#pragma unroll
        for (int e = 0; e < 4; ++e) { z[e] = a[e]; z[4 + e] = b[e]; }
    }
}
__device__ __forceinline__ void store8(void* row, int bf16, int i, const float (&g)[8]) {
    if (bf16) {
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(g[2 * e], g[2 * e + 1]);
            w[e] = *reinterpret_cast<const uint32_t*>(&h);
        }
        __stcs(reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(row) + i), make_uint4(w[0], w[1], w[2], w[3]));
    } else {      // streaming stores: the gradient is not read again and should not push the logits out of L2
        float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(row) + i);
        __stcs(dst, make_float4(g[0], g[1], g[2], g[3]));
        __stcs(dst + 1, make_float4(g[4], g[5], g[6], g[7]));
    }
}
__device__ __forceinline__ void store1(void* row, int bf16, int i, float g) {
    if (bf16) reinterpret_cast<__nv_bfloat16*>(row)[i] = __float2bfloat16_rn(g);
    else reinterpret_cast<float*>(row)[i] = g;
}

// persistent: CTA c takes rows c, c + gridDim.x, ...
__global__ void __launch_bounds__(LOSS_THREADS, LOSS_CTAS_PER_SM) block_loss_kernel(const LossParams p) {
    __shared__ float2 sh[LOSS_THREADS / 32];
    __shared__ float s_zt;
    ptx::pdl_trigger();
    ptx::pdl_wait();
    const int es_in = p.in_bf16 ? 2 : 4, es_out = p.out_bf16 ? 2 : 4;
    for (int row = blockIdx.x; row < p.n_rows; row += gridDim.x) {
        const int k = row % p.B;
        const char* z_row = reinterpret_cast<const char*>(p.logits) + (size_t)row * p.ld * es_in;
        char* g_row = p.dlogits ? reinterpret_cast<char*>(p.dlogits) + (size_t)row * p.d_ld * es_out : nullptr;
        int t = p.targets[row];
        if (t >= p.vocab) {
            if (threadIdx.x == 0 && p.status) atomicOr(p.status, DFLASH_DEV_BAD_TOKEN);
            t = -1;
        }
        const bool on = k > 0 && t >= 0;
        float w = 0.f, lse = 0.f;
        if (on) {
            __syncthreads();            // sh / s_zt of the previous row are no longer read
            if (threadIdx.x == 0) s_zt = ld_logit(z_row, p.in_bf16, t);      // before any store: dlogits may alias logits
            const float2 st = p.in_bf16 ? segment_stats(reinterpret_cast<const __nv_bfloat16*>(z_row), 0, p.vocab, LOG2E, sh)
                                        : segment_stats(reinterpret_cast<const float*>(z_row), 0, p.vocab, LOG2E, sh);
            w = expf(-(float)(k - 1) * p.inv_gamma);
            lse = st.x + logf(st.y);
        }
        if (threadIdx.x == 0) p.row_loss[row] = on ? w * (lse - s_zt) : 0.f;
        if (!g_row) continue;
        const float gw = p.grad_scale * w, neg_lc = -lse * LOG2E;
        const bool vec = ((reinterpret_cast<uintptr_t>(z_row) | reinterpret_cast<uintptr_t>(g_row)) & 15) == 0;
        const int n8 = vec ? p.vocab / 8 : 0;
        constexpr int U = 2;            // 8-element groups per thread in flight
        for (int v0 = threadIdx.x; v0 < n8; v0 += blockDim.x * U) {
            float z[U][8];
            if (on) {
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int v = v0 + u * blockDim.x;
                    if (v < n8) load8(z_row, p.in_bf16, v * 8, z[u]);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v0 + u * blockDim.x;
                if (v < n8) {
                    float g[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) g[e] = on ? gw * fast_exp2(fmaf(z[u][e], LOG2E, neg_lc)) : 0.f;
                    store8(g_row, p.out_bf16, v * 8, g);
                }
            }
        }
        for (int i = n8 * 8 + threadIdx.x; i < p.vocab; i += blockDim.x) {
            const float g = on ? gw * fast_exp2(fmaf(ld_logit(z_row, p.in_bf16, i), LOG2E, neg_lc)) : 0.f;
            store1(g_row, p.out_bf16, i, g);
        }
        if (on) {       // the target's entry: softmax - 1, from the logit read before the row was overwritten
            __syncthreads();
            if (threadIdx.x == 0) store1(g_row, p.out_bf16, t, gw * (fast_exp2(fmaf(s_zt, LOG2E, neg_lc)) - 1.f));
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Rows that allow 16-byte accesses: a cluster of CS CTAs per row, each CTA holding its 1/CS of the row in
// shared memory, so the logits cross HBM exactly once whatever L2 keeps. The CTAs exchange their (max, sum)
// through distributed shared memory around one cluster barrier per row.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {      // every thread of every CTA of the cluster
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void st_cluster_f2(const void* local_smem, uint32_t cta_rank, float2 v) {      // the same variable in CTA cta_rank
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(ptx::smem_u32(local_smem)), "r"(cta_rank));
    asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(remote), "f"(v.x), "f"(v.y) : "memory");
}

constexpr int CLU_THREADS = 1024, CLU_CTAS_PER_SM = 1, CLU_MAX = 4;      // (two 512-thread CTAs per SM in clusters of 4 / 8: measured 1.4 x slower)
constexpr int CLU_PART_BYTES = 160 * 1024;        // the most one CTA keeps of a row

// Running (max, sum of exponentials) of one thread; a finite floor instead of -inf keeps the updates branch-free
struct RunStat {
    float m, z, neg_mc;
    __device__ __forceinline__ void reset() { m = -1.0e30f; z = 0.f; neg_mc = 1.0e30f * LOG2E; }
    template <int N>
    __device__ __forceinline__ void add(const float (&f)[N]) {
        float mx = f[0];
#pragma unroll
        for (int e = 1; e < N; ++e) mx = fmaxf(mx, f[e]);
        if (mx > m) {                     // rare after the first entries
            z *= fast_exp2((m - mx) * LOG2E);
            m = mx;
            neg_mc = -mx * LOG2E;
        }
#pragma unroll
        for (int e = 0; e < N; ++e) z += fast_exp2(fmaf(f[e], LOG2E, neg_mc));
    }
};

template <typename IN, int CS>
__global__ void __launch_bounds__(CLU_THREADS, CLU_CTAS_PER_SM) block_loss_cluster_kernel(const LossParams p, int part) {      // part: elements per CTA
    constexpr int EI = 16 / (int)sizeof(IN), LB = 4;      // elements per 16-byte vector; vectors per thread in flight
    extern __shared__ uint4 buf[];                      // this CTA's part of the row (slot v belongs to thread v % T)
    __shared__ float2 sh[CLU_THREADS / 32];
    __shared__ float2 peer[2][CLU_MAX];                 // [row parity][CTA rank]: written by the peers
    ptx::pdl_wait();
    const int tid = threadIdx.x, T = blockDim.x;
    const int rank = (int)cluster_ctarank(), cid = blockIdx.x / CS, n_clusters = gridDim.x / CS;
    const int lo = min(rank * part, p.vocab), hi = min(p.vocab, lo + part), n_vec = (hi - lo) / EI;      // vocab is a multiple of 8 here
    const int es_out = p.out_bf16 ? 2 : 4;
    auto g_of = [&](int row) { return p.dlogits ? reinterpret_cast<char*>(p.dlogits) + (size_t)row * p.d_ld * es_out : nullptr; };
    auto src_of = [&](int row) { return reinterpret_cast<const uint4*>(reinterpret_cast<const IN*>(p.logits) + (size_t)row * p.ld + lo); };
    // The first row at or after `row` (in this cluster's sequence) that carries loss; the rows passed on the way get
    // their zeros. Every CTA of the cluster takes the same decisions.
    auto advance = [&](int row, int& t_out) {
        for (; row < p.n_rows; row += n_clusters) {
            int t = p.targets[row];
            if (t >= p.vocab) {
                if (rank == 0 && tid == 0 && p.status) atomicOr(p.status, DFLASH_DEV_BAD_TOKEN);
                t = -1;
            }
            if (row % p.B > 0 && t >= 0) { t_out = t; return row; }
            if (rank == 0 && tid == 0) p.row_loss[row] = 0.f;
            if (char* g_row = g_of(row)) {
                const float zero[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                for (int i = lo + tid * 8; i < hi; i += T * 8) store8(g_row, p.out_bf16, i, zero);      // hi - lo is a multiple of 8
            }
        }
        t_out = -1;
        return row;
    };
    cluster_sync_all();                                 // every CTA of the cluster is running before anyone writes into it
    int parity = 0, t = -1;
    int row = advance(cid, t);
    RunStat rs;
    rs.reset();
    if (row < p.n_rows) {                               // the first row: HBM -> registers -> shared memory, with the running statistics
        const uint4* src = src_of(row);
        for (int v0 = tid; v0 < n_vec; v0 += T * LB) {
            uint4 raw[LB];
#pragma unroll
            for (int u = 0; u < LB; ++u) raw[u] = v0 + u * T < n_vec ? src[v0 + u * T] : make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int u = 0; u < LB; ++u) {
                if (v0 + u * T < n_vec) {
                    buf[v0 + u * T] = raw[u];
                    float f[EI];
                    unpack16(raw[u], f, IN());
                    rs.add(f);
                }
            }
        }
    }
    while (row < p.n_rows) {
        // ---- this row's statistics: warp, CTA, cluster
        // (floors stay finite through the warp merge: exp2 of a huge negative number is 0, never inf - inf)
        float wm = rs.m, wz = rs.z;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float om = __shfl_xor_sync(0xffffffffu, wm, o), oz = __shfl_xor_sync(0xffffffffu, wz, o);
            const float nm = fmaxf(wm, om);
            wz = wz * fast_exp2((wm - nm) * LOG2E) + oz * fast_exp2((om - nm) * LOG2E);
            wm = nm;
        }
        if ((tid & 31) == 0) sh[tid >> 5] = make_float2(wz > 0.f ? wm : -CUDART_INF_F, wz);
        __syncthreads();
        if (tid < CS) {                                 // thread r tells CTA r this CTA's result
            float m = sh[0].x;
            for (int w = 1; w < (T >> 5); ++w) m = fmaxf(m, sh[w].x);
            float z = 0.f;
            if (m > -CUDART_INF_F)
                for (int w = 0; w < (T >> 5); ++w) z += sh[w].y > 0.f ? sh[w].y * fast_exp2((sh[w].x - m) * LOG2E) : 0.f;
            st_cluster_f2(&peer[parity][rank], (uint32_t)tid, make_float2(m, z));
        }
        __syncwarp();                                   // the aligned barrier below wants whole warps
        cluster_sync_all();                             // every CTA's result has arrived in every CTA (and sh is free again)
        float m = peer[parity][0].x;
#pragma unroll
        for (int r = 1; r < CS; ++r) m = fmaxf(m, peer[parity][r].x);
        float z = 0.f;
#pragma unroll
        for (int r = 0; r < CS; ++r) z += peer[parity][r].y > 0.f ? peer[parity][r].y * fast_exp2((peer[parity][r].x - m) * LOG2E) : 0.f;
        parity ^= 1;
        const float w_k = __expf(-(float)(row % p.B - 1) * p.inv_gamma);
        const float lse = m + __logf(z);
        const int t_loc = t - lo;                       // the target's place in this CTA's part, if it is here
        if (t_loc >= 0 && t_loc < hi - lo && (t_loc / EI) % T == tid)      // read by the slot's own thread, before that thread reuses the slot
            p.row_loss[row] = w_k * (lse - as_f(reinterpret_cast<const IN*>(buf)[t_loc]));
        // ---- the gradient of this row from shared memory; each slot, once read, takes the next row's logits
        char* g_row = g_of(row);
        const float gw = p.grad_scale * w_k, neg_lc = -lse * LOG2E;
        int t_next = -1;
        const int next = advance(row + n_clusters, t_next);
        const bool more = next < p.n_rows;
        const uint4* src = more ? src_of(next) : nullptr;
        rs.reset();
        for (int v0 = tid; v0 < n_vec; v0 += T * LB) {
            uint4 raw[LB];
            if (more) {
#pragma unroll
                for (int u = 0; u < LB; ++u) raw[u] = v0 + u * T < n_vec ? src[v0 + u * T] : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < LB; ++u) {
                const int v = v0 + u * T;
                if (v < n_vec) {
                    float f[EI];
                    if (g_row) {
                        float g[EI];
                        unpack16(buf[v], f, IN());
#pragma unroll
                        for (int e = 0; e < EI; ++e) g[e] = gw * fast_exp2(fmaf(f[e], LOG2E, neg_lc));
                        const int d = t_loc - v * EI;
                        if (d >= 0 && d < EI) {
#pragma unroll
                            for (int e = 0; e < EI; ++e)
                                if (e == d) g[e] -= gw;
                        }
                        const int i = lo + v * EI;
                        if constexpr (EI == 8) {
                            store8(g_row, p.out_bf16, i, g);
                        } else {
                            if (p.out_bf16) {
                                const __nv_bfloat162 h0 = __floats2bfloat162_rn(g[0], g[1]), h1 = __floats2bfloat162_rn(g[2], g[3]);
                                __stcs(reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(g_row) + i),
                                       make_uint2(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1)));
                            } else {
                                __stcs(reinterpret_cast<float4*>(reinterpret_cast<float*>(g_row) + i), make_float4(g[0], g[1], g[2], g[3]));
                            }
                        }
                    }
                    if (more) {
                        buf[v] = raw[u];
                        unpack16(raw[u], f, IN());
                        rs.add(f);
                    }
                }
            }
        }
        row = next;
        t = t_next;
    }
    cluster_sync_all();                                 // nobody leaves while a peer may still write into it
}

// CTAs per row for this element size and vocabulary, or 0 if the cluster kernel does not apply
int cluster_size_for(int vocab, int es) {
    for (int cs = 2; cs <= CLU_MAX; cs *= 2) {
        const int64_t part = (((int64_t)vocab + cs - 1) / cs + 7) / 8 * 8;
        if (part * es <= CLU_PART_BYTES) return cs;
    }
    return 0;
}

template <typename IN, int CS>
cudaError_t launch_cluster(const LossParams& p, int part, int sm_count, cudaStream_t st) {
    const size_t smem = (size_t)part * sizeof(IN);
    static bool attr_set[MAX_DEVICES] = {};
    static int resident[MAX_DEVICES] = {};
    const int dev = current_device_slot();
    if (dev < 0) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
        const cudaError_t e = cudaFuncSetAttribute(block_loss_cluster_kernel<IN, CS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                   CLU_PART_BYTES);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(sm_count / CS * CS);
    cfg.blockDim = dim3(CLU_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CS;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // as many clusters as can be resident at once (an SM left over in a GPC cannot host half a cluster):
    // the clusters are persistent, so one that had to wait for a free pair of SMs would run after all the others
    if (resident[dev] == 0) {
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, block_loss_cluster_kernel<IN, CS>, &cfg) != cudaSuccess || n < 1) n = sm_count / CS;
        resident[dev] = n;
    }
    const int n_clusters = std::max(1, std::min(p.n_rows, std::min(resident[dev], sm_count * CLU_CTAS_PER_SM / CS)));
    cfg.gridDim = dim3(n_clusters * CS);
    return cudaLaunchKernelEx(&cfg, block_loss_cluster_kernel<IN, CS>, p, part);
}

// one CTA: sum of the row losses and of the weights that count, in double, in a fixed order
__global__ void __launch_bounds__(256) block_loss_sum_kernel(const float* __restrict__ row_loss, const int32_t* __restrict__ targets,
                                                             int n_rows, int B, int vocab, float inv_gamma, float* __restrict__ out) {
    __shared__ double sh[2 * 8];
    ptx::pdl_trigger();
    ptx::pdl_wait();
    double a = 0.0, b = 0.0;
    for (int i = threadIdx.x; i < n_rows; i += blockDim.x) {
        const int k = i % B, t = targets[i];
        if (k > 0 && t >= 0 && t < vocab) {
            a += (double)row_loss[i];
            b += (double)expf(-(float)(k - 1) * inv_gamma);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        a += __shfl_xor_sync(0xffffffffu, a, o);
        b += __shfl_xor_sync(0xffffffffu, b, o);
    }
    if ((threadIdx.x & 31) == 0) { sh[2 * (threadIdx.x >> 5)] = a; sh[2 * (threadIdx.x >> 5) + 1] = b; }
    __syncthreads();
    if (threadIdx.x == 0) {
        a = 0.0; b = 0.0;
        for (int w = 0; w < 8; ++w) { a += sh[2 * w]; b += sh[2 * w + 1]; }
        out[0] = (float)a;
        out[1] = (float)b;
    }
}

}  // namespace
}  // namespace dflash

using namespace dflash;

extern "C" {

int32_t dflash_block_loss(dflash_handle* h, const dflash_block_loss_args* a, void* stream) {
    if (!h || !a) return DFLASH_ERR_INVALID_ARG;
    if (a->n_blocks < 0 || a->block_rows < 1 || a->vocab < 1 || !(a->gamma > 0.f)) return DFLASH_ERR_INVALID_ARG;
    if (a->logits_dtype != DFLASH_F32 && a->logits_dtype != DFLASH_BF16) return DFLASH_ERR_INVALID_ARG;
    if (a->dlogits && a->dlogits_dtype != DFLASH_F32 && a->dlogits_dtype != DFLASH_BF16) return DFLASH_ERR_INVALID_ARG;
    const int64_t n_rows = (int64_t)a->n_blocks * a->block_rows;
    if (n_rows > (1ll << 30)) return DFLASH_ERR_UNSUPPORTED;
    if (n_rows == 0) return DFLASH_OK;
    if (!a->logits || !a->targets || !a->row_loss) return DFLASH_ERR_INVALID_ARG;
    const int64_t ld = a->row_stride ? a->row_stride : a->vocab, d_ld = a->dlogits_row_stride ? a->dlogits_row_stride : a->vocab;
    if (ld < a->vocab || d_ld < a->vocab) return DFLASH_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    LossParams p{};
    p.logits = a->logits; p.targets = a->targets; p.dlogits = a->dlogits; p.row_loss = a->row_loss; p.status = a->dev_status;
    p.ld = ld; p.d_ld = d_ld; p.in_bf16 = a->logits_dtype == DFLASH_BF16; p.out_bf16 = a->dlogits_dtype == DFLASH_BF16;
    p.vocab = a->vocab; p.B = a->block_rows; p.n_rows = (int)n_rows;
    p.inv_gamma = 1.f / a->gamma; p.grad_scale = a->grad_scale;
    const int es_in = p.in_bf16 ? 2 : 4, es_out = p.out_bf16 ? 2 : 4;
    const bool aligned = (reinterpret_cast<uintptr_t>(a->logits) & 15) == 0 && (ld * es_in) % 16 == 0 && a->vocab % 8 == 0 &&
                         (!a->dlogits || ((reinterpret_cast<uintptr_t>(a->dlogits) & 15) == 0 && (d_ld * es_out) % 16 == 0));
    const int cs = aligned ? cluster_size_for(a->vocab, es_in) : 0;
    cudaError_t e;
    if (cs > 0) {
        const int part = ((a->vocab + cs - 1) / cs + 7) / 8 * 8;
        if (p.in_bf16)
            e = cs == 2 ? launch_cluster<__nv_bfloat16, 2>(p, part, h->sm_count, st) : launch_cluster<__nv_bfloat16, 4>(p, part, h->sm_count, st);
        else
            e = cs == 2 ? launch_cluster<float, 2>(p, part, h->sm_count, st) : launch_cluster<float, 4>(p, part, h->sm_count, st);
    } else {
        const int grid = (int)std::min<int64_t>(n_rows, (int64_t)h->sm_count * LOSS_CTAS_PER_SM);
        e = launch_pdl(block_loss_kernel, dim3(grid), dim3(LOSS_THREADS), 0, st, p);
    }
    if (e != cudaSuccess) return DFLASH_ERR_CUDA;
    g_launches += 1;
    if (a->loss_sum) {
        if (launch_pdl(block_loss_sum_kernel, dim3(1), dim3(256), 0, st, (const float*)a->row_loss, a->targets, (int)n_rows, a->block_rows,
                       a->vocab, p.inv_gamma, a->loss_sum) != cudaSuccess)
            return DFLASH_ERR_CUDA;
        g_launches += 1;
    }
    return DFLASH_OK;
}

}  // extern "C"
