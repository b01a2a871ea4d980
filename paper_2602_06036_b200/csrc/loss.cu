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
    const int grid = (int)std::min<int64_t>(n_rows, (int64_t)h->sm_count * LOSS_CTAS_PER_SM);
    const cudaError_t e = launch_pdl(block_loss_kernel, dim3(grid), dim3(LOSS_THREADS), 0, st, p);
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
