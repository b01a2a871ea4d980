// bf16 contractions with few tokens and large weights (QKV / O / SwiGLU / LM head / context K,V):
//   acc[token][feature] = sum_k X[token][k] * W[feature][k]
// The WEIGHT tile is the 128-row "M" operand of tcgen05.mma and the tokens are its "N" operand
// (16..256 columns), so the tensor core runs full-height instructions however few tokens there
// are. A CTA is one TMA producer warp, one MMA-issuing warp and four epilogue warps; operands
// stream through a ring of 128-byte-swizzled shared-memory stages, accumulators live in two TMEM
// buffers so the epilogue of one work unit overlaps the main loop of the next. Work units are
// (feature tile, token tile, K split), walked persistently; K splits meet in a fixed-order sum done
// by whichever CTA arrives last at a ticket counter (no waiting, bit-reproducible).
// Every wait on an mbarrier is bounded; on expiry the kernel raises DFLASH_DEV_TIMEOUT, drains its
// outstanding copies, frees its TMEM and returns.
#include "gemm_tc.cuh"

#include "ptx_sm100.cuh"

#include <math_constants.h>

#include <algorithm>

namespace dflash {
namespace {

using namespace ptx;

constexpr int TILE_F = 128;                      // weight rows per tile = MMA M
constexpr int BK = 64;                           // K elements per stage = one 128-byte swizzle row
constexpr int CH = 16;                           // token columns handled per epilogue pass
constexpr int W_STAGE_BYTES = TILE_F * BK * 2;   // 16 KiB
constexpr int MAX_STAGES = 12;
constexpr int ACC_LD = CH + 1;
constexpr int SMEM_FIXED = TILE_F * ACC_LD * 4 + 128 * 16 + (2 * MAX_STAGES + 4) * 8 + 64;
constexpr int SMEM_LIMIT = 227 * 1024;
constexpr int N_THREADS = 192;

struct KParams {
    int M, N, K, epi, splits, chunks_total, chunks_per_split, n_ftiles, n_ttiles, stages;
    float* part;
    int32_t* counters;
    float* out_f32;
    int ld_out;
    __nv_bfloat16 *q, *k, *v;
    const int32_t* ctx_len;
    int rows_per_seq, Hq, Hkv, hd, use_rope;
    const float *cs, *sn;
    int max_pos;
    __nv_bfloat16* h;
    int F;
    Top2Entry* top2;
    float* logits_out;
    __nv_bfloat16* pool;
    const int32_t* n_new;
    const int32_t* page_table;
    int max_new, max_pages, n_pages, PG, layer;
    int32_t* status;
};

// ---------------------------------------------------------------------------------------------
// epilogues: 128 threads, thread `row` owns feature f0 + row; sAcc[row][c] holds 16 token columns
// ---------------------------------------------------------------------------------------------
struct T2 {
    float v1;
    int i1;
    float v2;
};
__device__ __forceinline__ void t2_push(T2& t, float v, int i) {
    if (v > t.v1 || (v == t.v1 && i < t.i1)) { t.v2 = t.v1; t.v1 = v; t.i1 = i; }
    else if (v > t.v2) t.v2 = v;
}
__device__ __forceinline__ void t2_merge(T2& a, float v1, int i1, float v2) {
    if (v1 > a.v1 || (v1 == a.v1 && i1 < a.i1)) { a.v2 = fmaxf(a.v1, v2); a.v1 = v1; a.i1 = i1; }
    else a.v2 = fmaxf(a.v2, v1);
}

__device__ __forceinline__ void apply_epilogue(const KParams& p, const float* sAcc, Top2Entry* sRed, int ft, int tok0,
                                               int row) {
    const int f = ft * TILE_F + row;
    const int n_tok = min(CH, p.M - tok0);
    switch (p.epi) {
        case EPI_STORE_F32:
        case EPI_RESIDUAL: {
            if (f < p.N) {
                float* o = p.out_f32 + (size_t)tok0 * p.ld_out + f;
                float prev[CH];
                // all loads first: they are independent and must not queue behind the stores
#pragma unroll
                for (int c = 0; c < CH; ++c)
                    prev[c] = (p.epi == EPI_RESIDUAL && c < n_tok) ? __ldcg(o + (size_t)c * p.ld_out) : 0.f;
#pragma unroll
                for (int c = 0; c < CH; ++c)
                    if (c < n_tok) o[(size_t)c * p.ld_out] = prev[c] + sAcc[row * ACC_LD + c];
            }
        } break;
        case EPI_QKV_ROPE: {
            if (f < p.N) {
                const int hd = p.hd, half = hd >> 1;
                const int head = f / hd, hrow = f % hd, i = hrow % half;
                const int partner = row ^ half;
                const int qdim = p.Hq * hd, kdim = p.Hkv * hd;
                const bool rot = p.use_rope && head < p.Hq + p.Hkv;
                float cs[CH], sn[CH];
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    cs[c] = 1.f; sn[c] = 0.f;
                    if (rot && c < n_tok) {
                        const int tok = tok0 + c;
                        int pos = __ldg(p.ctx_len + tok / p.rows_per_seq) + tok % p.rows_per_seq;
                        if (pos < 0 || pos >= p.max_pos) {
                            if (row == 0 && p.status) atomicOr(p.status, DFLASH_DEV_CTX_OVERFLOW);
                            pos = pos < 0 ? 0 : p.max_pos - 1;
                        }
                        cs[c] = __ldg(p.cs + (size_t)pos * half + i);
                        sn[c] = __ldg(p.sn + (size_t)pos * half + i);
                    }
                }
                __nv_bfloat16* dst;
                int ld;
                if (head < p.Hq) { dst = p.q + f; ld = qdim; }
                else if (head < p.Hq + p.Hkv) { dst = p.k + (f - qdim); ld = kdim; }
                else { dst = p.v + (f - qdim - kdim); ld = kdim; }
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    if (c >= n_tok) break;
                    const float a = sAcc[row * ACC_LD + c], b = sAcc[partner * ACC_LD + c];
                    const float val = hrow < half ? (a * cs[c] - b * sn[c]) : (a * cs[c] + b * sn[c]);
                    dst[(size_t)(tok0 + c) * ld] = __float2bfloat16_rn(val);
                }
            }
        } break;
        case EPI_SWIGLU: {
            if ((row & 1) == 0 && f + 1 < p.N) {
                const int j = f >> 1;
                for (int c = 0; c < n_tok; ++c) {
                    const float g = sAcc[row * ACC_LD + c], u = sAcc[(row + 1) * ACC_LD + c];
                    p.h[(size_t)(tok0 + c) * p.F + j] = __float2bfloat16_rn(g / (1.f + __expf(-g)) * u);
                }
            }
        } break;
        case EPI_ARGMAX: {
            if (p.logits_out && f < p.N)
                for (int c = 0; c < n_tok; ++c) p.logits_out[(size_t)(tok0 + c) * p.N + f] = sAcc[row * ACC_LD + c];
            const int c = row & 15, g = row >> 4;
            T2 t{-CUDART_INF_F, 0x7fffffff, -CUDART_INF_F};
#pragma unroll
            for (int r = 0; r < 16; ++r) {
                const int rr = g * 16 + r, ff = ft * TILE_F + rr;
                if (ff < p.N) t2_push(t, sAcc[rr * ACC_LD + c], ff);
            }
            sRed[g * 16 + c] = Top2Entry{t.v1, t.i1, t.v2, 0};
            epi_bar();
            if (row < n_tok) {
                T2 m{sRed[row].v1, sRed[row].i1, sRed[row].v2};
#pragma unroll
                for (int gg = 1; gg < 8; ++gg) t2_merge(m, sRed[gg * 16 + row].v1, sRed[gg * 16 + row].i1, sRed[gg * 16 + row].v2);
                p.top2[(size_t)ft * p.M + tok0 + row] = Top2Entry{m.v1, m.i1, m.v2, 0};
            }
        } break;
        case EPI_CTX_KV: {
            if (f < p.N) {
                const int hd = p.hd, half = hd >> 1;
                const int kdim = p.Hkv * hd;
                const int is_v = f >= kdim ? 1 : 0;
                const int fh = f - is_v * kdim;
                const int head = fh / hd, hrow = fh % hd, i = hrow % half;
                const int partner = row ^ half;
                for (int c = 0; c < n_tok; ++c) {
                    const int tok = tok0 + c;
                    const int b = tok / p.max_new, r = tok % p.max_new;
                    const int nn = p.n_new ? p.n_new[b] : p.max_new;
                    if (r >= nn) continue;
                    const int pos = p.ctx_len[b] + r;
                    const int pidx = pos / p.PG;
                    if (pos < 0 || pidx >= p.max_pages || (p.use_rope && pos >= p.max_pos)) {
                        if (row == 0 && p.status) atomicOr(p.status, DFLASH_DEV_CTX_OVERFLOW);
                        continue;
                    }
                    const int page = p.page_table[(size_t)b * p.max_pages + pidx];
                    if (page < 0 || page >= p.n_pages) {
                        if (row == 0 && p.status) atomicOr(p.status, DFLASH_DEV_BAD_PAGE);
                        continue;
                    }
                    float val = sAcc[row * ACC_LD + c];
                    if (!is_v && p.use_rope) {
                        const float bb = sAcc[partner * ACC_LD + c];
                        const float cs = p.cs[(size_t)pos * half + i], sn = p.sn[(size_t)pos * half + i];
                        val = hrow < half ? (val * cs - bb * sn) : (val * cs + bb * sn);
                    }
                    const size_t dst = (((((size_t)p.layer * p.n_pages + page) * 2 + is_v) * p.Hkv + head) * p.PG +
                                        (pos % p.PG)) * hd + hrow;
                    p.pool[dst] = __float2bfloat16_rn(val);
                }
            }
        } break;
        default: break;
    }
}

// ---------------------------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------------------------
template <int NT>
__global__ void __launch_bounds__(N_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, const KParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    constexpr int X_STAGE_BYTES = NT * BK * 2;
    constexpr uint32_t TMEM_COLS = (2 * NT < 32) ? 32u : (uint32_t)(2 * NT);
    const int stages = p.stages;
    uint8_t* sW = smem;
    uint8_t* sX = sW + (size_t)stages * W_STAGE_BYTES;
    float* sAcc = reinterpret_cast<float*>(sX + (size_t)stages * X_STAGE_BYTES);
    Top2Entry* sRed = reinterpret_cast<Top2Entry*>(sAcc + TILE_F * ACC_LD);
    uint64_t* full = reinterpret_cast<uint64_t*>(sRed + 128);
    uint64_t* empty = full + MAX_STAGES;
    uint64_t* acc_full = empty + MAX_STAGES;
    uint64_t* acc_empty = acc_full + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    volatile int* flags = reinterpret_cast<volatile int*>(tmem_slot + 1);   // [0] abort, [1] last-arriver, [2] epilogue abort

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 4); }
        flags[0] = 0; flags[1] = 0; flags[2] = 0;
        fence_barrier_init();
        fence_proxy_async();
    }
    if (warp == 1) tmem_alloc(tmem_slot, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int total_units = p.n_ftiles * p.n_ttiles * p.splits;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            const uint64_t pol_w = policy_evict_first(), pol_x = policy_evict_last();
            uint32_t it = 0;
            bool ok = true;
            for (int u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
                const int s = u % p.splits, tt = (u / p.splits) % p.n_ttiles, ft = u / (p.splits * p.n_ttiles);
                const int c0 = s * p.chunks_per_split, c1 = min(c0 + p.chunks_per_split, p.chunks_total);
                for (int c = c0; c < c1; ++c, ++it) {
                    const int st = it % stages;
                    const uint32_t ph = (it / stages) & 1;
                    if (!mbar_wait(&empty[st], ph ^ 1, &flags[0])) { ok = false; break; }
                    mbar_expect_tx(&full[st], W_STAGE_BYTES + X_STAGE_BYTES);
                    tma_load_2d(sW + (size_t)st * W_STAGE_BYTES, &tmW, c * BK, ft * TILE_F, &full[st], pol_w);
                    tma_load_2d(sX + (size_t)st * X_STAGE_BYTES, &tmX, c * BK, tt * NT, &full[st], pol_x);
                }
            }
            if (!ok) {
                flags[0] = 1;
                if (p.status) atomicOr(p.status, DFLASH_DEV_TIMEOUT);
                // give copies already issued a chance to land before the CTA goes away
                const int n_out = min((int)it, stages);
                for (int j = 0; j < n_out; ++j) {
                    const uint32_t jt = it - 1 - j;
                    volatile int never = 0;
                    mbar_wait(&full[jt % stages], (jt / stages) & 1, &never, DRAIN_LIMIT);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc_bf16(TILE_F, NT);
            uint32_t it = 0, ui = 0;
            bool ok = true;
            for (int u = blockIdx.x; u < total_units && ok; u += gridDim.x, ++ui) {
                const int s = u % p.splits;
                const int c0 = s * p.chunks_per_split, c1 = min(c0 + p.chunks_per_split, p.chunks_total);
                const uint32_t buf = ui & 1, aph = (ui >> 1) & 1;
                if (!mbar_wait(&acc_empty[buf], aph ^ 1, &flags[0])) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * NT;
                for (int c = c0; c < c1; ++c, ++it) {
                    const int st = it % stages;
                    const uint32_t ph = (it / stages) & 1;
                    if (!mbar_wait(&full[st], ph, &flags[0])) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(sW + (size_t)st * W_STAGE_BYTES);
                    const uint32_t b_addr = smem_u32(sX + (size_t)st * X_STAGE_BYTES);
#pragma unroll
                    for (int kk = 0; kk < BK / 16; ++kk)
                        mma_bf16(d_tmem, smem_desc_sw128(a_addr + kk * 32), smem_desc_sw128(b_addr + kk * 32), idesc,
                                 (c > c0 || kk > 0) ? 1u : 0u);
                    mma_commit(&empty[st]);
                }
                if (ok) mma_commit(&acc_full[buf]);
            }
            if (!ok) {
                flags[0] = 1;
                if (p.status) atomicOr(p.status, DFLASH_DEV_TIMEOUT);
            }
        }
    } else {
        // ---------------- epilogue: warps 2..5, TMEM lane quadrant = warp % 4 ----------------
        const int ew = warp & 3;
        const int row = ew * 32 + lane;
        uint32_t ui = 0;
        for (int u = blockIdx.x; u < total_units; u += gridDim.x, ++ui) {
            const int s = u % p.splits, tt = (u / p.splits) % p.n_ttiles, ft = u / (p.splits * p.n_ttiles);
            const uint32_t buf = ui & 1, aph = (ui >> 1) & 1;
            const bool got = mbar_wait(&acc_full[buf], aph, &flags[0]);
            if (!got) flags[2] = 1;
            epi_bar();
            if (flags[2]) break;   // uniform over the four warps
            tc_fence_after();
            const int tok_base = tt * NT;
            const int n_ch = (min(NT, p.M - tok_base) + CH - 1) / CH;
            const int unit_tile = ft * p.n_ttiles + tt;
            for (int ch = 0; ch < n_ch; ++ch) {
                float v[CH];
                tmem_ld16(tmem_base + buf * NT + ch * CH + ((uint32_t)(ew * 32) << 16), v);
                if (p.splits > 1) {
                    float* dst = p.part + (((size_t)unit_tile * p.splits + s) * NT + ch * CH) * TILE_F + row;
#pragma unroll
                    for (int c = 0; c < CH; ++c) dst[(size_t)c * TILE_F] = v[c];
                } else {
#pragma unroll
                    for (int c = 0; c < CH; ++c) sAcc[row * ACC_LD + c] = v[c];
                    epi_bar();
                    apply_epilogue(p, sAcc, sRed, ft, tok_base + ch * CH, row);
                    epi_bar();
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
            if (p.splits > 1) {
                // ticket: the CTA that completes the set sums the slices in split order
                __threadfence();
                epi_bar();
                if (row == 0) {
                    const int old = atomicAdd(p.counters + unit_tile, 1);
                    flags[1] = (old == p.splits - 1) ? 1 : 0;
                    if (old == p.splits - 1) p.counters[unit_tile] = 0;   // ready for the next launch
                }
                epi_bar();
                if (flags[1]) {
                    __threadfence();
                    for (int ch = 0; ch < n_ch; ++ch) {
                        float acc[CH];
#pragma unroll
                        for (int c = 0; c < CH; ++c) acc[c] = 0.f;
                        for (int ss = 0; ss < p.splits; ++ss) {
                            const float* src = p.part + (((size_t)unit_tile * p.splits + ss) * NT + ch * CH) * TILE_F + row;
#pragma unroll
                            for (int c = 0; c < CH; ++c) acc[c] += __ldcg(src + (size_t)c * TILE_F);
                        }
#pragma unroll
                        for (int c = 0; c < CH; ++c) sAcc[row * ACC_LD + c] = acc[c];
                        epi_bar();
                        apply_epilogue(p, sAcc, sRed, ft, tok_base + ch * CH, row);
                        epi_bar();
                    }
                }
                epi_bar();   // flags[1] is rewritten by the next unit
            }
        }
        if (flags[2] && row == 0) {
            flags[0] = 1;
            if (p.status) atomicOr(p.status, DFLASH_DEV_TIMEOUT);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// one CTA per token: merge the per-tile winners in tile order (index-aware, so order-independent)
__global__ void __launch_bounds__(128) argmax_finish_kernel(const Top2Entry* __restrict__ top2, int n_tiles, int M,
                                                            int32_t* __restrict__ ids, float* __restrict__ top1,
                                                            float* __restrict__ margin) {
    __shared__ Top2Entry sh[4];
    const int tok = blockIdx.x;
    T2 t{-CUDART_INF_F, 0x7fffffff, -CUDART_INF_F};
    for (int i = threadIdx.x; i < n_tiles; i += blockDim.x) {
        const Top2Entry e = top2[(size_t)i * M + tok];
        t2_merge(t, e.v1, e.i1, e.v2);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float v1 = __shfl_xor_sync(0xffffffffu, t.v1, o);
        const int i1 = __shfl_xor_sync(0xffffffffu, t.i1, o);
        const float v2 = __shfl_xor_sync(0xffffffffu, t.v2, o);
        t2_merge(t, v1, i1, v2);
    }
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = Top2Entry{t.v1, t.i1, t.v2, 0};
    __syncthreads();
    if (threadIdx.x == 0) {
        T2 r{sh[0].v1, sh[0].i1, sh[0].v2};
        for (int w = 1; w < 4; ++w) t2_merge(r, sh[w].v1, sh[w].i1, sh[w].v2);
        ids[tok] = r.i1 == 0x7fffffff ? 0 : r.i1;
        if (top1) top1[tok] = r.v1;
        if (margin) margin[tok] = r.v1 - r.v2;
    }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
// [rows, K] bf16 row-major; box = 64 K-elements x box_rows rows
bool make_map(CUtensorMap* m, const void* base, int rows, int K, int box_rows) {
    const uint64_t dims[2] = {(uint64_t)K, (uint64_t)rows};
    const uint64_t strides[1] = {(uint64_t)K * 2};
    const uint32_t box[2] = {(uint32_t)BK, (uint32_t)box_rows};
    return tmap_encode_bf16(m, base, 2, dims, strides, box);
}

int pick_nt(int M) {
    for (int nt : {16, 32, 64, 128}) if (M <= nt) return nt;
    return 256;
}

template <int NT>
int launch_nt(const Launch& L, const CUtensorMap& tw, const CUtensorMap& tx, const KParams& p, int grid) {
    static bool attr_set = false;
    const int smem = 1024 + p.stages * (W_STAGE_BYTES + NT * BK * 2) + SMEM_FIXED;
    if (!attr_set) {
        if (cudaFuncSetAttribute(gemm_tc_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_LIMIT) != cudaSuccess)
            return DFLASH_ERR_CUDA;
        attr_set = true;
    }
    gemm_tc_kernel<NT><<<grid, N_THREADS, smem, L.st>>>(tw, tx, p);
    ++g_launches;
    return cudaPeekAtLastError() == cudaSuccess ? DFLASH_OK : DFLASH_ERR_CUDA;
}

}  // namespace

int gemm_tc_splits(int M, int N, int K, int sm_count) {
    const int nt = pick_nt(M);
    const int base = ((N + TILE_F - 1) / TILE_F) * ((M + nt - 1) / nt);
    const int chunks = (K + BK - 1) / BK;
    if (base >= 4 * sm_count) return 1;   // enough units: the tail imbalance is already small
    int best = 1;
    double best_eff = 0.0;
    for (int s = 1; s <= 16; ++s) {
        const int cps = (chunks + s - 1) / s;
        if (cps < 4 && s > 1) break;
        if ((chunks + cps - 1) / cps != s) continue;   // would leave an empty split
        const int units = base * s;
        const int waves = (units + sm_count - 1) / sm_count;
        const double eff = (double)units / ((double)waves * sm_count);
        if (eff > best_eff + 0.03) { best_eff = eff; best = s; }
    }
    return best;
}

int64_t gemm_tc_part_bytes(int M, int N, int K, int sm_count) {
    const int s = gemm_tc_splits(M, N, K, sm_count);
    if (s == 1) return 0;
    const int nt = pick_nt(M);
    const int64_t tiles = (int64_t)((N + TILE_F - 1) / TILE_F) * ((M + nt - 1) / nt);
    return tiles * s * nt * TILE_F * 4;
}

int64_t gemm_tc_counter_bytes(int M, int N) {
    const int nt = pick_nt(M);
    return (int64_t)((N + TILE_F - 1) / TILE_F) * ((M + nt - 1) / nt) * 4;
}

int launch_gemm_tc(const Launch& L, const GemmArgs& a) {
    if (a.M <= 0 || a.N <= 0) return DFLASH_OK;
    if (a.K % 8 != 0) return DFLASH_ERR_UNSUPPORTED;
    const dflash_config& c = L.h->cfg;
    const int nt = pick_nt(a.M);
    KParams p{};
    p.M = a.M; p.N = a.N; p.K = a.K; p.epi = a.epilogue;
    p.n_ftiles = (a.N + TILE_F - 1) / TILE_F;
    p.n_ttiles = (a.M + nt - 1) / nt;
    p.chunks_total = (a.K + BK - 1) / BK;
    p.splits = gemm_tc_splits(a.M, a.N, a.K, L.h->sm_count);
    if (p.splits > 1 && (!a.part || !a.counters)) p.splits = 1;
    p.chunks_per_split = (p.chunks_total + p.splits - 1) / p.splits;
    p.stages = std::min(MAX_STAGES, (SMEM_LIMIT - 1024 - SMEM_FIXED) / (W_STAGE_BYTES + nt * BK * 2));
    p.part = a.part; p.counters = a.counters;
    p.out_f32 = a.out_f32; p.ld_out = a.ld_out;
    p.q = a.q; p.k = a.k; p.v = a.v; p.ctx_len = a.ctx_len; p.rows_per_seq = a.rows_per_seq > 0 ? a.rows_per_seq : 1;
    p.Hq = c.n_q_heads; p.Hkv = c.n_kv_heads; p.hd = c.head_dim; p.use_rope = c.use_rope;
    p.cs = L.h->w.rope_cos; p.sn = L.h->w.rope_sin; p.max_pos = L.h->w.rope_max_pos;
    p.h = a.h; p.F = c.d_ffn;
    p.top2 = a.top2; p.logits_out = a.logits_out;
    if (a.ctx) {
        p.pool = (__nv_bfloat16*)a.ctx->kv_pool; p.n_new = a.ctx->n_new; p.page_table = a.ctx->page_table;
        p.ctx_len = a.ctx->ctx_len;
        p.max_new = a.ctx->max_new; p.max_pages = a.ctx->max_pages; p.n_pages = a.ctx->n_pool_pages;
    }
    p.PG = c.page_size; p.layer = a.layer;
    p.status = L.status;

    CUtensorMap tw, tx;
    if (!make_map(&tw, a.W, a.N, a.K, TILE_F) || !make_map(&tx, a.X, a.M, a.K, nt)) return DFLASH_ERR_CUDA;
    const int units = p.n_ftiles * p.n_ttiles * p.splits;
    const int grid = std::min(units, L.h->sm_count);
    switch (nt) {
        case 16: return launch_nt<16>(L, tw, tx, p, grid);
        case 32: return launch_nt<32>(L, tw, tx, p, grid);
        case 64: return launch_nt<64>(L, tw, tx, p, grid);
        case 128: return launch_nt<128>(L, tw, tx, p, grid);
        default: return launch_nt<256>(L, tw, tx, p, grid);
    }
}

int launch_argmax_finish(const Launch& L, const Top2Entry* top2, int n_tiles, int M, int32_t* ids, float* top1,
                         float* margin) {
    if (M <= 0) return DFLASH_OK;
    argmax_finish_kernel<<<M, 128, 0, L.st>>>(top2, n_tiles, M, ids, top1, margin);
    ++g_launches;
    return cudaPeekAtLastError() == cudaSuccess ? DFLASH_OK : DFLASH_ERR_CUDA;
}

}  // namespace dflash
