// Host side of the chained tensor-core contractions: phases and their tensor maps, the choice of the launch form
// (K-split clusters, plain CTAs, CTA pairs), the small kernels around them (argmax merge, embedding) and the
// host-side walk of the work split. The kernel itself is in gemm_tc_kernel.cuh.
#include "gemm_tc_kernel.cuh"

#include <utility>
#include <vector>

namespace dflash {
using namespace gemmk;
namespace {

// Merge of the per-tile winners (index-aware, so order-independent). The entries are laid out
// [tile][token]: a CTA takes 8 consecutive tokens (one full 128-byte line per tile) and 64 interleaved
// sub-sequences of the tiles, so every request is a whole line however few SMs the CTAs land on.
constexpr int FIN_TOK = 8, FIN_SUB = 64;
__global__ void __launch_bounds__(FIN_TOK * FIN_SUB) argmax_finish_kernel(const Top2Entry* __restrict__ top2, int n_tiles, int M,
                                                                          int32_t* __restrict__ ids, float* __restrict__ top1,
                                                                          float* __restrict__ margin, unsigned long long* trace) {
    __shared__ Top2Entry sh[FIN_TOK * FIN_SUB / 32][FIN_TOK];
    if (threadIdx.x == 0) trace_min(trace, 0);
    pdl_trigger();
    pdl_wait();
    if (threadIdx.x == 0) trace_min(trace, 1);
    const int tl = threadIdx.x & (FIN_TOK - 1), sub = threadIdx.x / FIN_TOK;
    const int tok = blockIdx.x * FIN_TOK + tl;
    T2 t{-CUDART_INF_F, 0x7fffffff, -CUDART_INF_F};
    if (tok < M) {
        constexpr int INFL = 8;             // entries requested together per thread
        for (int i0 = sub; i0 < n_tiles; i0 += INFL * FIN_SUB) {
            float4 e[INFL];
#pragma unroll
            for (int k = 0; k < INFL; ++k) {
                const int i = i0 + k * FIN_SUB;
                e[k] = i < n_tiles ? __ldcg(reinterpret_cast<const float4*>(top2 + (size_t)i * M + tok))
                                   : make_float4(-CUDART_INF_F, __int_as_float(0x7fffffff), -CUDART_INF_F, 0.f);
            }
#pragma unroll
            for (int k = 0; k < INFL; ++k) t2_merge(t, e[k].x, __float_as_int(e[k].y), e[k].z);
        }
    }
    // lanes tl, tl + 8, tl + 16, tl + 24 of a warp hold the same token
#pragma unroll
    for (int o = FIN_TOK; o < 32; o <<= 1) {
        const float v1 = __shfl_xor_sync(0xffffffffu, t.v1, o);
        const int i1 = __shfl_xor_sync(0xffffffffu, t.i1, o);
        const float v2 = __shfl_xor_sync(0xffffffffu, t.v2, o);
        t2_merge(t, v1, i1, v2);
    }
    if ((threadIdx.x & 31) < FIN_TOK) sh[threadIdx.x >> 5][tl] = Top2Entry{t.v1, t.i1, t.v2, 0};
    __syncthreads();
    if (threadIdx.x < FIN_TOK && tok < M) {
        T2 r{sh[0][tl].v1, sh[0][tl].i1, sh[0][tl].v2};
        for (int w = 1; w < FIN_TOK * FIN_SUB / 32; ++w) t2_merge(r, sh[w][tl].v1, sh[w][tl].i1, sh[w][tl].v2);
        ids[tok] = r.i1 == 0x7fffffff ? 0 : r.i1;
        if (top1) top1[tok] = r.v1;
        if (margin) margin[tok] = r.v1 - r.v2;
    }
    if (threadIdx.x == 0) trace_max(trace, 3);
}

// Few tokens: one CTA per token (more CTAs in flight matter more than whole-line requests).
__global__ void __launch_bounds__(128) argmax_finish_rows_kernel(const Top2Entry* __restrict__ top2, int n_tiles, int M,
                                                                 int32_t* __restrict__ ids, float* __restrict__ top1,
                                                                 float* __restrict__ margin, unsigned long long* trace) {
    __shared__ Top2Entry sh[4];
    if (threadIdx.x == 0) trace_min(trace, 0);
    pdl_trigger();
    pdl_wait();
    if (threadIdx.x == 0) trace_min(trace, 1);
    const int tok = blockIdx.x;
    T2 t{-CUDART_INF_F, 0x7fffffff, -CUDART_INF_F};
    constexpr int INFL = 12;
    for (int i0 = threadIdx.x; i0 < n_tiles; i0 += INFL * blockDim.x) {
        float4 e[INFL];
#pragma unroll
        for (int k = 0; k < INFL; ++k) {
            const int i = i0 + k * blockDim.x;
            e[k] = i < n_tiles ? __ldcg(reinterpret_cast<const float4*>(top2 + (size_t)i * M + tok))
                               : make_float4(-CUDART_INF_F, __int_as_float(0x7fffffff), -CUDART_INF_F, 0.f);
        }
#pragma unroll
        for (int k = 0; k < INFL; ++k) t2_merge(t, e[k].x, __float_as_int(e[k].y), e[k].z);
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
        trace_max(trace, 3);
    }
}

// block row 0 of each sequence = anchor, rows 1.. = mask token; also the first layer's norm inputs
__global__ void __launch_bounds__(256) embed_norm_kernel(const __nv_bfloat16* __restrict__ E,
                                                         const int32_t* __restrict__ anchor,
                                                         const int32_t* __restrict__ token_ids, float* __restrict__ x,
                                                         const __nv_bfloat16* __restrict__ g,
                                                         __nv_bfloat16* __restrict__ xn, float* __restrict__ ssq, int B,
                                                         int D, int V, int mask_id, int M, int32_t* status,
                                                         unsigned long long* trace) {
    if (threadIdx.x == 0) trace_min(trace, 0);
    pdl_trigger();
    pdl_wait();
    if (threadIdx.x == 0) trace_min(trace, 1);
    const int row = blockIdx.x, b = row / B, r = row % B;
    int id = token_ids ? token_ids[row] : ((r == 0) ? anchor[b] : mask_id);
    if (id < 0 || id >= V) {
        if (threadIdx.x == 0 && status) atomicOr(status, DFLASH_DEV_BAD_TOKEN);
        id = 0;
    }
    const __nv_bfloat16* src = E + (size_t)id * D;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles = (D + 127) / 128;
    for (int t = warp; t < n_tiles; t += (blockDim.x >> 5)) {
        float s = 0.f;
        for (int d = t * 128 + lane; d < min(D, (t + 1) * 128); d += 32) {
            const float v = __bfloat162float(src[d]);
            x[(size_t)row * D + d] = v;
            xn[(size_t)row * D + d] = __float2bfloat16_rn(v * __bfloat162float(g[d]));
            s += v * v;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (lane == 0) ssq[(size_t)t * M + row] = s;
    }
    if (threadIdx.x == 0) trace_max(trace, 3);
}

// [rows, K] bf16 row-major; box = 64 K-elements x box_rows rows (x `slabs` consecutive 64-element
// column blocks, through the view [64][rows][K/64], when slabs > 1: K must be a multiple of 64)
bool make_map(CUtensorMap* m, const void* base, int rows, int K, int box_rows, int slabs) {
    if (slabs == 1) {
        const uint64_t dims[2] = {(uint64_t)K, (uint64_t)rows};
        const uint64_t strides[1] = {(uint64_t)K * 2};
        const uint32_t box[2] = {(uint32_t)BK, (uint32_t)box_rows};
        return tmap_encode_bf16(m, base, 2, dims, strides, box);
    }
    const uint64_t dims[3] = {(uint64_t)BK, (uint64_t)rows, (uint64_t)(K / BK)};
    const uint64_t strides[2] = {(uint64_t)K * 2, (uint64_t)BK * 2};
    const uint32_t box[3] = {(uint32_t)BK, (uint32_t)box_rows, (uint32_t)slabs};
    return tmap_encode_bf16(m, base, 3, dims, strides, box);
}

// Token-tile width: up to 128 rows the smallest width that holds them; beyond that the width (a multiple of 32 up
// to 256) that pads the fewest token columns over all token tiles, the widest among equals (fewer token tiles =
// fewer passes over the weights through L2): 136 rows -> 160, 544 -> 3 x 192, 512 -> 2 x 256.
// The map of a weight matrix, from the handle's cache (encoded on first use; a full cache encodes without storing)
bool weight_map(dflash_handle* h, CUtensorMap* m, const void* base, int rows, int K, int slabs) {
    for (int i = 0; i < h->n_wmaps; ++i) {
        const dflash_wmap_entry& e = h->wmaps[i];
        if (e.base == base && e.rows == rows && e.K == K && e.slabs == slabs) { *m = e.map; return true; }
    }
    if (!make_map(m, base, rows, K, TILE_F, slabs)) return false;
    if (h->n_wmaps < DFLASH_WMAP_CACHE) h->wmaps[h->n_wmaps++] = dflash_wmap_entry{base, rows, K, slabs, *m};
    return true;
}

int pick_nt(int M) {
    for (int nt : {16, 32, 64, 128}) if (M <= nt) return nt;
    int best = 256;
    long long best_cols = (long long)((M + 255) / 256) * 256;
    for (int nt : {192, 160}) {
        const long long cols = (long long)((M + nt - 1) / nt) * nt;
        if (cols < best_cols) { best = nt; best_cols = cols; }
    }
    return best;
}

}  // namespace

// A workspace sized for M rows also serves launches with fewer rows, whose token tile may be WIDER than the one M
// rows get (520 rows take tiles of 192 columns, 640 rows tiles of 160): both sizes below are upper bounds over
// every row count up to M.
int64_t gemm_tc_part_bytes(int M, int N, int K, int n_groups, int sm_count) {
    (void)N; (void)K; (void)n_groups;
    const int nt_max = M > 128 ? 256 : pick_nt(M);
    return (int64_t)sm_count * 2 * nt_max * TILE_F * 4;    // two partial pieces per CTA at most
}

int64_t gemm_tc_counter_bytes(int M, int N, int n_groups) {
    // token tiles: rows beyond 128 use tiles of at least 160 columns, so ceil(M / 128) bounds every smaller row count too
    const int ttiles = M > 128 ? (M + 127) / 128 : 1;
    return (int64_t)std::max(n_groups, 1) * ((N + TILE_F - 1) / TILE_F) * ttiles * 4;
}

static int fill_phase(const Launch& L, const GemmArgs& a, int nt, int slabs, bool pair, KParams& p) {
    if (a.K % 8 != 0) return DFLASH_ERR_UNSUPPORTED;
    const dflash_config& c = L.h->cfg;
    const int groups = std::max(a.n_groups, 1);
    p = KParams{};
    p.M = a.M; p.N = a.N; p.K = a.K; p.epi = a.epilogue;
    p.n_groups = groups;
    p.n_ftiles_real = (a.N + TILE_F - 1) / TILE_F;
    p.n_ftiles = pair ? (p.n_ftiles_real + 1) / 2 : p.n_ftiles_real;
    p.n_ttiles = (a.M + nt - 1) / nt;
    p.chunks_total = (a.K + BK * slabs - 1) / (BK * slabs);
    p.n_tiles = groups * p.n_ftiles * p.n_ttiles;
    if (!a.part || !a.counters) return DFLASH_ERR_INVALID_ARG;
    p.part = a.part; p.counters = a.counters;
    p.ssq_in = a.ssq_in; p.n_parts_in = (a.K + 127) / 128; p.inv_dim_in = 1.f / (float)a.K; p.eps = c.rms_eps;
    p.g_next = (const __nv_bfloat16*)a.g_next; p.xn_out = a.xn_out; p.ssq_out = a.ssq_out;
    p.out_f32 = a.out_f32; p.ld_out = a.ld_out;
    p.q = a.q; p.k = a.k; p.v = a.v;
    p.gq = (const __nv_bfloat16*)a.g_q;
    p.gk[0] = (const __nv_bfloat16*)a.g_k;
    if (a.epilogue == EPI_CTX_KV) {
        for (int g = 0; g < groups; ++g) p.gk[g] = (const __nv_bfloat16*)a.g_k_group[g];
    }
    p.ctx_len = a.ctx_len;
    p.rows_per_seq = a.rows_per_seq > 0 ? a.rows_per_seq : 1;
    p.Hq = c.n_q_heads; p.Hkv = c.n_kv_heads; p.hd = c.head_dim; p.use_rope = c.use_rope;
    p.cs = L.h->w.rope_cos; p.sn = L.h->w.rope_sin; p.max_pos = L.h->w.rope_max_pos;
    p.h = a.h; p.F = c.d_ffn;
    p.top2 = a.top2; p.logits_out = a.logits_out;
    if (a.ctx) {
        p.pool = (__nv_bfloat16*)a.ctx->kv_pool; p.n_new = a.ctx->n_new; p.page_table = a.ctx->page_table;
        p.ctx_len = a.ctx->ctx_len;
        p.max_new = a.ctx->max_new; p.max_pages = a.ctx->max_pages; p.n_pages = a.ctx->n_pool_pages;
    }
    p.PG = c.page_size; p.first_layer = a.first_layer;
    p.status = L.status;
    return DFLASH_OK;
}

int launch_gemm_chain(const Launch& L, const GemmArgs* phases, int n_phases, int32_t* phase_done,
                      unsigned long long* const* traces) {
    if (n_phases < 1 || n_phases > MAX_PHASES) return DFLASH_ERR_INVALID_ARG;
    // phases may differ in their row count (the context projection's rows, then a draft block's); the
    // token tile is sized for the largest
    int M = 0;
    for (int i = 0; i < n_phases; ++i) M = std::max(M, phases[i].M);
    if (M <= 0) return DFLASH_OK;
    const int nt = pick_nt(M);
    MParams mp{};
    WMaps tw;
    XMaps tx;
    bool k64 = true;
    for (int i = 0; i < n_phases; ++i) k64 = k64 && phases[i].K % BK == 0;
    const int slabs = slabs_for(nt, k64);
    bool qkn = false;
    for (int i = 0; i < n_phases; ++i) {
        qkn = qkn || phases[i].g_q != nullptr || phases[i].g_k != nullptr;
        if (phases[i].epilogue == EPI_CTX_KV)
            for (int g = 0; g < std::max(phases[i].n_groups, 1); ++g) qkn = qkn || phases[i].g_k_group[g] != nullptr;
    }
    // Token tiles of 160 columns and more run as CTA pairs where the device keeps pairs resident
    int pair_cap = 0;
    if (nt >= 160 && L.h->sm_count >= 2) {
        pair_cap = gemm_pair_capacity(nt, qkn);
        pair_cap = std::min(pair_cap, L.h->sm_count / 2);
    }
    const bool pair = pair_cap >= 1;
    mp.n_phases = n_phases;
    mp.stages = pair ? pair_stages(nt)
                     : std::min(MAX_STAGES, (SMEM_LIMIT - 1024 - smem_fixed(nt)) / (slabs * (W_STAGE_BYTES + nt * BK * 2)));
    mp.phase_done = phase_done;
    mp.status = L.status;

    int n_maps = 0;
    long long min_pairs = -1;
    for (int i = 0; i < n_phases; ++i) {
        const GemmArgs& a = phases[i];
        if (a.M <= 0 || a.N <= 0) return DFLASH_ERR_INVALID_ARG;
        const int rc = fill_phase(L, a, nt, slabs, pair, mp.ph[i]);
        if (rc != DFLASH_OK) return rc;
        KParams& p = mp.ph[i];
        p.trace = traces ? traces[i] : nullptr;
        if (n_maps + p.n_groups > GEMM_MAX_GROUPS) return DFLASH_ERR_UNSUPPORTED;
        p.w_map0 = n_maps;
        for (int g = 0; g < p.n_groups; ++g)
            if (!weight_map(L.h, &tw.m[n_maps++], a.W[g], a.N, a.K, slabs)) return DFLASH_ERR_CUDA;
        p.x_map = i;
        if (!make_map(&tx.m[i], a.X, a.M, a.K, pair ? nt / 2 : nt, slabs)) return DFLASH_ERR_CUDA;
        const long long pairs = (long long)p.n_tiles * p.chunks_total;
        min_pairs = min_pairs < 0 ? pairs : std::min(min_pairs, pairs);
    }
    for (int g = n_maps; g < GEMM_MAX_GROUPS; ++g) tw.m[g] = tw.m[0];
    for (int i = n_phases; i < MAX_PHASES; ++i) tx.m[i] = tx.m[0];
    // one CTA per SM unless the smallest phase would leave ranges under 256 K-elements
    const int grid = (int)std::max<long long>(1, std::min<long long>(L.h->sm_count, min_pairs * slabs / 4));
    if (pair) {
        // one pair per two SMs unless the smallest phase would leave ranges under 256 K-elements
        const int pairs = (int)std::max<long long>(1, std::min<long long>(pair_cap, min_pairs / 4));
        return gemm_launch_pair(nt, qkn, L, tw, tx, mp, pairs);
    }
    switch (nt) {
        case 16: return gemm_launch_16(slabs, qkn, L, tw, tx, mp, grid);
        case 32: return gemm_launch_32(slabs, qkn, L, tw, tx, mp, grid);
        case 64:
        case 128: return gemm_launch_64_128(nt, qkn, L, tw, tx, mp, grid);
        default: return gemm_launch_160_256(nt, qkn, L, tw, tx, mp, grid);
    }
}

// The work split of one phase, walked on the host exactly as the kernel's roles walk it (the same PieceWalk code):
// every (tile, chunk) of the matrix covered once, at most two partial pieces per walker in different slots, the
// contributors of a shared tile and their slots as the finishing code derives them. 0 = consistent.
int gemm_plan_check(int M, int N, int K, int n_groups, int sm_count, int pair_cap, int cluster_cap, int32_t* info) {
    if (M <= 0 || N <= 0 || K <= 0 || sm_count <= 0) return -1;
    const int groups = std::max(n_groups, 1);
    const int nt = pick_nt(M);
    const int slabs = slabs_for(nt, K % BK == 0);
    pair_cap = std::min(pair_cap, sm_count / 2);
    const bool pair = nt >= 160 && sm_count >= 2 && pair_cap >= 1;
    KParams p{};
    p.M = M; p.N = N; p.K = K; p.n_groups = groups;
    p.n_ftiles_real = (N + TILE_F - 1) / TILE_F;
    p.n_ftiles = pair ? (p.n_ftiles_real + 1) / 2 : p.n_ftiles_real;
    p.n_ttiles = (M + nt - 1) / nt;
    p.chunks_total = (K + BK * slabs - 1) / (BK * slabs);
    p.n_tiles = groups * p.n_ftiles * p.n_ttiles;
    const long long pairs_tc = (long long)p.n_tiles * p.chunks_total;
    int grid, cs = 1, walkers;
    if (pair) {
        walkers = (int)std::max<long long>(1, std::min<long long>(pair_cap, pairs_tc / 4));
        grid = 2 * walkers;
    } else {
        grid = (int)std::max<long long>(1, std::min<long long>(sm_count, pairs_tc * slabs / 4));
        if (nt <= 32 && grid >= CS) {
            int cap = std::min(cluster_cap, MAX_CLUSTERS);      // as cluster_capacity() reports it
            if (cap < MIN_CLUSTERS) cap = 0;
            const int n_cl = std::min(cap, grid / CS);
            if (n_cl >= 1) { cs = CS; grid = n_cl * CS; }
        }
        p.cluster_k = (cs > 1 && p.n_tiles < grid && p.chunks_total >= CS) ? 1 : 0;
        walkers = grid;
    }
    if (info) { info[0] = nt; info[1] = pair ? 1 : 0; info[2] = grid; info[3] = cs; info[4] = shared_tiles(p, walkers); info[5] = p.cluster_k; }
    const int real_tiles = groups * p.n_ftiles_real * p.n_ttiles;
    std::vector<uint8_t> cover((size_t)real_tiles * p.chunks_total, 0);
    const int n_shared = shared_tiles(p, walkers);
    const long long T = (long long)n_shared * p.chunks_total;
    std::vector<std::vector<std::pair<int, int>>> contrib((size_t)std::max(n_shared, 0));
    for (int w = 0; w < walkers; ++w) {
        for (int prank = 0; prank < (pair ? 2 : 1); ++prank) {
            int n_partial = 0, slot_mask = 0;
            for (PieceWalk pw(p, w, walkers, cs); !pw.done(p);) {
                Unit u = pw.next(p);
                if (pair) own_tile<true>(p, u, prank);
                if (u.c0 < 0 || u.c1 > p.chunks_total || u.c0 >= u.c1) return 1;
                if (u.full && u.tile < n_shared && prank == 0) contrib[(size_t)u.tile].push_back({w, -1});   // whole tile, one walker
                if (!u.full && !u.cl) {
                    if (u.tile >= n_shared) return 2;
                    ++n_partial;
                    if (slot_mask & (1 << u.slot)) return 3;            // two pieces of one CTA in the same partial slot
                    slot_mask |= 1 << u.slot;
                    if (prank == 0) contrib[(size_t)u.tile].push_back({w, u.slot});
                }
                if (u.phantom) continue;
                if (u.ft >= p.n_ftiles_real || u.tt >= p.n_ttiles || u.g >= groups) return 4;
                if (u.ctr != (u.g * p.n_ftiles_real + u.ft) * p.n_ttiles + u.tt) return 5;
                for (int c = u.c0; c < u.c1; ++c) {
                    uint8_t& k = cover[(size_t)u.ctr * p.chunks_total + c];
                    if (k) return 6;                                    // a chunk of a tile handed out twice
                    k = 1;
                }
            }
            if (n_partial > 2) return 7;
        }
    }
    for (uint8_t k : cover)
        if (!k) return 8;                                               // a chunk nobody takes
    for (int t = 0; t < n_shared; ++t) {
        const long long x0 = (long long)t * p.chunks_total;
        const int j0 = cta_of_pair(x0, T, walkers), j1 = cta_of_pair(x0 + p.chunks_total - 1, T, walkers);
        const auto& cv = contrib[(size_t)t];
        if ((int)cv.size() != j1 - j0 + 1) return 9;                    // the finishing code expects other contributors
        if (cv.size() == 1 && cv[0].second == -1) {                     // a whole tile inside one walker's range: no exchange
            if (cv[0].first != j0) return 12;
            continue;
        }
        for (int j = j0; j <= j1; ++j) {
            if (cv[(size_t)(j - j0)].first != j) return 10;
            const int sa = ((long long)j * T / walkers >= x0) ? 0 : 1;
            if (cv[(size_t)(j - j0)].second != sa) return 11;           // ... or looks for a piece in the other slot
        }
    }
    return 0;
}

int launch_gemm_tc(const Launch& L, const GemmArgs& a, int32_t* phase_done) {
    if (a.M <= 0 || a.N <= 0) return DFLASH_OK;
    unsigned long long* tr[1] = {L.trace};
    return launch_gemm_chain(L, &a, 1, phase_done, tr);
}

int launch_argmax_finish(const Launch& L, const Top2Entry* top2, int n_tiles, int M, int32_t* ids, float* top1,
                         float* margin) {
    if (M <= 0) return DFLASH_OK;
    const cudaError_t e =
        M <= 32 ? launch_pdl(argmax_finish_rows_kernel, dim3(M), dim3(128), 0, L.st, top2, n_tiles, M, ids, top1, margin, L.trace)
                : launch_pdl(argmax_finish_kernel, dim3((M + FIN_TOK - 1) / FIN_TOK), dim3(FIN_TOK * FIN_SUB), 0, L.st, top2,
                             n_tiles, M, ids, top1, margin, L.trace);
    ++g_launches;
    return e == cudaSuccess ? DFLASH_OK : DFLASH_ERR_CUDA;
}

int launch_embed_norm(const Launch& L, const int32_t* anchor, const int32_t* token_ids, int batch, int block_rows, float* x,
                      const void* g, __nv_bfloat16* xn, float* ssq) {
    const dflash_config& c = L.h->cfg;
    const int rows = batch * block_rows;
    if (rows <= 0) return DFLASH_OK;
    const cudaError_t e = launch_pdl(embed_norm_kernel, dim3(rows), dim3(256), 0, L.st,
                                     (const __nv_bfloat16*)L.h->w.embed, anchor, token_ids, x, (const __nv_bfloat16*)g, xn, ssq,
                                     block_rows, c.d_model, c.vocab, c.mask_token_id, rows, L.status, L.trace);
    ++g_launches;
    return e == cudaSuccess ? DFLASH_OK : DFLASH_ERR_CUDA;
}

}  // namespace dflash
