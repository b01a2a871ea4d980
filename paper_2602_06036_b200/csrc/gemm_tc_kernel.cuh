// The chained tensor-core contraction kernel and its launch templates. Included by the translation units that
// instantiate it (one per group of token-tile widths, so that they compile side by side) and by gemm_tc.cu, which
// holds the host logic (phases, tensor maps, the choice of the launch form) and calls the entry points below.
// bf16 contractions with few tokens and large weights (QKV / O / SwiGLU / LM head / context K,V):
//   acc[token][feature] = sum_k X[token][k] * W[feature][k]
// The WEIGHT tile is the 128-row "M" operand of tcgen05.mma and the tokens are its "N" operand
// (16..256 columns), so the tensor core runs full-height instructions however few tokens there
// are. A CTA is one TMA producer warp, one MMA-issuing warp and four epilogue warps; operands
// stream through a ring of 128-byte-swizzled shared-memory stages, accumulators live in two TMEM
// buffers so the epilogue of one piece of work overlaps the main loop of the next.
// Work split ("stream-K" remainder first, whole tiles last): with at least one output tile per CTA,
// the n_tiles % n_ctas remainder tiles are cut into (tile, K chunk) pairs and shared out as one
// contiguous, equally long range per CTA; the other tiles go whole, the same number to every CTA. So
// every SM streams the same number of weight bytes whatever the tile count, the cross-CTA reduction
// of the shared tiles runs under the main loop of the whole tiles, and a phase ends with direct
// epilogues. With fewer tiles than CTAs all tiles are shared. A shared tile is finished by ALL of its
// contributors: each writes its partial sums and takes a ticket, waits (bounded) until the tile's
// tickets are complete, and then sums the pieces in CTA order for its own share of the tile's token
// passes (bit-reproducible, and the finishing work is spread over the CTAs instead of piling up on
// one). A ring stage holds one or two 64-element K slabs of both operands (two for small token tiles,
// fetched by one 3-D copy each: the single issuing thread, not HBM, is the limit there).
// RMSNorm never runs as a kernel of its own: epilogues that produce residual
// rows also emit the gain-scaled bf16 operand and per-tile sums of squares, and the consuming
// contraction scales its accumulator columns by the per-token rsqrt.
// One launch runs a CHAIN of up to four such contractions ("phases": e.g. output projection ->
// gate/up -> down -> next layer's QKV), each consuming what the previous one's epilogues wrote.
// The producer warp never stops streaming WEIGHT tiles: only the activation tile of a ring slot
// waits until every CTA has signalled the end of the previous phase (a counter in global memory,
// polled with a bound), so the tail of one phase - partial sums, tickets, epilogues - overlaps the
// weight stream of the next and HBM stays busy across the chain.
// Launched with programmatic dependent launch: barrier set-up and TMEM allocation happen before
// griddepcontrol.wait. (Filling the ring with weight tiles before that wait was measured slower: the
// copy queue is in order, so CTAs that start after the dependency resolved had their first
// activation tiles stuck behind a ring of HBM-bound weight copies.)
// Every wait on an mbarrier is bounded; on expiry the kernel raises DFLASH_DEV_TIMEOUT, drains its
// outstanding copies, frees its TMEM and returns.
#pragma once
#include "gemm_tc.cuh"

#include "ptx_sm100.cuh"

#include <math_constants.h>

#include <algorithm>

namespace dflash {
namespace gemmk {


using namespace ptx;

constexpr int TILE_F = 128;                      // weight rows per tile = MMA M
constexpr int BK = 64;                           // K elements per slab = one 128-byte swizzle row
constexpr int W_STAGE_BYTES = TILE_F * BK * 2;   // 16 KiB per slab
// A ring stage holds SL slabs (SL * 64 K-elements) of both operands, each fetched by ONE copy:
// with few tokens the tensor-core work per byte is tiny and the single issuing thread, not HBM,
// limits the stream, so small token tiles take two slabs per copy (a 3-D view [64][rows][K/64] of
// the row-major matrix lands as [slab][row][64], i.e. two canonical swizzled tiles back to back).
constexpr int slabs_for(int nt, bool k_mult_64) { return (nt <= 32 && k_mult_64) ? 2 : 1; }
constexpr int MAX_STAGES = 12;
// per-token scale / position / page kept for this many rows (token tiles of up to 32 rows only run with <= 32 rows)
constexpr int tok_cache(int nt) { return nt <= 32 ? 32 : 1024; }
// Thread-block clusters (token tiles of up to 32 rows): the CS CTAs of a cluster split the K range of one
// weight tile and exchange their partial sums through distributed shared memory. Every CTA finishes NT / CS
// token columns of the tile: it receives those columns from its CS - 1 peers into one of two buffers.
constexpr int CS = 4;
constexpr int xch_bytes(int nt) { return nt <= 32 ? 2 * (CS - 1) * (nt / CS) * TILE_F * 4 : 0; }
// token columns handled per epilogue pass (each of the 128 epilogue threads holds CH accumulators)
constexpr int pass_cols(int nt) { return nt <= 16 ? nt : (nt == 32 ? 16 : 32); }   // short passes: short dependent chains when finishing, fewer registers
constexpr int smem_fixed(int nt) {
    return TILE_F * (pass_cols(nt) + 1) * 4 + 128 * 16 + 3 * tok_cache(nt) * 4 + xch_bytes(nt) + (2 * MAX_STAGES + 6) * 8 + 64 +
           3 * MAX_STAGES * 4;
}
constexpr int SMEM_LIMIT = 227 * 1024;
constexpr int N_THREADS = 192;

struct WMaps {
    CUtensorMap m[GEMM_MAX_GROUPS];
};

struct KParams {
    int M, N, K, epi, chunks_total, n_groups, n_ftiles, n_ttiles, n_tiles, w_map0, x_map;
    // A launch of CTA pairs walks PAIRS of neighbouring weight tiles: n_ftiles and n_tiles then count those pairs and
    // n_ftiles_real the weight tiles themselves (an odd count leaves the last pair's odd CTA a tile beyond the matrix).
    int n_ftiles_real;
    int cluster_k;     // the phase splits every tile's K range over the CTAs of a cluster (partial sums through their shared memory)
    float* part;
    int32_t* counters;
    const float* ssq_in;
    int n_parts_in;
    float inv_dim_in, eps;
    const __nv_bfloat16* g_next;
    __nv_bfloat16* xn_out;
    float* ssq_out;
    float* out_f32;
    int ld_out;
    __nv_bfloat16 *q, *k, *v;
    const __nv_bfloat16* gq;                          // per-head norm gains [hd] (nullptr: no head norm)
    const __nv_bfloat16* gk[GEMM_MAX_GROUPS];         // QKV: [0]; context K/V: one per group (layer)
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
    int max_new, max_pages, n_pages, PG, first_layer;
    int32_t* status;
    unsigned long long* trace;   // this phase's timeline record
};

constexpr int MAX_PHASES = 4;
struct XMaps {
    CUtensorMap m[MAX_PHASES];
};
// A launch = a chain of phases that share the token tile size and the ring.
struct MParams {
    int n_phases, stages;
    int cs;                      // CTAs per cluster (1: launched without clusters)
    int32_t* phase_done;         // [MAX_PHASES] CTAs that finished each phase (zero on entry)
    int32_t* status;
    KParams ph[MAX_PHASES];
};

// One piece of a CTA's chunk range: chunks [c0, c1) of output tile `tile`.
struct Unit {
    int tile, g, ft, tt, c0, c1;
    int slot;      // 0 = first piece of this CTA's range, 1 = a later one (partial pieces only: first or last)
    int full;      // covers every chunk of the tile
    int cl;        // this CTA's K share of a tile that its cluster finishes together
    int ctr;       // index of the tile's ticket counter
    int phantom;   // CTA pairs: this CTA's weight tile lies beyond the matrix (it only keeps the pair's protocol going)
};
// CTA pairs: the walk hands out pairs of weight tiles; CTA `prank` of the pair takes tile 2 * pair + prank.
template <bool PAIR>
__host__ __device__ __forceinline__ void own_tile(const KParams& p, Unit& u, int prank) {
    if constexpr (PAIR) {
        u.ft = u.ft * 2 + prank;
        u.phantom = u.ft >= p.n_ftiles_real ? 1 : 0;
        u.ctr = (u.g * p.n_ftiles_real + u.ft) * p.n_ttiles + u.tt;
    }
}

// Work of CTA `cta` out of `n_ctas` in one phase. With at least one tile per CTA the tiles are split
// into a SHARED part (the first n_tiles % n_ctas tiles) and whole tiles, the same number per CTA:
//   1. the (tile, chunk) pairs of the shared part are cut into one contiguous, equally long range per
//      CTA ("stream-K"), processed FIRST: the cross-CTA reduction of those tiles then overlaps the
//      streaming of the whole tiles instead of sitting at the end of the phase;
//   2. whole tiles shared + k * n_ctas + cta, k = 0.., go straight from the accumulator to the epilogue.
// Every CTA streams the same number of chunks (+-1). With fewer tiles than CTAs everything is shared.
// Tiles are ordered token-tile fastest, so neighbouring CTAs share weight tiles through L2.
// The shared part never leaves a CTA an empty range (every CTA between the first and the last
// contributor of a tile publishes a piece): a remainder that small takes one more round of tiles with it.
__host__ __device__ __forceinline__ int shared_tiles(const KParams& p, int n_ctas) {
    if (p.cluster_k) return 0;      // every tile is finished inside a cluster
    if (p.n_tiles < n_ctas) return p.n_tiles;
    const int r = p.n_tiles % n_ctas;
    if (r == 0) return 0;
    if ((long long)r * p.chunks_total >= 4LL * n_ctas) return r;
    return p.n_tiles / n_ctas >= 2 ? r + n_ctas : p.n_tiles;
}
struct PieceWalk {
    long long cur, hi;
    int first, n_shared, dp_next, dp_stride;
    int cl_c0, cl_c1;      // cluster mode: this CTA's chunk range of every tile its cluster takes (cl_c1 = 0: not cluster mode)
    // cs: CTAs per cluster. A cluster-mode phase gives its tiles to the clusters in turn; rank r of a cluster
    // streams chunks [r * C / cs, (r + 1) * C / cs) of each of its tiles.
    __host__ __device__ __forceinline__ PieceWalk(const KParams& p, int cta, int n_ctas, int cs) {
        first = 1;
        n_shared = shared_tiles(p, n_ctas);
        const long long T = (long long)n_shared * p.chunks_total;
        cur = (long long)cta * T / n_ctas;
        hi = (long long)(cta + 1) * T / n_ctas;
        if (p.cluster_k) {
            const int rank = cta % cs;
            dp_next = n_shared + cta / cs;
            dp_stride = n_ctas / cs;
            cl_c0 = rank * p.chunks_total / cs;
            cl_c1 = (rank + 1) * p.chunks_total / cs;
        } else {
            cl_c0 = cl_c1 = 0;
            dp_next = n_shared + cta;
            dp_stride = n_ctas;
        }
    }
    __host__ __device__ __forceinline__ bool shared_done() const { return cur >= hi; }
    __host__ __device__ __forceinline__ bool done(const KParams& p) const { return cur >= hi && dp_next >= p.n_tiles; }
    __host__ __device__ __forceinline__ Unit next(const KParams& p) {
        Unit u;
        u.cl = 0;
        if (cur < hi) {
            u.tile = (int)(cur / p.chunks_total);
            u.c0 = (int)(cur % p.chunks_total);
            const long long left = hi - cur;
            u.c1 = (u.c0 + left < (long long)p.chunks_total) ? (int)(u.c0 + left) : p.chunks_total;
            u.full = (u.c0 == 0 && u.c1 == p.chunks_total) ? 1 : 0;
            u.slot = first ? 0 : 1;
            cur += u.c1 - u.c0;
            first = 0;
        } else {
            u.tile = dp_next;
            u.c0 = 0;
            u.c1 = p.chunks_total;
            u.full = 1;
            u.slot = 0;
            if (cl_c1 > 0) { u.c0 = cl_c0; u.c1 = cl_c1; u.full = 0; u.cl = 1; }
            dp_next += dp_stride;
        }
        int t = u.tile;
        u.tt = t % p.n_ttiles;
        t /= p.n_ttiles;
        u.ft = t % p.n_ftiles;
        u.g = t / p.n_ftiles;
        u.ctr = u.tile;
        u.phantom = 0;
        return u;
    }
};
// CTA that owns pair number x of the shared part (T pairs):  largest j with floor(j*T/G) <= x
__host__ __device__ __forceinline__ int cta_of_pair(long long x, long long T, int G) { return (int)(((x + 1) * G + T - 1) / T - 1); }

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

// Residual rows of one pass (x += ...) and the next norm's gain for this feature: loaded by the caller,
// ahead of whatever else it waits for.
// lim: token columns of this pass (<= CH)
template <int CH>
__device__ __forceinline__ void residual_load(const KParams& p, const Unit& un, int tok0, int row, float (&xres)[CH], float& gain,
                                              int lim = CH) {
    const int f = un.ft * TILE_F + row;
    const int n_tok = min(lim, p.M - tok0);
    gain = (p.g_next && (p.epi == EPI_RESIDUAL || p.epi == EPI_STORE_F32) && f < p.N) ? __bfloat162float(p.g_next[f]) : 0.f;
#pragma unroll
    for (int c = 0; c < CH; ++c) xres[c] = 0.f;
    if (p.epi == EPI_RESIDUAL && f < p.N) {
        const float* o = p.out_f32 + (size_t)tok0 * p.ld_out + f;
#pragma unroll
        for (int c = 0; c < CH; ++c)
            if (c < n_tok) xres[c] = __ldcg(o + (size_t)c * p.ld_out);
    }
}

// rn[c] = rsqrt(mean over this row's head of acc^2 + eps) for SB token columns of sAcc, all 128
// threads together (two named barriers): a head is the tile's 128 rows (hd = 128) or its half (hd = 64).
template <int SB>
__device__ __forceinline__ void head_rnorm(const KParams& p, const float* sAcc, int acc_ld, float* red, int row, int c0, int n_tok,
                                           bool active, float (&rn)[SB]) {
    float sq[SB];
#pragma unroll
    for (int c = 0; c < SB; ++c) {
        const float a = (active && c0 + c < n_tok) ? sAcc[row * acc_ld + c0 + c] : 0.f;
        sq[c] = a * a;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
#pragma unroll
        for (int c = 0; c < SB; ++c) sq[c] += __shfl_xor_sync(0xffffffffu, sq[c], o);
    if ((row & 31) == 0) {
#pragma unroll
        for (int c = 0; c < SB; ++c) red[(row >> 5) * SB + c] = sq[c];
    }
    epi_bar();
    const int w0 = p.hd == 128 ? 0 : (row >> 6) * 2, nw = p.hd == 128 ? 4 : 2;
    const float inv_hd = 1.f / (float)p.hd;
#pragma unroll
    for (int c = 0; c < SB; ++c) {
        float t = 0.f;
        for (int w = 0; w < nw; ++w) t += red[(w0 + w) * SB + c];
        rn[c] = rsqrtf(t * inv_hd + p.eps);
    }
    epi_bar();
}

// Every one of the 128 epilogue threads calls this (it contains named barriers).
// QKN: the launch has per-head q/k norms (a separate instantiation keeps the common path's registers down).
// val: this thread's accumulator row of the pass (already scaled by the per-token rsqrt of a folded norm). It goes
// through shared memory (sAcc) only where an epilogue needs other rows' values (rotation partners, per-tile
// reductions); the element-wise epilogues work from registers, with a lane exchange for the gate/up pairs.
// lim: token columns of this pass (<= CH; columns from lim on hold nothing and produce nothing)
template <int CH, bool QKN>
__device__ __forceinline__ void apply_epilogue(const KParams& p, float* sAcc, Top2Entry* sRed, const Unit& un, int tok0,
                                               int row, const int* tPos, const int* tPage, const float (&xres)[CH], float gain,
                                               const float (&val)[CH], int lim = CH) {
    // tPos / tPage: position and (context projection) pool row of the page slot of the tokens of this pass (-1 = skip)
    constexpr int ACC_LD = CH + 1;
    constexpr int GROUPS = 128 / CH;     // threads per token column in the cross-row reductions
    const int f = un.ft * TILE_F + row;
    const int n_tok = min(lim, p.M - tok0);
    if (p.epi == EPI_QKV_ROPE || p.epi == EPI_ARGMAX || p.epi == EPI_CTX_KV) {      // other rows read this one's values
#pragma unroll
        for (int c = 0; c < CH; ++c) sAcc[row * ACC_LD + c] = val[c];
        epi_bar();
    }
    switch (p.epi) {
        case EPI_STORE_F32:
        case EPI_RESIDUAL: {
            // New rows x (+)= acc go through a shared-memory tile [token][128 features], so that the global side is
            // 16-byte accesses of whole 128-byte lines: the number of memory requests a CTA has in flight, not
            // bytes, limits these epilogues (one 4-byte store per thread and token was measured several times slower).
            // A warp writes out whole tokens: lane l holds features 4l .. 4l+3 of the tile, also scales them into
            // the next contraction's bf16 operand and adds up the token's sum of squares by lane exchange.
            float* sOut = sAcc;                         // CH x 128 floats (<= 128 x (CH + 1))
#pragma unroll
            for (int c = 0; c < CH; ++c) {
                float x = (p.epi == EPI_RESIDUAL) ? xres[c] : 0.f;
                if (c < n_tok && f < p.N) x += val[c];
                sOut[c * TILE_F + row] = x;
            }
            epi_bar();
            const int we = row >> 5, ln = row & 31;
            const int f4 = un.ft * TILE_F + ln * 4;
            const bool vec = f4 + 3 < p.N;
            float g4[4] = {0.f, 0.f, 0.f, 0.f};
            if (p.g_next) {
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (f4 + e < p.N) g4[e] = __bfloat162float(p.g_next[f4 + e]);
            }
#pragma unroll
            for (int t = we; t < CH; t += 4) {
                if (t < n_tok) {                        // uniform over the warp
                    const float4 x4 = *reinterpret_cast<const float4*>(sOut + t * TILE_F + ln * 4);
                    const float xe[4] = {x4.x, x4.y, x4.z, x4.w};
                    const size_t tok = (size_t)(tok0 + t);
                    if (vec) {
                        if (p.out_f32) *reinterpret_cast<float4*>(p.out_f32 + tok * p.ld_out + f4) = x4;
                        if (p.g_next) {
                            __nv_bfloat162 lo = __floats2bfloat162_rn(g4[0] * xe[0], g4[1] * xe[1]);
                            __nv_bfloat162 hi = __floats2bfloat162_rn(g4[2] * xe[2], g4[3] * xe[3]);
                            uint2 w2;
                            w2.x = *reinterpret_cast<uint32_t*>(&lo);
                            w2.y = *reinterpret_cast<uint32_t*>(&hi);
                            *reinterpret_cast<uint2*>(p.xn_out + tok * p.N + f4) = w2;
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            if (f4 + e < p.N) {
                                if (p.out_f32) p.out_f32[tok * p.ld_out + f4 + e] = xe[e];
                                if (p.g_next) p.xn_out[tok * p.N + f4 + e] = __float2bfloat16_rn(g4[e] * xe[e]);
                            }
                        }
                    }
                    if (p.ssq_out) {                    // features past N hold zeros
                        float sq = (xe[0] * xe[0] + xe[1] * xe[1]) + (xe[2] * xe[2] + xe[3] * xe[3]);
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
                        if (ln == 0) p.ssq_out[(size_t)un.ft * p.M + tok0 + t] = sq;
                    }
                }
            }
            epi_bar();      // the next pass overwrites the tile
        } break;
        case EPI_QKV_ROPE: {
            // N is a multiple of 128 on this path (whole heads per tile), so every row is a real feature
            const int hd = p.hd, half = hd >> 1;
            const int head = f / hd, hrow = f % hd, i = hrow % half;
            const int partner = row ^ half;
            const int qdim = p.Hq * hd, kdim = p.Hkv * hd;
            const bool rot = p.use_rope && head < p.Hq + p.Hkv;
            // the tile's 128 features lie in one of q / k / v (their widths are multiples of 128)
            const int f0 = un.ft * TILE_F;
            __nv_bfloat16* dst0;
            int ld;
            if (f0 < qdim) { dst0 = p.q + f0; ld = qdim; }
            else if (f0 < qdim + kdim) { dst0 = p.k + (f0 - qdim); ld = kdim; }
            else { dst0 = p.v + (f0 - qdim - kdim); ld = kdim; }
            float rot_out[CH];
#pragma unroll
            for (int c = 0; c < CH; ++c) rot_out[c] = 0.f;
            // optional per-head RMSNorm of q and k before the rotation
            const __nv_bfloat16* gain = (!QKN || !p.gq) ? nullptr : (head < p.Hq ? p.gq : (head < p.Hq + p.Hkv ? p.gk[0] : nullptr));
            const float g_self = gain ? __bfloat162float(gain[hrow]) : 1.f;
            const float g_part = gain ? __bfloat162float(gain[hrow ^ half]) : 1.f;
            constexpr int SB = CH <= 16 ? 8 : 16;        // tokens per sub-block: their table loads are in flight together
#pragma unroll
            for (int c0 = 0; c0 < CH; c0 += SB) {
                if (c0 >= n_tok) break;
                float cs[SB], sn[SB];
#pragma unroll
                for (int c = 0; c < SB; ++c) { cs[c] = 1.f; sn[c] = 0.f; }
                if (p.use_rope) {       // unconditional loads (table row 0 when the token is unused)
#pragma unroll
                    for (int c = 0; c < SB; ++c) {
                        const int pos = (c0 + c < n_tok) ? tPos[c0 + c] : 0;      // entries past n_tok are not initialised
                        const size_t at = (size_t)max(pos, 0) * half + i;
                        cs[c] = __ldg(p.cs + at);
                        sn[c] = __ldg(p.sn + at);
                    }
                }
                float rn[SB];
#pragma unroll
                for (int c = 0; c < SB; ++c) rn[c] = 1.f;
                if (QKN && p.gq) {      // uniform over the 128 threads
                    head_rnorm<SB>(p, sAcc, ACC_LD, reinterpret_cast<float*>(sRed), row, c0, n_tok, gain != nullptr, rn);
                    if (!gain) {
#pragma unroll
                        for (int c = 0; c < SB; ++c) rn[c] = 1.f;
                    }
                }
#pragma unroll
                for (int c = 0; c < SB; ++c) {
                    if (c0 + c < n_tok) {
                        const bool on = rot && tPos[c0 + c] >= 0;
                        const float cc = on ? cs[c] : 1.f, ss = on ? sn[c] : 0.f;
                        const float a = sAcc[row * ACC_LD + c0 + c] * (rn[c] * g_self);
                        const float b = sAcc[partner * ACC_LD + c0 + c] * (rn[c] * g_part);
                        rot_out[c0 + c] = hrow < half ? (a * cc - b * ss) : (a * cc + b * ss);
                    }
                }
            }
            // out through a shared-memory tile [token][128] as 16-byte stores of whole lines (see the residual epilogue)
            epi_bar();                                  // every row has read its partner's accumulators
            __nv_bfloat16* sOut = reinterpret_cast<__nv_bfloat16*>(sAcc);
#pragma unroll
            for (int c = 0; c < CH; ++c) sOut[c * TILE_F + row] = __float2bfloat16_rn(rot_out[c]);
            epi_bar();
            for (int q = row; q < CH * 16; q += 128) {
                const int t = q >> 4, part = q & 15;
                if (t < n_tok)
                    *reinterpret_cast<uint4*>(dst0 + (size_t)(tok0 + t) * ld + part * 8) = *reinterpret_cast<const uint4*>(sOut + t * TILE_F + part * 8);
            }
            epi_bar();
        } break;
        case EPI_SWIGLU: {
            // rows 2j / 2j+1 hold gate_j / up_j. The even lane finishes token columns [0, CH/2), the odd lane
            // [CH/2, CH): each sends its partner the half it does not finish itself (one lane exchange per column
            // pair). The 64 outputs per token go through a shared-memory tile [token][64] and leave as 16-byte
            // stores of whole lines (see the residual epilogue).
            const bool odd = (row & 1) != 0;
            constexpr int HC = CH / 2;
            const int c_base = odd ? HC : 0;
            __nv_bfloat16* sOut = reinterpret_cast<__nv_bfloat16*>(sAcc);      // CH x 64 bf16
#pragma unroll
            for (int k = 0; k < HC; ++k) {
                const float other = __shfl_xor_sync(0xffffffffu, odd ? val[k] : val[k + HC], 1);
                const float g = odd ? other : val[k], u = odd ? val[k + HC] : other;
                sOut[(c_base + k) * 64 + (row >> 1)] = __float2bfloat16_rn(__fdividef(g, 1.f + __expf(-g)) * u);
            }
            epi_bar();
            const int j_tile = un.ft * 64;              // first FFN unit of this tile
            for (int q = row; q < CH * 8; q += 128) {
                const int t = q >> 3, part = q & 7;
                if (t < n_tok) {
                    const int j0 = j_tile + part * 8;
                    __nv_bfloat16* dst = p.h + (size_t)(tok0 + t) * p.F + j0;
                    if (j0 + 8 <= p.F) {
                        *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(sOut + t * 64 + part * 8);
                    } else {
                        for (int e = 0; e < 8; ++e)
                            if (j0 + e < p.F) dst[e] = sOut[t * 64 + part * 8 + e];
                    }
                }
            }
            epi_bar();
        } break;
        case EPI_ARGMAX: {
            if (p.logits_out && f < p.N)
                for (int c = 0; c < n_tok; ++c) p.logits_out[(size_t)(tok0 + c) * p.N + f] = sAcc[row * ACC_LD + c];
            const int c = row % CH, g = row / CH;
            // largest value, its first row and the second largest value of CH rows of one token column, without
            // branches (rows come in increasing order, so a strict comparison keeps the smallest index among equals;
            // data-dependent branches made this scan the slowest part of a wide token tile's epilogue)
            float v1 = -CUDART_INF_F, v2 = -CUDART_INF_F;
            int i1 = 0x7fffffff;
            const int f_base = un.ft * TILE_F + g * CH;
#pragma unroll
            for (int r = 0; r < CH; ++r) {
                const float x = (f_base + r < p.N) ? sAcc[(g * CH + r) * ACC_LD + c] : -CUDART_INF_F;
                i1 = (x > v1) ? f_base + r : i1;
                v2 = fmaxf(v2, fminf(v1, x));
                v1 = fmaxf(v1, x);
            }
            sRed[g * CH + c] = Top2Entry{v1, i1, v2, 0};
            epi_bar();
            if (row < n_tok) {
                T2 m{sRed[row].v1, sRed[row].i1, sRed[row].v2};
#pragma unroll
                for (int gg = 1; gg < GROUPS; ++gg) t2_merge(m, sRed[gg * CH + row].v1, sRed[gg * CH + row].i1, sRed[gg * CH + row].v2);
                p.top2[(size_t)un.ft * p.M + tok0 + row] = Top2Entry{m.v1, m.i1, m.v2, 0};
            }
            epi_bar();
        } break;
        case EPI_CTX_KV: {
            // N = 2 * Hkv * hd is a multiple of 128 on this path
            const int hd = p.hd, half = hd >> 1;
            const int kdim = p.Hkv * hd;
            const int is_v = f >= kdim ? 1 : 0;
            const int fh = f - is_v * kdim;
            const int head = fh / hd, hrow = fh % hd, i = hrow % half;
            const int partner = row ^ half;
            const int layer = p.first_layer + un.g;
            const bool rot = !is_v && p.use_rope;
            const __nv_bfloat16* gk = QKN ? p.gk[un.g] : nullptr;         // per-head norm of the keys, or nullptr
            const __nv_bfloat16* gain = is_v ? nullptr : gk;
            const float g_self = gain ? __bfloat162float(gain[hrow]) : 1.f;
            const float g_part = gain ? __bfloat162float(gain[hrow ^ half]) : 1.f;
            // pool[layer][page][K|V][head][slot][hd]: tPage[c] = row of (page, K, head 0, slot)
            __nv_bfloat16* base = p.pool + (((size_t)layer * p.n_pages * 2 + is_v) * p.Hkv + head) * p.PG * hd + hrow;
            constexpr int SB = CH <= 16 ? 8 : 16;
#pragma unroll
            for (int c0 = 0; c0 < CH; c0 += SB) {
                if (c0 >= n_tok) break;
                float cs[SB], sn[SB];
#pragma unroll
                for (int c = 0; c < SB; ++c) { cs[c] = 1.f; sn[c] = 0.f; }
                if (rot) {
#pragma unroll
                    for (int c = 0; c < SB; ++c) {
                        const int pos = (c0 + c < n_tok) ? tPos[c0 + c] : 0;      // entries past n_tok are not initialised
                        const size_t at = (size_t)max(pos, 0) * half + i;
                        cs[c] = __ldg(p.cs + at);
                        sn[c] = __ldg(p.sn + at);
                    }
                }
                float rn[SB];
#pragma unroll
                for (int c = 0; c < SB; ++c) rn[c] = 1.f;
                if (QKN && gk) {        // uniform over the 128 threads
                    head_rnorm<SB>(p, sAcc, ACC_LD, reinterpret_cast<float*>(sRed), row, c0, n_tok, gain != nullptr, rn);
                    if (!gain) {
#pragma unroll
                        for (int c = 0; c < SB; ++c) rn[c] = 1.f;
                    }
                }
#pragma unroll
                for (int c = 0; c < SB; ++c) {
                    const int prow = (c0 + c < n_tok) ? tPage[c0 + c] : -1;
                    if (prow >= 0) {
                        float kv_v = sAcc[row * ACC_LD + c0 + c] * (rn[c] * g_self);
                        if (rot) {
                            const float bb = sAcc[partner * ACC_LD + c0 + c] * (rn[c] * g_part);
                            kv_v = hrow < half ? (kv_v * cs[c] - bb * sn[c]) : (kv_v * cs[c] + bb * sn[c]);
                        }
                        base[(size_t)prow * hd] = __float2bfloat16_rn(kv_v);
                    }
                }
            }
            epi_bar();
        } break;
        default: break;
    }
}

// ---------------------------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------------------------
// Position (and, for the context projection, the pool row of its page slot) of every token of a token
// tile, worked out once per phase by the epilogue threads: the per-pass epilogues then carry no
// dependent loads and little address arithmetic (with one warp per scheduler every instruction of a
// dependent chain costs its full latency).
__device__ __forceinline__ void token_info(const KParams& p, int tok_base, int nt, int row, int* sPos, int* sPage) {
    for (int t = row; t < nt; t += 128) {      // sPos[t] describes token tok_base + t
        const int tok = tok_base + t;
        int pos = -1, page = -1;
        if (tok < p.M) {
            if (p.epi == EPI_QKV_ROPE) {
                pos = __ldcg(p.ctx_len + tok / p.rows_per_seq) + tok % p.rows_per_seq;
                if (p.use_rope && (pos < 0 || pos >= p.max_pos)) {
                    if (p.status) atomicOr(p.status, DFLASH_DEV_CTX_OVERFLOW);
                    pos = pos < 0 ? 0 : p.max_pos - 1;
                }
            } else if (p.epi == EPI_CTX_KV) {
                const int b = tok / p.max_new, r = tok % p.max_new;
                const int nn = p.n_new ? __ldcg(p.n_new + b) : p.max_new;
                if (r < nn) {
                    pos = __ldcg(p.ctx_len + b) + r;
                    const int pidx = pos / p.PG;
                    if (pos < 0 || pidx >= p.max_pages || (p.use_rope && pos >= p.max_pos)) {
                        if (p.status) atomicOr(p.status, DFLASH_DEV_CTX_OVERFLOW);
                        pos = -1;
                    } else {
                        page = __ldcg(p.page_table + (size_t)b * p.max_pages + pidx);
                        if (page < 0 || page >= p.n_pages) {
                            if (p.status) atomicOr(p.status, DFLASH_DEV_BAD_PAGE);
                            pos = -1;
                            page = -1;
                        } else {
                            page = page * 2 * p.Hkv * p.PG + pos % p.PG;     // row of (page, K, head 0, slot) in the layer's pool
                        }
                    }
                }
            }
        }
        sPos[t] = pos;
        sPage[t] = page;
    }
}

// rsqrt(mean square) of operand rows tok_base .. tok_base+nt-1 from the per-tile sums of squares:
// eight threads per token, sixteen loads in flight per thread-group of a pass (64 tokens per pass).
__device__ __forceinline__ void token_rstd(const KParams& p, int tok_base, int nt, int row, float* sRstd) {
    const int sub = row & 7, tl = row >> 3;
    for (int t0 = 0; t0 < nt; t0 += 64) {
        float s[4];
        bool on[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            s[u] = 0.f;
            const int t = t0 + u * 16 + tl;
            on[u] = t < nt && tok_base + t < p.M;
        }
        for (int q0 = sub; q0 < p.n_parts_in; q0 += 32) {
            float v[4][4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int q = q0 + 8 * k;
                    v[u][k] = (on[u] && q < p.n_parts_in) ? __ldcg(p.ssq_in + (size_t)q * p.M + tok_base + t0 + u * 16 + tl) : 0.f;
                }
#pragma unroll
            for (int u = 0; u < 4; ++u) s[u] += (v[u][0] + v[u][1]) + (v[u][2] + v[u][3]);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            s[u] += __shfl_xor_sync(0xffffffffu, s[u], 1);
            s[u] += __shfl_xor_sync(0xffffffffu, s[u], 2);
            s[u] += __shfl_xor_sync(0xffffffffu, s[u], 4);
            const int t = t0 + u * 16 + tl;
            if (sub == 0 && t < nt) sRstd[t] = on[u] ? rsqrtf(s[u] * p.inv_dim_in + p.eps) : 1.f;
        }
    }
}

// Counter increment that publishes what this CTA wrote: the CTA's threads meet at a barrier, then ONE thread adds
// with release semantics at GPU scope (cumulative over the writes ordered before it by the barrier); readers poll
// with ld_acquire. Cheaper than a fence by each of the 128 threads.
__device__ __forceinline__ void red_release_add(int32_t* p, int v) {
    asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Bounded poll of a global counter written by other CTAs (release/acquire through L2).
__device__ __forceinline__ int ld_acquire(const int32_t* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Register cap: with small token tiles the kernel is kept at 232 registers, so that a warp of a small dependent
// kernel (merge, finish) still fits into the register file partition that holds two of this CTA's six warps and
// can become resident before this grid has drained.
// PAIR: the launch runs as clusters of two CTAs that share every MMA (cta_group::2, M = 256): each CTA streams its own
// 128-row weight tile but only HALF of the token tile, so a ring stage is a third smaller and the ring deeper - with
// 160 to 256 token columns the single-CTA form is limited by the operand bytes an SM keeps in flight, not by the tensor
// pipe. The even CTA's MMA thread issues for both; its commits arrive on both CTAs' barriers. Each CTA holds its own
// 128 rows x NT columns of the accumulator in its own TMEM, so the epilogues are those of the single-CTA form.
template <int NT, int SL, bool QKN, bool PAIR>
__global__ void __maxnreg__(NT <= 32 ? 232 : 255)
gemm_tc_kernel(const __grid_constant__ WMaps tmW, const __grid_constant__ XMaps tmX, const __grid_constant__ MParams mp) {
    if (threadIdx.x == 0) trace_min(mp.ph[0].trace, 0);
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    constexpr int W_STAGE = W_STAGE_BYTES * SL;
    constexpr int XR = PAIR ? NT / 2 : NT;           // token rows of the activation tile this CTA loads
    constexpr int X_SLAB = XR * BK * 2;
    constexpr int X_STAGE = X_SLAB * SL;
    static_assert(!PAIR || (SL == 1 && NT % 32 == 0 && NT >= 64), "CTA pairs: one slab per stage, halves of whole 16-row groups");
    constexpr int CH = pass_cols(NT);
    constexpr int ACC_LD = CH + 1;
    // partial pieces fetched together when finishing. More would shorten the tail further, but the register
    // count must leave room for the CTAs of the next kernel to become resident beside this one: a
    // dependent kernel that cannot start early was measured 30 us slower.
    constexpr int PF = (NT == 256) ? 1 : (CH <= 16 ? 4 : (CH <= 32 ? 3 : 1));
    constexpr uint32_t TMEM_COLS = (2 * NT <= 32) ? 32u : (2 * NT <= 64) ? 64u : (2 * NT <= 128) ? 128u : (2 * NT <= 256) ? 256u : 512u;   // a power of two
    const int stages = mp.stages;
    uint8_t* sW = smem;
    uint8_t* sX = sW + (size_t)stages * W_STAGE;
    float* sAcc = reinterpret_cast<float*>(sX + (size_t)stages * X_STAGE);
    Top2Entry* sRed = reinterpret_cast<Top2Entry*>(sAcc + TILE_F * ACC_LD);
    constexpr int TOK_CACHE = tok_cache(NT);
    float* sRstd = reinterpret_cast<float*>(sRed + 128);          // [TOK_CACHE] per-token rsqrt(mean square)
    int* sPos = reinterpret_cast<int*>(sRstd + TOK_CACHE);        // [TOK_CACHE] per-token position (-1: skip)
    int* sPage = sPos + TOK_CACHE;                                // [TOK_CACHE] per-token physical page
    float* sXch = reinterpret_cast<float*>(sPage + TOK_CACHE);    // [2][CS - 1][128][NT / CS] columns received from cluster peers
    uint64_t* full = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(sXch) + xch_bytes(NT));
    uint64_t* empty = full + MAX_STAGES;
    uint64_t* acc_full = empty + MAX_STAGES;
    uint64_t* acc_empty = acc_full + 2;
    uint64_t* xch_bar = acc_empty + 2;                            // [2] one per receive buffer: counts the bytes the peers' stores deliver
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(xch_bar + 2);
    volatile int* flags = reinterpret_cast<volatile int*>(tmem_slot + 1);   // [0] abort, [2] epilogue abort
    int* sPend = const_cast<int*>(flags) + 4;                               // [3 * MAX_STAGES] producer's queue

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        // a pair's leader frees an accumulator buffer when the epilogue warps of BOTH CTAs have read it
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], PAIR ? 8 : 4); mbar_init(&xch_bar[b], 1); }
        flags[0] = 0; flags[2] = 0;
        fence_barrier_init();
        fence_proxy_async();
    }
    if (warp == 1) tmem_alloc(tmem_slot, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_trigger();
    // Peers must not write into this CTA's receive buffers or count bytes on its barriers before they exist: every
    // thread arrives on the cluster barrier here and waits on it later, where its role has nothing better to do (the
    // epilogue warps before their first tile, the two single-thread roles at their end).
    if (mp.cs > 1) cluster_arrive();

    const int G = gridDim.x;
    // CTA pairs: the pair is the unit that walks the work; both CTAs take the same pieces
    const int prank = PAIR ? (int)cluster_ctarank() : 0;
    const int wid = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int WG = PAIR ? G >> 1 : G;
    bool run = true;
    if constexpr (PAIR) {
        // Both CTAs' barriers exist before anyone arrives on a peer's; the MMA addresses both accumulators by ONE
        // TMEM address, so the two allocations must have come out at the same columns (each CTA allocates once from
        // an empty TMEM, so they do; checked, not assumed).
        cluster_sync_all();
        run = ld_shared_cluster_u32(mapa_shared(smem_u32(tmem_slot), (uint32_t)(prank ^ 1))) == tmem_base;
        if (!run && threadIdx.x == 0 && mp.status) atomicOr(mp.status, DFLASH_DEV_TIMEOUT);
    }

    if (!run) {
        // nothing: the other pairs' waits run out and the call reports the status word
    } else if (warp == 0) {
        // ---------------- TMA producer ----------------
        // WEIGHT tiles are issued as soon as a ring slot is free. The ACTIVATION tile of a slot needs
        // the phase's inputs (phase 0: the grid dependency; later phases: every CTA has finished the
        // previous phase). While they are missing, the slot is queued and the weight stream goes on;
        // queued slots are completed, in order, as soon as the inputs exist. In the steady state the
        // queue is empty and both tiles are issued back to back.
        if (lane == 0) {
            const uint64_t pol_w = policy_evict_first(), pol_x = policy_evict_last();
            // chunk c of rows y.. : SL slabs of 64 K-elements
            // CTA pairs: both CTAs' copies count their bytes on the LEADER's barrier of the stage
            const uint32_t full_leader = PAIR ? mapa_shared(smem_u32(full), 0u) : 0u;
            auto load = [&](void* dst, const CUtensorMap* m, int c, int y, int slot, uint64_t pol) {
                if constexpr (PAIR) tma_load_2d_pair(dst, m, c * BK, y, full_leader + (uint32_t)slot * 8u, pol);
                else if constexpr (SL == 1) tma_load_2d(dst, m, c * BK, y, &full[slot], pol);
                else tma_load_3d(dst, m, 0, y, c * SL, &full[slot], pol);
            };
            int* q_ph = sPend;                      // queued slots: phase, chunk, token tile (ring order)
            int* q_c = sPend + MAX_STAGES;
            int* q_tt = sPend + 2 * MAX_STAGES;
            int q_head = 0, q_count = 0;            // q_head = ring slot of the oldest queued entry
            int ready_ph = -1;                      // phases 0..ready_ph have their inputs
            int st = 0;
            uint32_t par = 0;
            bool ok = true;
            // completes queued slots while their phase is ready; returns false if the head still waits
            auto flush = [&]() {
                while (q_count > 0) {
                    const int ph = q_ph[q_head];
                    if (ph > ready_ph) {
                        if (ph == 0) {
                            pdl_wait();
                            trace_min(mp.ph[0].trace, 1);
                        } else {
                            if (ld_acquire(mp.phase_done + ph - 1) < G) return;
                            fence_proxy_async_all();      // other CTAs' stores -> this CTA's TMA reads
                            trace_min(mp.ph[ph].trace, 0);
                            trace_min(mp.ph[ph].trace, 1);
                        }
                        ready_ph = ph;
                    }
                    load(sX + (size_t)q_head * X_STAGE, &tmX.m[mp.ph[ph].x_map], q_c[q_head], q_tt[q_head] * NT + prank * XR, q_head, pol_x);
                    q_head = (q_head + 1 == stages) ? 0 : q_head + 1;
                    --q_count;
                }
            };
            for (int ph = 0; ph < mp.n_phases && ok; ++ph) {
                const KParams& p = mp.ph[ph];
                const CUtensorMap* xm = &tmX.m[p.x_map];
                for (PieceWalk w(p, wid, WG, mp.cs); !w.done(p) && ok;) {
                    Unit un = w.next(p);
                    own_tile<PAIR>(p, un, prank);
                    const CUtensorMap* wm = &tmW.m[p.w_map0 + un.g];
                    const int y_w = un.ft * TILE_F, y_x = un.tt * NT + prank * XR;      // rows beyond the matrix arrive as zeros
                    for (int c = un.c0; c < un.c1; ++c) {
                        if (!mbar_try_wait(&empty[st], par ^ 1)) {
                            const long long t0 = clock64();
                            while (!mbar_try_wait(&empty[st], par ^ 1)) {
                                flush();                  // a full ring of queued slots frees nothing by itself
                                if (flags[0] || clock64() - t0 > SPIN_LIMIT) { ok = false; break; }
                            }
                            if (!ok) break;
                        }
                        if (!PAIR || prank == 0) mbar_expect_tx(&full[st], (PAIR ? 2 : 1) * (W_STAGE + X_STAGE));
                        load(sW + (size_t)st * W_STAGE, wm, c, y_w, st, pol_w);
                        if (q_count == 0 && ph <= ready_ph) {
                            load(sX + (size_t)st * X_STAGE, xm, c, y_x, st, pol_x);
                        } else {
                            if (q_count == 0) q_head = st;
                            q_ph[st] = ph; q_c[st] = c; q_tt[st] = un.tt;
                            ++q_count;
                            flush();
                        }
                        if (++st == stages) { st = 0; par ^= 1; }
                    }
                }
            }
            if (ok && q_count > 0) {
                const long long t0 = clock64();
                while (q_count > 0) {
                    flush();
                    if (flags[0] || clock64() - t0 > SPIN_LIMIT) { ok = false; break; }
                }
            }
            if (!ok) {
                flags[0] = 1;
                if (mp.status) atomicOr(mp.status, DFLASH_DEV_TIMEOUT);
                // weight tiles already in flight must land before the CTA goes away; their barriers
                // never complete without the activation tile, so wait on time instead
                const long long t0 = clock64();
                while (clock64() - t0 < DRAIN_LIMIT) {}
            }
        }
        __syncwarp();     // the whole warp must reach the closing barrier together
        if (mp.cs > 1) cluster_wait();
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        // (the odd CTA of a pair issues nothing: the leader's MMAs read both CTAs' operands and write both accumulators)
        if (lane == 0 && !(PAIR && prank == 1)) {
            constexpr uint32_t idesc = instr_desc_bf16(PAIR ? 2 * TILE_F : TILE_F, NT);
            uint32_t it = 0, ui = 0;
            bool ok = true;
            for (int ph = 0; ph < mp.n_phases && ok; ++ph) {
                const KParams& p = mp.ph[ph];
                for (PieceWalk w(p, wid, WG, mp.cs); !w.done(p) && ok; ++ui) {
                    const Unit un = w.next(p);
                    const uint32_t buf = ui & 1, aph = (ui >> 1) & 1;
                    if (!mbar_wait(&acc_empty[buf], aph ^ 1, &flags[0])) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + buf * NT;
                    for (int c = un.c0; c < un.c1; ++c, ++it) {
                        const int st = it % stages;
                        const uint32_t phs = (it / stages) & 1;
                        if (!mbar_wait(&full[st], phs, &flags[0])) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t a_addr = smem_u32(sW + (size_t)st * W_STAGE);
                        const uint32_t b_addr = smem_u32(sX + (size_t)st * X_STAGE);
#pragma unroll
                        for (int kk = 0; kk < SL * (BK / 16); ++kk) {
                            const uint64_t da = smem_desc_sw128(a_addr + (kk >> 2) * W_STAGE_BYTES + (kk & 3) * 32);
                            const uint64_t db = smem_desc_sw128(b_addr + (kk >> 2) * X_SLAB + (kk & 3) * 32);
                            const uint32_t acc = (c > un.c0 || kk > 0) ? 1u : 0u;
                            if constexpr (PAIR) mma_bf16_pair(d_tmem, da, db, idesc, acc);
                            else mma_bf16(d_tmem, da, db, idesc, acc);
                        }
                        if constexpr (PAIR) mma_commit_pair(&empty[st], 3);
                        else mma_commit(&empty[st]);
                    }
                    if (ok) {
                        if constexpr (PAIR) mma_commit_pair(&acc_full[buf], 3);
                        else mma_commit(&acc_full[buf]);
                    }
                }
                trace_max(p.trace, 2);
            }
            if (!ok) {
                flags[0] = 1;
                if (mp.status) atomicOr(mp.status, DFLASH_DEV_TIMEOUT);
            }
        }
        __syncwarp();
        if (mp.cs > 1) cluster_wait();
    } else {
        // ---------------- epilogue: warps 2..5, TMEM lane quadrant = warp % 4 ----------------
        const int ew = warp & 3;
        const int row = ew * 32 + lane;
        uint32_t ui = 0;
        bool alive = true;
        // cluster exchange: this CTA's rank, the peers' views of the receive buffers and of their barriers
        const int rank = mp.cs > 1 ? (int)cluster_ctarank() : 0;
        uint32_t xch_remote[CS], xbar_remote[CS];
#pragma unroll
        for (int q = 0; q < CS; ++q) {
            xch_remote[q] = mp.cs > 1 ? mapa_shared(smem_u32(sXch), (uint32_t)q) : 0u;
            xbar_remote[q] = mp.cs > 1 ? mapa_shared(smem_u32(xch_bar), (uint32_t)q) : 0u;
        }
        uint32_t cl_units = 0;       // cluster-shared tiles finished so far (the same number in every CTA of the cluster)
        pdl_wait();      // lengths, page tables, residual rows ... come from earlier kernels
        if (mp.cs > 1) cluster_wait();      // every peer has set up its barriers (they arrived after doing so)
        for (int ph = 0; ph < mp.n_phases && alive; ++ph) {
            const KParams& p = mp.ph[ph];
            const long long T = (long long)shared_tiles(p, WG) * p.chunks_total;     // (tile, chunk) pairs of the shared part
            const bool all_tok = p.M <= TOK_CACHE;   // per-token data cached for the whole phase (else per token tile)
            const bool need_info = p.epi == EPI_QKV_ROPE || p.epi == EPI_CTX_KV;
            int rstd_tt = -1, info_tt = -1;
            // token positions / pages do not depend on this chain: work them out while the main loop runs
            if (need_info && all_tok) {
                token_info(p, 0, p.M, row, sPos, sPage);
                info_tt = 0;             // visible after the next barrier
            }
            // per-token scales: as soon as the previous phase is complete (its sums of squares are final),
            // long before this phase's first accumulator
            if (p.ssq_in && all_tok) {
                if (ph > 0) {
                    if (row == 0) {
                        const long long t0 = clock64();
                        while (ld_acquire(mp.phase_done + ph - 1) < G) {
                            if (flags[0] || clock64() - t0 > SPIN_LIMIT) { flags[2] = 1; break; }
                        }
                    }
                    epi_bar();
                    if (flags[2]) { alive = false; break; }
                }
                token_rstd(p, 0, p.M, row, sRstd);
                rstd_tt = 0;
            }
            Unit pend[2];            // this CTA's pieces of shared tiles (at most its first and its last piece)
            int n_pend = 0;
            // ---- shared tiles: wait for every contributor's piece, then do this CTA's share of the passes.
            // Runs as soon as this CTA's shared pieces are published: while whole tiles remain, the
            // reduction overlaps their streaming.
            auto finish_shared = [&]() {
                for (int pi = 0; pi < n_pend && alive; ++pi) {
                    const Unit un = pend[pi];
                    const int tok_base = un.tt * NT;
                    const int tok_off = all_tok ? tok_base : 0;
                    const long long x0 = (long long)un.tile * p.chunks_total;
                    const int j0 = cta_of_pair(x0, T, WG), j1 = cta_of_pair(x0 + p.chunks_total - 1, T, WG);
                    const int n_contrib = j1 - j0 + 1, my_q = wid - j0;
                    const int n_ch = (min(NT, p.M - tok_base) + CH - 1) / CH;
                    if (my_q >= n_ch) continue;                      // more contributors than passes: nothing for this one
                    // residual rows of the first pass travel while the tickets are polled
                    float xres[CH], gain = 0.f;
                    if constexpr (CH <= 32) residual_load<CH>(p, un, tok_base + my_q * CH, row, xres, gain);
                    if (row == 0) {
                        const long long t0 = clock64();
                        while (ld_acquire(p.counters + un.ctr) < n_contrib) {
                            if (flags[0] || clock64() - t0 > SPIN_LIMIT) { flags[2] = 1; break; }
                        }
                    }
                    epi_bar();               // row 0's acquire, then the barrier: every piece is visible to all rows
                    if (flags[2]) { alive = false; return; }
                    if (!all_tok) {      // caches hold one token tile at a time
                        if (need_info && info_tt != un.tt) { token_info(p, tok_base, NT, row, sPos, sPage); info_tt = un.tt; }
                        if (p.ssq_in && rstd_tt != un.tt) { token_rstd(p, tok_base, NT, row, sRstd); rstd_tt = un.tt; }
                        epi_bar();
                    }
                    for (int ch = my_q; ch < n_ch; ch += n_contrib) {
                        if constexpr (CH <= 32) {
                            if (ch != my_q) residual_load<CH>(p, un, tok_base + ch * CH, row, xres, gain);
                        }
                        float acc[CH];
#pragma unroll
                        for (int c = 0; c < CH; ++c) acc[c] = 0.f;
                        // pieces are summed in CTA order; the loads of PF pieces are all in flight together
                        for (int jb = j0; jb <= j1; jb += PF) {
                            float va[PF][CH];
#pragma unroll
                            for (int u = 0; u < PF; ++u) {
                                const int j = jb + u;
                                if (j <= j1) {
                                    const int sa = ((long long)j * T / WG >= x0) ? 0 : 1;
                                    const size_t jc = PAIR ? (size_t)j * 2 + prank : (size_t)j;      // the contributing CTA
                                    const float* pa = p.part + ((jc * 2 + sa) * NT + ch * CH) * TILE_F + row;
#pragma unroll
                                    for (int c = 0; c < CH; ++c) va[u][c] = __ldcg(pa + (size_t)c * TILE_F);
                                } else {
#pragma unroll
                                    for (int c = 0; c < CH; ++c) va[u][c] = 0.f;
                                }
                            }
#pragma unroll
                            for (int u = 0; u < PF; ++u)
#pragma unroll
                                for (int c = 0; c < CH; ++c) acc[c] += va[u][c];
                        }
                        if (p.ssq_in) {
#pragma unroll
                            for (int c = 0; c < CH; ++c) acc[c] *= sRstd[tok_off + ch * CH + c];
                        }
                        if constexpr (CH > 32) residual_load<CH>(p, un, tok_base + ch * CH, row, xres, gain);
                        apply_epilogue<CH, QKN>(p, sAcc, sRed, un, tok_base + ch * CH, row, sPos + tok_off + ch * CH, sPage + tok_off + ch * CH, xres, gain, acc);
                    }
                }
                n_pend = 0;
            };
            for (PieceWalk w(p, wid, WG, mp.cs); !w.done(p); ++ui) {
                Unit un = w.next(p);
                own_tile<PAIR>(p, un, prank);
                const int tok_base = un.tt * NT;
                const uint32_t buf = ui & 1, aph = (ui >> 1) & 1;
                const int tok_off = all_tok ? tok_base : 0;          // index of this tile's first token in the caches
                if (need_info && !all_tok && info_tt != un.tt) {
                    token_info(p, tok_base, NT, row, sPos, sPage);
                    info_tt = un.tt;
                }
                const bool got = mbar_wait(&acc_full[buf], aph, &flags[0]);
                if (!got) flags[2] = 1;
                epi_bar();
                if (flags[2]) { alive = false; break; }   // uniform over the four warps
                tc_fence_after();
                // the leader of a pair counts both CTAs' epilogue warps before it overwrites an accumulator buffer
                auto release_acc = [&]() {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        if (PAIR && prank == 1) mbar_arrive_cluster(mapa_shared(smem_u32(&acc_empty[buf]), 0u));
                        else mbar_arrive(&acc_empty[buf]);
                    }
                };
                if (un.phantom) { release_acc(); continue; }
                // The accumulator exists, so the previous phase is complete and its sums of squares are final.
                if (p.ssq_in && !all_tok && rstd_tt != un.tt) {
                    token_rstd(p, tok_base, NT, row, sRstd);
                    rstd_tt = un.tt;
                    epi_bar();
                }
                if constexpr (NT <= 32) {
                    if (un.cl) {
                        // ---- the tile is shared by the CTAs of this cluster, each holding the sums over its K share.
                        // Rank q finishes token columns [q * GC, (q + 1) * GC): every CTA sends those columns of its
                        // accumulator into rank q's receive buffer with asynchronous stores into distributed shared
                        // memory that count as transactions on q's barrier; q adds the four pieces in rank order
                        // (bit-reproducible) and runs the epilogue. Every CTA sends every column and waits for all its
                        // peers whether or not its columns hold tokens, which keeps the cluster in step: a peer sends
                        // its (i+2)-th tile only after it has received this CTA's (i+1)-th, which is sent after the
                        // i-th was read, so two buffers suffice; phases are separated by the phase counter.
                        constexpr int GC = NT / CS;
                        static_assert(GC % 4 == 0, "columns per rank travel as groups of four floats");
                        const uint32_t xb = cl_units & 1, xpar = (cl_units >> 1) & 1;
                        ++cl_units;
                        const int tok0 = tok_base + rank * GC;
                        if (row == 0) mbar_expect_tx(&xch_bar[xb], (uint32_t)((CS - 1) * GC * TILE_F * 4));
                        float own[GC];
#pragma unroll
                        for (int c = 0; c < GC; ++c) own[c] = 0.f;
#pragma unroll
                        for (int ch = 0; ch < NT / CH; ++ch) {
                            float v[CH];
                            tmem_ld_cols<CH>(tmem_base + buf * NT + ch * CH + ((uint32_t)(ew * 32) << 16), v);
#pragma unroll
                            for (int c4 = 0; c4 < CH; c4 += 4) {
                                const int col = ch * CH + c4, q = col / GC, lc = col % GC;      // compile-time after unrolling
                                if (q == rank) {
#pragma unroll
                                    for (int e = 0; e < 4; ++e) own[lc + e] = v[c4 + e];
                                } else {
                                    const int slot = rank - (rank > q ? 1 : 0);
                                    st_async_f32x4(xch_remote[q] + (uint32_t)((((xb * (CS - 1) + slot) * TILE_F + row) * GC + lc) * 4), v[c4],
                                                   v[c4 + 1], v[c4 + 2], v[c4 + 3], xbar_remote[q] + xb * 8);
                                }
                            }
                        }
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&acc_empty[buf]);
                        // residual rows travel while the peers' columns arrive
                        float xres[CH], gain = 0.f;
                        residual_load<CH>(p, un, tok0, row, xres, gain, GC);
                        if (!mbar_wait_cluster(&xch_bar[xb], xpar, &flags[0])) flags[2] = 1;
                        epi_bar();
                        if (flags[2]) { alive = false; break; }
                        if (tok0 < p.M) {
                            const float* rx = sXch + ((size_t)xb * (CS - 1) * TILE_F + row) * GC;
                            float val[CH];
#pragma unroll
                            for (int c = 0; c < CH; ++c) val[c] = 0.f;
#pragma unroll
                            for (int l4 = 0; l4 < GC; l4 += 4) {
                                float a[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                                for (int j = 0; j < CS; ++j) {
                                    float4 t;
                                    if (j == rank) t = make_float4(own[l4], own[l4 + 1], own[l4 + 2], own[l4 + 3]);
                                    else t = *reinterpret_cast<const float4*>(rx + (size_t)(j - (j > rank ? 1 : 0)) * TILE_F * GC + l4);
                                    a[0] += t.x; a[1] += t.y; a[2] += t.z; a[3] += t.w;
                                }
#pragma unroll
                                for (int e = 0; e < 4; ++e) val[l4 + e] = p.ssq_in ? a[e] * sRstd[tok_off + rank * GC + l4 + e] : a[e];
                            }
                            apply_epilogue<CH, QKN>(p, sAcc, sRed, un, tok0, row, sPos + tok_off + rank * GC, sPage + tok_off + rank * GC,
                                                    xres, gain, val, GC);
                        }
                        continue;
                    }
                }
                const int n_ch = (min(NT, p.M - tok_base) + CH - 1) / CH;
                for (int ch = 0; ch < n_ch; ++ch) {
                    float v[CH];
                    tmem_ld_cols<CH>(tmem_base + buf * NT + ch * CH + ((uint32_t)(ew * 32) << 16), v);
                    if (!un.full) {
                        float* dst = p.part + (((size_t)blockIdx.x * 2 + un.slot) * NT + ch * CH) * TILE_F + row;
#pragma unroll
                        for (int c = 0; c < CH; ++c) dst[(size_t)c * TILE_F] = v[c];
                    } else {
                        if (p.ssq_in) {
#pragma unroll
                            for (int c = 0; c < CH; ++c) v[c] *= sRstd[tok_off + ch * CH + c];
                        }
                        float xres[CH], gain;
                        residual_load<CH>(p, un, tok_base + ch * CH, row, xres, gain);
                        apply_epilogue<CH, QKN>(p, sAcc, sRed, un, tok_base + ch * CH, row, sPos + tok_off + ch * CH, sPage + tok_off + ch * CH, xres, gain, v);
                    }
                }
                release_acc();
                if (!un.full) {
                    // the tile is shared: publish the piece, take a ticket, finish the tile at the end of the phase
                    epi_bar();
                    if (row == 0) red_release_add(p.counters + un.ctr, 1);
                    pend[n_pend++] = un;
                    if (w.shared_done() && !w.done(p)) {      // whole tiles follow: reduce now, under their main loop
                        finish_shared();
                        if (!alive) break;
                    }
                }
            }
            if (!alive) break;
            if (n_pend > 0) finish_shared();
            if (!alive) break;
            // this CTA's share of the phase is done and visible: tell the others
            epi_bar();
            if (row == 0) {
                trace_max(p.trace, 3);
                red_release_add(mp.phase_done + ph, 1);
            }
        }
        if (flags[2] && row == 0) {
            flags[0] = 1;
            if (mp.status) atomicOr(mp.status, DFLASH_DEV_TIMEOUT);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
    // no CTA of a cluster may go away while a peer can still write into its shared memory; every wait above is
    // bounded, so every CTA gets here
    if (mp.cs > 1 || PAIR) cluster_sync_all();
}

// Largest grid of clusters of CS CTAs whose CTAs are all resident at once (the CTAs of a launch wait for each
// other), asked of the runtime once per device and kernel; 0 = run without clusters. Capped at 32 clusters: with
// one CTA per SM the B200 co-schedules 32 clusters of 4 (its GPCs hold 16 to 20 usable SMs), and 128 CTAs
// already draw the full HBM bandwidth (measured: a plain streaming kernel reads at the same rate with 74 CTAs
// as with 148).
constexpr int MAX_CLUSTERS = 32, MIN_CLUSTERS = 16;
template <int NT, int SL, bool QKN>
int cluster_capacity(int stages) {
    constexpr bool PAIR = false;
    static int memo[MAX_DEVICES];
    static bool known[MAX_DEVICES] = {};
    const int dev = current_device_slot();
    if (dev >= 0 && known[dev]) return memo[dev];
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(CS * MAX_CLUSTERS);
    cfg.blockDim = dim3(N_THREADS);
    cfg.dynamicSmemBytes = (size_t)(1024 + stages * SL * (W_STAGE_BYTES + NT * BK * 2) + smem_fixed(NT));
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = CS;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, gemm_tc_kernel<NT, SL, QKN, PAIR>, &cfg) != cudaSuccess) {
        (void)cudaGetLastError();
        n = 0;
    }
    n = std::min(n, MAX_CLUSTERS);
    if (n < MIN_CLUSTERS) n = 0;
    if (dev >= 0) { memo[dev] = n; known[dev] = true; }
    return n;
}

constexpr int pair_smem(int nt, int stages) { return 1024 + stages * (W_STAGE_BYTES + (nt / 2) * BK * 2) + smem_fixed(nt); }
constexpr int pair_stages(int nt) { return std::min(MAX_STAGES, (SMEM_LIMIT - 1024 - smem_fixed(nt)) / (W_STAGE_BYTES + (nt / 2) * BK * 2)); }

template <int NT, int SL, bool QKN, bool PAIR>
int set_attr();

// CTA pairs the device keeps resident at once for the pair form of a kernel (its CTAs wait for each other), asked of
// the runtime once per device and kernel.
template <int NT, bool QKN>
int pair_capacity() {
    static int memo[MAX_DEVICES];
    static bool known[MAX_DEVICES] = {};
    const int dev = current_device_slot();
    if (dev >= 0 && known[dev]) return memo[dev];
    int n = 0;
    if (set_attr<NT, 1, QKN, true>() == DFLASH_OK) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * 1024);
        cfg.blockDim = dim3(N_THREADS);
        cfg.dynamicSmemBytes = (size_t)pair_smem(NT, pair_stages(NT));
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 2;
        at[0].val.clusterDim.y = 1;
        at[0].val.clusterDim.z = 1;
        cfg.attrs = at;
        cfg.numAttrs = 1;
        if (cudaOccupancyMaxActiveClusters(&n, gemm_tc_kernel<NT, 1, QKN, true>, &cfg) != cudaSuccess) {
            (void)cudaGetLastError();
            n = 0;
        }
    }
    if (dev >= 0) { memo[dev] = n; known[dev] = true; }
    return n;
}

template <int NT, int SL, bool QKN, bool PAIR>
int set_attr() {
    static bool attr_set[MAX_DEVICES] = {};
    const int dev = current_device_slot();
    if (dev < 0 || !attr_set[dev]) {
        if (cudaFuncSetAttribute(gemm_tc_kernel<NT, SL, QKN, PAIR>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_LIMIT) != cudaSuccess)
            return DFLASH_ERR_CUDA;
        if (dev >= 0) attr_set[dev] = true;
    }
    return DFLASH_OK;
}

// `grid_free`: CTAs the work itself asks for (one per SM, fewer for tiny problems). With token tiles of up to
// 32 rows the launch runs in clusters of CS CTAs when the device co-schedules enough of them: phases with fewer
// tiles than CTAs then split each tile's K range inside a cluster instead of through global memory.
template <int NT, int SL, bool QKN>
int launch_nt(const Launch& L, const WMaps& tw, const XMaps& tx, MParams& mp, int grid_free) {
    constexpr bool PAIR = false;
    if (set_attr<NT, SL, QKN, PAIR>() != DFLASH_OK) return DFLASH_ERR_CUDA;
    const int smem = 1024 + mp.stages * SL * (W_STAGE_BYTES + NT * BK * 2) + smem_fixed(NT);
    int grid = grid_free;
    mp.cs = 1;
    if (NT <= 32 && grid_free >= CS) {
        const int n_cl = std::min(cluster_capacity<NT, SL, QKN>(mp.stages), grid_free / CS);
        if (n_cl >= 1) { mp.cs = CS; grid = n_cl * CS; }
    }
    // Cluster mode for every phase with fewer tiles than CTAs (all its tiles would be shared anyway): the clusters
    // take the tiles in rounds. Tile counts that do not fill whole rounds (48 QKV tiles or 80 context K/V tiles over
    // 32 clusters) leave some CTAs up to twice the bytes of others and stretch the main loop (QKV: 9.9 us against 7.4
    // with an even split), but the exchange inside a cluster ends the phase ~4 us sooner than partial tiles through
    // global memory do: measured 12.1 against 13.6 us (QKV) and 17.8 against 22.6 us (context K/V).
    for (int i = 0; i < mp.n_phases; ++i) {
        const KParams& p = mp.ph[i];
        mp.ph[i].cluster_k = (mp.cs > 1 && p.n_tiles < grid && p.chunks_total >= CS) ? 1 : 0;
    }
    const cudaError_t e =
        mp.cs > 1 ? launch_pdl_cluster(gemm_tc_kernel<NT, SL, QKN, PAIR>, dim3(grid), dim3(N_THREADS), (size_t)smem, L.st, CS, tw, tx, mp)
                  : launch_pdl(gemm_tc_kernel<NT, SL, QKN, PAIR>, dim3(grid), dim3(N_THREADS), (size_t)smem, L.st, tw, tx, mp);
    ++g_launches;
    return e == cudaSuccess ? DFLASH_OK : DFLASH_ERR_CUDA;
}

// The pair form: `pairs` clusters of two CTAs (the phases were filled for pairs of weight tiles, the activation maps
// for half token tiles).
template <int NT, bool QKN>
int launch_pair(const Launch& L, const WMaps& tw, const XMaps& tx, MParams& mp, int pairs) {
    if (set_attr<NT, 1, QKN, true>() != DFLASH_OK) return DFLASH_ERR_CUDA;
    mp.cs = 1;
    for (int i = 0; i < mp.n_phases; ++i) mp.ph[i].cluster_k = 0;
    const cudaError_t e = launch_pdl_cluster(gemm_tc_kernel<NT, 1, QKN, true>, dim3(2 * pairs), dim3(N_THREADS),
                                             (size_t)pair_smem(NT, mp.stages), L.st, 2, tw, tx, mp);
    ++g_launches;
    return e == cudaSuccess ? DFLASH_OK : DFLASH_ERR_CUDA;
}


// Entry points of the instantiating translation units (token-tile width groups).
int gemm_launch_16(int slabs, bool qkn, const Launch& L, const WMaps& tw, const XMaps& tx, MParams& mp, int grid);
int gemm_launch_32(int slabs, bool qkn, const Launch& L, const WMaps& tw, const XMaps& tx, MParams& mp, int grid);
int gemm_launch_64_128(int nt, bool qkn, const Launch& L, const WMaps& tw, const XMaps& tx, MParams& mp, int grid);
int gemm_launch_160_256(int nt, bool qkn, const Launch& L, const WMaps& tw, const XMaps& tx, MParams& mp, int grid);
int gemm_launch_pair(int nt, bool qkn, const Launch& L, const WMaps& tw, const XMaps& tx, MParams& mp, int pairs);
int gemm_pair_capacity(int nt, bool qkn);

}  // namespace gemmk
}  // namespace dflash
