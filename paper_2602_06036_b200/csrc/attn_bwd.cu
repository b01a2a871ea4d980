// Backward pass of the block attention on tcgen05 tensor cores (bf16, head_dim 128, 64-token pages): the
// training side of the method, where many anchor blocks of one sequence are processed in one forward and one
// backward pass under a mask that is open inside a block and towards the injected context before the block's
// anchor (Sec. 4.2). Per query head, with keys = [context ; block] and P the forward's probabilities:
//     dV = P^T dO      dP = dO V^T      dS = P * (dP - D),  D = rowsum(dO * O)      dQ = scale dS K      dK = scale dS^T Q
// The forward hands over O and the log-sum-exp of every row, so P is recomputed tile by tile as
// exp(scale * S - lse) and no probability matrix ever exists in memory. Two kernels, both deterministic:
//   attn_bwd_q_kernel    one CTA per (block, kv head): walks the block's key tiles, accumulates dQ in TMEM, and on the
//                        block's own tile also produces dK_blk, dV_blk; writes D for the second kernel.
//   attn_bwd_kv_kernel   one CTA per (context tile of 64 keys, kv head): walks the blocks that see the tile in batch
//                        order and accumulates the tile's dK, dV in TMEM, so the context gradients of all blocks add
//                        up in a fixed order (bit-reproducible) without atomics.
// Operands are staged by TMA in the 128-byte-swizzled layouts of the forward kernel. The 64 query rows of a kv
// head (block rows x q heads of the group) are loaded twice to fill the 128-row operand, so that all four TMEM lane
// quadrants share the row arithmetic (the second copy takes keys 32..63 of every tile); P and dS are written for rows
// 0..63 only and rows 64..127 of their tiles stay zero, so contractions over the row index count every row once. Transposed
// products (P^T dO, dS^T Q) cost nothing: the tensor core reads the same shared-memory tiles through MN-major
// descriptors and produces dV^T, dK^T with head_dim on the TMEM lanes. One thread issues copies and tensor-core
// instructions, 128 threads (one per TMEM lane) do the row arithmetic; every mbarrier wait is bounded.
#include "attn_tc.cuh"

#include "ptx_sm100.cuh"

#include <math_constants.h>

#include <algorithm>

namespace dflash {
namespace {

using namespace ptx;

constexpr int HD = 128;
constexpr int PG = 64;
constexpr int QD_BYTES = 128 * HD * 2;           // one 128-row operand tile (Q or dO): two 64-column halves of 16 KiB
constexpr int KV_TILE_BYTES = PG * HD * 2;       // K or V tile: two 64-column halves of 8 KiB
constexpr int PS_BYTES = 128 * PG * 2;           // P or dS tile: 128 rows x 64 keys
constexpr int N_THREADS = 224;                   // 4 row warps (TMEM lane quadrants 0..3) + three single-thread roles: copies, scores, products
constexpr uint32_t TMEM_COLS = 512;
// S and dP are double-buffered (the contractions of the next key tile run under the row arithmetic of the current one)
constexpr uint32_t COL_S = 0, COL_DP = 64, COL_DQ = 128, COL_DVT = 256, COL_DKT = 320, COL_SDP2 = 384;
__device__ __forceinline__ uint32_t sdp_col(int buf) { return buf ? COL_SDP2 : 0u; }
constexpr int KV_STAGES = 3;
constexpr float LOG2E = 1.4426950408889634f;

struct BParams {
    int S, R, Hq, Hkv, group, max_pages, n_pages, layer, causal, rows_valid, max_ctx_len, shared_row;
    float scale, scale_log2;
    const int32_t* ctx_len;
    const int32_t* page_table;
    const __nv_bfloat16* out;      // forward output
    const __nv_bfloat16* dout;
    const float* lse;              // forward log-sum-exp (natural log)
    float* D;                      // [S, R, Hq] rowsum(dO * O): written by the first kernel, read by the second
    const int32_t* order;          // [S] blocks by falling context length (ties by index): written by order_kernel
    __nv_bfloat16 *dq, *dk_blk, *dv_blk;
    float* dkv_ctx;                // [page][K|V][kv head][slot][hd] fp32 of the layer
    int32_t* status;
};

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// MN-major operand in 128-byte-swizzled rows of 64 elements: `lbo` = bytes between the 64-element groups along the
// MN dimension (one tile half to the next), stride byte offset = 1 KiB between 8-row groups along K.
__device__ __forceinline__ uint64_t smem_desc_mn(uint32_t addr, uint32_t lbo) {
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
           (2ull << 61);
}
// instruction descriptors: D fp32, A and B bf16; major bits: 15 = A is MN-major, 16 = B is MN-major
__host__ __device__ constexpr uint32_t idesc_kk(int m, int n) { return instr_desc_bf16(m, n); }
__host__ __device__ constexpr uint32_t idesc_k_mn(int m, int n) { return instr_desc_bf16(m, n) | (1u << 16); }
__host__ __device__ constexpr uint32_t idesc_mn_mn(int m, int n) { return instr_desc_bf16(m, n) | (1u << 15) | (1u << 16); }

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 t = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&t);
}
__device__ __forceinline__ void rows_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// Q and dO of block b, kv head g: the 64 rows twice (rows 0..63 and 64..127 of each 64-column half)
__device__ __forceinline__ void load_q_do(uint8_t* sQ, uint8_t* sDO, const CUtensorMap* tmQ, const CUtensorMap* tmDO, int g, int row0,
                                          uint64_t* bar, uint64_t pol) {
    mbar_expect_tx(bar, 2 * QD_BYTES);
    for (int hf = 0; hf < 2; ++hf)
        for (int cp = 0; cp < 2; ++cp) {
            tma_load_4d(sQ + hf * (QD_BYTES / 2) + cp * (QD_BYTES / 4), tmQ, hf * 64, 0, g, row0, bar, pol);
            tma_load_4d(sDO + hf * (QD_BYTES / 2) + cp * (QD_BYTES / 4), tmDO, hf * 64, 0, g, row0, bar, pol);
        }
}

// Q and dO of TWO blocks: rows 0..63 of the operand tiles hold block A's 64 rows, rows 64..127 block B's
__device__ __forceinline__ void load_q_do_pair(uint8_t* sQ, uint8_t* sDO, const CUtensorMap* tmQ, const CUtensorMap* tmDO, int g, int rowA,
                                               int rowB, uint64_t* bar, uint64_t pol) {
    mbar_expect_tx(bar, 2 * QD_BYTES);
    for (int hf = 0; hf < 2; ++hf)
        for (int cp = 0; cp < 2; ++cp) {
            const int row0 = cp ? rowB : rowA;
            tma_load_4d(sQ + hf * (QD_BYTES / 2) + cp * (QD_BYTES / 4), tmQ, hf * 64, 0, g, row0, bar, pol);
            tma_load_4d(sDO + hf * (QD_BYTES / 2) + cp * (QD_BYTES / 4), tmDO, hf * 64, 0, g, row0, bar, pol);
        }
}

// S = Q K^T and dP = dO V^T of one 64-key tile (16 instructions)
__device__ __forceinline__ void issue_s_dp(uint32_t tmem_base, uint32_t q_addr, uint32_t do_addr, uint32_t k_addr, uint32_t v_addr) {
    // tmem_base already includes the S / dP buffer's first column
    constexpr uint32_t idesc = idesc_kk(128, PG);
#pragma unroll
    for (int kk = 0; kk < HD / 16; ++kk)
        mma_bf16(tmem_base + COL_S, smem_desc_sw128(q_addr + (kk >> 2) * (QD_BYTES / 2) + (kk & 3) * 32),
                 smem_desc_sw128(k_addr + (kk >> 2) * (KV_TILE_BYTES / 2) + (kk & 3) * 32), idesc, kk > 0 ? 1u : 0u);
#pragma unroll
    for (int kk = 0; kk < HD / 16; ++kk)
        mma_bf16(tmem_base + COL_DP, smem_desc_sw128(do_addr + (kk >> 2) * (QD_BYTES / 2) + (kk & 3) * 32),
                 smem_desc_sw128(v_addr + (kk >> 2) * (KV_TILE_BYTES / 2) + (kk & 3) * 32), idesc, kk > 0 ? 1u : 0u);
}
// dV^T (+)= dO^T P and dK^T (+)= Q^T dS: contraction over the 128 operand rows (16 instructions)
__device__ __forceinline__ void issue_dkv_t(uint32_t tmem_base, uint32_t q_addr, uint32_t do_addr, uint32_t p_addr, uint32_t ds_addr,
                                            uint32_t accumulate) {
    constexpr uint32_t idesc = idesc_mn_mn(128, PG);
#pragma unroll
    for (int kk = 0; kk < 128 / 16; ++kk)
        mma_bf16(tmem_base + COL_DVT, smem_desc_mn(do_addr + kk * 2048, QD_BYTES / 2), smem_desc_mn(p_addr + kk * 2048, PS_BYTES), idesc,
                 (accumulate || kk > 0) ? 1u : 0u);
#pragma unroll
    for (int kk = 0; kk < 128 / 16; ++kk)
        mma_bf16(tmem_base + COL_DKT, smem_desc_mn(q_addr + kk * 2048, QD_BYTES / 2), smem_desc_mn(ds_addr + kk * 2048, PS_BYTES), idesc,
                 (accumulate || kk > 0) ? 1u : 0u);
}

// Row arithmetic of one tile. The 64 query rows sit twice in the operand (TMEM lanes 0..63 and 64..127 hold the same
// S and dP rows): the thread of lane l works on query row l & 63 and on keys [32 (l >> 6), +32) of the tile, so all
// four lane quadrants (one warp each) share the work. It reads its half rows of S and dP from TMEM and writes P
// and dS (bf16) into rows 0..63 of the swizzled tiles; rows 64..127 of those tiles stay zero (zeroed once at the
// start), which is what makes contractions over the 128 operand rows count every query row once.
// vis = keys of this tile the query row sees (0 for rows that hold no query).
__device__ __forceinline__ void row_math(uint32_t tmem_row, uint8_t* sP, uint8_t* sDS, int lane_row, int vis, float lse2, float Dr,
                                         float scale, float scale_log2) {
    const int qrow = lane_row & 63, h = lane_row >> 6;
    uint8_t* prow = sP + qrow * 128;
    uint8_t* drow = sDS + qrow * 128;
    float s[32], dp[32];
    tmem_ld32(tmem_row + COL_S + h * 32, s);          // tmem_row includes the S / dP buffer's first column
    tmem_ld32(tmem_row + COL_DP + h * 32, dp);
#pragma unroll
    for (int c = 0; c < 32; ++c) {
        const bool on = h * 32 + c < vis;
        const float p = on ? fast_exp2(fmaf(s[c], scale_log2, -lse2)) : 0.f;
        s[c] = p;
        dp[c] = on ? p * (dp[c] - Dr) * scale : 0.f;
    }
#pragma unroll
    for (int ck = 0; ck < 4; ++ck) {
        uint4 w4, d4;
        w4.x = pack_bf16(s[ck * 8 + 0], s[ck * 8 + 1]);
        w4.y = pack_bf16(s[ck * 8 + 2], s[ck * 8 + 3]);
        w4.z = pack_bf16(s[ck * 8 + 4], s[ck * 8 + 5]);
        w4.w = pack_bf16(s[ck * 8 + 6], s[ck * 8 + 7]);
        d4.x = pack_bf16(dp[ck * 8 + 0], dp[ck * 8 + 1]);
        d4.y = pack_bf16(dp[ck * 8 + 2], dp[ck * 8 + 3]);
        d4.z = pack_bf16(dp[ck * 8 + 4], dp[ck * 8 + 5]);
        d4.w = pack_bf16(dp[ck * 8 + 6], dp[ck * 8 + 7]);
        const int off = ((h * 4 + ck) ^ (qrow & 7)) << 4;
        *reinterpret_cast<uint4*>(prow + off) = w4;
        *reinterpret_cast<uint4*>(drow + off) = d4;
    }
}
// Row arithmetic of one tile when the 128 operand rows are 64 query rows of each of TWO blocks (the context-gradient
// kernel): the thread of lane l owns operand row l - all 64 keys of the tile - and writes row l of P and dS.
__device__ __forceinline__ void row_math_full(uint32_t tmem_row, uint8_t* sP, uint8_t* sDS, int row, int vis, float lse2, float Dr,
                                              float scale, float scale_log2) {
    uint8_t* prow = sP + row * 128;
    uint8_t* drow = sDS + row * 128;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        float s[32], dp[32];
        tmem_ld32(tmem_row + COL_S + h * 32, s);
        tmem_ld32(tmem_row + COL_DP + h * 32, dp);
#pragma unroll
        for (int c = 0; c < 32; ++c) {
            const bool on = h * 32 + c < vis;
            const float p = on ? fast_exp2(fmaf(s[c], scale_log2, -lse2)) : 0.f;
            s[c] = p;
            dp[c] = on ? p * (dp[c] - Dr) * scale : 0.f;
        }
#pragma unroll
        for (int ck = 0; ck < 4; ++ck) {
            uint4 w4, d4;
            w4.x = pack_bf16(s[ck * 8 + 0], s[ck * 8 + 1]);
            w4.y = pack_bf16(s[ck * 8 + 2], s[ck * 8 + 3]);
            w4.z = pack_bf16(s[ck * 8 + 4], s[ck * 8 + 5]);
            w4.w = pack_bf16(s[ck * 8 + 6], s[ck * 8 + 7]);
            d4.x = pack_bf16(dp[ck * 8 + 0], dp[ck * 8 + 1]);
            d4.y = pack_bf16(dp[ck * 8 + 2], dp[ck * 8 + 3]);
            d4.z = pack_bf16(dp[ck * 8 + 4], dp[ck * 8 + 5]);
            d4.w = pack_bf16(dp[ck * 8 + 6], dp[ck * 8 + 7]);
            const int off = ((h * 4 + ck) ^ (row & 7)) << 4;
            *reinterpret_cast<uint4*>(prow + off) = w4;
            *reinterpret_cast<uint4*>(drow + off) = d4;
        }
    }
}
// rows 64..127 of both P / dS buffer pairs := 0 (128 threads; visible to the tensor core after the first
// fence.proxy.async + barrier arrival that follows)
__device__ __forceinline__ void zero_upper_rows(uint8_t* sPS, int tid) {
    for (int t = 0; t < 4; ++t) {
        uint4* dst = reinterpret_cast<uint4*>(sPS + (size_t)t * PS_BYTES + 64 * 128);
        for (int e = tid; e < 64 * 128 / 16; e += 128) dst[e] = make_uint4(0, 0, 0, 0);
    }
}

// Blocks by falling context length, ties by index (every thread ranks some blocks against all others; one CTA).
// The first kernel takes its blocks in this order: the longest first, and - two blocks per CTA - neighbours of
// similar length together.
// More than ORDER_MAX blocks (the ranking is quadratic): index order.
constexpr int ORDER_MAX = 4096;
__global__ void __launch_bounds__(1024) order_kernel(const int32_t* __restrict__ ctx_len, int S, int32_t* __restrict__ order) {
    extern __shared__ int32_t s_len[];
    if (S > ORDER_MAX) {
        for (int i = threadIdx.x; i < S; i += blockDim.x) order[i] = i;
        return;
    }
    for (int i = threadIdx.x; i < S; i += blockDim.x) s_len[i] = ctx_len[i];
    __syncthreads();
    for (int t = threadIdx.x; t < S; t += blockDim.x) {
        const int mine = s_len[t];
        int rank = 0;
        for (int j = 0; j < S; ++j) {
            const int l = s_len[j];
            rank += (l > mine || (l == mine && j < t)) ? 1 : 0;
        }
        order[rank] = t;
    }
}

// ------------------------------------------------------------------------------------------------------------
// dQ, dK_blk, dV_blk: one CTA per (kv head, block)
// ------------------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(N_THREADS, 1)
attn_bwd_q_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmDO,
                  const __grid_constant__ CUtensorMap tmPool, const __grid_constant__ CUtensorMap tmKb,
                  const __grid_constant__ CUtensorMap tmVb, const BParams p) {
    pdl_trigger();
    // Blocks are taken by falling context length (p.order). Blocks that share one page-table row (the training layout)
    // go TWO per CTA: operand rows 0..63 are block A's query rows, rows 64..127 block B's; both walk the same key
    // tiles (a row past its own context sees no key) and each block's own keys take a tile of their own. Otherwise
    // one block per CTA, its rows loaded twice.
    const int g = blockIdx.x;
    const bool two = p.shared_row != 0;
    const int ia0 = two ? 2 * (int)blockIdx.y : (int)blockIdx.y;
    const int b = p.order[ia0];                                              // block A
    const int bB = (two && ia0 + 1 < p.S) ? p.order[ia0 + 1] : -1;           // block B (or none)
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem;
    uint8_t* sDO = sQ + QD_BYTES;
    uint8_t* sKV = sDO + QD_BYTES;                       // KV_STAGES x (K, V)
    uint8_t* sPS = sKV + KV_STAGES * 2 * KV_TILE_BYTES;  // 2 x (P, dS)
    uint64_t* bars = reinterpret_cast<uint64_t*>(sPS + 2 * 2 * PS_BYTES);
    uint64_t* q_full = bars;
    uint64_t* kv_full = bars + 1;                  // [KV_STAGES]
    uint64_t* kv_empty = kv_full + KV_STAGES;      // [KV_STAGES]
    uint64_t* s_full = kv_empty + KV_STAGES;       // [2] S / dP buffer written by the tensor core
    uint64_t* ds_full = s_full + 2;                // [2] P / dS buffer written by the row threads (and S / dP buffer read)
    uint64_t* acc_done = ds_full + 2;              // [2] the products that read P / dS buffer are complete
    uint64_t* blk_read = acc_done + 2;             // [1] block A's own-key gradients have been read out of TMEM
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(blk_read + 1);
    volatile int* flags = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        mbar_init(blk_read, 4);
        for (int s = 0; s < KV_STAGES; ++s) { mbar_init(&kv_full[s], 1); mbar_init(&kv_empty[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&s_full[s], 1); mbar_init(&ds_full[s], 4); mbar_init(&acc_done[s], 1); }
        flags[0] = 0;
        fence_barrier_init();
        fence_proxy_async();
    }
    if (warp == 4) tmem_alloc(tmem_slot, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();

    const int LA_given = p.ctx_len[b], LB_given = bB >= 0 ? p.ctx_len[bB] : 0;
    const int LA = min(max(LA_given, 0), p.max_ctx_len), LB = min(max(LB_given, 0), p.max_ctx_len);
    if ((LA_given > p.max_ctx_len || LB_given > p.max_ctx_len) && threadIdx.x == 0 && g == 0 && p.status)
        atomicOr(p.status, DFLASH_DEV_CTX_OVERFLOW);
    const int L = max(LA, LB);                           // keys the CTA walks
    const int n_ctx_tiles = (L + PG - 1) / PG;
    const int n_tiles = n_ctx_tiles + 1 + (bB >= 0 ? 1 : 0);      // + block A's own keys (+ block B's)

    // Three single-thread roles, each with its own chain of waits, so that a copy in flight never holds up a
    // contraction whose operands are ready: copies (warp 4), S / dP of the next tile (warp 5), the accumulating
    // products of the current tile (warp 6).
    if (warp == 4) {
        if (lane == 0) {
            const uint64_t pol_kv = policy_evict_last(), pol_q = policy_evict_first();
            bool ok = true;
            if (two) load_q_do_pair(sQ, sDO, &tmQ, &tmDO, g, b * p.R, (bB >= 0 ? bB : b) * p.R, q_full, pol_q);
            else load_q_do(sQ, sDO, &tmQ, &tmDO, g, b * p.R, q_full, pol_q);
            for (int i = 0; i < n_tiles && ok; ++i) {
                const int st = i % KV_STAGES;
                // the stage held tile i - KV_STAGES: wait for that tile's products
                if (i >= KV_STAGES && !mbar_wait(&kv_empty[st], ((i / KV_STAGES) - 1) & 1, &flags[0])) { ok = false; break; }
                uint8_t* dK = sKV + (size_t)st * 2 * KV_TILE_BYTES;
                uint8_t* dV = dK + KV_TILE_BYTES;
                mbar_expect_tx(&kv_full[st], 2 * KV_TILE_BYTES);
                if (i < n_ctx_tiles) {
                    int page = i < p.max_pages ? __ldg(p.page_table + (size_t)(p.shared_row ? 0 : b) * p.max_pages + i) : -1;
                    if (page < 0 || page >= p.n_pages) {
                        if (p.status) atomicOr(p.status, DFLASH_DEV_BAD_PAGE);
                        page = 0;
                    }
                    const int rowK = ((((p.layer * p.n_pages + page) * 2 + 0) * p.Hkv + g) * PG);
                    const int rowV = rowK + p.Hkv * PG;
                    tma_load_2d(dK, &tmPool, 0, rowK, &kv_full[st], pol_kv);
                    tma_load_2d(dK + KV_TILE_BYTES / 2, &tmPool, 64, rowK, &kv_full[st], pol_kv);
                    tma_load_2d(dV, &tmPool, 0, rowV, &kv_full[st], pol_kv);
                    tma_load_2d(dV + KV_TILE_BYTES / 2, &tmPool, 64, rowV, &kv_full[st], pol_kv);
                } else {
                    const int bo = (i == n_ctx_tiles ? b : bB) * p.R;      // the own keys of block A, then of block B
                    tma_load_2d(dK, &tmKb, g * HD, bo, &kv_full[st], pol_q);
                    tma_load_2d(dK + KV_TILE_BYTES / 2, &tmKb, g * HD + 64, bo, &kv_full[st], pol_q);
                    tma_load_2d(dV, &tmVb, g * HD, bo, &kv_full[st], pol_q);
                    tma_load_2d(dV + KV_TILE_BYTES / 2, &tmVb, g * HD + 64, bo, &kv_full[st], pol_q);
                }
            }
            if (!ok) {
                flags[0] = 1;
                if (p.status) atomicOr(p.status, DFLASH_DEV_TIMEOUT);
            }
        }
        __syncwarp();
    } else if (warp == 5) {
        if (lane == 0) {
            const uint32_t q_addr = smem_u32(sQ), do_addr = smem_u32(sDO);
            bool ok = mbar_wait(q_full, 0, &flags[0]);
            for (int i = 0; i < n_tiles && ok; ++i) {
                const int st = i % KV_STAGES, buf = i & 1;
                if (!mbar_wait(&kv_full[st], (i / KV_STAGES) & 1, &flags[0])) { ok = false; break; }
                // S / dP buffer `buf` was last read by the row threads of tile i - 2
                if (i >= 2 && !mbar_wait(&ds_full[buf], ((i - 2) >> 1) & 1, &flags[0])) { ok = false; break; }
                tc_fence_after();
                const uint32_t k_addr = smem_u32(sKV + (size_t)st * 2 * KV_TILE_BYTES);
                issue_s_dp(tmem_base + sdp_col(buf), q_addr, do_addr, k_addr, k_addr + KV_TILE_BYTES);
                mma_commit(&s_full[buf]);
            }
            if (!ok) {
                flags[0] = 1;
                if (p.status) atomicOr(p.status, DFLASH_DEV_TIMEOUT);
            }
        }
        __syncwarp();
    } else if (warp == 6) {
        if (lane == 0) {
            const uint32_t q_addr = smem_u32(sQ), do_addr = smem_u32(sDO);
            bool ok = true;
            for (int i = 0; i < n_tiles && ok; ++i) {
                const int st = i % KV_STAGES, buf = i & 1;
                if (!mbar_wait(&ds_full[buf], (i >> 1) & 1, &flags[0])) { ok = false; break; }
                tc_fence_after();
                const uint32_t k_addr = smem_u32(sKV + (size_t)st * 2 * KV_TILE_BYTES);
                const uint32_t p_addr = smem_u32(sPS + (size_t)buf * 2 * PS_BYTES), ds_addr = p_addr + PS_BYTES;
                constexpr uint32_t idesc_dq = idesc_k_mn(128, HD);
#pragma unroll
                for (int kk = 0; kk < PG / 16; ++kk)
                    mma_bf16(tmem_base + COL_DQ, smem_desc_sw128(ds_addr + kk * 32), smem_desc_mn(k_addr + kk * 2048, KV_TILE_BYTES / 2),
                             idesc_dq, (i > 0 || kk > 0) ? 1u : 0u);
                if (i >= n_ctx_tiles) {      // a block's own keys (the other block's rows hold zeros in P / dS)
                    // block B's gradients take the columns of block A's: those must have been read out
                    if (i > n_ctx_tiles && !mbar_wait(blk_read, 0, &flags[0])) { ok = false; break; }
                    tc_fence_after();
                    issue_dkv_t(tmem_base, q_addr, do_addr, p_addr, ds_addr, 0u);
                }
                mma_commit(&acc_done[buf]);
                mma_commit(&kv_empty[st]);
            }
            if (!ok) {
                flags[0] = 1;
                if (p.status) atomicOr(p.status, DFLASH_DEV_TIMEOUT);
            }
        }
        __syncwarp();
    } else {
        const int row = warp * 32 + lane;                       // TMEM lane
        const uint32_t tmem_row = tmem_base + ((uint32_t)(warp * 32) << 16);
        const int lrow = row & 63;                              // query row (one block: lanes 64..127 repeat rows 0..63)
        const int mine = (two && row >= 64) ? bB : b;           // the block this thread's operand row belongs to
        const bool real = lrow < p.rows_valid && mine >= 0;
        const int r = real ? lrow / p.group : 0, j = real ? lrow % p.group : 0;
        const size_t qrow = ((size_t)max(mine, 0) * p.R + r) * p.Hq + g * p.group + j;
        const int L_mine = (two && row >= 64) ? LB : LA;
        if (!two) zero_upper_rows(sPS, row);
        // D = rowsum(dO * O) and the row's log-sum-exp in the log2 domain
        float Dr = 0.f, lse2 = 0.f;
        if (real) {
            const uint4* po = reinterpret_cast<const uint4*>(p.out + qrow * HD);
            const uint4* pd = reinterpret_cast<const uint4*>(p.dout + qrow * HD);
#pragma unroll 4
            for (int i = 0; i < HD / 8; ++i) {
                const uint4 a = __ldg(po + i), c = __ldg(pd + i);
                const __nv_bfloat162* a2 = reinterpret_cast<const __nv_bfloat162*>(&a);
                const __nv_bfloat162* c2 = reinterpret_cast<const __nv_bfloat162*>(&c);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 x = __bfloat1622float2(a2[e]), y = __bfloat1622float2(c2[e]);
                    Dr = fmaf(x.x, y.x, Dr);
                    Dr = fmaf(x.y, y.y, Dr);
                }
            }
            if (two || row < 64) p.D[qrow] = Dr;
            lse2 = __ldg(p.lse + qrow) * LOG2E;
        }
        // a block's own-key gradients leave TMEM as soon as their tile's products are complete
        auto write_own = [&](int blk) {
            float tv[32], tk[32];      // dV_blk^T, dK_blk^T: lane = head_dim index, column = block row
            tmem_ld32(tmem_row + COL_DVT, tv);
            tmem_ld32(tmem_row + COL_DKT, tk);
#pragma unroll
            for (int c = 0; c < 32; ++c) {
                if (c < p.R) {
                    const size_t at = (((size_t)blk * p.R + c) * p.Hkv + g) * HD + row;
                    p.dv_blk[at] = __float2bfloat16_rn(tv[c]);
                    p.dk_blk[at] = __float2bfloat16_rn(tk[c]);
                }
            }
        };
        bool ok = true;
        for (int i = 0; i < n_tiles; ++i) {
            const int buf = i & 1;
            int n_valid, vis;
            if (i < n_ctx_tiles) {
                n_valid = min(PG, L - i * PG);
                vis = min(max(L_mine - i * PG, 0), PG);
            } else {
                n_valid = p.R;
                const int owner = i == n_ctx_tiles ? b : bB;      // whose own keys these are
                vis = mine == owner ? (p.causal ? min(r + 1, p.R) : p.R) : 0;
            }
            if (!real) vis = 0;
            if (!mbar_wait(&s_full[buf], (i >> 1) & 1, &flags[0])) { ok = false; break; }
            tc_fence_after();
            // P / dS buffer `buf` is still being read by the products of tile i - 2 until their acc_done
            if (i >= 2 && !mbar_wait(&acc_done[buf], ((i - 2) >> 1) & 1, &flags[0])) { ok = false; break; }
            uint8_t* sP = sPS + (size_t)buf * 2 * PS_BYTES;
            if (two) row_math_full(tmem_row + sdp_col(buf), sP, sP + PS_BYTES, row, vis, lse2, Dr, p.scale, p.scale_log2);
            else row_math(tmem_row + sdp_col(buf), sP, sP + PS_BYTES, row, vis, lse2, Dr, p.scale, p.scale_log2);
            // keys that do not exist must not poison dS K with whatever the page holds there
            if (n_valid < PG) {
                uint8_t* dK = sKV + (size_t)(i % KV_STAGES) * 2 * KV_TILE_BYTES;
                const int n_bad = PG - n_valid;
                for (int e = row; e < n_bad * 16; e += 128) {
                    const int kr = n_valid + e / 16, part = e % 16;
                    *reinterpret_cast<uint4*>(dK + (part >> 3) * (KV_TILE_BYTES / 2) + kr * 128 + (part & 7) * 16) = make_uint4(0, 0, 0, 0);
                }
            }
            tc_fence_before();
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(&ds_full[buf]);
            if (bB >= 0 && i == n_tiles - 1) {
                // block A's own-key tile was the one before: its products are complete once its acc_done fires;
                // read its gradients out, then block B's products (waiting on blk_read) may take the columns
                const int ia = n_ctx_tiles;
                if (!mbar_wait(&acc_done[ia & 1], (ia >> 1) & 1, &flags[0])) { ok = false; break; }
                tc_fence_after();
                write_own(b);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(blk_read);
            }
        }
        // the tensor pipe completes in order: the last tile's products close the accumulators
        if (ok && !mbar_wait(&acc_done[(n_tiles - 1) & 1], ((n_tiles - 1) >> 1) & 1, &flags[0])) ok = false;
        if (!ok) {
            flags[0] = 1;
            if (lane == 0 && p.status) atomicOr(p.status, DFLASH_DEV_TIMEOUT);
        }
        tc_fence_after();
        rows_bar();                  // a row that gave up told the others through flags[0]
        if (!flags[0]) {
            // dQ row (every thread of a warp executes the same tensor-memory loads; only real rows store)
            __nv_bfloat16* dst = p.dq + qrow * HD;
#pragma unroll
            for (int c4 = 0; c4 < HD / 32; ++c4) {
                float o[32];
                tmem_ld32(tmem_row + COL_DQ + c4 * 32, o);
                if (real && (two || row < 64)) {
#pragma unroll
                    for (int d = 0; d < 32; d += 8) {
                        uint4 w4;
                        w4.x = pack_bf16(o[d], o[d + 1]);
                        w4.y = pack_bf16(o[d + 2], o[d + 3]);
                        w4.z = pack_bf16(o[d + 4], o[d + 5]);
                        w4.w = pack_bf16(o[d + 6], o[d + 7]);
                        *reinterpret_cast<uint4*>(dst + c4 * 32 + d) = w4;
                    }
                }
            }
            write_own(bB >= 0 ? bB : b);      // the own-key gradients of the last own tile
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ------------------------------------------------------------------------------------------------------------
// dK_ctx, dV_ctx: one CTA per (context tile, kv head, page-table row); the blocks that see the tile in batch order,
// TWO per step: the 128 operand rows are the 64 query rows of two consecutive contributing blocks, so a step's
// contractions over the operand rows add both blocks' terms (half the steps, no duplicated rows; the order of the
// sums is still fixed by the batch order). An odd block out rides with rows that see no key.
// ------------------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(N_THREADS, 1)
attn_bwd_kv_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmDO,
                   const __grid_constant__ CUtensorMap tmPool, const BParams p) {
    pdl_trigger();
    // kv head fastest, key tile next: CTAs reach the SMs in index order, and a tile is seen by at least as many blocks
    // as every later one, so the longest CTAs (the first tiles, seen by every block) all start first
    const int g = blockIdx.x, t = blockIdx.y, owner = blockIdx.z;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sKV = smem;                                  // K tile, V tile
    uint8_t* sQD = sKV + 2 * KV_TILE_BYTES;               // 2 stages x (Q, dO)
    uint8_t* sPS = sQD + 2 * 2 * QD_BYTES;                // 2 x (P, dS)
    uint64_t* bars = reinterpret_cast<uint64_t*>(sPS + 2 * 2 * PS_BYTES);
    uint64_t* kv_full = bars;
    uint64_t* qd_full = bars + 1;      // [2]
    uint64_t* qd_empty = bars + 3;     // [2]
    uint64_t* s_full = bars + 5;       // [2]
    uint64_t* ds_full = bars + 7;      // [2]
    uint64_t* acc_done = bars + 9;     // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 11);
    volatile int* flags = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        mbar_init(kv_full, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&qd_full[s], 1); mbar_init(&qd_empty[s], 1);
            mbar_init(&s_full[s], 1); mbar_init(&ds_full[s], 4); mbar_init(&acc_done[s], 1);
        }
        flags[0] = 0;
        fence_barrier_init();
        fence_proxy_async();
    }
    if (warp == 4) tmem_alloc(tmem_slot, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();

    const int b_lo = p.shared_row ? 0 : owner, b_hi = p.shared_row ? p.S : owner + 1;
    const int key0 = t * PG;
    int page = t < p.max_pages ? __ldg(p.page_table + (size_t)(p.shared_row ? 0 : owner) * p.max_pages + t) : -1;
    // a block sees this tile if its context is longer than the tile's first key
    auto sees = [&](int b) { return min(max(__ldg(p.ctx_len + b), 0), p.max_ctx_len) > key0; };
    int n_contrib = 0;       // blocks that see this tile
    for (int b = b_lo; b < b_hi; ++b) n_contrib += sees(b) ? 1 : 0;
    bool any = n_contrib > 0;
    const bool page_ok = page >= 0 && page < p.n_pages;
    if (any && !page_ok) {
        if (threadIdx.x == 0 && p.status) atomicOr(p.status, DFLASH_DEV_BAD_PAGE);
        any = false;
    }

    const int n_steps = (n_contrib + 1) / 2;      // two contributing blocks per step
    int n_done = 0;      // steps processed (uniform over the CTA)
    bool ok = true;
    if (any) {
        if (warp == 4) {
            if (lane == 0) {      // copies: the key tile once, then Q / dO of every block that sees it
                const uint64_t pol_kv = policy_evict_last(), pol_q = policy_evict_first();
                const int rowK = ((((p.layer * p.n_pages + page) * 2 + 0) * p.Hkv + g) * PG);
                const int rowV = rowK + p.Hkv * PG;
                mbar_expect_tx(kv_full, 2 * KV_TILE_BYTES);
                tma_load_2d(sKV, &tmPool, 0, rowK, kv_full, pol_kv);
                tma_load_2d(sKV + KV_TILE_BYTES / 2, &tmPool, 64, rowK, kv_full, pol_kv);
                tma_load_2d(sKV + KV_TILE_BYTES, &tmPool, 0, rowV, kv_full, pol_kv);
                tma_load_2d(sKV + KV_TILE_BYTES + KV_TILE_BYTES / 2, &tmPool, 64, rowV, kv_full, pol_kv);
                int b = b_lo;
                for (int k = 0; k < n_steps && ok; ++k) {
                    while (!sees(b)) ++b;
                    const int bA = b++;
                    while (b < b_hi && !sees(b)) ++b;
                    const int bB = b < b_hi ? b++ : bA;      // odd block out: its partner's rows see no key
                    const int st = k & 1;
                    if (k >= 2 && !mbar_wait(&qd_empty[st], ((k >> 1) - 1) & 1, &flags[0])) { ok = false; break; }
                    load_q_do_pair(sQD + (size_t)st * 2 * QD_BYTES, sQD + (size_t)st * 2 * QD_BYTES + QD_BYTES, &tmQ, &tmDO, g, bA * p.R,
                                   bB * p.R, &qd_full[st], pol_q);
                }
                if (!ok) {
                    flags[0] = 1;
                    if (p.status) atomicOr(p.status, DFLASH_DEV_TIMEOUT);
                }
            }
            __syncwarp();
        } else if (warp == 5) {
            if (lane == 0) {      // scores of the k-th pair of contributing blocks into buffer k & 1
                const uint32_t k_addr = smem_u32(sKV), v_addr = k_addr + KV_TILE_BYTES;
                ok = mbar_wait(kv_full, 0, &flags[0]);
                for (int k = 0; k < n_steps && ok; ++k) {
                    const int st = k & 1;
                    if (!mbar_wait(&qd_full[st], (k >> 1) & 1, &flags[0])) { ok = false; break; }
                    if (k >= 2 && !mbar_wait(&ds_full[st], ((k - 2) >> 1) & 1, &flags[0])) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t q_addr = smem_u32(sQD + (size_t)st * 2 * QD_BYTES);
                    issue_s_dp(tmem_base + sdp_col(st), q_addr, q_addr + QD_BYTES, k_addr, v_addr);
                    mma_commit(&s_full[st]);
                }
                if (!ok) {
                    flags[0] = 1;
                    if (p.status) atomicOr(p.status, DFLASH_DEV_TIMEOUT);
                }
            }
            __syncwarp();
        } else if (warp == 6) {
            if (lane == 0) {      // accumulating products of the k-th pair of contributing blocks
                for (int k = 0; k < n_steps && ok; ++k) {
                    const int st = k & 1;
                    if (!mbar_wait(&ds_full[st], (k >> 1) & 1, &flags[0])) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t q_addr = smem_u32(sQD + (size_t)st * 2 * QD_BYTES), do_addr = q_addr + QD_BYTES;
                    const uint32_t p_addr = smem_u32(sPS + (size_t)st * 2 * PS_BYTES), ds_addr = p_addr + PS_BYTES;
                    issue_dkv_t(tmem_base, q_addr, do_addr, p_addr, ds_addr, k > 0 ? 1u : 0u);
                    mma_commit(&acc_done[st]);
                    mma_commit(&qd_empty[st]);
                }
                if (!ok) {
                    flags[0] = 1;
                    if (p.status) atomicOr(p.status, DFLASH_DEV_TIMEOUT);
                }
            }
            __syncwarp();
        } else {
            const int row = warp * 32 + lane;
            const uint32_t tmem_row = tmem_base + ((uint32_t)(warp * 32) << 16);
            const int lrow = row & 63;
            const bool real = lrow < p.rows_valid;
            const int r = real ? lrow / p.group : 0, j = real ? lrow % p.group : 0;
            int bn = b_lo;
            for (int i = 0; i < n_steps; ++i) {
                while (!sees(bn)) ++bn;
                const int bA = bn++;
                while (bn < b_hi && !sees(bn)) ++bn;
                const int bB = bn < b_hi ? bn++ : -1;
                n_done = i + 1;
                // operand rows 0..63: block A, rows 64..127: block B (none: rows that see nothing)
                const int b = row < 64 ? bA : bB;
                const bool on = real && b >= 0;
                const int Lb = on ? min(max(__ldg(p.ctx_len + b), 0), p.max_ctx_len) : 0;
                const size_t qrow = on ? ((size_t)b * p.R + r) * p.Hq + g * p.group + j : 0;
                const float Dr = on ? __ldcg(p.D + qrow) : 0.f;
                const float lse2 = on ? __ldg(p.lse + qrow) * LOG2E : 0.f;
                const int vis = on ? min(PG, Lb - key0) : 0;
                const int buf = i & 1;
                if (!mbar_wait(&s_full[buf], (i >> 1) & 1, &flags[0])) { ok = false; break; }
                tc_fence_after();
                if (i >= 2 && !mbar_wait(&acc_done[buf], ((i - 2) >> 1) & 1, &flags[0])) { ok = false; break; }
                uint8_t* sP = sPS + (size_t)buf * 2 * PS_BYTES;
                row_math_full(tmem_row + sdp_col(buf), sP, sP + PS_BYTES, row, vis, lse2, Dr, p.scale, p.scale_log2);
                tc_fence_before();
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(&ds_full[buf]);
            }
            if (ok && n_done > 0 && !mbar_wait(&acc_done[(n_done - 1) & 1], ((n_done - 1) >> 1) & 1, &flags[0])) ok = false;
            if (!ok) {
                flags[0] = 1;
                if (lane == 0 && p.status) atomicOr(p.status, DFLASH_DEV_TIMEOUT);
            }
            tc_fence_after();
        }
    }
    // write the tile's gradients (zeros if no block sees it): lane = head_dim index, column = key
    if (warp < 4 && page_ok) {
        const int row = warp * 32 + lane;
        const uint32_t tmem_row = tmem_base + ((uint32_t)(warp * 32) << 16);
        float* dK = p.dkv_ctx + ((((size_t)page * 2 + 0) * p.Hkv + g) * PG) * HD + row;
        float* dV = dK + (size_t)p.Hkv * PG * HD;
        if (any) rows_bar();         // a row that gave up told the others through flags[0]
        const bool have = any && n_done > 0 && !flags[0];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float tk[32], tv[32];
            if (have) {
                tmem_ld32(tmem_row + COL_DKT + h * 32, tk);
                tmem_ld32(tmem_row + COL_DVT + h * 32, tv);
            } else {
#pragma unroll
                for (int c = 0; c < 32; ++c) { tk[c] = 0.f; tv[c] = 0.f; }
            }
#pragma unroll
            for (int c = 0; c < 32; ++c) {
                dK[(size_t)(h * 32 + c) * HD] = tk[c];
                dV[(size_t)(h * 32 + c) * HD] = tv[c];
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

constexpr int SMEM_Q = 1024 + 2 * QD_BYTES + KV_STAGES * 2 * KV_TILE_BYTES + 2 * 2 * PS_BYTES + 256;
constexpr int SMEM_KV = 1024 + 2 * KV_TILE_BYTES + 2 * 2 * QD_BYTES + 2 * 2 * PS_BYTES + 256;
static_assert(SMEM_Q <= 227 * 1024 && SMEM_KV <= 227 * 1024, "shared memory of one CTA");

}  // namespace

bool attn_bwd_supported(const dflash_config& c, int rows) {
    if (c.dtype != DFLASH_BF16 || c.head_dim != HD || c.page_size != PG) return false;
    const int group = c.n_q_heads / c.n_kv_heads;
    return group >= 1 && 64 % group == 0 && rows * group <= 64 && rows <= 32;
}

int launch_attention_bwd(const Launch& L, const dflash_attn_bwd_args& a, float* D) {
    const dflash_config& c = L.h->cfg;
    if (a.batch == 0 || a.rows == 0) return DFLASH_OK;
    BParams p{};
    p.S = a.batch; p.R = a.rows; p.Hq = c.n_q_heads; p.Hkv = c.n_kv_heads; p.group = c.n_q_heads / c.n_kv_heads;
    p.max_pages = a.max_pages; p.n_pages = a.n_pool_pages; p.layer = a.layer;
    p.causal = a.mode == DFLASH_ATTN_CAUSAL ? 1 : 0;
    p.rows_valid = a.rows * p.group;
    p.max_ctx_len = a.max_ctx_len;
    p.shared_row = a.shared_page_row ? 1 : 0;
    p.scale = c.softmax_scale;
    p.scale_log2 = c.softmax_scale * LOG2E;
    p.ctx_len = a.ctx_len; p.page_table = a.page_table;
    p.out = (const __nv_bfloat16*)a.out; p.dout = (const __nv_bfloat16*)a.dout; p.lse = a.lse; p.D = D;
    p.dq = (__nv_bfloat16*)a.dq; p.dk_blk = (__nv_bfloat16*)a.dk_blk; p.dv_blk = (__nv_bfloat16*)a.dv_blk;
    p.dkv_ctx = a.dkv_ctx; p.status = L.status;

    CUtensorMap tq, tdo, tpool, tkb, tvb;
    {   // q / dout as [S*R][Hkv][group][hd]: box of 64 rows (block rows x group), one kv head, 64 columns
        const uint64_t dims[4] = {(uint64_t)HD, (uint64_t)p.group, (uint64_t)p.Hkv, (uint64_t)a.batch * a.rows};
        const uint64_t str[3] = {(uint64_t)HD * 2, (uint64_t)p.group * HD * 2, (uint64_t)p.Hq * HD * 2};
        const uint32_t box[4] = {64, (uint32_t)p.group, 1, (uint32_t)(64 / p.group)};
        if (!tmap_encode_bf16(&tq, a.q, 4, dims, str, box)) return DFLASH_ERR_CUDA;
        if (!tmap_encode_bf16(&tdo, a.dout, 4, dims, str, box)) return DFLASH_ERR_CUDA;
    }
    {
        const uint64_t rows = (uint64_t)c.n_layers * a.n_pool_pages * 2 * p.Hkv * PG;
        const uint64_t dims[2] = {(uint64_t)HD, rows};
        const uint64_t str[1] = {(uint64_t)HD * 2};
        const uint32_t box[2] = {64, (uint32_t)PG};
        if (!tmap_encode_bf16(&tpool, a.kv_pool, 2, dims, str, box)) return DFLASH_ERR_CUDA;
    }
    {
        const uint64_t dims[2] = {(uint64_t)p.Hkv * HD, (uint64_t)a.batch * a.rows};
        const uint64_t str[1] = {(uint64_t)p.Hkv * HD * 2};
        const uint32_t box[2] = {64, (uint32_t)PG};
        if (!tmap_encode_bf16(&tkb, a.k_blk, 2, dims, str, box)) return DFLASH_ERR_CUDA;
        if (!tmap_encode_bf16(&tvb, a.v_blk, 2, dims, str, box)) return DFLASH_ERR_CUDA;
    }
    static bool attr_set[MAX_DEVICES] = {};
    const int dev = current_device_slot();
    if (dev < 0 || !attr_set[dev]) {
        if (cudaFuncSetAttribute(attn_bwd_q_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_Q) != cudaSuccess ||
            cudaFuncSetAttribute(attn_bwd_kv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_KV) != cudaSuccess)
            return DFLASH_ERR_CUDA;
        if (dev >= 0) attr_set[dev] = true;
    }
    // the blocks by falling context length, behind D in the scratch (a.batch ints)
    int32_t* order = reinterpret_cast<int32_t*>(D + (((size_t)a.batch * a.rows * c.n_q_heads + 63) / 64) * 64);
    p.order = order;
    if (launch_ordered(order_kernel, dim3(1), dim3(1024), (size_t)std::min(a.batch, ORDER_MAX) * 4, L.st, a.ctx_len, a.batch, order) !=
        cudaSuccess)
        return DFLASH_ERR_CUDA;
    ++g_launches;
    const int q_ctas = p.shared_row ? (a.batch + 1) / 2 : a.batch;      // blocks sharing one page-table row: two per CTA
    if (launch_ordered(attn_bwd_q_kernel, dim3(p.Hkv, q_ctas), dim3(N_THREADS), (size_t)SMEM_Q, L.st, tq, tdo, tpool, tkb, tvb, p) !=
        cudaSuccess)
        return DFLASH_ERR_CUDA;
    ++g_launches;
    const int n_ctx_tiles = (a.max_ctx_len + PG - 1) / PG;
    if (n_ctx_tiles > 0 && a.dkv_ctx) {
        const dim3 grid(p.Hkv, n_ctx_tiles, p.shared_row ? 1 : a.batch);
        if (launch_pdl(attn_bwd_kv_kernel, grid, dim3(N_THREADS), (size_t)SMEM_KV, L.st, tq, tdo, tpool, p) != cudaSuccess)
            return DFLASH_ERR_CUDA;
        ++g_launches;
    }
    return DFLASH_OK;
}

}  // namespace dflash
