// Block attention on tcgen05 tensor cores (bf16, head_dim 128, 64-token pages):
//   every block row of a sequence attends over [paged context K/V ; the block's own K/V].
// One CTA works on one (sequence, kv head, range of KV tiles). The queries of all block rows and of
// the q heads that share the kv head (rows x group <= 128) are the 128-row "M" operand; a KV tile
// is one 64-token page (or the block's own rows). Roles: a TMA producer warp (5-deep K/V ring that
// runs ahead of the math) and TWO independent pipelines that take alternate tiles, each made of one
// MMA-issuing warp and one softmax warpgroup with their own S buffers (two, so the next S is ready
// before the current softmax ends), P buffer and output accumulator:
//   S_w = Q K^T          tcgen05.mma into TMEM
//   softmax              one thread per query row reads its S row from TMEM (no cross-thread
//                        reduction), exponentials in the log2 domain against a running maximum that
//                        is only raised when a tile exceeds it by more than 2^8 (then the row of O_w
//                        in TMEM is rescaled in place), P -> shared memory (bf16)
//   O_w += P V           tcgen05.mma accumulating in TMEM, V as an MN-major operand straight from
//                        the page layout
// When the query rows fill at most half of the 128-row operand (the draft block: 16 rows x 4 heads) they
// are loaded twice; the threads of the second copy sit on the other two TMEM lane quadrants (hence the
// other two warp schedulers) and take keys 32..63 of every tile, so no issue slot idles on padding.
// So the softmax of one tile overlaps the contractions of the next, and the output never leaves
// TMEM until the end, where the two accumulators are merged. Long contexts are split across CTAs;
// each writes its partial (acc, max, sum) and a small second kernel merges them in range order
// (bit-reproducible). DRAFT mode: no mask inside the block; VERIFY mode: block row r sees block
// rows <= r. Every mbarrier wait is bounded.
#include "attn_tc.cuh"

#include "ptx_sm100.cuh"

#include <math_constants.h>

#include <algorithm>

namespace dflash {
namespace {

using namespace ptx;

constexpr int HD = 128;          // head_dim
constexpr int PG = 64;           // tokens per page = keys per tile
constexpr int LPT_MAX = 256;      // batches up to this size are taken longest sequence first
constexpr int NS = 5;            // K/V ring depth (the kernel is bound by the bytes it keeps in flight: 3 stages ran 1.37x slower than 4)
constexpr int Q_BYTES = 128 * HD * 2;            // 32 KiB: two 64-wide halves of 128 rows
constexpr int KV_STAGE_BYTES = 2 * PG * HD * 2;  // K (16 KiB) + V (16 KiB)
constexpr int P_BYTES = 128 * PG * 2;            // 16 KiB per warpgroup
constexpr int PART_LD = HD + 4;                  // acc[128], running max, running sum, 2 pad (16-byte rows)
constexpr int SMEM_BYTES = 1024 + Q_BYTES + NS * KV_STAGE_BYTES + 2 * P_BYTES + 512;
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory of one CTA");
constexpr uint32_t TMEM_COLS = 512;              // S[w][2] (4 x 64) | O0 | O1 (128 each)
constexpr int N_THREADS = 352;                   // producer, MMA issuer 0, 2 x 4 softmax warps, MMA issuer 1
constexpr uint32_t TMEM_O = 256;                 // first column of the output accumulators
constexpr float RESCALE_GAP = 8.f;               // log2 units

struct AParams {
    int S, R, Hq, Hkv, group, max_pages, n_pages, layer, causal, tiles_per_unit, n_chunks, rows_valid;
    int max_ctx_len;   // the caller's bound the KV split was sized for: longer lengths are clamped to it and flagged
    int dup;     // rows_valid <= 64: the query rows are loaded twice and each copy handles 32 of a tile's 64 keys
    int early_kv;   // the cached context of this layer was written before the previous kernel's dependencies:
                    // its first tiles may be requested before the grid dependency resolves
    float scale_log2;
    const int32_t* ctx_len;
    const int32_t* early_len;   // with early_kv: rows [0, early_len[b]) are the final ones (nullptr: all of ctx_len[b])
    const int32_t* page_table;
    __nv_bfloat16* out;
    float* lse;       // [S, R, Hq] natural-log sum of exponentials per query row, or nullptr
    float* part;
    int32_t* status;
    unsigned long long* trace;
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
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float* v) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(taddr),
        "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
        "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
        "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
        "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])),
        "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
        "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
        "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])),
        "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// MN-major operand (V: [key][head_dim], head_dim contiguous) in two 64-column halves of 64 rows x
// 128 bytes, 128-byte swizzle: leading byte offset = distance between the halves (8 KiB), stride
// byte offset = distance between 8-key groups (1 KiB).
__device__ __forceinline__ uint64_t smem_desc_sw128_mn(uint32_t addr) {
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(8192 >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}
// D fp32, A bf16 K-major, B bf16 MN-major
__host__ __device__ constexpr uint32_t instr_desc_bf16_bmn(int m, int n) {
    return instr_desc_bf16(m, n) | (1u << 16);
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 t = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&t);
}
// named barrier over the 128 threads of one softmax warpgroup (ids 1 and 2), and over both (id 3)
__device__ __forceinline__ void wg_bar(int wg) { asm volatile("bar.sync %0, 128;" ::"r"(wg + 1) : "memory"); }
__device__ __forceinline__ void both_bar() { asm volatile("bar.sync 3, 256;" ::: "memory"); }

__global__ void __launch_bounds__(N_THREADS, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmPool,
               const __grid_constant__ CUtensorMap tmKb, const __grid_constant__ CUtensorMap tmVb, const AParams p) {
    // ---- which work unit ----
    // Lengths and the page table are inputs of the call (no kernel writes them), so the work unit, the
    // barriers, the TMEM allocation and the first page numbers are ready before the grid dependency
    // (q and the block's k/v from the contraction before this kernel) resolves.
    if (threadIdx.x == 0) trace_min(p.trace, 0);
    pdl_trigger();
    const int chunk = blockIdx.x % p.n_chunks;
    const int g = (blockIdx.x / p.n_chunks) % p.Hkv;
    // CTAs are handed to the SMs in index order, so the sequences are taken longest first (a long sequence that
    // starts in the last wave would hold the tail alone): the CTA group with number s works on the sequence whose
    // length has rank s, ties by index. Every CTA finds that sequence itself from the call's lengths.
    int b = blockIdx.x / (p.n_chunks * p.Hkv);
    if (p.S > 1 && p.S <= LPT_MAX) {
        __shared__ int s_len[LPT_MAX];
        __shared__ int s_seq;
        const int want = b;
        for (int t = threadIdx.x; t < p.S; t += N_THREADS) s_len[t] = p.ctx_len[t];
        __syncthreads();
        if ((int)threadIdx.x < p.S) {
            const int t = threadIdx.x, mine = s_len[t];
            int rank = 0;
            for (int j = 0; j < p.S; ++j) {
                const int l = s_len[j];
                rank += (l > mine || (l == mine && j < t)) ? 1 : 0;
            }
            if (rank == want) s_seq = t;
        }
        __syncthreads();
        b = s_seq;
    }
    const int L_given = p.ctx_len[b];
    const int L = min(max(L_given, 0), p.max_ctx_len);   // the ranges (and the partials buffer) cover max_ctx_len keys
    if (L_given > p.max_ctx_len && threadIdx.x == 0 && chunk == 0 && p.status) atomicOr(p.status, DFLASH_DEV_CTX_OVERFLOW);
    const int n_ctx_tiles = (L + PG - 1) / PG;
    const int T = n_ctx_tiles + 1;                       // + the block's own rows
    const int t_lo = chunk * p.tiles_per_unit;
    if (t_lo >= T) return;                               // whole CTA leaves before touching any barrier
    const int t_hi = min(t_lo + p.tiles_per_unit, T);
    const int n_tiles = t_hi - t_lo;
    const int n_splits = (T + p.tiles_per_unit - 1) / p.tiles_per_unit;   // CTAs sharing this (sequence, kv head)

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem;
    uint8_t* sKV = sQ + Q_BYTES;
    uint8_t* sP = sKV + NS * KV_STAGE_BYTES;             // two P tiles
    uint64_t* bars = reinterpret_cast<uint64_t*>(sP + 2 * P_BYTES);
    uint64_t* q_full = bars;
    uint64_t* kv_full = bars + 1;
    uint64_t* kv_empty = kv_full + NS;
    uint64_t* s_full = kv_empty + NS;      // [2][2] S buffer (pipeline w, buffer) written by the tensor core
    uint64_t* s_free = s_full + 4;         // [2][2] S buffer read by its warpgroup
    uint64_t* p_full = s_free + 4;         // [2] P_w written (and O_w rescaled if needed)
    uint64_t* pv_done = p_full + 2;        // [2] O_w += P_w V finished (P_w reusable, O_w consistent)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(pv_done + 2);
    volatile int* flags = reinterpret_cast<volatile int*>(tmem_slot + 1);   // [0] abort
    volatile int* tile_ok = flags + 2;      // [NS] 0 if the ring stage holds a page that must be ignored

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int s = 0; s < NS; ++s) { mbar_init(&kv_full[s], 1); mbar_init(&kv_empty[s], 1); }
        for (int s = 0; s < 4; ++s) { mbar_init(&s_full[s], 1); mbar_init(&s_free[s], 4); }
        for (int s = 0; s < 2; ++s) { mbar_init(&p_full[s], 4); mbar_init(&pv_done[s], 1); }
        flags[0] = 0;
        fence_barrier_init();
        fence_proxy_async();
    }
    if (warp == 1) tmem_alloc(tmem_slot, TMEM_COLS);      // warp 1 owns the allocation
    constexpr int PAGE_PRE = 4;                           // page numbers fetched ahead of the dependency
    int page_pre[PAGE_PRE];
    if (threadIdx.x == 0) {
#pragma unroll
        for (int i = 0; i < PAGE_PRE; ++i) {
            const int t = t_lo + i;
            page_pre[i] = (i < n_tiles && t < n_ctx_tiles && t < p.max_pages) ? __ldg(p.page_table + (size_t)b * p.max_pages + t) : -1;
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // Context K/V tiles of the first ring stages travel while the previous kernel (which produces q and
    // the block's own k/v, not the cache) is still running.
    int n_early = 0;
    if (threadIdx.x == 0 && p.early_kv) {
        const uint64_t pol_kv = policy_evict_first();
        // only pages that lie wholly below the rows an earlier kernel of this call may still be writing
        const int n_final_tiles = p.early_len ? min(__ldg(p.early_len + b), L) / PG : n_ctx_tiles;
#pragma unroll
        for (int i = 0; i < PAGE_PRE; ++i) {
            const int t = t_lo + i;
            const int page = page_pre[i];
            if (i == n_early && i < n_tiles && i < NS && t < n_ctx_tiles && t < n_final_tiles && page >= 0 && page < p.n_pages) {
                uint8_t* dK = sKV + (size_t)i * KV_STAGE_BYTES;
                uint8_t* dV = dK + KV_STAGE_BYTES / 2;
                mbar_expect_tx(&kv_full[i], KV_STAGE_BYTES);
                tile_ok[i] = 1;
                const int rowK = ((((p.layer * p.n_pages + page) * 2 + 0) * p.Hkv + g) * PG);
                const int rowV = rowK + p.Hkv * PG;
                tma_load_2d(dK, &tmPool, 0, rowK, &kv_full[i], pol_kv);
                tma_load_2d(dK + 8192, &tmPool, 64, rowK, &kv_full[i], pol_kv);
                tma_load_2d(dV, &tmPool, 0, rowV, &kv_full[i], pol_kv);
                tma_load_2d(dV + 8192, &tmPool, 64, rowV, &kv_full[i], pol_kv);
                n_early = i + 1;
            }
        }
    }
    pdl_wait();
    if (threadIdx.x == 0) trace_min(p.trace, 1);

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            const uint64_t pol_kv = policy_evict_first(), pol_q = policy_evict_last();
            mbar_expect_tx(q_full, Q_BYTES);
            // q viewed as [S*R][Hkv][group][hd]: box = 64 x group x 1 x (128/group) -> rows ordered (r, j)
            if (p.dup) {     // box of 64 rows, placed at rows 0..63 and again at rows 64..127 of each K half
                for (int hf = 0; hf < 2; ++hf)
                    for (int cp = 0; cp < 2; ++cp)
                        tma_load_4d(sQ + hf * (Q_BYTES / 2) + cp * (Q_BYTES / 4), &tmQ, hf * 64, 0, g, b * p.R, q_full, pol_q);
            } else {
                tma_load_4d(sQ, &tmQ, 0, 0, g, b * p.R, q_full, pol_q);
                tma_load_4d(sQ + Q_BYTES / 2, &tmQ, 64, 0, g, b * p.R, q_full, pol_q);
            }
            bool ok = true;
            for (int i = n_early; i < n_tiles; ++i) {      // the first n_early tiles are already on their way
                const int st = i % NS;
                const uint32_t ph = (i / NS) & 1;
                if (!mbar_wait(&kv_empty[st], ph ^ 1, &flags[0])) { ok = false; break; }
                uint8_t* dK = sKV + (size_t)st * KV_STAGE_BYTES;
                uint8_t* dV = dK + KV_STAGE_BYTES / 2;
                mbar_expect_tx(&kv_full[st], KV_STAGE_BYTES);
                const int t = t_lo + i;
                if (t < n_ctx_tiles) {
                    int page;
                    if (i < PAGE_PRE) {
                        page = page_pre[0];
#pragma unroll
                        for (int q = 1; q < PAGE_PRE; ++q)
                            if (i == q) page = page_pre[q];
                    } else {
                        page = t < p.max_pages ? __ldg(p.page_table + (size_t)b * p.max_pages + t) : -1;
                    }
                    tile_ok[st] = 1;
                    if (page < 0 || page >= p.n_pages) {
                        if (p.status) atomicOr(p.status, DFLASH_DEV_BAD_PAGE);
                        page = 0;      // loaded but fully masked by the softmax warps
                        tile_ok[st] = 0;
                    }
                    // pool rows: ((((layer*n_pages + page)*2 + kv)*Hkv + head)*PG + slot), hd contiguous
                    const int rowK = ((((p.layer * p.n_pages + page) * 2 + 0) * p.Hkv + g) * PG);
                    const int rowV = rowK + p.Hkv * PG;
                    tma_load_2d(dK, &tmPool, 0, rowK, &kv_full[st], pol_kv);
                    tma_load_2d(dK + 8192, &tmPool, 64, rowK, &kv_full[st], pol_kv);
                    tma_load_2d(dV, &tmPool, 0, rowV, &kv_full[st], pol_kv);
                    tma_load_2d(dV + 8192, &tmPool, 64, rowV, &kv_full[st], pol_kv);
                } else {
                    // the block's own k/v: [S*R][Hkv*hd]; rows past this sequence are masked
                    tma_load_2d(dK, &tmKb, g * HD, b * p.R, &kv_full[st], pol_q);
                    tma_load_2d(dK + 8192, &tmKb, g * HD + 64, b * p.R, &kv_full[st], pol_q);
                    tma_load_2d(dV, &tmVb, g * HD, b * p.R, &kv_full[st], pol_q);
                    tma_load_2d(dV + 8192, &tmVb, g * HD + 64, b * p.R, &kv_full[st], pol_q);
                }
            }
            if (!ok) {
                flags[0] = 1;
                if (p.status) atomicOr(p.status, DFLASH_DEV_TIMEOUT);
            }
        }
        __syncwarp();     // the whole warp must reach the closing barrier together
    } else if (warp == 1 || warp == 10) {
        // ---------------- MMA issuers: warp 1 drives pipeline 0 (even tiles), warp 10 pipeline 1 ----------------
        if (lane == 0) {
            constexpr uint32_t idesc_s = instr_desc_bf16(128, PG);
            constexpr uint32_t idesc_o = instr_desc_bf16_bmn(128, HD);
            const uint32_t w = (warp == 1) ? 0u : 1u;
            const int n_mine = (n_tiles - (int)w + 1) / 2;          // tiles w, w+2, ...
            const uint32_t q_addr = smem_u32(sQ), p_addr = smem_u32(sP + w * P_BYTES);
            bool ok = mbar_wait(q_full, 0, &flags[0]);
            // S of this pipeline's k-th tile into its buffer k & 1
            auto issue_s = [&](int k) -> bool {
                const int i = 2 * k + (int)w, st = i % NS;
                const uint32_t bsel = k & 1;
                if (!mbar_wait(&kv_full[st], (i / NS) & 1, &flags[0])) return false;
                if (!mbar_wait(&s_free[w * 2 + bsel], ((k >> 1) & 1) ^ 1, &flags[0])) return false;
                tc_fence_after();
                const uint32_t k_addr = smem_u32(sKV + (size_t)st * KV_STAGE_BYTES);
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk)
                    mma_bf16(tmem_base + (w * 2 + bsel) * PG, smem_desc_sw128(q_addr + (kk >> 2) * (Q_BYTES / 2) + (kk & 3) * 32),
                             smem_desc_sw128(k_addr + (kk >> 2) * 8192 + (kk & 3) * 32), idesc_s, kk > 0 ? 1u : 0u);
                mma_commit(&s_full[w * 2 + bsel]);
                return true;
            };
            if (ok && n_mine > 0) ok = issue_s(0);
            if (ok && n_mine > 1) ok = issue_s(1);
            for (int k = 0; k < n_mine && ok; ++k) {
                const int i = 2 * k + (int)w, st = i % NS;
                if (!mbar_wait(&p_full[w], k & 1, &flags[0])) { ok = false; break; }
                tc_fence_after();
                const uint32_t v_addr = smem_u32(sKV + (size_t)st * KV_STAGE_BYTES + KV_STAGE_BYTES / 2);
#pragma unroll
                for (int kk = 0; kk < PG / 16; ++kk)
                    mma_bf16(tmem_base + TMEM_O + w * HD, smem_desc_sw128(p_addr + kk * 32), smem_desc_sw128_mn(v_addr + kk * 2048),
                             idesc_o, (k > 0 || kk > 0) ? 1u : 0u);      // a pipeline's first tile starts its accumulator
                mma_commit(&pv_done[w]);
                mma_commit(&kv_empty[st]);
                if (k + 2 < n_mine) ok = issue_s(k + 2);
            }
            if (!ok) {
                flags[0] = 1;
                if (p.status) atomicOr(p.status, DFLASH_DEV_TIMEOUT);
            }
        }
        __syncwarp();
    } else {
        // ---------------- softmax warpgroups: thread = query row ----------------
        const int wg = (warp - 2) >> 2;                     // 0: even tiles, 1: odd tiles
        const int ew = warp & 3;                            // TMEM lane quadrant of this warp
        const int row = ew * 32 + lane;                     // TMEM lane
        const int dup = p.dup;
        const int half = dup ? (row >> 6) : 0;              // dup: which 32 keys of a tile this thread takes
        const int lrow = dup ? (row & 63) : row;            // query row
        const int ncol = dup ? 32 : PG;                     // keys per thread and tile
        const int r = lrow / p.group, j = lrow % p.group;   // block row, q head inside the group
        const uint32_t lane_sel = (uint32_t)(ew * 32) << 16;
        const uint32_t tmem_O = tmem_base + TMEM_O + wg * HD + lane_sel;
        uint8_t* myP = sP + wg * P_BYTES;
        // [3][128] exchange between the two copies of a row (dup only): it lives in rows 64..127 of this
        // pipeline's P tile, which in that mode hold nothing (their products land in ignored output rows)
        float* xch = reinterpret_cast<float*>(myP + 64 * 128);
        float m_run = -CUDART_INF_F, l_run = 0.f;           // log2-domain reference maximum, running sum
        bool ok = true;
        int k = 0;                                          // index of this warpgroup's tile
        for (int i = wg; i < n_tiles; i += 2, ++k) {
            const int t = t_lo + i;
            const int st = i % NS;
            // how many keys of this tile exist, and from which one on they are hidden from this row
            int n_valid, n_vis;
            if (t < n_ctx_tiles) {
                n_valid = min(PG, L - t * PG);
                n_vis = n_valid;
            } else {
                n_valid = p.R;
                n_vis = p.causal ? min(r + 1, p.R) : p.R;
            }
            const uint32_t bsel = k & 1;
            const uint32_t tmem_S = tmem_base + (wg * 2 + bsel) * PG + half * 32 + lane_sel;
            if (!mbar_wait(&s_full[wg * 2 + bsel], (k >> 1) & 1, &flags[0])) { ok = false; break; }
            tc_fence_after();
            if (t < n_ctx_tiles && !tile_ok[st]) { n_valid = 0; n_vis = 0; }   // written by the producer before the tile's copy
            const int vis_here = n_vis - half * 32;          // visible keys among this thread's columns
            // pass 1 over this thread's part of the S row (32 columns at a time, straight from TMEM): the maximum
            float mx4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
            for (int h = 0; h * 32 < ncol; ++h) {
                float s[32];
                tmem_ld32(tmem_S + h * 32, s);
                if (vis_here >= (h + 1) * 32) {
#pragma unroll
                    for (int c = 0; c < 32; ++c) mx4[c & 3] = fmaxf(mx4[c & 3], s[c]);
                } else {
#pragma unroll
                    for (int c = 0; c < 32; ++c)
                        if (h * 32 + c < vis_here) mx4[c & 3] = fmaxf(mx4[c & 3], s[c]);
                }
            }
            float mx_raw = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
            if (dup) {       // the other copy of this row looked at the other 32 keys
                xch[bsel * 128 + row] = mx_raw;
                wg_bar(wg);
                mx_raw = fmaxf(mx_raw, xch[bsel * 128 + (row ^ 64)]);
            }
            const float mx = mx_raw * p.scale_log2;          // scale > 0
            // raise the reference maximum only when this tile tops it by more than the gap
            const bool raise = mx > m_run + RESCALE_GAP || (m_run == -CUDART_INF_F && mx > -CUDART_INF_F);
            const float m_new = raise ? mx : m_run;
            const float alpha = (raise && m_run > -CUDART_INF_F) ? fast_exp2(m_run - m_new) : 1.f;
            const float m_use = (m_new > -CUDART_INF_F) ? m_new : 0.f;
            m_run = m_new;
            // the previous P_w V of this warpgroup must be finished before P_w is rewritten or O_w rescaled
            if (!mbar_wait(&pv_done[wg], (k & 1) ^ 1, &flags[0])) { ok = false; break; }
            if (k > 0 && half == 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
                tc_fence_after();
#pragma unroll
                for (int c4 = 0; c4 < HD / 32; ++c4) {
                    float o[32];
                    tmem_ld32(tmem_O + c4 * 32, o);
#pragma unroll
                    for (int d = 0; d < 32; ++d) o[d] *= alpha;
                    tmem_st32(tmem_O + c4 * 32, o);
                }
                tmem_st_wait();
                tc_fence_before();
            }
            // pass 2: exponentials, row sum, P (bf16) into the swizzled K-major tile
            float ps4[4] = {0.f, 0.f, 0.f, 0.f};
            uint8_t* prow = myP + lrow * 128;
            for (int h = 0; h * 32 < ncol; ++h) {
                float s[32];
                tmem_ld32(tmem_S + h * 32, s);
                if (vis_here >= (h + 1) * 32) {
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        s[c] = fast_exp2(fmaf(s[c], p.scale_log2, -m_use));
                        ps4[c & 3] += s[c];
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        s[c] = (h * 32 + c < vis_here) ? fast_exp2(fmaf(s[c], p.scale_log2, -m_use)) : 0.f;
                        ps4[c & 3] += s[c];
                    }
                }
#pragma unroll
                for (int ck = 0; ck < 4; ++ck) {
                    uint4 w4;
                    w4.x = pack_bf16(s[ck * 8 + 0], s[ck * 8 + 1]);
                    w4.y = pack_bf16(s[ck * 8 + 2], s[ck * 8 + 3]);
                    w4.z = pack_bf16(s[ck * 8 + 4], s[ck * 8 + 5]);
                    w4.w = pack_bf16(s[ck * 8 + 6], s[ck * 8 + 7]);
                    *reinterpret_cast<uint4*>(prow + ((((half + h) * 4 + ck) ^ (lrow & 7)) << 4)) = w4;
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&s_free[wg * 2 + bsel]);   // this S buffer may be overwritten (tile k + 2)
            l_run = l_run * alpha + ((ps4[0] + ps4[1]) + (ps4[2] + ps4[3]));
            // keys that do not exist must not poison P.V with whatever the page holds there
            if (n_valid < PG) {
                uint8_t* dV = sKV + (size_t)st * KV_STAGE_BYTES + KV_STAGE_BYTES / 2;
                const int n_bad = PG - n_valid;                  // rows n_valid..63, two halves, 8 chunks each
                for (int e = row; e < n_bad * 16; e += 128) {
                    const int kr = n_valid + e / 16, part = e % 16;
                    *reinterpret_cast<uint4*>(dV + (part >> 3) * 8192 + kr * 128 + (part & 7) * 16) = make_uint4(0, 0, 0, 0);
                }
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(&p_full[wg]);
        }
        // this warpgroup's last P.V
        if (ok && k > 0 && !mbar_wait(&pv_done[wg], (k & 1) ^ 1, &flags[0])) ok = false;
        if (!ok) {
            flags[0] = 1;
            if (lane == 0 && p.status) atomicOr(p.status, DFLASH_DEV_TIMEOUT);
        }
        tc_fence_after();
        if (dup) {               // whole-row sum: the two copies add their parts
            xch[256 + row] = l_run;
            wg_bar(wg);
            l_run += xch[256 + (row ^ 64)];
        }
        // ---- merge the two accumulators: warpgroup 1 hands (max, sum, O_1 row) over through the idle ring
        float* stage = reinterpret_cast<float*>(sKV);
        const bool row_valid = r < p.R;
        both_bar();              // every contraction of both warpgroups is complete: the ring is idle
        if (wg == 1 && half == 0 && !flags[0]) {
            float4* srow = reinterpret_cast<float4*>(stage + row * PART_LD);
            if (k > 0) {
#pragma unroll
                for (int c4 = 0; c4 < HD / 32; ++c4) {
                    float o[32];
                    tmem_ld32(tmem_O + c4 * 32, o);
#pragma unroll
                    for (int d = 0; d < 32; d += 4) srow[(c4 * 32 + d) >> 2] = make_float4(o[d], o[d + 1], o[d + 2], o[d + 3]);
                }
            }
            srow[HD >> 2] = make_float4(k > 0 ? m_run : -CUDART_INF_F, k > 0 ? l_run : 0.f, 0.f, 0.f);
        }
        both_bar();
        if (wg == 0 && half == 0 && !flags[0]) {
            const float4* orow = reinterpret_cast<const float4*>(stage + row * PART_LD);
            const float4 ml1 = orow[HD >> 2];
            const float M = fmaxf(m_run, ml1.x);
            const float w0 = (m_run > -CUDART_INF_F) ? fast_exp2(m_run - M) : 0.f;
            const float w1 = (ml1.x > -CUDART_INF_F) ? fast_exp2(ml1.x - M) : 0.f;
            const float l_tot = l_run * w0 + ml1.y * w1;
            __nv_bfloat16* dst = p.out + (((size_t)b * p.R + r) * p.Hq + g * p.group + j) * HD;
            const float inv = l_tot > 0.f ? 1.f / l_tot : 0.f;
            const float f0 = (n_splits == 1) ? w0 * inv : w0, f1 = (n_splits == 1) ? w1 * inv : w1;
            float4* srow = reinterpret_cast<float4*>(stage + row * PART_LD);     // this thread's own row
            // 32 columns at a time: merged values go straight to the output (one range) or back into this
            // thread's staging row (several ranges: unnormalised partial, copied out below)
#pragma unroll
            for (int c4 = 0; c4 < HD / 32; ++c4) {
                float o[32];
                tmem_ld32(tmem_O + c4 * 32, o);
#pragma unroll
                for (int d = 0; d < 32; d += 4) {
                    float4 o1 = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (w1 > 0.f) o1 = orow[(c4 * 32 + d) >> 2];
                    o[d + 0] = o[d + 0] * f0 + o1.x * f1;
                    o[d + 1] = o[d + 1] * f0 + o1.y * f1;
                    o[d + 2] = o[d + 2] * f0 + o1.z * f1;
                    o[d + 3] = o[d + 3] * f0 + o1.w * f1;
                }
                if (n_splits == 1) {
                    if (row_valid) {
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
                } else {
#pragma unroll
                    for (int d = 0; d < 32; d += 4) srow[(c4 * 32 + d) >> 2] = make_float4(o[d], o[d + 1], o[d + 2], o[d + 3]);
                }
            }
            if (n_splits > 1) srow[HD >> 2] = make_float4(M, l_tot, 0.f, 0.f);
            else if (p.lse && row_valid)      // M and the sum are in the log2 domain
                p.lse[((size_t)b * p.R + r) * p.Hq + g * p.group + j] = (l_tot > 0.f) ? (M + log2f(l_tot)) * 0.6931471805599453f : -CUDART_INF_F;
        }
        if (wg == 0 && n_splits > 1 && !flags[0]) {
            wg_bar(0);
            const int bg = b * p.Hkv + g;
            float4* dst4 = reinterpret_cast<float4*>(p.part + ((size_t)bg * p.n_chunks + chunk) * p.rows_valid * PART_LD);
            const float4* src4 = reinterpret_cast<const float4*>(stage);
            for (int e = row; e < p.rows_valid * (PART_LD / 4); e += 128) dst4[e] = src4[e];
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
    if (threadIdx.x == 0) trace_max(p.trace, 3);
}

// Merge of the per-range partials of one (sequence, kv head): one warp per query row, lanes over
// head_dim, ranges visited in order. Sequences whose context fitted one range were already written.
__global__ void __launch_bounds__(128) attn_combine_kernel(const AParams p) {
    unsigned long long* trace = p.trace ? p.trace + 4 : nullptr;   // the record after the main kernel's
    if (threadIdx.x == 0) trace_min(trace, 0);
    pdl_trigger();
    const int rows_valid = p.rows_valid;
    const int row_blocks = (rows_valid + 3) / 4;
    const int bg = blockIdx.x / row_blocks;
    const int row = (blockIdx.x % row_blocks) * 4 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    const int b = bg / p.Hkv, g = bg % p.Hkv;
    const int L = min(max(__ldg(p.ctx_len + b), 0), p.max_ctx_len);      // an input of the call: no kernel writes it
    const int T = (L + PG - 1) / PG + 1;
    const int n_splits = (T + p.tiles_per_unit - 1) / p.tiles_per_unit;
    pdl_wait();
    if (threadIdx.x == 0) trace_min(trace, 1);
    if (n_splits <= 1 || row >= rows_valid) return;
    const float* base = p.part + ((size_t)bg * p.n_chunks * rows_valid + row) * PART_LD;
    const size_t unit_stride = (size_t)rows_valid * PART_LD;
    // One round trip in the common case: the accumulator rows of the first KF ranges and every
    // range's (max, sum) are requested together; the weights then travel by shuffle.
    // More than 32 ranges: a first pass over (max, sum) finds the global maximum.
    constexpr int KF = 20;
    float4 a[KF];
    auto fetch = [&](int s_first, int n) {
#pragma unroll
        for (int k = 0; k < KF; ++k)
            a[k] = (k < n) ? __ldcg(reinterpret_cast<const float4*>(base + (size_t)(s_first + k) * unit_stride) + lane)
                           : make_float4(0.f, 0.f, 0.f, 0.f);
    };
    fetch(0, min(KF, n_splits));
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float Lsum = 0.f;
    float M = -CUDART_INF_F;
    float2 ml0 = make_float2(-CUDART_INF_F, 0.f);
    for (int s0 = 0; s0 < n_splits; s0 += 32) {
        const int s = s0 + lane;
        if (s < n_splits) {
            const float2 ml = __ldcg(reinterpret_cast<const float2*>(base + s * unit_stride + HD));
            if (s0 == 0) ml0 = ml;
            M = fmaxf(M, ml.x);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    for (int s0 = 0; s0 < n_splits; s0 += 32) {
        const int s = s0 + lane;
        float2 ml = ml0;
        if (s0 > 0) ml = (s < n_splits) ? __ldcg(reinterpret_cast<const float2*>(base + s * unit_stride + HD))
                                        : make_float2(-CUDART_INF_F, 0.f);
        const float w_mine = (s < n_splits && ml.x > -CUDART_INF_F) ? exp2f(ml.x - M) : 0.f;
        float l_mine = ml.y * w_mine;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) l_mine += __shfl_xor_sync(0xffffffffu, l_mine, o);
        Lsum += l_mine;
        const int n_here = min(32, n_splits - s0);
        for (int k0 = 0; k0 < n_here; k0 += KF) {
            if (s0 + k0 > 0) fetch(s0 + k0, min(KF, n_here - k0));
#pragma unroll
            for (int k = 0; k < KF; ++k) {
                const float w = __shfl_sync(0xffffffffu, w_mine, (k0 + k) & 31);
                if (k0 + k < n_here) { acc.x += a[k].x * w; acc.y += a[k].y * w; acc.z += a[k].z * w; acc.w += a[k].w * w; }
            }
        }
    }
    const float inv = Lsum > 0.f ? 1.f / Lsum : 0.f;
    const int r = row / p.group, j = row % p.group;
    if (p.lse && lane == 0) p.lse[((size_t)b * p.R + r) * p.Hq + g * p.group + j] = (Lsum > 0.f) ? (M + log2f(Lsum)) * 0.6931471805599453f : -CUDART_INF_F;
    __nv_bfloat16* dst = p.out + (((size_t)b * p.R + r) * p.Hq + g * p.group + j) * HD + lane * 4;
    uint2 w2;
    w2.x = pack_bf16(acc.x * inv, acc.y * inv);
    w2.y = pack_bf16(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2*>(dst) = w2;
    if (threadIdx.x == 0) trace_max(trace, 3);
}

}  // namespace

bool attn_tc_supported(const dflash_config& c, int rows) {
    if (c.dtype != DFLASH_BF16 || c.head_dim != HD || c.page_size != PG) return false;
    const int group = c.n_q_heads / c.n_kv_heads;
    return group >= 1 && 128 % group == 0 && rows * group <= 128 && rows <= PG;
}

// Keys are split into ranges of `tiles_per_unit` 64-key tiles. One sequence: about one wave of equal
// CTAs. A batch: lengths differ (shorter sequences leave empty units that exit at once).
static int tiles_per_unit(int batch, int Hkv, int max_ctx_len, int sm_count) {
    const int Tmax = (max_ctx_len + PG - 1) / PG + 1;
    const int64_t bh = (int64_t)batch * Hkv;
    if (batch > 1) {
        // measured on the serving-mix shapes: with at least one (sequence, kv head) per SM, whole sequences per
        // CTA win (no partials, no merge kernel); with fewer, ranges of >= 16 tiles sized for about two waves
        // (ranges capped at 128 tiles so that one very long sequence among short ones cannot hold the tail)
        if (bh >= sm_count) return std::min(std::max(2, Tmax), 128);
        const int64_t c = (bh * Tmax + 2 * (int64_t)sm_count - 1) / (2 * (int64_t)sm_count);
        return (int)std::min<int64_t>(std::max<int64_t>(16, c), std::max(2, Tmax));
    }
    for (int c = 2; c < Tmax; ++c)
        if (bh * ((Tmax + c - 1) / c) <= sm_count) return c;
    return std::max(2, Tmax);
}

// Partials the workspace holds: one per (sequence, kv head, range). One sequence: <= SMs (+ rounding); a batch:
// <= 2*SMs + 2*batch*Hkv (ranges of >= total/(2*SMs) tiles); kept generous. attn_tc_plan never exceeds it.
static int64_t part_units(const dflash_config& c, int batch, int sm_count) {
    return 8 * (int64_t)sm_count + 2 * (int64_t)batch * c.n_kv_heads;
}
int64_t attn_tc_part_bytes(const dflash_config& c, int batch, int rows, int sm_count) {
    const int rows_valid = std::min(128, rows * (c.n_q_heads / c.n_kv_heads));
    return part_units(c, batch, sm_count) * rows_valid * PART_LD * 4;
}
AttnPlan attn_tc_plan(const dflash_config& c, int batch, int max_ctx_len, int sm_count) {
    AttnPlan pl{};
    const int Tmax = (max_ctx_len + PG - 1) / PG + 1;
    pl.tiles_per_unit = tiles_per_unit(batch, c.n_kv_heads, max_ctx_len, sm_count);
    pl.capacity_units = part_units(c, batch, sm_count);
    const int64_t bh = (int64_t)batch * c.n_kv_heads;
    // The heuristic caps a range at 128 tiles; a large batch of very long contexts would then need more
    // partials than the workspace holds. Longer ranges instead: two per (sequence, kv head) always fit.
    const int64_t max_chunks = std::max<int64_t>(1, pl.capacity_units / std::max<int64_t>(bh, 1));
    if ((Tmax + pl.tiles_per_unit - 1) / pl.tiles_per_unit > max_chunks)
        pl.tiles_per_unit = (int)((Tmax + max_chunks - 1) / max_chunks);
    pl.n_chunks = (Tmax + pl.tiles_per_unit - 1) / pl.tiles_per_unit;
    pl.units = bh * pl.n_chunks;
    return pl;
}
int64_t attn_tc_counter_bytes(const dflash_config& c, int batch) { return (int64_t)batch * c.n_kv_heads * 4; }

int launch_attention_tc(const Launch& L, const dflash_attn_args& a, float* part, int32_t* counters, bool early_kv,
                        const int32_t* early_len, bool first_of_call) {
    const dflash_config& c = L.h->cfg;
    if (a.batch == 0 || a.rows == 0) return DFLASH_OK;
    AParams p{};
    p.S = a.batch; p.R = a.rows; p.Hq = c.n_q_heads; p.Hkv = c.n_kv_heads; p.group = c.n_q_heads / c.n_kv_heads;
    p.max_pages = a.max_pages; p.n_pages = a.n_pool_pages; p.layer = a.layer;
    p.causal = a.mode == DFLASH_ATTN_CAUSAL ? 1 : 0;
    const AttnPlan plan = attn_tc_plan(c, a.batch, a.max_ctx_len, L.h->sm_count);
    if (plan.units > plan.capacity_units) return DFLASH_ERR_WORKSPACE;      // cannot happen: the plan lengthens the ranges
    p.tiles_per_unit = plan.tiles_per_unit;
    p.max_ctx_len = a.max_ctx_len;
    p.rows_valid = std::min(128, a.rows * p.group);
    p.dup = (p.rows_valid <= 64 && 64 % p.group == 0) ? 1 : 0;
    p.early_kv = early_kv ? 1 : 0;
    p.early_len = early_len;
    p.n_chunks = plan.n_chunks;
    p.scale_log2 = c.softmax_scale * 1.4426950408889634f;
    p.ctx_len = a.ctx_len; p.page_table = a.page_table;
    p.out = (__nv_bfloat16*)a.out; p.lse = a.lse_out; p.part = part; p.status = L.status; p.trace = L.trace;
    (void)counters;

    CUtensorMap tq, tpool, tkb, tvb;
    {   // q as [S*R][Hkv][group][hd]
        const uint64_t dims[4] = {(uint64_t)HD, (uint64_t)p.group, (uint64_t)p.Hkv, (uint64_t)a.batch * a.rows};
        const uint64_t str[3] = {(uint64_t)HD * 2, (uint64_t)p.group * HD * 2, (uint64_t)p.Hq * HD * 2};
        const uint32_t box[4] = {64, (uint32_t)p.group, 1, (uint32_t)((p.dup ? 64 : 128) / p.group)};
        if (!tmap_encode_bf16(&tq, a.q, 4, dims, str, box)) return DFLASH_ERR_CUDA;
    }
    {   // the whole pool as rows of head_dim
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
        if (cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess)
            return DFLASH_ERR_CUDA;
        if (dev >= 0) attr_set[dev] = true;
    }
    const int grid = a.batch * p.Hkv * p.n_chunks;
    // the kernel reads lengths and page numbers ahead of its grid dependency: as the first kernel of a call
    // it therefore starts in plain stream order (the caller's previous call may have produced them)
    const cudaError_t e = first_of_call
        ? launch_ordered(attn_tc_kernel, dim3(grid), dim3(N_THREADS), (size_t)SMEM_BYTES, L.st, tq, tpool, tkb, tvb, p)
        : launch_pdl(attn_tc_kernel, dim3(grid), dim3(N_THREADS), (size_t)SMEM_BYTES, L.st, tq, tpool, tkb, tvb, p);
    if (e != cudaSuccess) return DFLASH_ERR_CUDA;
    ++g_launches;
    if (p.n_chunks > 1) {
        const int rows_valid = p.rows_valid;
        if (launch_pdl(attn_combine_kernel, dim3(a.batch * p.Hkv * ((rows_valid + 3) / 4)), dim3(128), 0, L.st, p) != cudaSuccess)
            return DFLASH_ERR_CUDA;
        ++g_launches;
    }
    return DFLASH_OK;
}

}  // namespace dflash
