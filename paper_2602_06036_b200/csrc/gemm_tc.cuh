// Interface of the bf16 tensor-core contraction family (tcgen05 / TMEM / TMA).
#pragma once

#include "dflash_internal.h"

namespace dflash {

// What happens to a finished [128 features x tokens] fp32 accumulator tile.
enum GemmEpilogue : int {
    EPI_STORE_F32 = 0,  // out[token][feature] = acc                         (+ optional norm outputs)
    EPI_RESIDUAL = 1,   // out[token][feature] += acc  (x += W_o a, x += W_down h) (+ optional norm outputs)
    EPI_QKV_ROPE = 2,   // split into q, k, v (bf16), rotate q and k
    EPI_SWIGLU = 3,     // h[token][j] = silu(acc[2j]) * acc[2j+1]
    EPI_ARGMAX = 4,     // per (feature tile, token): top-2 over the tile's features
    EPI_CTX_KV = 5,     // rotate K, scatter K and V rows into the paged pool (one group per layer)
};

struct Top2Entry {  // 16 bytes
    float v1;
    int32_t i1;
    float v2;
    int32_t pad;
};

constexpr int GEMM_MAX_GROUPS = 8;

// RMSNorm is folded into the contractions around it (App. A.3 norm, pre-norm layers):
//   producer side ("norm_out"): an epilogue that has the new residual row values also writes
//     xn[token][f] = bf16(g_next[f] * value) and, per 128-feature tile, sum(value^2) per token;
//   consumer side ("norm_in"): the next contraction multiplies each token column of its
//     accumulator by rsqrt(sum over tiles / dim + eps), which equals W * RMSNorm(x) because the
//     per-token scale commutes with the contraction.
struct GemmArgs {
    // problem: acc[token][feature] = sum_k X[token][k] * W[g][feature][k]
    const void* X;                      // [M, K] bf16 row-major
    const void* W[GEMM_MAX_GROUPS];     // n_groups weight matrices [N, K] bf16 row-major
    int n_groups;                       // 0 or 1 = a single matrix
    int M, N, K;
    int epilogue;
    // split-K scratch (needed when the chooser returns more than one split)
    float* part;
    int32_t* counters;
                           // tickets: zero on entry, one slice per launch (the kernel leaves them non-zero)
    // norm_in
    const float* ssq_in;   // [ceil(K/128), M] or nullptr
    // norm_out (EPI_STORE_F32 / EPI_RESIDUAL)
    const void* g_next;    // bf16 [N] or nullptr
    __nv_bfloat16* xn_out; // [M, N]
    float* ssq_out;        // [ceil(N/128), M]
    // EPI_STORE_F32 / EPI_RESIDUAL
    float* out_f32;        // may be nullptr for EPI_STORE_F32 with norm_out
    int ld_out;
    // EPI_QKV_ROPE (g_q / g_k: gains of the per-head norm of q and k, or nullptr)
    const void *g_q, *g_k;
    __nv_bfloat16 *q, *k, *v;
    const int32_t* ctx_len;
    int rows_per_seq;
    // EPI_SWIGLU
    __nv_bfloat16* h;
    // EPI_ARGMAX
    Top2Entry* top2;    // [n_feature_tiles, M]
    float* logits_out;  // optional [M, N]
    // EPI_CTX_KV (group g writes pool layer first_layer + g; g_k_group[g]: that layer's k-head norm gain or nullptr)
    const dflash_ctx_args* ctx;
    int first_layer;
    const void* g_k_group[GEMM_MAX_GROUPS];
};

// Scratch the launcher needs: partial accumulators of tiles shared by several CTAs, and their tickets.
int64_t gemm_tc_part_bytes(int M, int N, int K, int n_groups, int sm_count);
int64_t gemm_tc_counter_bytes(int M, int N, int n_groups);

// `phase_done`: GEMM_MAX_PHASES int32 counters in device memory, zero on entry (the kernel leaves
// them non-zero: one launch per zeroing).
constexpr int GEMM_MAX_PHASES = 4;
int launch_gemm_tc(const Launch& L, const GemmArgs& a, int32_t* phase_done);
// Host-only consistency check of the work split of one contraction (see dflash_gemm_plan_check in dflash.h).
int gemm_plan_check(int M, int N, int K, int n_groups, int sm_count, int pair_cap, int cluster_cap, int32_t* info);
// A chain of contractions in ONE launch: phase i+1 may read what phase i's epilogues wrote. The
// phases share the token-tile size (chosen for the largest row count) but not the row count. traces[i] (may be nullptr) = timeline record of phase i.
int launch_gemm_chain(const Launch& L, const GemmArgs* phases, int n_phases, int32_t* phase_done,
                      unsigned long long* const* traces);
int launch_argmax_finish(const Launch& L, const Top2Entry* top2, int n_tiles, int M, int32_t* ids, float* top1,
                         float* margin);
// x[row] = E[id] (fp32), xn[row] = bf16(g * x[row]), ssq[tile][row] = sum over the tile of x^2
int launch_embed_norm(const Launch& L, const int32_t* anchor, const int32_t* token_ids, int batch, int block_rows, float* x,
                      const void* g, __nv_bfloat16* xn, float* ssq);

}  // namespace dflash
