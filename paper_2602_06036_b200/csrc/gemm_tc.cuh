// Interface of the bf16 tensor-core contraction family (tcgen05 / TMEM / TMA).
#pragma once

#include "dflash_internal.h"

namespace dflash {

// What happens to a finished [128 features x tokens] fp32 accumulator tile.
enum GemmEpilogue : int {
    EPI_STORE_F32 = 0,  // out[token][feature] = acc
    EPI_RESIDUAL = 1,   // out[token][feature] += acc            (x += W_o a,  x += W_down h)
    EPI_QKV_ROPE = 2,   // split into q, k, v (bf16), rotate q and k
    EPI_SWIGLU = 3,     // h[token][j] = silu(acc[2j]) * acc[2j+1]
    EPI_ARGMAX = 4,     // per (feature tile, token): top-2 over the tile's features
    EPI_CTX_KV = 5,     // rotate K, scatter K and V rows into the paged pool
};

struct Top2Entry {  // 16 bytes
    float v1;
    int32_t i1;
    float v2;
    int32_t pad;
};

struct GemmArgs {
    // problem: acc[token][feature] = sum_k X[token][k] * W[feature][k]
    const void* X;   // [M, K] bf16 row-major
    const void* W;   // [N, K] bf16 row-major
    int M, N, K;
    int epilogue;
    // split-K scratch (needed when the chooser returns more than one split)
    float* part;
    int32_t* counters;
    // EPI_STORE_F32 / EPI_RESIDUAL
    float* out_f32;
    int ld_out;
    // EPI_QKV_ROPE
    __nv_bfloat16 *q, *k, *v;
    const int32_t* ctx_len;
    int rows_per_seq;
    // EPI_SWIGLU
    __nv_bfloat16* h;
    // EPI_ARGMAX
    Top2Entry* top2;    // [n_feature_tiles, M]
    float* logits_out;  // optional [M, N]
    // EPI_CTX_KV
    const dflash_ctx_args* ctx;
    int layer;
};

// Number of K splits the launcher will use for this shape (1 = none), and scratch it then needs.
int gemm_tc_splits(int M, int N, int K, int sm_count);
int64_t gemm_tc_part_bytes(int M, int N, int K, int sm_count);
int64_t gemm_tc_counter_bytes(int M, int N);

int launch_gemm_tc(const Launch& L, const GemmArgs& a);
int launch_argmax_finish(const Launch& L, const Top2Entry* top2, int n_tiles, int M, int32_t* ids, float* top1,
                         float* margin);

}  // namespace dflash
