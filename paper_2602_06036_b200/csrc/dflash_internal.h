// Internal declarations shared by the translation units of the library (not part of the ABI).
#pragma once

#include <cuda.h>  // CUtensorMap only
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "dflash.h"

#define DFLASH_MAX_LAYERS 64

enum DflashFamily : int {
    FAM_EMBED = 0, FAM_RMSNORM, FAM_GEMM_QKV, FAM_ATTENTION, FAM_GEMM_O, FAM_GEMM_GATEUP, FAM_GEMM_DOWN,
    FAM_LMHEAD, FAM_ARGMAX_FINISH, FAM_ROW_ARGMAX, FAM_ACCEPT, FAM_CTX_FUSE, FAM_CTX_KV, FAM_MISC, FAM_GEMM_CHAIN,
};
static_assert(FAM_GEMM_CHAIN + 1 == DFLASH_N_FAMILIES, "family table out of step with the header");

struct dflash_profile_rec {
    cudaEvent_t e0, e1;
    int family;
};

// Encoded tensor maps of weight matrices, kept per handle: the weights of a handle do not move between
// dflash_set_weights calls, so a launch looks its maps up instead of encoding 6-8 of them (about 13 us of host
// time per step for callers that launch eagerly).
struct dflash_wmap_entry {
    const void* base;
    int rows, K, slabs;
    CUtensorMap map;
};
constexpr int DFLASH_WMAP_CACHE = 8 * 64 + 8;      // per layer: QKV, K/V rows of QKV, O, gate/up, down (x slab variants) + fusion, LM head

struct dflash_handle {
    dflash_config cfg;
    dflash_wmap_entry* wmaps;      // [DFLASH_WMAP_CACHE], allocated at create
    int n_wmaps;
    dflash_layer_weights layers[DFLASH_MAX_LAYERS];
    dflash_weights w;
    bool has_weights;
    int sm_count;
    // optional per-launch event pairs
    bool prof_on;
    dflash_profile_rec* prof;
    int prof_cap, prof_used;
    // optional device-side timeline
    unsigned long long* trace_buf;
    int trace_cap, trace_used;
    int* trace_fam;
};

namespace dflash {

// Counts kernel launches issued by the library (reported by dflash_launch_count).
extern long long g_launches;

// Per-device memo for settings a launcher makes once per (kernel, device): function attributes are per
// device, so a process that drives several GPUs must make them on each. Indexed by the current device.
constexpr int MAX_DEVICES = 64;
inline int current_device_slot() {
    int d = 0;
    if (cudaGetDevice(&d) != cudaSuccess || d < 0 || d >= MAX_DEVICES) return -1;
    return d;
}

inline int64_t align_up(int64_t v, int64_t a) { return (v + a - 1) / a * a; }
inline int elem_size(int dtype) { return dtype == DFLASH_F32 ? 4 : 2; }

// Bump allocator over the caller's workspace; the same walk sizes it (base == nullptr).
struct Arena {
    char* base;
    int64_t off;
    explicit Arena(void* b) : base(static_cast<char*>(b)), off(0) {}
    void* take(int64_t bytes) {
        void* p = base ? base + off : nullptr;
        off += align_up(bytes, 256);
        return p;
    }
};

// Activation buffers of one pass over `rows` rows (rows = batch * rows-per-sequence).
struct Workspace {
    float* x;        // [rows, D]   fp32 residual stream
    void*  u;        // [rows, max(D, k*D_t?)] normalised operand, config dtype
    float* tmp;      // [rows, max(QKV, 2F, D)] fp32 GEMM output before its epilogue
    void*  q;        // [rows, Hq*hd]
    void*  k_blk;    // [rows, Hkv*hd]
    void*  v_blk;    // [rows, Hkv*hd]
    void*  attn;     // [rows, Hq*hd]
    void*  h;        // [rows, F]
    float* logits;   // [min(rows, LOGIT_ROWS), V] fp32 (only the fp32 path stages logits)
    int32_t* ids;    // [rows]
    float* part;     // split-K partial sums of the tensor-core contractions
    enum { CNT_QKV = 0, CNT_O, CNT_GATEUP, CNT_DOWN, CNT_LM, CNT_FUSE, CNT_KV, CNT_N };
    int32_t* counters;   // tickets of shared output tiles (zeroed at the start of each call)
    int cnt_off[CNT_N];  // first ticket of each contraction shape (int32 units)
    int cnt_stride[CNT_N];   // tickets per use of that shape within one call (QKV / O / gate-up / down: one slice per layer)
    int32_t* flags;      // [n_flag_sets][4] phase-completion counters of chained launches
    int n_flag_sets;
    int64_t counter_bytes;
    int32_t* attn_counters;   // split-KV tickets of the attention kernel (inside the same region)
    void* top2;      // [vocab tiles, rows] per-tile winners of the fused LM-head argmax
    float* attn_part;    // attention split-KV partials
    float4* seg;         // [rows, 64] per-segment winners of the row argmax over given logits
    float* ssq;          // [D/128, rows] per-tile sums of squares feeding the folded RMSNorm
    int64_t bytes;
};
Workspace carve(const dflash_handle* h, void* base, int batch, int rows);

constexpr int LOGIT_ROWS = 64;

struct Launch {
    dflash_handle* h;
    cudaStream_t st;
    int32_t* status;
    unsigned long long* trace;   // 4-word timeline record of the launch being issued, or nullptr
};

// ---- generic (any dtype) kernels: the whole fp32 path, and the small steps of the bf16 path ----
// token of row r of sequence b: token_ids[b * block_rows + r] if token_ids, else anchor[b] (r = 0) or the mask token
int launch_embed(const Launch& L, const int32_t* anchor, const int32_t* token_ids, float* x, int batch, int block_rows);
// block rows' k / v [batch * rows_per_seq, Hkv * hd] -> pool layer `layer` at positions ctx_len[b] + r
int launch_kv_commit(const Launch& L, const void* k_blk, const void* v_blk, int batch, int rows_per_seq, const int32_t* ctx_len,
                     const int32_t* page_table, int max_pages, void* pool, int n_pages, int layer);
// feats[row, off .. off + D) = x[row, :] in the config dtype
int launch_tap_copy(const Launch& L, const float* x, void* feats, int rows, int D, int ld_out, int off);
int launch_rmsnorm(const Launch& L, const void* in, bool in_is_f32, const void* g, bool apply,
                   void* out, int rows, int dim);
int launch_gemm_simt(const Launch& L, const void* X, const void* W, float* Y, int M, int N, int K,
                     bool accumulate);
// g_q / g_k: gains of the per-head q / k norm applied before the rotation, or nullptr
int launch_rope_split(const Launch& L, const float* qkv, const int32_t* ctx_len, int rows_per_seq,
                      int rows, void* q, void* k, void* v, const void* g_q, const void* g_k);
int launch_swiglu(const Launch& L, const float* gu, void* h, int rows);
int launch_attention_simt(const Launch& L, const dflash_attn_args& a);
int launch_ctx_scatter(const Launch& L, const float* kv, const dflash_ctx_args& a, int layer, const void* g_k);
// two-stage row argmax; seg_scratch holds rows * 64 float4 entries
int launch_row_argmax(const Launch& L, const void* logits, int dtype, int64_t row_stride, int rows,
                      int vocab, float4* seg_scratch, int32_t* ids, float* top1, float* margin);
int launch_accept(const Launch& L, const dflash_verify_args& a, const int32_t* target_ids);
// greedy verification from logits: segment arg-max pass, then per sequence the row merge and the accept rule
int launch_verify_logits(const Launch& L, const dflash_verify_args& a, int64_t row_stride, float4* seg_scratch);
int launch_copy_f32(const Launch& L, const float* src, float* dst, int64_t n);
int launch_zero(const Launch& L, void* dst, int64_t bytes);

}  // namespace dflash
