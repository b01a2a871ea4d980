// C ABI of the library: argument validation, workspace carving and the launch sequence of each call.
#include "dflash_internal.h"
#include "gemm_tc.cuh"
#include "attn_tc.cuh"

#include <algorithm>
#include <cstring>
#include <new>

using namespace dflash;

namespace dflash {

Workspace carve(const dflash_handle* h, void* base, int batch, int rows) {
    const dflash_config& c = h->cfg;
    Arena a(base);
    Workspace w{};
    const int es = elem_size(c.dtype);
    const int64_t R = std::max(rows, 1);
    const int qdim = c.n_q_heads * c.head_dim, kdim = c.n_kv_heads * c.head_dim;
    const int feat = c.n_feat_layers * c.d_target;
    const bool tc = c.dtype == DFLASH_BF16;
    // fp32 staging of a projection before its element-wise epilogue (fp32 path), or the fused
    // context projection's un-normalised output (both paths)
    const int64_t wide = tc ? (int64_t)c.d_model
                            : std::max<int64_t>(std::max<int64_t>(qdim + 2 * kdim, 2 * (int64_t)c.d_ffn), c.d_model);
    w.x = (float*)a.take(R * c.d_model * 4);
    w.u = a.take(R * std::max(c.d_model, qdim) * es);
    w.tmp = (float*)a.take(R * wide * 4);
    w.q = a.take(R * qdim * es);
    w.k_blk = a.take(R * kdim * es);
    w.v_blk = a.take(R * kdim * es);
    w.attn = a.take(R * qdim * es);
    w.h = a.take(R * c.d_ffn * es);
    w.logits = (float*)a.take(tc ? 256 : std::min<int64_t>(R, LOGIT_ROWS) * c.vocab * 4);
    w.ids = (int32_t*)a.take(R * 4);
    int64_t part = 0, counters = 0;
    if (tc) {
        const int M = (int)R, sm = h->sm_count;
        // context K/V: one ticket range per layer (launches of up to GEMM_MAX_GROUPS - 1 layers each take their own
        // slice)
        const int kv_groups = c.n_layers;
        // order = Workspace::CNT_* : every contraction shape has its own ticket range
        const int shapes[Workspace::CNT_N][3] = {{qdim + 2 * kdim, c.d_model, 1}, {c.d_model, qdim, 1}, {2 * c.d_ffn, c.d_model, 1},
                                                 {c.d_model, c.d_ffn, 1},         {c.vocab, c.d_model, 1}, {c.d_model, feat, 1},
                                                 {2 * kdim, c.d_model, kv_groups}};
        // Every launch that uses a shape within one call takes its own slice of tickets (one per layer for
        // the four per-layer contractions): tickets are zeroed once per call and never shared between
        // launches, whose tile splits may differ (a chained launch and a single one size their grids apart).
        for (int i = 0; i < Workspace::CNT_N; ++i) {
            part = std::max(part, gemm_tc_part_bytes(M, shapes[i][0], shapes[i][1], shapes[i][2], sm));
            const bool per_layer = i == Workspace::CNT_QKV || i == Workspace::CNT_O || i == Workspace::CNT_GATEUP ||
                                   i == Workspace::CNT_DOWN;
            const int64_t one = align_up(gemm_tc_counter_bytes(M, shapes[i][0], shapes[i][2]), 256);
            w.cnt_off[i] = (int)(counters / 4);
            w.cnt_stride[i] = (int)(one / 4);
            counters += one * (per_layer ? c.n_layers : 1);
        }
    }
    w.part = (float*)a.take(std::max<int64_t>(part, 256));
    // one zeroing per call clears: tickets of the contractions, chain phase flags, attention tickets
    const int64_t gemm_counters = std::max<int64_t>(counters, 256);
    w.n_flag_sets = 2 * c.n_layers + 8;
    const int64_t flag_bytes = tc ? align_up((int64_t)w.n_flag_sets * GEMM_MAX_PHASES * 4, 256) : 0;
    const int64_t attn_counters = tc ? align_up(attn_tc_counter_bytes(c, std::max(batch, 1)), 256) : 0;
    w.counter_bytes = gemm_counters + flag_bytes + attn_counters;
    w.counters = (int32_t*)a.take(w.counter_bytes);
    w.flags = w.counters ? (int32_t*)((char*)w.counters + gemm_counters) : nullptr;
    w.attn_counters = w.counters ? (int32_t*)((char*)w.counters + gemm_counters + flag_bytes) : nullptr;
    w.top2 = a.take(tc ? (int64_t)((c.vocab + 127) / 128) * R * (int64_t)sizeof(Top2Entry) : 256);
    w.attn_part = (float*)a.take(tc ? attn_tc_part_bytes(c, std::max(batch, 1), (int)std::min<int64_t>(32, (R + std::max(batch, 1) - 1) / std::max(batch, 1)), h->sm_count) : 256);
    w.seg = (float4*)a.take(R * 64 * 16);
    w.ssq = (float*)a.take((int64_t)((c.d_model + 127) / 128) * R * 4);
    w.bytes = a.off;
    return w;
}

}  // namespace dflash

static bool is_pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }

static const char* kFamilyNames[DFLASH_N_FAMILIES] = {
    "embed", "rmsnorm", "gemm_qkv", "attention", "gemm_o", "gemm_gateup", "gemm_down", "lmhead_argmax",
    "argmax_finish", "row_argmax", "accept", "ctx_fuse", "ctx_kv", "misc", "gemm_chain"};

// ---- per-launch event pairs -------------------------------------------------------------------
static void prof_begin(const Launch& L, int fam) {
    dflash_handle* h = L.h;
    if (!h->prof_on) return;
    if (h->prof_used == h->prof_cap) {
        const int cap = h->prof_cap ? h->prof_cap * 2 : 256;
        dflash_profile_rec* n = new (std::nothrow) dflash_profile_rec[cap];
        if (!n) { h->prof_on = false; return; }
        for (int i = 0; i < h->prof_cap; ++i) n[i] = h->prof[i];
        for (int i = h->prof_cap; i < cap; ++i) {
            cudaEventCreate(&n[i].e0);
            cudaEventCreate(&n[i].e1);
        }
        delete[] h->prof;
        h->prof = n;
        h->prof_cap = cap;
    }
    h->prof[h->prof_used].family = fam;
    cudaEventRecord(h->prof[h->prof_used].e0, L.st);
}
static void prof_end(const Launch& L) {
    dflash_handle* h = L.h;
    if (!h->prof_on) return;
    cudaEventRecord(h->prof[h->prof_used].e1, L.st);
    ++h->prof_used;
}

// next timeline record (attention takes two: main kernel + combine)
static unsigned long long* trace_slot(dflash_handle* h, int fam) {
    if (!h->trace_buf) return nullptr;
    const int n = fam == FAM_ATTENTION ? 2 : 1;
    if (h->trace_used + n > h->trace_cap) return nullptr;
    unsigned long long* r = h->trace_buf + (size_t)h->trace_used * 4;
    for (int i = 0; i < n; ++i) h->trace_fam[h->trace_used + i] = fam;
    h->trace_used += n;
    return r;
}

#define DFLASH_TRY(expr)                    \
    do {                                    \
        int rc__ = (expr);                  \
        if (rc__ != DFLASH_OK) return rc__; \
    } while (0)

#define RUN(fam, expr)              \
    do {                            \
        L.trace = trace_slot(L.h, fam); \
        prof_begin(L, fam);         \
        int rc2__ = (expr);         \
        prof_end(L);                \
        if (rc2__ != DFLASH_OK) return rc2__; \
    } while (0)

static int check_ws(const dflash_handle* h, void* ws, int64_t bytes, int batch, int rows, Workspace* out) {
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255)) return DFLASH_ERR_WORKSPACE;
    *out = carve(h, ws, batch, rows);
    if (out->bytes > bytes) return DFLASH_ERR_WORKSPACE;
    return DFLASH_OK;
}

static int zero_counters(const Launch& L, const Workspace& ws) {
    if (L.h->cfg.dtype != DFLASH_BF16) return DFLASH_OK;
    return launch_zero(L, ws.counters, ws.counter_bytes);      // counter_bytes is a multiple of 256
}

// LM head + argmax over `rows` normalised rows z (config dtype)
// (bf16 path: if ssq_in is given, z holds gain-scaled rows and the per-token rsqrt is applied inside)
static int lmhead_rows(Launch& L, const Workspace& ws, const void* z, const float* ssq_in, int rows, int32_t* ids,
                       float* top1, float* margin, float* logits_out) {
    const dflash_config& c = L.h->cfg;
    if (c.dtype == DFLASH_BF16) {
        GemmArgs g{};
        g.X = z; g.W[0] = L.h->w.W_lm; g.M = rows; g.N = c.vocab; g.K = c.d_model;
        g.epilogue = EPI_ARGMAX; g.part = ws.part; g.counters = ws.counters + ws.cnt_off[Workspace::CNT_LM]; g.ssq_in = ssq_in;
        g.top2 = (Top2Entry*)ws.top2; g.logits_out = logits_out;
        RUN(FAM_LMHEAD, launch_gemm_tc(L, g, ws.flags + GEMM_MAX_PHASES * (ws.n_flag_sets - 1)));
        RUN(FAM_ARGMAX_FINISH, launch_argmax_finish(L, (const Top2Entry*)ws.top2, (c.vocab + 127) / 128, rows, ids, top1, margin));
        return DFLASH_OK;
    }
    const int es = elem_size(c.dtype);
    for (int r0 = 0; r0 < rows; r0 += LOGIT_ROWS) {
        const int n = std::min(LOGIT_ROWS, rows - r0);
        float* lg = logits_out ? logits_out + (size_t)r0 * c.vocab : ws.logits;
        RUN(FAM_LMHEAD, launch_gemm_simt(L, (const char*)z + (size_t)r0 * c.d_model * es, L.h->w.W_lm, lg, n, c.vocab,
                                         c.d_model, false));
        RUN(FAM_ROW_ARGMAX, launch_row_argmax(L, lg, DFLASH_F32, c.vocab, n, c.vocab, ws.seg, ids + r0, top1 ? top1 + r0 : nullptr,
                                              margin ? margin + r0 : nullptr));
    }
    return DFLASH_OK;
}

extern "C" {

const char* dflash_status_string(int32_t code) {
    switch (code) {
        case DFLASH_OK: return "ok";
        case DFLASH_ERR_INVALID_ARG: return "invalid argument";
        case DFLASH_ERR_UNSUPPORTED: return "unsupported shape or dtype";
        case DFLASH_ERR_WORKSPACE: return "workspace too small or misaligned";
        case DFLASH_ERR_CUDA: return "CUDA launch failed";
        case DFLASH_ERR_NOT_READY: return "weights not set";
        default: return "unknown status";
    }
}

const char* dflash_family_name(int32_t f) { return (f >= 0 && f < DFLASH_N_FAMILIES) ? kFamilyNames[f] : "?"; }

int64_t dflash_launch_count(void) { return (int64_t)g_launches; }

int32_t dflash_create(const dflash_config* cfg, dflash_handle** out) {
    if (!cfg || !out) return DFLASH_ERR_INVALID_ARG;
    *out = nullptr;
    const dflash_config& c = *cfg;
    if (c.n_layers < 1 || c.d_model < 1 || c.n_q_heads < 1 || c.n_kv_heads < 1 || c.head_dim < 1 ||
        c.d_ffn < 1 || c.vocab < 2 || c.n_feat_layers < 1 || c.d_target < 1 || c.block_size < 1 ||
        c.page_size < 1 || !(c.rms_eps >= 0.f) || !(c.softmax_scale > 0.f))
        return DFLASH_ERR_INVALID_ARG;
    if (c.mask_token_id < 0 || c.mask_token_id >= c.vocab) return DFLASH_ERR_INVALID_ARG;
    if (c.qk_norm != 0 && c.qk_norm != 1) return DFLASH_ERR_INVALID_ARG;
    if (c.dtype != DFLASH_F32 && c.dtype != DFLASH_BF16) return DFLASH_ERR_UNSUPPORTED;
    if (c.n_layers > DFLASH_MAX_LAYERS) return DFLASH_ERR_UNSUPPORTED;
    if (c.head_dim != 64 && c.head_dim != 128) return DFLASH_ERR_UNSUPPORTED;
    if (c.n_q_heads % c.n_kv_heads != 0) return DFLASH_ERR_UNSUPPORTED;
    if (c.block_size > 32) return DFLASH_ERR_UNSUPPORTED;
    if (!is_pow2(c.page_size) || c.page_size > 256) return DFLASH_ERR_UNSUPPORTED;
    if (c.d_model % 8 || c.d_ffn % 8 || (c.n_feat_layers * c.d_target) % 8) return DFLASH_ERR_UNSUPPORTED;
    // the bf16 epilogues pair rows of whole heads inside a 128-row weight tile
    if (c.dtype == DFLASH_BF16 && ((c.n_q_heads * c.head_dim) % 128 || (c.n_kv_heads * c.head_dim) % 128))
        return DFLASH_ERR_UNSUPPORTED;
    dflash_handle* h = new (std::nothrow) dflash_handle();
    if (!h) return DFLASH_ERR_INVALID_ARG;
    h->cfg = c;
    h->wmaps = new (std::nothrow) dflash_wmap_entry[DFLASH_WMAP_CACHE];
    h->n_wmaps = 0;
    if (!h->wmaps) { delete h; return DFLASH_ERR_INVALID_ARG; }
    h->has_weights = false;
    // SMs of the current device (grids of one CTA per SM, split heuristics and the partial-tile workspace follow
    // it); without a device - sizing queries on a host with no GPU - the B200's count
    h->sm_count = 148;
    {
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0)
            h->sm_count = n;
        else
            (void)cudaGetLastError();
    }
    h->prof_on = false;
    h->prof = nullptr;
    h->prof_cap = h->prof_used = 0;
    h->trace_buf = nullptr;
    h->trace_cap = h->trace_used = 0;
    h->trace_fam = nullptr;
    *out = h;
    return DFLASH_OK;
}

void dflash_destroy(dflash_handle* h) {
    if (!h) return;
    for (int i = 0; i < h->prof_cap; ++i) {
        cudaEventDestroy(h->prof[i].e0);
        cudaEventDestroy(h->prof[i].e1);
    }
    delete[] h->prof;
    delete[] h->trace_fam;
    delete[] h->wmaps;
    delete h;
}

int32_t dflash_profile_enable(dflash_handle* h, int32_t on) {
    if (!h) return DFLASH_ERR_INVALID_ARG;
    h->prof_on = on != 0;
    return DFLASH_OK;
}

int32_t dflash_profile_read(dflash_handle* h, float* ms, int32_t* launches) {
    if (!h || !ms || !launches) return DFLASH_ERR_INVALID_ARG;
    if (h->prof_used > 0 && cudaEventSynchronize(h->prof[h->prof_used - 1].e1) != cudaSuccess) return DFLASH_ERR_CUDA;
    for (int i = 0; i < h->prof_used; ++i) {
        float t = 0.f;
        if (cudaEventElapsedTime(&t, h->prof[i].e0, h->prof[i].e1) != cudaSuccess) return DFLASH_ERR_CUDA;
        ms[h->prof[i].family] += t;
        launches[h->prof[i].family] += 1;
    }
    h->prof_used = 0;
    return DFLASH_OK;
}

int32_t dflash_trace_enable(dflash_handle* h, uint64_t* dev_buf, int32_t capacity_records) {
    if (!h || capacity_records < 0) return DFLASH_ERR_INVALID_ARG;
    delete[] h->trace_fam;
    h->trace_fam = nullptr;
    h->trace_buf = nullptr;
    h->trace_cap = h->trace_used = 0;
    if (dev_buf && capacity_records > 0) {
        h->trace_fam = new (std::nothrow) int[capacity_records];
        if (!h->trace_fam) return DFLASH_ERR_INVALID_ARG;
        h->trace_buf = reinterpret_cast<unsigned long long*>(dev_buf);
        h->trace_cap = capacity_records;
    }
    return DFLASH_OK;
}

int32_t dflash_trace_read(dflash_handle* h, int32_t* families, int32_t* n_records) {
    if (!h || !families || !n_records) return DFLASH_ERR_INVALID_ARG;
    for (int i = 0; i < h->trace_used; ++i) families[i] = h->trace_fam[i];
    *n_records = h->trace_used;
    h->trace_used = 0;
    return DFLASH_OK;
}

int32_t dflash_set_weights(dflash_handle* h, const dflash_weights* w) {
    if (!h || !w || !w->layers) return DFLASH_ERR_INVALID_ARG;
    if (!w->embed || !w->W_c || !w->g_c || !w->g_f || !w->W_lm) return DFLASH_ERR_INVALID_ARG;
    if (h->cfg.use_rope && (!w->rope_cos || !w->rope_sin || w->rope_max_pos < 1)) return DFLASH_ERR_INVALID_ARG;
    for (int i = 0; i < h->cfg.n_layers; ++i) {
        const dflash_layer_weights& l = w->layers[i];
        if (!l.g1 || !l.W_qkv || !l.W_o || !l.g2 || !l.W_gateup || !l.W_down) return DFLASH_ERR_INVALID_ARG;
        if (h->cfg.qk_norm && (!l.g_q || !l.g_k)) return DFLASH_ERR_INVALID_ARG;
        h->layers[i] = l;
    }
    h->w = *w;
    h->w.layers = h->layers;
    h->n_wmaps = 0;      // maps of the previous weights are stale
    h->has_weights = true;
    return DFLASH_OK;
}

int64_t dflash_workspace_bytes(const dflash_handle* h, int32_t max_batch, int32_t max_rows) {
    if (!h || max_batch < 0 || max_rows < 0) return DFLASH_ERR_INVALID_ARG;
    return carve(h, nullptr, max_batch, max_rows).bytes;
}

int32_t dflash_ctx_project(dflash_handle* h, const dflash_ctx_args* a, void* stream) {
    if (!h || !a) return DFLASH_ERR_INVALID_ARG;
    if (!h->has_weights) return DFLASH_ERR_NOT_READY;
    if (a->batch < 0 || a->max_new < 0 || a->max_pages < 1 || a->n_pool_pages < 1) return DFLASH_ERR_INVALID_ARG;
    const int64_t rows64 = (int64_t)a->batch * a->max_new;
    if (rows64 > (1 << 24)) return DFLASH_ERR_UNSUPPORTED;
    const int rows = (int)rows64;
    if (rows == 0) return DFLASH_OK;
    if (!a->feats || !a->ctx_len || !a->page_table || !a->kv_pool) return DFLASH_ERR_INVALID_ARG;
    Workspace ws;
    DFLASH_TRY(check_ws(h, a->workspace, a->workspace_bytes, a->batch, rows, &ws));
    const dflash_config& c = h->cfg;
    Launch L{h, (cudaStream_t)stream, a->dev_status, nullptr};
    const int kdim = c.n_kv_heads * c.head_dim, feat = c.n_feat_layers * c.d_target;
    const bool tc = c.dtype == DFLASH_BF16;
    DFLASH_TRY(zero_counters(L, ws));
    // y = W_c [h^(l1); ...; h^(lk)]  ->  H_t = RMSNorm(y)  ->  per layer K = RoPE(W^K H_t), V = W^V H_t
    const size_t kv_off = (size_t)c.n_q_heads * c.head_dim * c.d_model * elem_size(c.dtype);   // rows Hq*hd.. of W_qkv
    if (tc) {
        // the norm is folded: the first contraction emits g_c*y (bf16) and sums of squares, the second
        // scales its accumulator by the per-token rsqrt
        GemmArgs g{};
        g.X = a->feats; g.W[0] = h->w.W_c; g.M = rows; g.N = c.d_model; g.K = feat;
        g.epilogue = EPI_STORE_F32; g.g_next = h->w.g_c; g.xn_out = (__nv_bfloat16*)ws.u; g.ssq_out = ws.ssq;
        g.part = ws.part; g.counters = ws.counters + ws.cnt_off[Workspace::CNT_FUSE];
        int flag_set = 0;
        bool fused_done = false;
        for (int i0 = 0; i0 < c.n_layers; i0 += GEMM_MAX_GROUPS - 1) {
            GemmArgs k{};
            k.n_groups = std::min(GEMM_MAX_GROUPS - 1, c.n_layers - i0);
            for (int j = 0; j < k.n_groups; ++j) {
                k.W[j] = (const char*)h->layers[i0 + j].W_qkv + kv_off;
                k.g_k_group[j] = c.qk_norm ? h->layers[i0 + j].g_k : nullptr;
            }
            k.X = ws.u; k.M = rows; k.N = 2 * kdim; k.K = c.d_model; k.ssq_in = ws.ssq;
            k.epilogue = EPI_CTX_KV; k.ctx = a; k.first_layer = i0; k.part = ws.part;
            k.counters = ws.counters + ws.cnt_off[Workspace::CNT_KV] + (int64_t)i0 * (gemm_tc_counter_bytes(rows, 2 * kdim, 1) / 4);
            if (flag_set >= ws.n_flag_sets - 1) return DFLASH_ERR_UNSUPPORTED;
            if (!fused_done) {
                // one launch: the fusion contraction, then the K/V contractions of the first layers as its second phase
                GemmArgs ph[2] = {g, k};
                unsigned long long* tr[2] = {trace_slot(h, FAM_CTX_FUSE), trace_slot(h, FAM_CTX_KV)};
                prof_begin(L, FAM_GEMM_CHAIN);
                const int rc = launch_gemm_chain(L, ph, 2, ws.flags + GEMM_MAX_PHASES * flag_set++, tr);
                prof_end(L);
                if (rc != DFLASH_OK) return rc;
                fused_done = true;
            } else {
                RUN(FAM_CTX_KV, launch_gemm_tc(L, k, ws.flags + GEMM_MAX_PHASES * flag_set++));
            }
        }
        return DFLASH_OK;
    }
    RUN(FAM_CTX_FUSE, launch_gemm_simt(L, a->feats, h->w.W_c, ws.tmp, rows, c.d_model, feat, false));
    RUN(FAM_RMSNORM, launch_rmsnorm(L, ws.tmp, true, h->w.g_c, true, ws.u, rows, c.d_model));
    for (int i = 0; i < c.n_layers; ++i) {
        const char* Wkv = (const char*)h->layers[i].W_qkv + kv_off;
        RUN(FAM_CTX_KV, launch_gemm_simt(L, ws.u, Wkv, ws.tmp, rows, 2 * kdim, c.d_model, false));
        RUN(FAM_CTX_KV, launch_ctx_scatter(L, ws.tmp, *a, i, c.qk_norm ? h->layers[i].g_k : nullptr));
    }
    return DFLASH_OK;
}

}  // extern "C"

// One pass of a stack of pre-norm layers over `rows_per_seq` rows per sequence on top of a paged KV
// cache: the draft block (row 0 = anchor, the rest mask tokens, no mask inside the block) and the
// target's verify pass (given tokens, causal inside the block, block K/V written behind the committed
// context, hidden states of chosen layers tapped) are the same launches with different options.
struct BlockRun {
    const int32_t* anchor_ids;   // draft: token of row 0 of each sequence (rows 1.. embed the mask token)
    const int32_t* token_ids;    // verify: token of every row [batch * rows_per_seq]; overrides anchor_ids
    int batch, rows_per_seq, causal;
    const int32_t* ctx_len;
    int max_ctx_len;
    const int32_t* page_table;
    int max_pages;
    const void* kv_pool;
    int n_pool_pages;
    bool commit_kv;              // write the block's K/V of every layer at positions L .. L + rows_per_seq - 1
    void* workspace;
    int64_t workspace_bytes;
    int32_t* ids;
    float *top1, *margin, *hidden_out, *logits_out;
    int32_t* dev_status;
    const int32_t* tap_layers;   // [host] ascending layer indices whose output rows go to feats_out
    int n_taps;
    void* feats_out;             // [batch * rows_per_seq, n_taps * D] config dtype
    const dflash_ctx_args* ctx;  // draft: context projection to run inside this call (chained with the first QKV), or nullptr
};

static int block_forward(dflash_handle* h, const BlockRun* a, void* stream) {
    const dflash_config& c = h->cfg;
    const int B = a->rows_per_seq, rows = a->batch * B;
    const bool tc = c.dtype == DFLASH_BF16;
    // A context projection handed in with the draft: fused into the first chained launch when its weight
    // maps fit one launch (fusion + one K/V group per layer + QKV), else run first as its own launches.
    const dflash_ctx_args* cx = a->ctx;
    if (cx && (cx->batch < 0 || cx->max_new < 0)) return DFLASH_ERR_INVALID_ARG;
    const int rows_ctx = cx ? cx->batch * cx->max_new : 0;
    if (cx && rows_ctx > 0 && (!cx->feats || !cx->ctx_len || !cx->page_table || !cx->kv_pool || cx->batch != a->batch ||
                               cx->max_pages < 1 || cx->n_pool_pages < 1))
        return DFLASH_ERR_INVALID_ARG;
    const bool fuse_ctx = tc && cx && rows_ctx > 0 && c.n_layers + 2 <= GEMM_MAX_GROUPS;
    if (cx && rows_ctx > 0 && !fuse_ctx) {
        dflash_ctx_args own = *cx;
        own.workspace = a->workspace; own.workspace_bytes = a->workspace_bytes;
        if (!own.dev_status) own.dev_status = a->dev_status;
        DFLASH_TRY(dflash_ctx_project(h, &own, stream));
    }
    Workspace ws;
    DFLASH_TRY(check_ws(h, a->workspace, a->workspace_bytes, a->batch, fuse_ctx ? std::max(rows, rows_ctx) : rows, &ws));
    Launch L{h, (cudaStream_t)stream, a->dev_status, nullptr};
    const int qdim = c.n_q_heads * c.head_dim, kdim = c.n_kv_heads * c.head_dim;
    DFLASH_TRY(zero_counters(L, ws));
    // after layer i: tapped hidden rows, and (verify) the block's K/V into the cache
    int next_tap = 0;
    auto after_attention = [&](int i) -> int {
        if (a->commit_kv) RUN(FAM_MISC, launch_kv_commit(L, ws.k_blk, ws.v_blk, a->batch, B, a->ctx_len, a->page_table, a->max_pages,
                                                         const_cast<void*>(a->kv_pool), a->n_pool_pages, i));
        return DFLASH_OK;
    };
    auto after_layer = [&](int i) -> int {
        if (next_tap < a->n_taps && a->tap_layers[next_tap] == i) {
            RUN(FAM_MISC, launch_tap_copy(L, ws.x, a->feats_out, rows, c.d_model, a->n_taps * c.d_model, next_tap * c.d_model));
            ++next_tap;
        }
        return DFLASH_OK;
    };

    dflash_attn_args at{};
    at.mode = a->causal ? DFLASH_ATTN_CAUSAL : DFLASH_ATTN_FULL;
    at.q = ws.q; at.k_blk = ws.k_blk; at.v_blk = ws.v_blk;
    at.batch = a->batch; at.rows = B;
    at.ctx_len = a->ctx_len; at.max_ctx_len = a->max_ctx_len;
    at.page_table = a->page_table; at.max_pages = a->max_pages;
    at.kv_pool = a->kv_pool; at.n_pool_pages = a->n_pool_pages;
    at.out = ws.attn;

    if (tc) {
        // bf16: tensor-core contractions with the norms folded into their epilogues.
        // ws.u always holds bf16(gain * x) of the rows about to be projected, ws.ssq their sums of squares.
        // Launches: embed | QKV_0 | attention_0 | [O_0, gate/up_0, down_0, QKV_1] | attention_1 | ... |
        //           [O_last, gate/up_last, down_last, LM head] | argmax finish. Each [...] is one chained launch
        //           that keeps the weight stream running across its phases.
        __nv_bfloat16* xn = (__nv_bfloat16*)ws.u;
        int flag_set = 0;
        auto qkv_args = [&](int i) {
            GemmArgs g{};      // q,k,v = W_qkv RMSNorm(x), rotated
            g.X = xn; g.W[0] = h->layers[i].W_qkv; g.M = rows; g.N = qdim + 2 * kdim; g.K = c.d_model; g.ssq_in = ws.ssq;
            g.epilogue = EPI_QKV_ROPE; g.q = (__nv_bfloat16*)ws.q; g.k = (__nv_bfloat16*)ws.k_blk;
            g.v = (__nv_bfloat16*)ws.v_blk; g.ctx_len = a->ctx_len; g.rows_per_seq = B;
            if (c.qk_norm) { g.g_q = h->layers[i].g_q; g.g_k = h->layers[i].g_k; }
            g.part = ws.part; g.counters = ws.counters + ws.cnt_off[Workspace::CNT_QKV] + i * ws.cnt_stride[Workspace::CNT_QKV];
            return g;
        };
        RUN(FAM_EMBED, launch_embed_norm(L, a->anchor_ids, a->token_ids, a->batch, B, ws.x, h->layers[0].g1, xn, ws.ssq));
        if (fuse_ctx) {
            // [context fusion, context K/V of every layer, QKV of layer 0] in one launch. The projection's
            // normalised operand and sums of squares live in buffers the draft only uses later (tmp, h).
            __nv_bfloat16* cxn = (__nv_bfloat16*)ws.tmp;
            float* cssq = (float*)ws.h;
            const int feat = c.n_feat_layers * c.d_target;
            const size_t kv_off = (size_t)qdim * c.d_model * elem_size(c.dtype);
            GemmArgs ph[3];
            GemmArgs& g = ph[0];
            g = GemmArgs{};
            g.X = cx->feats; g.W[0] = h->w.W_c; g.M = rows_ctx; g.N = c.d_model; g.K = feat;
            g.epilogue = EPI_STORE_F32; g.g_next = h->w.g_c; g.xn_out = cxn; g.ssq_out = cssq;
            g.part = ws.part; g.counters = ws.counters + ws.cnt_off[Workspace::CNT_FUSE];
            GemmArgs& k = ph[1];
            k = GemmArgs{};
            k.n_groups = c.n_layers;
            for (int j = 0; j < c.n_layers; ++j) {
                k.W[j] = (const char*)h->layers[j].W_qkv + kv_off;
                k.g_k_group[j] = c.qk_norm ? h->layers[j].g_k : nullptr;
            }
            k.X = cxn; k.M = rows_ctx; k.N = 2 * kdim; k.K = c.d_model; k.ssq_in = cssq;
            k.epilogue = EPI_CTX_KV; k.ctx = cx; k.first_layer = 0; k.part = ws.part;
            k.counters = ws.counters + ws.cnt_off[Workspace::CNT_KV];
            ph[2] = qkv_args(0);
            unsigned long long* tr[3] = {trace_slot(h, FAM_CTX_FUSE), trace_slot(h, FAM_CTX_KV), trace_slot(h, FAM_GEMM_QKV)};
            prof_begin(L, FAM_GEMM_CHAIN);
            const int rc = launch_gemm_chain(L, ph, 3, ws.flags + GEMM_MAX_PHASES * flag_set++, tr);
            prof_end(L);
            if (rc != DFLASH_OK) return rc;
        } else {
            const GemmArgs g = qkv_args(0);
            RUN(FAM_GEMM_QKV, launch_gemm_tc(L, g, ws.flags + GEMM_MAX_PHASES * flag_set++));
        }
        for (int i = 0; i < c.n_layers; ++i) {
            const dflash_layer_weights& lw = h->layers[i];
            const bool last = i + 1 == c.n_layers;
            at.layer = i;
            // layers after the first: the cache they read was final before this call's first attention ran
            // (not so in the verify pass, which writes the cache as it goes)
            if (attn_tc_supported(c, B)) RUN(FAM_ATTENTION, launch_attention_tc(L, at, ws.attn_part, ws.attn_counters, i > 0 && !a->commit_kv,
                                                                              fuse_ctx ? cx->ctx_len : nullptr));
            else RUN(FAM_ATTENTION, launch_attention_simt(L, at));
            DFLASH_TRY(after_attention(i));
            GemmArgs ph[4];
            int fam[4];
            GemmArgs& o = ph[0];      // x += W_o attn; emits the FFN norm inputs
            o = GemmArgs{};
            o.X = ws.attn; o.W[0] = lw.W_o; o.M = rows; o.N = c.d_model; o.K = qdim;
            o.epilogue = EPI_RESIDUAL; o.out_f32 = ws.x; o.ld_out = c.d_model; o.part = ws.part;
            o.counters = ws.counters + ws.cnt_off[Workspace::CNT_O] + i * ws.cnt_stride[Workspace::CNT_O];
            o.g_next = lw.g2; o.xn_out = xn; o.ssq_out = ws.ssq;
            fam[0] = FAM_GEMM_O;
            GemmArgs& u = ph[1];      // h = silu(W_gate u) * (W_up u)
            u = GemmArgs{};
            u.X = xn; u.W[0] = lw.W_gateup; u.M = rows; u.N = 2 * c.d_ffn; u.K = c.d_model; u.ssq_in = ws.ssq;
            u.epilogue = EPI_SWIGLU; u.h = (__nv_bfloat16*)ws.h; u.part = ws.part;
            u.counters = ws.counters + ws.cnt_off[Workspace::CNT_GATEUP] + i * ws.cnt_stride[Workspace::CNT_GATEUP];
            fam[1] = FAM_GEMM_GATEUP;
            GemmArgs& d = ph[2];      // x += W_down h; emits the next layer's (or the final) norm inputs
            d = GemmArgs{};
            d.X = ws.h; d.W[0] = lw.W_down; d.M = rows; d.N = c.d_model; d.K = c.d_ffn;
            d.epilogue = EPI_RESIDUAL; d.out_f32 = ws.x; d.ld_out = c.d_model; d.part = ws.part;
            d.counters = ws.counters + ws.cnt_off[Workspace::CNT_DOWN] + i * ws.cnt_stride[Workspace::CNT_DOWN];
            d.g_next = last ? h->w.g_f : h->layers[i + 1].g1; d.xn_out = xn; d.ssq_out = ws.ssq;
            fam[2] = FAM_GEMM_DOWN;
            if (!last) {
                ph[3] = qkv_args(i + 1);
                fam[3] = FAM_GEMM_QKV;
            } else {              // LM head on the final-normed rows, fused with the per-tile argmax
                GemmArgs& g = ph[3];
                g = GemmArgs{};
                g.X = xn; g.W[0] = h->w.W_lm; g.M = rows; g.N = c.vocab; g.K = c.d_model; g.ssq_in = ws.ssq;
                g.epilogue = EPI_ARGMAX; g.part = ws.part; g.counters = ws.counters + ws.cnt_off[Workspace::CNT_LM];
                g.top2 = (Top2Entry*)ws.top2; g.logits_out = a->logits_out;
                fam[3] = FAM_LMHEAD;
            }
            unsigned long long* tr[4];
            for (int k = 0; k < 4; ++k) tr[k] = trace_slot(h, fam[k]);
            if (flag_set >= ws.n_flag_sets - 1) return DFLASH_ERR_UNSUPPORTED;
            prof_begin(L, FAM_GEMM_CHAIN);
            const int rc = launch_gemm_chain(L, ph, 4, ws.flags + GEMM_MAX_PHASES * flag_set++, tr);
            prof_end(L);
            if (rc != DFLASH_OK) return rc;
            DFLASH_TRY(after_layer(i));      // x is final for layer i after the chain's third phase; the fourth does not touch it
        }
        RUN(FAM_ARGMAX_FINISH, launch_argmax_finish(L, (const Top2Entry*)ws.top2, (c.vocab + 127) / 128, rows, a->ids,
                                                    a->top1, a->margin));
        if (a->hidden_out) RUN(FAM_MISC, launch_copy_f32(L, ws.x, a->hidden_out, (int64_t)rows * c.d_model));
        return DFLASH_OK;
    }

    // fp32: CUDA-core kernels, one step per launch
    RUN(FAM_EMBED, launch_embed(L, a->anchor_ids, a->token_ids, ws.x, a->batch, B));
    for (int i = 0; i < c.n_layers; ++i) {
        const dflash_layer_weights& lw = h->layers[i];
        // attention half: u = RMSNorm(x); q,k,v = W u (+RoPE); x += W_o attention(q, [K_ctx; k], [V_ctx; v])
        RUN(FAM_RMSNORM, launch_rmsnorm(L, ws.x, true, lw.g1, true, ws.u, rows, c.d_model));
        RUN(FAM_GEMM_QKV, launch_gemm_simt(L, ws.u, lw.W_qkv, ws.tmp, rows, qdim + 2 * kdim, c.d_model, false));
        RUN(FAM_GEMM_QKV, launch_rope_split(L, ws.tmp, a->ctx_len, B, rows, ws.q, ws.k_blk, ws.v_blk, c.qk_norm ? lw.g_q : nullptr,
                                                c.qk_norm ? lw.g_k : nullptr));
        at.layer = i;
        RUN(FAM_ATTENTION, launch_attention_simt(L, at));
        DFLASH_TRY(after_attention(i));
        RUN(FAM_GEMM_O, launch_gemm_simt(L, ws.attn, lw.W_o, ws.x, rows, c.d_model, qdim, true));
        // FFN half: u = RMSNorm(x); x += W_down (silu(W_gate u) * W_up u)
        RUN(FAM_RMSNORM, launch_rmsnorm(L, ws.x, true, lw.g2, true, ws.u, rows, c.d_model));
        RUN(FAM_GEMM_GATEUP, launch_gemm_simt(L, ws.u, lw.W_gateup, ws.tmp, rows, 2 * c.d_ffn, c.d_model, false));
        RUN(FAM_GEMM_GATEUP, launch_swiglu(L, ws.tmp, ws.h, rows));
        RUN(FAM_GEMM_DOWN, launch_gemm_simt(L, ws.h, lw.W_down, ws.x, rows, c.d_model, c.d_ffn, true));
        DFLASH_TRY(after_layer(i));
    }
    if (a->hidden_out) RUN(FAM_MISC, launch_copy_f32(L, ws.x, a->hidden_out, (int64_t)rows * c.d_model));
    RUN(FAM_RMSNORM, launch_rmsnorm(L, ws.x, true, h->w.g_f, true, ws.u, rows, c.d_model));
    return lmhead_rows(L, ws, ws.u, nullptr, rows, a->ids, a->top1, a->margin, a->logits_out);
}

extern "C" {

int32_t dflash_draft_block(dflash_handle* h, const dflash_draft_args* a, void* stream) {
    if (!h || !a) return DFLASH_ERR_INVALID_ARG;
    if (!h->has_weights) return DFLASH_ERR_NOT_READY;
    if (a->batch < 0 || a->max_pages < 1 || a->n_pool_pages < 1 || a->max_ctx_len < 0) return DFLASH_ERR_INVALID_ARG;
    if (a->batch == 0) return DFLASH_OK;
    if (!a->anchor_ids || !a->ctx_len || !a->page_table || !a->kv_pool || !a->draft_ids) return DFLASH_ERR_INVALID_ARG;
    const dflash_config& c = h->cfg;
    if ((int64_t)a->batch * c.block_size > (1 << 20)) return DFLASH_ERR_UNSUPPORTED;
    if (a->block_rows < 0 || a->block_rows > c.block_size) return DFLASH_ERR_INVALID_ARG;
    BlockRun r{};
    r.anchor_ids = a->anchor_ids;
    r.batch = a->batch; r.rows_per_seq = a->block_rows > 0 ? a->block_rows : c.block_size; r.causal = 0;
    r.ctx_len = a->ctx_len; r.max_ctx_len = a->max_ctx_len; r.page_table = a->page_table; r.max_pages = a->max_pages;
    r.kv_pool = a->kv_pool; r.n_pool_pages = a->n_pool_pages;
    r.workspace = a->workspace; r.workspace_bytes = a->workspace_bytes;
    r.ids = a->draft_ids; r.top1 = a->top1; r.margin = a->margin; r.hidden_out = a->hidden_out; r.logits_out = a->logits_out;
    r.dev_status = a->dev_status;
    r.ctx = a->ctx;
    return block_forward(h, &r, stream);
}

int32_t dflash_target_verify(dflash_handle* h, const dflash_target_args* a, void* stream) {
    if (!h || !a) return DFLASH_ERR_INVALID_ARG;
    if (!h->has_weights) return DFLASH_ERR_NOT_READY;
    if (a->batch < 0 || a->rows < 1 || a->rows > 32 || a->max_pages < 1 || a->n_pool_pages < 1 || a->max_ctx_len < 0 ||
        a->n_taps < 0 || a->n_taps > DFLASH_MAX_LAYERS)
        return DFLASH_ERR_INVALID_ARG;
    if (a->batch == 0) return DFLASH_OK;
    if (!a->token_ids || !a->ctx_len || !a->page_table || !a->kv_pool || !a->ids_out) return DFLASH_ERR_INVALID_ARG;
    if (a->n_taps > 0 && (!a->tap_layers || !a->feats_out)) return DFLASH_ERR_INVALID_ARG;
    for (int t = 0; t < a->n_taps; ++t)
        if (a->tap_layers[t] < 0 || a->tap_layers[t] >= h->cfg.n_layers || (t > 0 && a->tap_layers[t] <= a->tap_layers[t - 1]))
            return DFLASH_ERR_INVALID_ARG;
    if ((int64_t)a->batch * a->rows > (1 << 20)) return DFLASH_ERR_UNSUPPORTED;
    BlockRun r{};
    r.token_ids = a->token_ids;
    r.batch = a->batch; r.rows_per_seq = a->rows; r.causal = 1;
    r.ctx_len = a->ctx_len; r.max_ctx_len = a->max_ctx_len; r.page_table = a->page_table; r.max_pages = a->max_pages;
    r.kv_pool = a->kv_pool; r.n_pool_pages = a->n_pool_pages; r.commit_kv = true;
    r.workspace = a->workspace; r.workspace_bytes = a->workspace_bytes;
    r.ids = a->ids_out; r.logits_out = a->logits_out; r.dev_status = a->dev_status;
    r.tap_layers = a->tap_layers; r.n_taps = a->n_taps; r.feats_out = a->feats_out;
    return block_forward(h, &r, stream);
}

int32_t dflash_verify_accept(dflash_handle* h, const dflash_verify_args* a, void* stream) {
    if (!h || !a) return DFLASH_ERR_INVALID_ARG;
    if (a->batch < 0 || a->gamma < 1 || a->gamma > 64 || a->draft_stride < a->gamma) return DFLASH_ERR_INVALID_ARG;
    if (a->batch == 0) return DFLASH_OK;
    if (!a->draft_ids || !a->ctx_len || !a->accept_len || !a->out_tokens || !a->bonus || !a->new_ctx_len)
        return DFLASH_ERR_INVALID_ARG;
    Launch L{h, (cudaStream_t)stream, a->dev_status, nullptr};
    const int rows = a->batch * (a->gamma + 1);
    if (a->mode == DFLASH_VERIFY_IDS) {
        if (!a->target_ids) return DFLASH_ERR_INVALID_ARG;
        RUN(FAM_ACCEPT, launch_accept(L, *a, a->target_ids));
        return DFLASH_OK;
    }
    if (a->mode != DFLASH_VERIFY_LOGITS) return DFLASH_ERR_INVALID_ARG;
    if (!a->logits || a->vocab < 2) return DFLASH_ERR_INVALID_ARG;
    if (a->logits_dtype != DFLASH_F32 && a->logits_dtype != DFLASH_BF16) return DFLASH_ERR_UNSUPPORTED;
    const int64_t stride = a->logits_row_stride ? a->logits_row_stride : a->vocab;
    if (stride < a->vocab) return DFLASH_ERR_INVALID_ARG;
    Workspace ws;
    DFLASH_TRY(check_ws(h, a->workspace, a->workspace_bytes, a->batch, rows, &ws));
    RUN(FAM_ROW_ARGMAX, launch_verify_logits(L, *a, stride, ws.seg));
    return DFLASH_OK;
}

int32_t dflash_block_attention(dflash_handle* h, const dflash_attn_args* a, void* stream) {
    if (!h || !a) return DFLASH_ERR_INVALID_ARG;
    if (a->batch < 0 || a->rows < 0 || a->rows > 32 || a->max_pages < 1 || a->n_pool_pages < 1 ||
        a->layer < 0 || a->layer >= h->cfg.n_layers || a->max_ctx_len < 0)
        return DFLASH_ERR_INVALID_ARG;
    if (a->mode != DFLASH_ATTN_FULL && a->mode != DFLASH_ATTN_CAUSAL) return DFLASH_ERR_INVALID_ARG;
    if (a->batch == 0 || a->rows == 0) return DFLASH_OK;
    if (!a->q || !a->k_blk || !a->v_blk || !a->ctx_len || !a->page_table || !a->kv_pool || !a->out)
        return DFLASH_ERR_INVALID_ARG;
    Launch L{h, (cudaStream_t)stream, a->dev_status, nullptr};
    if (attn_tc_supported(h->cfg, a->rows)) {
        Workspace ws;
        DFLASH_TRY(check_ws(h, a->workspace, a->workspace_bytes, a->batch, a->batch * a->rows, &ws));
        RUN(FAM_ATTENTION, launch_attention_tc(L, *a, ws.attn_part, ws.attn_counters, false, nullptr, true));
    } else {
        RUN(FAM_ATTENTION, launch_attention_simt(L, *a));
    }
    return DFLASH_OK;
}

int32_t dflash_block_attention_bwd(dflash_handle* h, const dflash_attn_bwd_args* a, void* stream) {
    if (!h || !a) return DFLASH_ERR_INVALID_ARG;
    if (a->batch < 0 || a->rows < 0 || a->rows > 32 || a->max_pages < 1 || a->n_pool_pages < 1 || a->layer < 0 ||
        a->layer >= h->cfg.n_layers || a->max_ctx_len < 0)
        return DFLASH_ERR_INVALID_ARG;
    if (a->mode != DFLASH_ATTN_FULL && a->mode != DFLASH_ATTN_CAUSAL) return DFLASH_ERR_INVALID_ARG;
    if (a->batch == 0 || a->rows == 0) return DFLASH_OK;
    if (!a->q || !a->k_blk || !a->v_blk || !a->out || !a->lse || !a->dout || !a->ctx_len || !a->page_table || !a->kv_pool ||
        !a->dq || !a->dk_blk || !a->dv_blk)
        return DFLASH_ERR_INVALID_ARG;
    if ((int64_t)a->batch * a->rows > (1 << 20)) return DFLASH_ERR_UNSUPPORTED;
    if (!attn_bwd_supported(h->cfg, a->rows)) return DFLASH_ERR_UNSUPPORTED;
    Workspace ws;
    DFLASH_TRY(check_ws(h, a->workspace, a->workspace_bytes, a->batch, a->batch * a->rows, &ws));
    Launch L{h, (cudaStream_t)stream, a->dev_status, nullptr};
    // ws.tmp holds rows * d_model floats: room for one float per (row, q head)
    RUN(FAM_ATTENTION, launch_attention_bwd(L, *a, ws.tmp));
    return DFLASH_OK;
}

int32_t dflash_gemm_plan_check(int32_t M, int32_t N, int32_t K, int32_t n_groups, int32_t sm_count, int32_t pair_cap,
                               int32_t cluster_cap, int32_t* info) {
    return dflash::gemm_plan_check(M, N, K, n_groups, sm_count, pair_cap, cluster_cap, info);
}

int32_t dflash_attention_plan(const dflash_handle* h, int32_t batch, int32_t max_ctx_len, int64_t* out) {
    if (!h || !out || batch < 1 || max_ctx_len < 0) return DFLASH_ERR_INVALID_ARG;
    const AttnPlan pl = attn_tc_plan(h->cfg, batch, max_ctx_len, h->sm_count);
    out[0] = pl.tiles_per_unit; out[1] = pl.n_chunks; out[2] = pl.units; out[3] = pl.capacity_units;
    return DFLASH_OK;
}

int32_t dflash_lmhead_argmax(dflash_handle* h, const dflash_lmhead_args* a, void* stream) {
    if (!h || !a) return DFLASH_ERR_INVALID_ARG;
    if (!h->has_weights) return DFLASH_ERR_NOT_READY;
    if (a->n_rows < 0) return DFLASH_ERR_INVALID_ARG;
    if (a->n_rows == 0) return DFLASH_OK;
    if (!a->hidden || !a->ids) return DFLASH_ERR_INVALID_ARG;
    if (a->n_rows > (1 << 20)) return DFLASH_ERR_UNSUPPORTED;
    Workspace ws;
    DFLASH_TRY(check_ws(h, a->workspace, a->workspace_bytes, 1, a->n_rows, &ws));
    Launch L{h, (cudaStream_t)stream, a->dev_status, nullptr};
    const dflash_config& c = h->cfg;
    const bool f32in = a->hidden_is_f32 || c.dtype == DFLASH_F32;
    DFLASH_TRY(zero_counters(L, ws));
    RUN(FAM_RMSNORM, launch_rmsnorm(L, a->hidden, f32in, h->w.g_f, a->apply_norm != 0, ws.u, a->n_rows, c.d_model));
    return lmhead_rows(L, ws, ws.u, nullptr, a->n_rows, a->ids, a->top1, a->margin, a->logits_out);
}

}  // extern "C"
