// C ABI of the library: argument validation, workspace carving and the launch sequence of each call.
#include "dflash_internal.h"

#include <algorithm>
#include <cstring>
#include <new>

using namespace dflash;

namespace dflash {

Workspace carve(const dflash_config& c, void* base, int batch, int rows) {
    Arena a(base);
    Workspace w{};
    const int es = elem_size(c.dtype);
    const int64_t R = std::max(rows, 1);
    const int qdim = c.n_q_heads * c.head_dim, kdim = c.n_kv_heads * c.head_dim;
    const int64_t wide = std::max<int64_t>(std::max<int64_t>(qdim + 2 * kdim, 2 * (int64_t)c.d_ffn),
                                           (int64_t)c.d_model);
    w.x = (float*)a.take(R * c.d_model * 4);
    w.u = a.take(R * std::max(c.d_model, qdim) * es);
    w.tmp = (float*)a.take(R * wide * 4);
    w.q = a.take(R * qdim * es);
    w.k_blk = a.take(R * kdim * es);
    w.v_blk = a.take(R * kdim * es);
    w.attn = a.take(R * qdim * es);
    w.h = a.take(R * c.d_ffn * es);
    w.logits = (float*)a.take(std::min<int64_t>(R, LOGIT_ROWS) * c.vocab * 4);
    w.ids = (int32_t*)a.take(R * 4);
    w.part = (float*)a.take(256);
    (void)batch;
    w.bytes = a.off;
    return w;
}

}  // namespace dflash

static bool is_pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }

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
    if (c.dtype != DFLASH_F32 && c.dtype != DFLASH_BF16) return DFLASH_ERR_UNSUPPORTED;
    if (c.n_layers > DFLASH_MAX_LAYERS) return DFLASH_ERR_UNSUPPORTED;
    if (c.head_dim != 64 && c.head_dim != 128) return DFLASH_ERR_UNSUPPORTED;
    if (c.n_q_heads % c.n_kv_heads != 0) return DFLASH_ERR_UNSUPPORTED;
    if (c.block_size > 32) return DFLASH_ERR_UNSUPPORTED;
    if (!is_pow2(c.page_size) || c.page_size > 256) return DFLASH_ERR_UNSUPPORTED;
    if (c.d_model % 8 || c.d_ffn % 8 || (c.n_feat_layers * c.d_target) % 8) return DFLASH_ERR_UNSUPPORTED;
    dflash_handle* h = new (std::nothrow) dflash_handle();
    if (!h) return DFLASH_ERR_INVALID_ARG;
    h->cfg = c;
    h->has_weights = false;
    h->sm_count = 148;
    *out = h;
    return DFLASH_OK;
}

void dflash_destroy(dflash_handle* h) { delete h; }

int32_t dflash_set_weights(dflash_handle* h, const dflash_weights* w) {
    if (!h || !w || !w->layers) return DFLASH_ERR_INVALID_ARG;
    if (!w->embed || !w->W_c || !w->g_c || !w->g_f || !w->W_lm) return DFLASH_ERR_INVALID_ARG;
    if (h->cfg.use_rope && (!w->rope_cos || !w->rope_sin || w->rope_max_pos < 1)) return DFLASH_ERR_INVALID_ARG;
    for (int i = 0; i < h->cfg.n_layers; ++i) {
        const dflash_layer_weights& l = w->layers[i];
        if (!l.g1 || !l.W_qkv || !l.W_o || !l.g2 || !l.W_gateup || !l.W_down) return DFLASH_ERR_INVALID_ARG;
        h->layers[i] = l;
    }
    h->w = *w;
    h->w.layers = h->layers;
    h->has_weights = true;
    return DFLASH_OK;
}

int64_t dflash_workspace_bytes(const dflash_handle* h, int32_t max_batch, int32_t max_rows) {
    if (!h || max_batch < 0 || max_rows < 0) return DFLASH_ERR_INVALID_ARG;
    return carve(h->cfg, nullptr, max_batch, max_rows).bytes;
}

static int check_ws(const dflash_handle* h, void* ws, int64_t bytes, int batch, int rows, Workspace* out) {
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255)) return DFLASH_ERR_WORKSPACE;
    *out = carve(h->cfg, ws, batch, rows);
    if (out->bytes > bytes) return DFLASH_ERR_WORKSPACE;
    return DFLASH_OK;
}

#define DFLASH_TRY(expr)            \
    do {                            \
        int rc__ = (expr);          \
        if (rc__ != DFLASH_OK) return rc__; \
    } while (0)

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
    Launch L{h, (cudaStream_t)stream, a->dev_status};
    const int kdim = c.n_kv_heads * c.head_dim;
    // y = W_c [h^(l1); ...; h^(lk)]  ->  H_t = RMSNorm(y)
    DFLASH_TRY(launch_gemm_simt(L, a->feats, h->w.W_c, ws.tmp, rows, c.d_model, c.n_feat_layers * c.d_target, false));
    DFLASH_TRY(launch_rmsnorm(L, ws.tmp, true, h->w.g_c, true, ws.u, rows, c.d_model));
    for (int i = 0; i < c.n_layers; ++i) {
        // rows Hq*hd .. of W_qkv are W_i^K then W_i^V
        const char* Wkv = (const char*)h->layers[i].W_qkv + (size_t)c.n_q_heads * c.head_dim * c.d_model * elem_size(c.dtype);
        DFLASH_TRY(launch_gemm_simt(L, ws.u, Wkv, ws.tmp, rows, 2 * kdim, c.d_model, false));
        DFLASH_TRY(launch_ctx_scatter(L, ws.tmp, *a, i));
    }
    return DFLASH_OK;
}

static int lmhead_rows(const Launch& L, const Workspace& ws, const void* z, int rows, int32_t* ids, float* top1,
                       float* margin, float* logits_out) {
    const dflash_config& c = L.h->cfg;
    const int es = elem_size(c.dtype);
    for (int r0 = 0; r0 < rows; r0 += LOGIT_ROWS) {
        const int n = std::min(LOGIT_ROWS, rows - r0);
        float* lg = logits_out ? logits_out + (size_t)r0 * c.vocab : ws.logits;
        DFLASH_TRY(launch_gemm_simt(L, (const char*)z + (size_t)r0 * c.d_model * es, L.h->w.W_lm, lg, n, c.vocab,
                                    c.d_model, false));
        DFLASH_TRY(launch_row_argmax(L, lg, DFLASH_F32, c.vocab, n, c.vocab, ids + r0, top1 ? top1 + r0 : nullptr,
                                     margin ? margin + r0 : nullptr));
    }
    return DFLASH_OK;
}

int32_t dflash_draft_block(dflash_handle* h, const dflash_draft_args* a, void* stream) {
    if (!h || !a) return DFLASH_ERR_INVALID_ARG;
    if (!h->has_weights) return DFLASH_ERR_NOT_READY;
    if (a->batch < 0 || a->max_pages < 1 || a->n_pool_pages < 1 || a->max_ctx_len < 0) return DFLASH_ERR_INVALID_ARG;
    if (a->batch == 0) return DFLASH_OK;
    if (!a->anchor_ids || !a->ctx_len || !a->page_table || !a->kv_pool || !a->draft_ids) return DFLASH_ERR_INVALID_ARG;
    const dflash_config& c = h->cfg;
    if ((int64_t)a->batch * c.block_size > (1 << 20)) return DFLASH_ERR_UNSUPPORTED;
    const int B = c.block_size, rows = a->batch * B;
    Workspace ws;
    DFLASH_TRY(check_ws(h, a->workspace, a->workspace_bytes, a->batch, rows, &ws));
    Launch L{h, (cudaStream_t)stream, a->dev_status};
    const int qdim = c.n_q_heads * c.head_dim;

    DFLASH_TRY(launch_embed(L, a->anchor_ids, ws.x, a->batch));
    for (int i = 0; i < c.n_layers; ++i) {
        const dflash_layer_weights& lw = h->layers[i];
        DFLASH_TRY(launch_rmsnorm(L, ws.x, true, lw.g1, true, ws.u, rows, c.d_model));
        DFLASH_TRY(launch_gemm_simt(L, ws.u, lw.W_qkv, ws.tmp, rows, qdim + 2 * c.n_kv_heads * c.head_dim, c.d_model, false));
        DFLASH_TRY(launch_rope_split(L, ws.tmp, a->ctx_len, B, rows, ws.q, ws.k_blk, ws.v_blk));
        dflash_attn_args at{};
        at.mode = DFLASH_ATTN_FULL;
        at.q = ws.q; at.k_blk = ws.k_blk; at.v_blk = ws.v_blk;
        at.batch = a->batch; at.rows = B;
        at.ctx_len = a->ctx_len; at.max_ctx_len = a->max_ctx_len;
        at.page_table = a->page_table; at.max_pages = a->max_pages;
        at.kv_pool = a->kv_pool; at.n_pool_pages = a->n_pool_pages; at.layer = i;
        at.out = ws.attn;
        DFLASH_TRY(launch_attention_simt(L, at));
        DFLASH_TRY(launch_gemm_simt(L, ws.attn, lw.W_o, ws.x, rows, c.d_model, qdim, true));
        DFLASH_TRY(launch_rmsnorm(L, ws.x, true, lw.g2, true, ws.u, rows, c.d_model));
        DFLASH_TRY(launch_gemm_simt(L, ws.u, lw.W_gateup, ws.tmp, rows, 2 * c.d_ffn, c.d_model, false));
        DFLASH_TRY(launch_swiglu(L, ws.tmp, ws.h, rows));
        DFLASH_TRY(launch_gemm_simt(L, ws.h, lw.W_down, ws.x, rows, c.d_model, c.d_ffn, true));
    }
    if (a->hidden_out) DFLASH_TRY(launch_copy_f32(L, ws.x, a->hidden_out, (int64_t)rows * c.d_model));
    DFLASH_TRY(launch_rmsnorm(L, ws.x, true, h->w.g_f, true, ws.u, rows, c.d_model));
    DFLASH_TRY(lmhead_rows(L, ws, ws.u, rows, a->draft_ids, a->top1, a->margin, a->logits_out));
    return DFLASH_OK;
}

int32_t dflash_verify_accept(dflash_handle* h, const dflash_verify_args* a, void* stream) {
    if (!h || !a) return DFLASH_ERR_INVALID_ARG;
    if (a->batch < 0 || a->gamma < 1 || a->gamma > 64 || a->draft_stride < a->gamma) return DFLASH_ERR_INVALID_ARG;
    if (a->batch == 0) return DFLASH_OK;
    if (!a->draft_ids || !a->ctx_len || !a->accept_len || !a->out_tokens || !a->bonus || !a->new_ctx_len)
        return DFLASH_ERR_INVALID_ARG;
    Launch L{h, (cudaStream_t)stream, a->dev_status};
    const int rows = a->batch * (a->gamma + 1);
    if (a->mode == DFLASH_VERIFY_IDS) {
        if (!a->target_ids) return DFLASH_ERR_INVALID_ARG;
        return launch_accept(L, *a, a->target_ids);
    }
    if (a->mode != DFLASH_VERIFY_LOGITS) return DFLASH_ERR_INVALID_ARG;
    if (!a->logits || a->vocab < 2) return DFLASH_ERR_INVALID_ARG;
    if (a->logits_dtype != DFLASH_F32 && a->logits_dtype != DFLASH_BF16) return DFLASH_ERR_UNSUPPORTED;
    const int64_t stride = a->logits_row_stride ? a->logits_row_stride : a->vocab;
    if (stride < a->vocab) return DFLASH_ERR_INVALID_ARG;
    int32_t* ids = a->target_ids_out;
    if (!ids) {
        Workspace ws;
        DFLASH_TRY(check_ws(h, a->workspace, a->workspace_bytes, a->batch, rows, &ws));
        ids = ws.ids;
    }
    DFLASH_TRY(launch_row_argmax(L, a->logits, a->logits_dtype, stride, rows, a->vocab, ids, nullptr, nullptr));
    return launch_accept(L, *a, ids);
}

int32_t dflash_block_attention(dflash_handle* h, const dflash_attn_args* a, void* stream) {
    if (!h || !a) return DFLASH_ERR_INVALID_ARG;
    if (a->batch < 0 || a->rows < 0 || a->rows > 32 || a->max_pages < 1 || a->n_pool_pages < 1 ||
        a->layer < 0 || a->max_ctx_len < 0)
        return DFLASH_ERR_INVALID_ARG;
    if (a->mode != DFLASH_ATTN_FULL && a->mode != DFLASH_ATTN_CAUSAL) return DFLASH_ERR_INVALID_ARG;
    if (a->batch == 0 || a->rows == 0) return DFLASH_OK;
    if (!a->q || !a->k_blk || !a->v_blk || !a->ctx_len || !a->page_table || !a->kv_pool || !a->out)
        return DFLASH_ERR_INVALID_ARG;
    Launch L{h, (cudaStream_t)stream, a->dev_status};
    return launch_attention_simt(L, *a);
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
    Launch L{h, (cudaStream_t)stream, a->dev_status};
    const dflash_config& c = h->cfg;
    const bool f32in = a->hidden_is_f32 || c.dtype == DFLASH_F32;
    DFLASH_TRY(launch_rmsnorm(L, a->hidden, f32in, h->w.g_f, a->apply_norm != 0, ws.u, a->n_rows, c.d_model));
    return lmhead_rows(L, ws, ws.u, a->n_rows, a->ids, a->top1, a->margin, a->logits_out);
}

}  // extern "C"
