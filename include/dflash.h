/*
 * dflash.h -- C ABI of the B200 (sm_100a) DFlash draft-block / verify-accept library.
 *
 * What the calls compute follows the paper "DFlash: Block Diffusion for Flash Speculative
 * Decoding": Sec. 3.1 (speculative cycle, Eq. 1), Sec. 4.1 (context features, KV injection,
 * single-pass block drafting) and App. A.3 (KV-injection equations).
 *
 * Conventions
 *   - Plain C. Every pointer is tagged [host] or [device] below. The library allocates NO device
 *     memory: weights, KV pool, page tables, lengths, outputs and the workspace are caller-owned
 *     device buffers; the library keeps only borrowed pointers (dflash_set_weights) which must
 *     stay valid while they are in use.
 *   - Every compute call is asynchronous on the caller's stream (`stream` is a cudaStream_t passed
 *     as void*; NULL = the legacy default stream) and never synchronises. Errors the host can see
 *     (bad arguments, unsupported shapes, small workspace, launch failures) come back as a negative
 *     return code and nothing is launched. Errors only the device can see (token id >= vocab, page
 *     index outside the pool, a bounded wait that ran out) OR bits into `*dev_status` (caller
 *     zeroes it; may be NULL) and the affected work is skipped or clamped; no kernel traps.
 *   - Lengths that chain from one call to the next (ctx_len, n_new, accept lengths) live in device
 *     memory, so a decode cycle needs no host round trip.
 *   - dtype: DFLASH_F32 or DFLASH_BF16 selects the storage type of weights, features, KV pool,
 *     and activations handed across the ABI. Accumulation, norms and softmax are fp32 either way.
 *   - All matrices are row-major [out_features, in_features].
 *
 * Paged KV pool layout (element type = config dtype):
 *     pool[layer][page][K=0|V=1][kv_head][slot 0..page_size-1][head_dim]
 *   Logical position p of sequence b lives in physical page page_table[b*max_pages + p/page_size],
 *   slot p % page_size. Pages need not be contiguous or ordered. Context keys are stored already
 *   position-encoded.
 */
#ifndef DFLASH_H_
#define DFLASH_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- return codes (host-visible) ---- */
#define DFLASH_OK                    0
#define DFLASH_ERR_INVALID_ARG      -1
#define DFLASH_ERR_UNSUPPORTED      -2
#define DFLASH_ERR_WORKSPACE        -3
#define DFLASH_ERR_CUDA             -4
#define DFLASH_ERR_NOT_READY        -5   /* weights not set */

/* ---- bits OR-ed into *dev_status by kernels ---- */
#define DFLASH_DEV_BAD_TOKEN         1   /* token id outside [0, vocab): row embedded as token 0 */
#define DFLASH_DEV_BAD_PAGE          2   /* page index outside the pool: tile skipped            */
#define DFLASH_DEV_CTX_OVERFLOW      4   /* position beyond page table capacity: row skipped     */
#define DFLASH_DEV_TIMEOUT           8   /* a bounded on-chip wait expired: output invalid       */

#define DFLASH_F32   0
#define DFLASH_BF16  1

#define DFLASH_ATTN_FULL    0   /* draft mode: block rows see each other in both directions */
#define DFLASH_ATTN_CAUSAL  1   /* verify mode: block row r sees block rows <= r            */

#define DFLASH_VERIFY_LOGITS 0
#define DFLASH_VERIFY_IDS    1

typedef struct dflash_handle dflash_handle;

/* Shape of the drafter. Notation: N layers, D, Hq, Hkv, hd, F, V, k tapped target layers of width
 * D_t (App. A.3: W_c is D x k*D_t), block size B. */
typedef struct {
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
    int32_t n_feat_layers, d_target, block_size, page_size;
    int32_t dtype;          /* DFLASH_F32 | DFLASH_BF16 */
    int32_t mask_token_id;  /* id embedded at block rows 1..B-1 */
    int32_t use_rope;       /* 1: rotary positions (rotate-half pairing) on q and k; 0: none */
    float   rms_eps;
    float   softmax_scale;  /* usually head_dim^-1/2 */
    int32_t qk_norm;        /* 1: every q and k head is RMS-normalised over head_dim (gains g_q, g_k, same rms_eps)
                               before the rotation, for block rows and for the injected context keys. The paper's
                               App. A.3 shows plain projections; the Qwen3 layers the draft shares its
                               architecture with carry this norm. 0: off. */
} dflash_config;

typedef struct {
    const void* g1;        /* [device] [D]            pre-attention norm gain            */
    const void* W_qkv;     /* [device] [(Hq+2Hkv)*hd, D]  rows: q heads, k heads, v heads */
    const void* W_o;       /* [device] [D, Hq*hd]                                         */
    const void* g2;        /* [device] [D]            pre-FFN norm gain                  */
    const void* W_gateup;  /* [device] [2F, D]        row 2j = gate_j, row 2j+1 = up_j   */
    const void* W_down;    /* [device] [D, F]                                             */
    const void* g_q;       /* [device] [hd] gain of the q-head norm (qk_norm = 1, else ignored / NULL) */
    const void* g_k;       /* [device] [hd] gain of the k-head norm (qk_norm = 1, else ignored / NULL) */
} dflash_layer_weights;

typedef struct {
    const void* embed;                    /* [device] [V, D] token embedding (shared with target) */
    const void* W_c;                      /* [device] [D, k*D_t] context fusion (App. A.3)        */
    const void* g_c;                      /* [device] [D] gain of the fusion RMSNorm              */
    const dflash_layer_weights* layers;   /* [host]   array of n_layers entries (copied)          */
    const void* g_f;                      /* [device] [D] final norm gain                         */
    const void* W_lm;                     /* [device] [V, D] LM head (shared with target)         */
    const float* rope_cos;                /* [device] [rope_max_pos, hd/2] fp32                   */
    const float* rope_sin;                /* [device] [rope_max_pos, hd/2] fp32                   */
    int32_t rope_max_pos;
} dflash_weights;

/* ---- life cycle (host only, no CUDA work) ---- */

/* Validates the configuration and builds a handle. Returns DFLASH_ERR_UNSUPPORTED for shapes the
 * kernels do not cover (head_dim not in {64,128}, Hq % Hkv != 0, block_size > 32, ...).
 * The handle remembers the SM count of the device that is current at this call (148 when the host has no
 * GPU): grids, work splits and workspace sizes follow it, so use the handle on that device (or an equal one).
 * bf16 attention runs on the tensor cores for head_dim = 128 with 64-token pages; head_dim = 64 (and other
 * page sizes) take a CUDA-core kernel, as does everything in fp32.
 * The chained contraction kernels run one CTA per SM and their CTAs wait for each other (bounded): two
 * library calls must not overlap in time on one GPU (issue them on one stream, or order them with
 * events), and the GPU's SMs must all be available to the process (no MPS / green-context SM limit);
 * otherwise waits expire after ~1.5 s, DFLASH_DEV_TIMEOUT is set and the output is invalid. */
int32_t dflash_create(const dflash_config* cfg /*[host]*/, dflash_handle** out /*[host]*/);
void    dflash_destroy(dflash_handle* h);

/* Borrow the weight pointers. The `layers` array is copied; the device buffers are not. */
int32_t dflash_set_weights(dflash_handle* h, const dflash_weights* w /*[host]*/);

/* Bytes of device workspace that any call below needs for up to `max_rows` rows in flight
 * (rows = batch * block_size for a draft, batch * (gamma+1) for verify-side calls, batch * max_new
 * for the context projection) and `max_batch` sequences. */
int64_t dflash_workspace_bytes(const dflash_handle* h, int32_t max_batch, int32_t max_rows);

/* ---- context-feature fusion and KV injection (App. A.3, first and second display) ----
 * For each valid row (b, r), r < n_new[b]:
 *   y = W_c * feats[b, r, :]                       (feats = k tapped hidden states, concatenated)
 *   H_t = g_c * y / sqrt(mean(y^2) + eps)
 *   for each draft layer i: K = RoPE(W_i^K H_t, pos), V = W_i^V H_t, pos = ctx_len[b] + r
 *   written to pool[i][page_table[b][pos/page]][K|V][:][pos % page][:].
 * ctx_len is read, never updated (the accept step produces the next value). */
typedef struct {
    const void*    feats;        /* [device] [batch, max_new, k*D_t], config dtype            */
    int32_t        batch;
    int32_t        max_new;      /* row slots per sequence                                    */
    const int32_t* n_new;        /* [device] [batch] valid rows per sequence; NULL = max_new  */
    const int32_t* ctx_len;      /* [device] [batch] position of row 0                        */
    const int32_t* page_table;   /* [device] [batch, max_pages]                               */
    int32_t        max_pages;
    void*          kv_pool;      /* [device] pool, see layout above                           */
    int32_t        n_pool_pages;
    void*          workspace;    /* [device] >= dflash_workspace_bytes(h, batch, batch*max_new), 256-byte aligned */
    int64_t        workspace_bytes;
    int32_t*       dev_status;   /* [device] may be NULL                                      */
} dflash_ctx_args;
int32_t dflash_ctx_project(dflash_handle* h, const dflash_ctx_args* a /*[host]*/, void* stream);

/* ---- single-pass block draft (Sec. 4.1 "Parallel diffusion drafting"; App. A.3) ----
 * Per sequence b: rows r = 0..B-1 at positions ctx_len[b]+r; row 0 embeds anchor_ids[b], the others
 * the mask token. N pre-norm layers: q,k,v projections (+RoPE), attention of every row over the
 * ctx_len[b] cached context entries and ALL B block rows, output projection, SwiGLU FFN; final
 * norm; LM head; draft_ids[b, r] = argmax_v logits (lowest index among equal maxima). Logits are
 * never written unless logits_out is given. */
typedef struct {
    const int32_t* anchor_ids;   /* [device] [batch]                                          */
    int32_t        batch;
    const int32_t* ctx_len;      /* [device] [batch]                                          */
    int32_t        max_ctx_len;  /* [host value] upper bound of ctx_len (sizes the KV split)  */
    const int32_t* page_table;   /* [device] [batch, max_pages]                               */
    int32_t        max_pages;
    const void*    kv_pool;      /* [device]                                                  */
    int32_t        n_pool_pages;
    void*          workspace;    /* [device] >= dflash_workspace_bytes(h, batch, batch*B)     */
    int64_t        workspace_bytes;
    int32_t*       draft_ids;    /* [device] out [batch, B]                                   */
    float*         top1;         /* [device] out [batch, B] winning logit; may be NULL        */
    float*         margin;       /* [device] out [batch, B] top-1 minus top-2; may be NULL    */
    float*         hidden_out;   /* [device] out [batch*B, D] fp32 residual stream after the last layer; may be NULL */
    float*         logits_out;   /* [device] out [batch*B, V] fp32; may be NULL (tests only)  */
    int32_t*       dev_status;   /* [device] may be NULL                                      */
    int32_t        block_rows;   /* rows per sequence in THIS call: 0 = the handle's block_size B, else 1..B
                                    (a drafter trained at B = 16 also runs blocks of 8 or 10, Sec. 5.3); every
                                    [batch, B] / [batch*B, ...] shape above then uses block_rows in place of B */
    const dflash_ctx_args* ctx;  /* [host] may be NULL. When given, the context projection described by *ctx (same
                                    result as dflash_ctx_project with these arguments; same batch and pool as this
                                    call; its workspace fields are ignored, this call's workspace must hold
                                    dflash_workspace_bytes(h, batch, max(batch*B, batch*max_new))) runs inside this
                                    call, chained in ONE launch with the first layer's QKV contraction: the draft's
                                    first weights stream while the projection's last tiles finish. The draft sees
                                    ctx_len[b] cached entries: pass the lengths AFTER the projection there if the
                                    new rows are to be visible (ctx->ctx_len holds the lengths before it). */
} dflash_draft_args;
int32_t dflash_draft_block(dflash_handle* h, const dflash_draft_args* a /*[host]*/, void* stream);

/* ---- the target's verify pass over the same kernels (Sec. 3.1: the target scores all gamma drafts in
 * one parallel pass; Sec. 4.1: hidden states of k of its layers are the drafter's context features) ----
 * A handle created with the TARGET's shape runs its stack over `rows` given tokens per sequence
 * (anchor, d_1 .. d_gamma) on top of the target's own paged KV cache (same pool layout): causal
 * inside the block, full over the cached context. Outputs: logits and their row argmax (the p_j of
 * the accept rule), the hidden rows after the layers listed in tap_layers laid out as
 * [batch, rows, n_taps * D] = the operand of dflash_ctx_project (no concatenation pass), and the
 * block's K/V of every layer written into the cache at positions ctx_len .. ctx_len + rows - 1:
 * after the accept step the caller only raises ctx_len by tau (rows past it stay invisible and are
 * overwritten by the next cycle). The handle's W_c / g_c / mask token are not used.
 * rows <= 32 and rows * (Hq / Hkv) <= 128 on the bf16 path; tap_layers ascending. */
typedef struct {
    const int32_t* token_ids;    /* [device] [batch, rows]                                     */
    int32_t        batch, rows;
    const int32_t* ctx_len;      /* [device] [batch] committed length of every sequence        */
    int32_t        max_ctx_len;  /* [host value] upper bound of ctx_len                        */
    const int32_t* page_table;   /* [device] [batch, max_pages]; must cover ctx_len + rows     */
    int32_t        max_pages;
    void*          kv_pool;      /* [device] the target's pool; read, and written at the block's positions */
    int32_t        n_pool_pages;
    const int32_t* tap_layers;   /* [host] n_taps layer indices (0-based, ascending); may be NULL if n_taps = 0 */
    int32_t        n_taps;
    void*          feats_out;    /* [device] out [batch, rows, n_taps * D] config dtype; may be NULL if n_taps = 0 */
    float*         logits_out;   /* [device] out [batch * rows, V] fp32; may be NULL           */
    int32_t*       ids_out;      /* [device] out [batch, rows] argmax of every row             */
    void*          workspace;    /* [device] >= dflash_workspace_bytes(h, batch, batch * rows)  */
    int64_t        workspace_bytes;
    int32_t*       dev_status;   /* [device] may be NULL                                       */
} dflash_target_args;
int32_t dflash_target_verify(dflash_handle* h, const dflash_target_args* a /*[host]*/, void* stream);

/* ---- greedy verify / accept (Sec. 3.1: tau in [1, gamma+1] incl. the bonus token) ----
 * One launch in either mode. Mode LOGITS counts, per sequence, the CTAs that have finished scanning in a small
 * ticket array inside the library image (16 KB per GPU, self-resetting; up to 4096 sequences per call, more take two
 * launches): like all calls of this library, verify calls on one GPU must not overlap in time.
 * p_j = argmax_v logits[b, j, :] (mode LOGITS) or target_ids[b, j] (mode IDS), j = 0..gamma.
 * a = length of the longest prefix with draft[b, i] == p_i, i < a;  tau = a + 1;
 * out_tokens[b] = draft[b, 0..a-1], p_a, then -1; bonus[b] = p_a; new_ctx_len[b] = ctx_len[b]+tau. */
typedef struct {
    int32_t        mode;             /* DFLASH_VERIFY_LOGITS | DFLASH_VERIFY_IDS               */
    const void*    logits;           /* [device] mode LOGITS: [batch, gamma+1, vocab]          */
    int32_t        logits_dtype;     /* DFLASH_F32 | DFLASH_BF16                               */
    int64_t        logits_row_stride;/* elements between rows j and j+1 (0 = vocab)            */
    const int32_t* target_ids;       /* [device] mode IDS: [batch, gamma+1]                    */
    const int32_t* draft_ids;        /* [device] first draft of sequence b at draft_ids + b*draft_stride */
    int32_t        draft_stride;     /* elements                                               */
    int32_t        batch, gamma, vocab;
    const int32_t* ctx_len;          /* [device] [batch]                                       */
    int32_t*       accept_len;       /* [device] out [batch] tau                               */
    int32_t*       out_tokens;       /* [device] out [batch, gamma+1]                          */
    int32_t*       bonus;            /* [device] out [batch]                                   */
    int32_t*       new_ctx_len;      /* [device] out [batch]; may alias ctx_len                */
    int32_t*       target_ids_out;   /* [device] out [batch, gamma+1] the p_j; may be NULL     */
    void*          workspace;        /* [device] >= dflash_workspace_bytes(h, batch, batch*(gamma+1)) */
    int64_t        workspace_bytes;
    int32_t*       dev_status;
} dflash_verify_args;
int32_t dflash_verify_accept(dflash_handle* h, const dflash_verify_args* a /*[host]*/, void* stream);

/* ---- verify/accept from logits without any caller-provided scratch ----
 * (No counterpart in the paper: this entry point exists for integration reasons only.)
 * Same result as dflash_verify_accept in mode DFLASH_VERIFY_LOGITS, for callers that cannot allocate
 * device memory for a workspace (all GPU memory already committed to a cache pool, no tolerance for
 * cudaMalloc's device-wide synchronisation, or a stream being captured into a graph). The scratch
 * is a fixed array inside the library image: about 1.1 MB that every GPU loading the library holds
 * until the process exits. `workspace` / `workspace_bytes` are ignored.
 *   - at most DFLASH_STATIC_MAX_ROWS = batch * (gamma+1) rows; more returns DFLASH_ERR_UNSUPPORTED
 *   - the array is shared by all calls on a device and keeps the previous call's contents (no entry
 *     needs to start at zero); calls that overlap on the GPU race on it, so order them on one stream
 *     or with events
 *   - the first call on each device resolves the array's device address on the host: issue it
 *     before any stream capture begins
 *   - allocates and frees nothing */
#define DFLASH_STATIC_MAX_ROWS 1088
int32_t dflash_verify_accept_static(dflash_handle* h, const dflash_verify_args* a /*[host]*/, void* stream);

/* ---- sampling (temperature > 0): drafting draws and speculative-sampling verification ----
 * The paper reports T = 1 results (Sec. 5.1) and relies on standard speculative sampling (Sec. 2)
 * without restating the rule; it is, with p_j = softmax(target_logits[b, j] / T) and
 * q_j = softmax(draft_logits[b, j] / T):
 *   draft j (j = 0..gamma-1, in order) is kept while  u_accept[b, j] * q_j(d_j) < p_j(d_j);
 *   at the first rejection a:  one token drawn from max(p_a - q_a, 0) (from p_a if that is all zero);
 *   with every draft kept (a = gamma): one token drawn from p_gamma;   tau = a + 1.
 * A draw maps a uniform u in [0, 1) to the first vocabulary index (with non-zero weight) whose running
 * sum of weights reaches u * total. The uniforms are INPUTS: the library draws no random numbers, so a
 * caller (and the CPU oracle) reproduces a result from the same uniforms. Sums that decide an index are
 * accumulated in double in a fixed order; against exact arithmetic a result can only differ when
 * u * total lies within ~1e-6 (relative) of an interval edge.
 * Scratch: `workspace` of dflash_sample_workspace_bytes(n_logit_rows, vocab) bytes, 256-byte aligned,
 * n_logit_rows = n_rows (dflash_sample_rows) or batch * (2 * gamma + 1) (dflash_verify_accept_sample).
 * Each call is two launches (segment statistics of every row; then per draw the weights of each segment,
 * the last segment to finish drawing the index). At most 65535 logit rows per call and gamma <= 64,
 * else DFLASH_ERR_UNSUPPORTED.
 * Errors: DFLASH_ERR_INVALID_ARG (null pointer, T <= 0, bad dtype or sizes), DFLASH_ERR_WORKSPACE;
 * a draft id outside [0, vocab) counts as rejected and sets DFLASH_DEV_BAD_TOKEN in *dev_status. */
typedef struct {
    const void*    logits;        /* [device] [n_rows, vocab]                                   */
    int32_t        logits_dtype;  /* DFLASH_F32 | DFLASH_BF16                                   */
    int64_t        row_stride;    /* elements between rows (0 = vocab)                          */
    int32_t        n_rows, vocab;
    float          temperature;   /* > 0                                                        */
    const float*   u;             /* [device] [n_rows] uniforms in [0, 1)                       */
    int32_t*       ids;           /* [device] out [n_rows] drawn index                          */
    float*         prob;          /* [device] out [n_rows] its probability; may be NULL         */
    void*          workspace;     /* [device]                                                   */
    int64_t        workspace_bytes;
    int32_t*       dev_status;    /* [device] may be NULL                                       */
} dflash_sample_args;
int32_t dflash_sample_rows(dflash_handle* h, const dflash_sample_args* a /*[host]*/, void* stream);

typedef struct {
    const void*    target_logits;      /* [device] [batch, gamma+1, vocab]                      */
    int32_t        target_dtype;       /* DFLASH_F32 | DFLASH_BF16                              */
    int64_t        target_row_stride;  /* elements (0 = vocab)                                  */
    const void*    draft_logits;       /* [device] draft j of sequence b = row b*draft_rows_per_seq + j */
    int32_t        draft_dtype;
    int64_t        draft_row_stride;   /* elements (0 = vocab)                                  */
    int32_t        draft_rows_per_seq; /* stored rows per sequence (>= gamma), e.g. the block size */
    const int32_t* draft_ids;          /* [device] first draft of sequence b at draft_ids + b*draft_stride */
    int32_t        draft_stride;
    int32_t        batch, gamma, vocab; /* gamma <= 64, else DFLASH_ERR_UNSUPPORTED               */
    float          temperature;        /* > 0, applied to both distributions                    */
    const float*   u_accept;           /* [device] [batch, gamma] uniforms in [0, 1)            */
    const float*   u_final;            /* [device] [batch] uniform of the emitted token         */
    const int32_t* ctx_len;            /* [device] [batch]                                      */
    int32_t*       accept_len;         /* [device] out [batch] tau                              */
    int32_t*       out_tokens;         /* [device] out [batch, gamma+1]: kept drafts, the emitted token, then -1 */
    int32_t*       bonus;              /* [device] out [batch] the emitted token (next anchor)  */
    int32_t*       new_ctx_len;        /* [device] out [batch]; may alias ctx_len               */
    void*          workspace;          /* [device]                                              */
    int64_t        workspace_bytes;
    int32_t*       dev_status;         /* [device] may be NULL                                  */
} dflash_verify_sample_args;
int32_t dflash_verify_accept_sample(dflash_handle* h, const dflash_verify_sample_args* a /*[host]*/, void* stream);
int64_t dflash_sample_workspace_bytes(int32_t n_logit_rows, int32_t vocab);

/* ---- building block: attention of `rows` block rows per sequence over paged context + the block
 * itself (App. A.3: K = [K_ctx ; K_block]_seq). FULL = draft mode, CAUSAL = the target's verify
 * pass over (gamma+1) rows. Head geometry and dtype come from the handle. q and k_blk must already
 * be position-encoded. */
typedef struct {
    int32_t        mode;         /* DFLASH_ATTN_FULL | DFLASH_ATTN_CAUSAL                     */
    const void*    q;            /* [device] [batch, rows, Hq, hd]                            */
    const void*    k_blk;        /* [device] [batch, rows, Hkv, hd]                           */
    const void*    v_blk;        /* [device] [batch, rows, Hkv, hd]                           */
    int32_t        batch, rows;  /* rows <= 32                                                */
    const int32_t* ctx_len;      /* [device] [batch]                                          */
    int32_t        max_ctx_len;  /* [host value] upper bound of ctx_len                       */
    const int32_t* page_table;   /* [device] [batch, max_pages]                               */
    int32_t        max_pages;
    const void*    kv_pool;      /* [device] pool with the layout above                       */
    int32_t        n_pool_pages;
    int32_t        layer;        /* which pool layer to read                                  */
    void*          out;          /* [device] [batch, rows, Hq, hd]                            */
    void*          workspace;
    int64_t        workspace_bytes;
    int32_t*       dev_status;
    float*         lse_out;      /* [device] out [batch, rows, Hq] fp32; may be NULL. Natural-log sum of exponentials
                                    of every row's scaled scores (what dflash_block_attention_bwd takes back)  */
} dflash_attn_args;
int32_t dflash_block_attention(dflash_handle* h, const dflash_attn_args* a /*[host]*/, void* stream);

/* ---- training side: backward pass of the block attention (Sec. 4.2: all anchor blocks of a sequence are trained
 * in one forward and one backward pass; a block attends in both directions to itself and to the injected context
 * before its anchor, never to another block) ----
 * The forward of that mask is dflash_block_attention over a batch of blocks with ctx_len[b] = position of block
 * b's anchor (mode FULL), all blocks sharing one page-table row. Given dout = d loss / d out, per query head h
 * (kv head h / (Hq/Hkv)), with P the forward's probabilities over keys = [context ; block]:
 *     dV = P^T dout     dP = dout V^T     dS = P * (dP - rowsum(dout * out))     dq = scale dS K     dK = scale dS^T q
 * P is recomputed from q, the keys and the forward's log-sum-exp (lse_out of dflash_block_attention); no
 * probability matrix is stored. Gradients of a kv head add up over the q heads of its group.
 * dkv_ctx receives the context gradients of ONE layer in the pool's own layout, fp32:
 *     dkv_ctx[page][K=0|V=1][kv_head][slot][head_dim]
 * for every page that holds positions below max_ctx_len of a page-table row in use (whole pages are written,
 * zeros where no block sees a key); other pages are not touched. shared_page_row = 1 (the training layout): every
 * block reads page-table row 0 and the gradients of a position add up over all blocks that see it in an order fixed
 * by the batch order (two blocks at a time; bit-reproducible, no atomics). shared_page_row = 0: block b uses row b and owns its pages.
 * bf16 handles with head_dim 128, 64-token pages and rows * (Hq/Hkv) <= 64 only (DFLASH_ERR_UNSUPPORTED else).
 * Workspace as for dflash_block_attention. Errors as there; a ctx_len above max_ctx_len is clamped and flagged. */
typedef struct {
    int32_t        mode;          /* DFLASH_ATTN_FULL | DFLASH_ATTN_CAUSAL (as in the forward)          */
    const void*    q;             /* [device] [batch, rows, Hq, hd]                                    */
    const void*    k_blk;         /* [device] [batch, rows, Hkv, hd]                                   */
    const void*    v_blk;         /* [device] [batch, rows, Hkv, hd]                                   */
    const void*    out;           /* [device] [batch, rows, Hq, hd] the forward's output               */
    const float*   lse;           /* [device] [batch, rows, Hq] the forward's lse_out                  */
    const void*    dout;          /* [device] [batch, rows, Hq, hd] gradient of the loss w.r.t. out    */
    int32_t        batch, rows;
    const int32_t* ctx_len;       /* [device] [batch]                                                  */
    int32_t        max_ctx_len;   /* [host value] upper bound of ctx_len                               */
    const int32_t* page_table;    /* [device] [batch, max_pages] (row 0 only if shared_page_row)       */
    int32_t        max_pages;
    const void*    kv_pool;       /* [device] pool, layout at the top of this file                     */
    int32_t        n_pool_pages;
    int32_t        layer;
    int32_t        shared_page_row;
    void*          dq;            /* [device] out [batch, rows, Hq, hd] config dtype                   */
    void*          dk_blk;        /* [device] out [batch, rows, Hkv, hd]                               */
    void*          dv_blk;        /* [device] out [batch, rows, Hkv, hd]                               */
    float*         dkv_ctx;       /* [device] out fp32 [n_pool_pages, 2, Hkv, page_size, hd]; may be NULL (then the
                                     context gradients are not computed)                               */
    void*          workspace;     /* [device] >= dflash_workspace_bytes(h, batch, batch * rows)        */
    int64_t        workspace_bytes;
    int32_t*       dev_status;    /* [device] may be NULL                                              */
} dflash_attn_bwd_args;
int32_t dflash_block_attention_bwd(dflash_handle* h, const dflash_attn_bwd_args* a /*[host]*/, void* stream);

/* ---- building block: LM head fused with row-wise argmax (Sec. 4.2: LM head shared with the
 * target). ids[m] = argmax_v (W_lm z_m)_v with z = hidden (apply_norm = 0) or
 * z = g_f * hidden / rms(hidden) (apply_norm = 1). */
typedef struct {
    const void* hidden;          /* [device] [n_rows, D]; config dtype, or fp32 if hidden_is_f32 */
    int32_t     hidden_is_f32;
    int32_t     n_rows;
    int32_t     apply_norm;
    int32_t*    ids;             /* [device] out [n_rows]                                     */
    float*      top1;            /* [device] out [n_rows]; may be NULL                        */
    float*      margin;          /* [device] out [n_rows]; may be NULL                        */
    float*      logits_out;      /* [device] out [n_rows, V] fp32; may be NULL                */
    void*       workspace;
    int64_t     workspace_bytes;
    int32_t*    dev_status;
} dflash_lmhead_args;
int32_t dflash_lmhead_argmax(dflash_handle* h, const dflash_lmhead_args* a /*[host]*/, void* stream);

/* ---- training side: position-weighted cross entropy of draft blocks (Sec. 4.2 "Loss weighting", Eq. 4) ----
 * Row k of a block (k = 0 .. block_rows-1) holds the logits of block position k; position 0 is the clean
 * anchor and carries no loss, position k >= 1 has weight w_k = exp(-(k-1)/gamma) (gamma = 7 / 5 / 4 for
 * blocks of 16 / 10 / 8, App. A.1). Per row:  row_loss = w_k * (logsumexp(z) - z[target]);  optionally the
 * gradient  dlogits = grad_scale * w_k * (softmax(z) - onehot(target))  (zeros for rows without loss).
 * A negative target marks a position without loss (a block cut short by the end of its sequence); a target
 * >= vocab is treated the same and sets DFLASH_DEV_BAD_TOKEN. loss_sum = {sum of row_loss, sum of the w_k
 * that count}, added in double in a fixed order: the caller divides by whichever normaliser it trains with
 * (the paper does not state one) and passes the matching grad_scale.
 * Arithmetic: fp32 per row (maximum, sum of exponentials, logarithm). A row is held in the shared memory of a
 * small thread-block cluster between the statistics and the gradient pass (rows that do not allow 16-byte
 * accesses are instead read twice by one CTA): HBM traffic is one read of the logits plus one write of the
 * gradient. `dlogits` may alias `logits` when dtype and stride agree. No scratch memory.
 * Errors: DFLASH_ERR_INVALID_ARG (null pointer, gamma <= 0, bad dtype or sizes). */
typedef struct {
    const void*    logits;             /* [device] [n_blocks * block_rows, vocab]                       */
    int32_t        logits_dtype;       /* DFLASH_F32 | DFLASH_BF16                                      */
    int64_t        row_stride;         /* elements (0 = vocab)                                          */
    int32_t        n_blocks, block_rows, vocab;
    const int32_t* targets;            /* [device] [n_blocks, block_rows]; entry 0 of a block is unused */
    float          gamma;              /* > 0                                                           */
    float*         row_loss;           /* [device] out [n_blocks * block_rows]                          */
    float*         loss_sum;           /* [device] out [2]; may be NULL                                 */
    void*          dlogits;            /* [device] out [n_blocks * block_rows, vocab]; may be NULL      */
    int32_t        dlogits_dtype;      /* DFLASH_F32 | DFLASH_BF16                                      */
    int64_t        dlogits_row_stride; /* elements (0 = vocab)                                          */
    float          grad_scale;
    int32_t*       dev_status;         /* [device] may be NULL                                          */
} dflash_block_loss_args;
int32_t dflash_block_loss(dflash_handle* h, const dflash_block_loss_args* a /*[host]*/, void* stream);

/* ---- per-kernel-family timing (host-side CUDA events; off by default) ----
 * While enabled, every launch the library issues is bracketed by an event pair on the caller's
 * stream. dflash_profile_read synchronises on the last event, adds the elapsed milliseconds and the
 * launch counts per family into the two host arrays (DFLASH_N_FAMILIES entries each) and clears
 * the record. Event pairs cost a little time per launch: never time a step with profiling on. */
#define DFLASH_N_FAMILIES 15
int32_t dflash_profile_enable(dflash_handle* h, int32_t on);
int32_t dflash_profile_read(dflash_handle* h, float* ms /*[host]*/, int32_t* launches /*[host]*/);
const char* dflash_family_name(int32_t family);

/* ---- device-side timeline (off by default) ----
 * While a trace buffer is set, every tensor-core kernel the library launches records four device
 * timestamps (nanoseconds of the GPU's global timer) into the next 4-word record of `dev_buf`:
 *   [0] ~(earliest CTA start)   [1] ~(earliest moment a CTA saw its grid dependency resolved)
 *   [2] latest end of a CTA's main loop   [3] latest CTA exit
 * (the first two are stored complemented so that every word is a running maximum and the caller
 * only has to zero the buffer). dflash_trace_read returns, per record written since the last read,
 * the kernel family that wrote it, and rewinds. Passing NULL switches tracing off. */
int32_t dflash_trace_enable(dflash_handle* h, uint64_t* dev_buf /*[device]*/, int32_t capacity_records);
int32_t dflash_trace_read(dflash_handle* h, int32_t* families /*[host] capacity entries*/, int32_t* n_records /*[host]*/);

/* How dflash_block_attention / the draft and verify passes split the keys of a call on the bf16 tensor-core
 * path (host arithmetic only, no CUDA work): out[0] = 64-key tiles per range, out[1] = ranges per (sequence,
 * kv head) at max_ctx_len, out[2] = partial-result slots the kernels index (batch * Hkv * ranges), out[3] =
 * slots the workspace of dflash_workspace_bytes(h, batch, ...) provides. out[2] <= out[3] for every input:
 * when many long sequences would need more, the ranges get longer instead. A ctx_len[b] above max_ctx_len is
 * clamped to it by the kernels and sets DFLASH_DEV_CTX_OVERFLOW. */
int32_t dflash_attention_plan(const dflash_handle* h, int32_t batch, int32_t max_ctx_len, int64_t* out /*[host] [4]*/);

/* How the chained contraction kernel splits one [M, K] x [N, K]^T product (n_groups weight matrices of N rows) over
 * its CTAs, walked on the host with the kernel's own arithmetic (no CUDA work, no handle): sm_count CTAs at most,
 * pair_cap = CTA pairs the device keeps resident (token tiles of 160+ columns run as pairs when >= 1; 74 on a B200),
 * cluster_cap = 4-CTA clusters it keeps resident (token tiles of up to 32 columns; 33 on a B200). Returns 0 when
 * every (tile, K chunk) is taken exactly once, no CTA holds more than two partial pieces (in different slots) and
 * the contributors of every shared tile are the ones the finishing code looks for; a positive code names the first
 * check that failed, -1 bad arguments. info (may be NULL): token tile width, pair form (0/1), grid size, CTAs per
 * K-split cluster, tiles split across CTAs, K-split-cluster phase (0/1). The paper has no counterpart: a test aid. */
int32_t dflash_gemm_plan_check(int32_t M, int32_t N, int32_t K, int32_t n_groups, int32_t sm_count, int32_t pair_cap,
                               int32_t cluster_cap, int32_t* info /*[host] [6] or NULL*/);

/* Static description of a return code. */
const char* dflash_status_string(int32_t code);

/* Number of kernel launches the library has issued since it was loaded (all handles). */
int64_t dflash_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* DFLASH_H_ */
