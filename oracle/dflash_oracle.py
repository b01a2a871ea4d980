"""CPU oracle for the DFlash draft-block forward and greedy verify/accept step.

TEST INFRASTRUCTURE ONLY. This file is the slow, plain definition that the CUDA library is
checked against; nothing in the product path may import or call it. It imports nothing from the
CUDA package and shares no code, table or constant generator with it.

Everything is float64 numpy, one sequence at a time, in the order and notation of the paper:

  App. A.3, first display:   H_t = RMSNorm(W_c [H^(l1); ...; H^(lk)])             -> ctx_fuse
  App. A.3, second display:  Q_i = W_i^Q H_d,  K_i = [W_i^K H_t ; W_i^K H_d]_seq,
                             V_i = [W_i^V H_t ; W_i^V H_d]_seq                     -> ctx_kv, draft_layer
  Sec. 4.1 "Parallel diffusion drafting": one forward pass over [anchor, mask x (B-1)],
  bidirectional inside the block and full over the injected context                -> draft_block
  Sec. 4.2 / Sec. 5: embedding and LM head shared with the target                  -> lm_head
  Sec. 3.1 (Eq. 1 and the sentence after it): gamma drafts verified in parallel,
  tau in [1, gamma+1] including the bonus token; lossless under greedy decoding    -> verify_accept

Readings taken where the paper is silent (each is listed in the design notes): optional per-head
RMSNorm of q and k before the rotation (cfg.qk_norm; App. A.3 shows plain projections, the Qwen3 layers
the draft shares its architecture with carry it); pre-norm residual
layers; RMSNorm y * (mean(y^2)+eps)^-1/2 * g; no biases; SwiGLU FFN; rotary position encoding with
rotate-half pairing (i, i + hd/2), context token p at position p and block row r at position L+r;
softmax scale hd^-1/2; argmax takes the lowest index among equal maxima and NaN never wins.

Pins (tests/test_oracle_*.py): closed forms for RMSNorm / SiLU / RoPE, the App. A.3 worked memory
figures for the layouts, brute-force loops for attention and matmul on tiny inputs, attention
special cases (uniform keys -> mean of V, dominant key -> its V, permutation invariance, GQA =
replicated MHA, causal last row = full last row), accept-rule enumeration of all match patterns,
equality of speculative output with plain greedy decoding of a toy target, and for one layer
(tests/test_oracle_draft_block.py) the SwiGLU half written out with scalar loops (SiLU on the gate
branch, gate 0 closes a unit, a large gate passes the up value), the first norm feeding q, k, v and
the second norm reading the hidden after the attention residual with its own gain.
The composed forward `draft_block` has no external value to compare with: parity unpinned beyond
its parts (each step above is pinned separately).

The target's side of a cycle (Sec. 3.1: one parallel pass scores all drafts; Sec. 4.1: hidden states of
k target layers become the context features): a causal stack over [anchor, d_1 .. d_gamma] on top of
its cached K/V, returning logits, tapped rows and the block's cache entries       -> target_verify
(pinned by equality with the plain full-sequence causal forward, continued from its own cache).

Sampling (temperature > 0) verification, the setting of the paper's T = 1 results (Sec. 5.1, Table 2):
the paper relies on standard speculative sampling (Sec. 2 related work) without restating it, so
the rule is written out here                                     -> softmax_t, sample_cdf, verify_accept_sample
  p_j = softmax(target_logits[j] / T),  q_j = softmax(draft_logits[j] / T);
  draft d_{j+1} is kept while  u_j * q_j(d_{j+1}) < p_j(d_{j+1})   (probability min(1, p/q));
  at the first rejection a the cycle emits one token drawn from max(p_a - q_a, 0) / sum (from p_a if
  that sum is zero); with all gamma kept it emits one token drawn from p_gamma;  tau = a + 1.
  Every draw maps a uniform u in [0, 1) to the first vocabulary index whose running sum of weights
  reaches u * total (inverse CDF in vocabulary order). Uniforms are inputs.
Pins (tests/test_oracle_sampling.py): the first emitted token is distributed exactly as p_0 (measure
of the uniform cube, computed cell by cell on small vocabularies), a hand-worked two-token case,
p = q keeps everything, T -> 0 reduces to the greedy rule, rejected positions only emit tokens
with p > q.

Training loss of a block (Sec. 4.2 "Loss weighting", Eq. 4; App. A.1 for gamma)   -> loss_weights, block_loss
  position k = 1 .. B-1 of a block (k = 0 is the clean anchor and carries no loss) has weight
  w_k = exp(-(k - 1) / gamma); the loss of a block is sum_k w_k CE(logits_k, target_k), CE the plain
  cross entropy logsumexp(z) - z[target]; its gradient w.r.t. the logits is w_k (softmax(z) - onehot).
  Readings: the anchor row is skipped (the paper trains the B - 1 masked positions); a negative target
  marks a position to ignore (a block cut short by the end of the sequence); the normalisation of the
  sum (by the number of positions or by the sum of weights) is left to the caller: the functions return
  the weighted sum and the sum of weights.
Pins (tests/test_oracle_loss.py): w_1 = 1 and the constant ratio exp(-1/gamma), the printed gamma of
each block size, uniform logits -> ln V, a dominant logit -> 0, gradient rows summing to zero, central
finite differences of the summed loss, gamma -> infinity = unweighted sum.

Training-side attention of anchor blocks (Sec. 4.2 "Random sampling of masked blocks": all blocks of a sequence
in one forward and backward pass under a mask that is bidirectional inside a block, open towards the injected
context before the block's anchor and closed between blocks)      -> block_attention_lse, block_attention_backward
  The forward of that mask is block_attention per block with L = the anchor's position; the backward is the
  plain softmax-attention gradient; context gradients of the blocks add up per position.
Pins (tests/test_oracle_attention_bwd.py): central finite differences of block_attention in every input,
torch autograd of an independently written attention, sum over keys of dV = sum over rows of dout, key
gradients of a kv head summing to zero, a lone key passes dout straight to its value, exp(lse) = sum of exp,
context gradients of two blocks over one sequence against finite differences of the joint loss.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64
_CHUNK_ROWS = 8192


def _f64(a):
    return np.asarray(a, dtype=F64)


# --------------------------------------------------------------------------------------------
# elementary steps
# --------------------------------------------------------------------------------------------
def linear(x, W):
    """y = x W^T for a row-major [out, in] weight; the weight is widened to float64 in row chunks
    only to bound memory (each output element is still one plain dot product)."""
    x = _f64(x)
    n_out = W.shape[0]
    y = np.empty(x.shape[:-1] + (n_out,), dtype=F64)
    for n0 in range(0, n_out, _CHUNK_ROWS):
        n1 = min(n_out, n0 + _CHUNK_ROWS)
        y[..., n0:n1] = x @ _f64(W[n0:n1]).T
    return y


def rmsnorm(y, g, eps):
    """RMSNorm of App. A.3: g * y / sqrt(mean_j y_j^2 + eps), statistics over the last axis."""
    y = _f64(y)
    ms = np.mean(y * y, axis=-1, keepdims=True)
    return _f64(g) * (y / np.sqrt(ms + eps))


def silu(x):
    x = _f64(x)
    return x / (1.0 + np.exp(-x))


def rope(x, pos, theta):
    """Rotary position encoding, rotate-half pairing. x: [T, H, hd]; pos: [T] absolute positions.

    Pair (x_i, x_{i+hd/2}) is rotated by the angle pos * theta^(-2i/hd)."""
    x = _f64(x)
    hd = x.shape[-1]
    half = hd // 2
    inv_freq = F64(theta) ** (-2.0 * np.arange(half, dtype=F64) / hd)
    ang = _f64(pos)[:, None] * inv_freq[None, :]
    c = np.cos(ang)[:, None, :]
    s = np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate((x1 * c - x2 * s, x2 * c + x1 * s), axis=-1)


def argmax_top2(logits):
    """Row-wise greedy choice: (index of the maximum with the lowest index among ties, its value,
    margin to the runner-up value). NaN never wins; an all-NaN row yields index 0."""
    z = _f64(logits)
    z = np.where(np.isnan(z), -np.inf, z)
    idx = np.argmax(z, axis=-1)                      # first occurrence
    top1 = np.take_along_axis(z, idx[..., None], axis=-1)[..., 0]
    rest = z.copy()
    np.put_along_axis(rest, idx[..., None], -np.inf, axis=-1)
    top2 = np.max(rest, axis=-1)
    with np.errstate(invalid="ignore"):
        margin = top1 - top2
    return idx.astype(np.int64), top1, margin


# --------------------------------------------------------------------------------------------
# context features -> injected K/V   (App. A.3)
# --------------------------------------------------------------------------------------------
def ctx_fuse(feats, W_c, g_c, eps):
    """H_t = RMSNorm(W_c [H^(l1); ...; H^(lk)]). feats: [T, k*D_t], the k tapped hidden states of
    each token concatenated along the feature axis (W_c is D x kD_t)."""
    return rmsnorm(linear(feats, W_c), g_c, eps)


def ctx_kv(H_t, W_k, W_v, pos, cfg, g_k=None):
    """K^ctx = RoPE(W_i^K H_t), V^ctx = W_i^V H_t for one draft layer. Returns [T, Hkv, hd] each.
    With cfg.qk_norm, every key head is RMS-normalised with gain g_k before the rotation."""
    T = H_t.shape[0]
    k = linear(H_t, W_k).reshape(T, cfg.n_kv_heads, cfg.head_dim)
    v = linear(H_t, W_v).reshape(T, cfg.n_kv_heads, cfg.head_dim)
    if getattr(cfg, "qk_norm", 0):
        k = rmsnorm(k, g_k, cfg.rms_eps)
    if cfg.use_rope:
        k = rope(k, pos, cfg.rope_theta)
    return k, v


def ctx_project(feats, pos, weights, cfg):
    """Fusion + injection for every draft layer. Returns K, V of shape [N, T, Hkv, hd]."""
    H_t = ctx_fuse(feats, weights["W_c"], weights["g_c"], cfg.rms_eps)
    Ks, Vs = [], []
    for lw in weights["layers"]:
        k, v = ctx_kv(H_t, lw["W_k"], lw["W_v"], pos, cfg, lw.get("g_k"))
        Ks.append(k)
        Vs.append(v)
    return np.stack(Ks), np.stack(Vs)


# --------------------------------------------------------------------------------------------
# paged KV pool  [layer][page][K|V][kv_head][slot][hd]
# --------------------------------------------------------------------------------------------
def pool_write(pool, page_table_row, positions, K, V, page_size):
    """Store K, V ([N, T, Hkv, hd]) of tokens at logical `positions` into the pool."""
    for t, p in enumerate(positions):
        page = int(page_table_row[p // page_size])
        slot = p % page_size
        pool[:, page, 0, :, slot, :] = K[:, t]
        pool[:, page, 1, :, slot, :] = V[:, t]


def pool_read(pool, page_table_row, L, layer, page_size):
    """Gather the first L logical positions of one sequence: K, V of shape [L, Hkv, hd]."""
    Hkv, hd = pool.shape[3], pool.shape[5]
    K = np.empty((L, Hkv, hd), dtype=F64)
    V = np.empty((L, Hkv, hd), dtype=F64)
    for p0 in range(0, L, page_size):
        n = min(page_size, L - p0)
        page = int(page_table_row[p0 // page_size])
        K[p0:p0 + n] = np.transpose(_f64(pool[layer, page, 0, :, :n, :]), (1, 0, 2))
        V[p0:p0 + n] = np.transpose(_f64(pool[layer, page, 1, :, :n, :]), (1, 0, 2))
    return K, V


# --------------------------------------------------------------------------------------------
# attention over [context ; block]
# --------------------------------------------------------------------------------------------
def block_attention(q, k_ctx, v_ctx, k_blk, v_blk, scale, causal=False):
    """q: [R, Hq, hd]; k_ctx/v_ctx: [L, Hkv, hd]; k_blk/v_blk: [R, Hkv, hd]. Returns [R, Hq, hd].

    Every query row sees all L context entries. Draft mode (causal=False): it also sees all R block
    rows (bidirectional inside the block). Verify mode (causal=True): block row r sees block rows
    <= r only. Query head h reads kv head h // (Hq/Hkv)."""
    q = _f64(q)
    R, Hq, hd = q.shape
    Hkv = k_blk.shape[1]
    group = Hq // Hkv
    L = k_ctx.shape[0]
    out = np.empty((R, Hq, hd), dtype=F64)
    for h in range(Hq):
        kv = h // group
        keys = np.concatenate((_f64(k_ctx[:, kv]), _f64(k_blk[:, kv])), axis=0)   # [L+R, hd]
        vals = np.concatenate((_f64(v_ctx[:, kv]), _f64(v_blk[:, kv])), axis=0)
        s = (q[:, h] @ keys.T) * scale                                              # [R, L+R]
        if causal:
            r = np.arange(R)
            s[:, L:][r[None, :] > r[:, None]] = -np.inf
        s = s - np.max(s, axis=-1, keepdims=True)
        p = np.exp(s)
        p = p / np.sum(p, axis=-1, keepdims=True)
        out[:, h] = p @ vals
    return out


def block_attention_lse(q, k_ctx, v_ctx, k_blk, v_blk, scale, causal=False):
    """The log-sum-exp of every query row's scaled scores, [R, Hq] (natural logarithm): what a backward pass
    keeps from the forward instead of the probabilities."""
    q = _f64(q)
    R, Hq, hd = q.shape
    group = Hq // k_blk.shape[1]
    L = k_ctx.shape[0]
    lse = np.empty((R, Hq), dtype=F64)
    for h in range(Hq):
        kv = h // group
        keys = np.concatenate((_f64(k_ctx[:, kv]), _f64(k_blk[:, kv])), axis=0)
        s = (q[:, h] @ keys.T) * scale
        if causal:
            r = np.arange(R)
            s[:, L:][r[None, :] > r[:, None]] = -np.inf
        m = np.max(s, axis=-1)
        lse[:, h] = m + np.log(np.sum(np.exp(s - m[:, None]), axis=-1))
    return lse


def block_attention_backward(q, k_ctx, v_ctx, k_blk, v_blk, dout, scale, causal=False):
    """Gradient of block_attention for one block (training side, Sec. 4.2: many anchor blocks of one sequence are
    trained in a single forward and backward pass; a block attends to the injected context before its anchor and,
    in both directions, to itself). Given dout = d loss / d out [R, Hq, hd], returns
    (dq [R, Hq, hd], dk_ctx [L, Hkv, hd], dv_ctx [L, Hkv, hd], dk_blk [R, Hkv, hd], dv_blk [R, Hkv, hd]).

    Plain softmax-attention calculus per query head h (kv head h // group), keys = [context ; block]:
      P = softmax(scale * q K^T)            dV  = P^T dout
      dP = dout V^T                         dS  = P * (dP - rowsum(dP * P))
      dq = scale * dS K                     dK  = scale * dS^T q
    The gradients of a kv head add up over the query heads of its group. With many blocks over one cached
    sequence the context gradients of the blocks add up position by position (the caller sums them)."""
    q = _f64(q)
    dout = _f64(dout)
    R, Hq, hd = q.shape
    Hkv = k_blk.shape[1]
    group = Hq // Hkv
    L = k_ctx.shape[0]
    dq = np.zeros((R, Hq, hd), dtype=F64)
    dk = np.zeros((L + R, Hkv, hd), dtype=F64)
    dv = np.zeros((L + R, Hkv, hd), dtype=F64)
    for h in range(Hq):
        kv = h // group
        keys = np.concatenate((_f64(k_ctx[:, kv]), _f64(k_blk[:, kv])), axis=0)   # [L+R, hd]
        vals = np.concatenate((_f64(v_ctx[:, kv]), _f64(v_blk[:, kv])), axis=0)
        s = (q[:, h] @ keys.T) * scale
        if causal:
            r = np.arange(R)
            s[:, L:][r[None, :] > r[:, None]] = -np.inf
        s = s - np.max(s, axis=-1, keepdims=True)
        p = np.exp(s)
        p = p / np.sum(p, axis=-1, keepdims=True)                                  # [R, L+R]
        dv[:, kv] += p.T @ dout[:, h]
        dp = dout[:, h] @ vals.T
        ds = p * (dp - np.sum(dp * p, axis=-1, keepdims=True))
        dq[:, h] = (ds @ keys) * scale
        dk[:, kv] += (ds.T @ q[:, h]) * scale
    return dq, dk[:L], dv[:L], dk[L:], dv[L:]


# --------------------------------------------------------------------------------------------
# draft forward
# --------------------------------------------------------------------------------------------
def draft_layer(x, lw, k_ctx, v_ctx, pos, cfg, causal=False, return_kv=False):
    """One pre-norm layer on the block hidden states x [R, D] (H_d = the normalised hidden).
    return_kv: also return the block's own (position-encoded) k and v [R, Hkv, hd]."""
    R = x.shape[0]
    u = rmsnorm(x, lw["g1"], cfg.rms_eps)
    q = linear(u, lw["W_q"]).reshape(R, cfg.n_q_heads, cfg.head_dim)
    k = linear(u, lw["W_k"]).reshape(R, cfg.n_kv_heads, cfg.head_dim)
    v = linear(u, lw["W_v"]).reshape(R, cfg.n_kv_heads, cfg.head_dim)
    if getattr(cfg, "qk_norm", 0):       # per-head RMSNorm over head_dim (the target family's attention variant)
        q = rmsnorm(q, lw["g_q"], cfg.rms_eps)
        k = rmsnorm(k, lw["g_k"], cfg.rms_eps)
    if cfg.use_rope:
        q = rope(q, pos, cfg.rope_theta)
        k = rope(k, pos, cfg.rope_theta)
    a = block_attention(q, k_ctx, v_ctx, k, v, cfg.softmax_scale, causal=causal)
    x = x + linear(a.reshape(R, cfg.q_dim), lw["W_o"])
    u2 = rmsnorm(x, lw["g2"], cfg.rms_eps)
    h = silu(linear(u2, lw["W_gate"])) * linear(u2, lw["W_up"])
    out = x + linear(h, lw["W_down"])
    return (out, k, v) if return_kv else out


def lm_head(x, g_f, W_lm, eps):
    """Final norm and shared LM head: logits [R, V]."""
    return linear(rmsnorm(x, g_f, eps), W_lm)


def draft_block(anchor, L, ctx_K, ctx_V, weights, cfg, return_logits=False):
    """Single-pass draft of one block for one sequence.

    anchor: token id (the previous cycle's bonus token); L: context length; ctx_K/ctx_V: per-layer
    injected context [N][L, Hkv, hd] (already position-encoded). Rows r = 0..B-1 sit at positions
    L + r; row 0 embeds the anchor, rows 1.. embed the mask token."""
    B = cfg.block_size
    ids = np.full((B,), cfg.mask_token_id, dtype=np.int64)
    ids[0] = int(anchor)
    x = _f64(weights["embed"][ids])
    pos = L + np.arange(B)
    for i, lw in enumerate(weights["layers"]):
        x = draft_layer(x, lw, ctx_K[i], ctx_V[i], pos, cfg, causal=False)
    logits = lm_head(x, weights["g_f"], weights["W_lm"], cfg.rms_eps)
    tok, top1, margin = argmax_top2(logits)
    out = {"hidden": x, "ids": tok, "top1": top1, "margin": margin}
    if return_logits:
        out["logits"] = logits
    return out


# --------------------------------------------------------------------------------------------
# greedy verify / accept   (Sec. 3.1)
# --------------------------------------------------------------------------------------------
def verify_accept(draft_ids, target_ids, ctx_len):
    """draft_ids d_1..d_gamma; target_ids p_0..p_gamma = the target's greedy choice after
    [anchor, d_1..d_j]. a = longest prefix with d_i == p_{i-1}; tau = a + 1 in [1, gamma+1];
    emitted tokens d_1..d_a, p_a; the bonus p_a is the next anchor; KV commit length ctx_len + tau.

    Returns (tau, out_tokens [gamma+1] padded with -1, bonus, new_ctx_len)."""
    gamma = len(draft_ids)
    assert len(target_ids) == gamma + 1
    a = 0
    while a < gamma and int(draft_ids[a]) == int(target_ids[a]):
        a += 1
    out = np.full((gamma + 1,), -1, dtype=np.int64)
    out[:a] = np.asarray(draft_ids[:a], dtype=np.int64)
    out[a] = int(target_ids[a])
    return a + 1, out, int(target_ids[a]), int(ctx_len) + a + 1


def verify_accept_logits(draft_ids, target_logits, ctx_len):
    """Same, starting from the target's logits [gamma+1, V]."""
    p, _, _ = argmax_top2(target_logits)
    return verify_accept(draft_ids, p, ctx_len)


# --------------------------------------------------------------------------------------------
# sampling verify / accept (speculative sampling; the rule is stated in the header)
# --------------------------------------------------------------------------------------------
def softmax_t(logits, T):
    """softmax(logits / T) along the last axis, T > 0."""
    z = _f64(logits) / float(T)
    z = z - z.max(axis=-1, keepdims=True)
    e = np.exp(z)
    return e / e.sum(axis=-1, keepdims=True)


def sample_cdf(w, u):
    """Inverse-CDF draw from non-negative weights w (need not be normalised), u in [0, 1):
    the first index i with w_0 + ... + w_i >= u * sum(w) among indices with w_i > 0.
    Returns (index, margin): margin = distance of u * sum(w) to the nearest edge of that index's
    interval, relative to sum(w) (how far u is from changing the answer)."""
    w = _f64(w)
    c = np.cumsum(w)
    total = c[-1]
    assert total > 0
    x = float(u) * total
    i = int(np.searchsorted(c, x, side="left"))
    i = min(i, len(w) - 1)
    while w[i] <= 0 and i + 1 < len(w):   # u * total landed exactly on an edge shared with empty entries
        i += 1
    while w[i] <= 0:                      # ... at the very end of the vocabulary
        i -= 1
    lo = c[i] - w[i]
    return i, float(min(x - lo, c[i] - x) / total)


def verify_accept_sample(draft_ids, draft_logits, target_logits, T, u_accept, u_final, ctx_len):
    """Speculative-sampling verification of gamma drafts (rule in the header).
    draft_ids [gamma]; draft_logits [gamma, V]; target_logits [gamma+1, V]; u_accept [gamma];
    u_final scalar. Returns (tau, out_tokens [gamma+1] padded with -1, final token, new_ctx_len,
    info) where info = dict(accept_margin=[...], final_margin=..., a=..., residual=bool)."""
    gamma = len(draft_ids)
    p = softmax_t(target_logits, T)
    q = softmax_t(draft_logits, T) if gamma else np.zeros((0, p.shape[-1]))
    assert p.shape[0] == gamma + 1
    a = 0
    margins = []
    while a < gamma:
        d = int(draft_ids[a])
        lhs, rhs = float(u_accept[a]) * q[a, d], p[a, d]
        margins.append(abs(rhs - lhs) / max(rhs, lhs, 1e-300))
        if not lhs < rhs:
            break
        a += 1
    residual = a < gamma
    if residual:
        w = np.maximum(p[a] - q[a], 0.0)
        if w.sum() <= 0:
            w = p[a]
    else:
        w = p[gamma]
    tok, fm = sample_cdf(w, u_final)
    out = np.full((gamma + 1,), -1, dtype=np.int64)
    out[:a] = np.asarray(draft_ids[:a], dtype=np.int64)
    out[a] = tok
    return a + 1, out, tok, int(ctx_len) + a + 1, dict(accept_margin=margins, final_margin=fm, a=a, residual=residual)


# --------------------------------------------------------------------------------------------
# the target's verify pass (Sec. 3.1: all drafts scored in one parallel pass; Sec. 4.1: hidden states
# of k target layers are the drafter's context features)
# --------------------------------------------------------------------------------------------
def target_verify(tokens, L, ctx_K, ctx_V, weights, cfg, tap_layers):
    """A causal stack over the rows `tokens` (anchor, d_1 .. d_gamma) at positions L .. L+R-1, on top of
    the cached context ctx_K / ctx_V ([N][L, Hkv, hd], position-encoded): causal inside the block,
    full over the context. Returns dict(logits [R, V], ids, feats [R, len(tap_layers) * D] = hidden rows
    after the tapped layers side by side, K / V [N][R, Hkv, hd] = the block's entries for the cache)."""
    R = len(tokens)
    x = _f64(weights["embed"][np.asarray(tokens, dtype=np.int64)])
    pos = L + np.arange(R)
    taps, Ks, Vs = [], [], []
    for i, lw in enumerate(weights["layers"]):
        x, k, v = draft_layer(x, lw, ctx_K[i], ctx_V[i], pos, cfg, causal=True, return_kv=True)
        Ks.append(k)
        Vs.append(v)
        if i in tap_layers:
            taps.append(x)
    logits = lm_head(x, weights["g_f"], weights["W_lm"], cfg.rms_eps)
    ids, top1, margin = argmax_top2(logits)
    feats = np.concatenate(taps, axis=-1) if taps else np.zeros((R, 0))
    return dict(logits=logits, ids=ids, margin=margin, feats=feats, K=Ks, V=Vs)


# --------------------------------------------------------------------------------------------
# training loss of a block (Sec. 4.2 "Loss weighting", Eq. 4)
# --------------------------------------------------------------------------------------------
def loss_weights(B, gamma):
    """w[k], k = 0 .. B-1: 0 for the anchor row, exp(-(k-1)/gamma) for the predicted positions (Eq. 4)."""
    w = np.zeros((B,), dtype=F64)
    for k in range(1, B):
        w[k] = np.exp(-(k - 1) / F64(gamma))
    return w


def block_loss(logits, targets, gamma, want_grad=True):
    """logits [B, V] of one block (row 0 = anchor), targets [B] (entry 0 unused; negative = ignore).
    Returns dict(row_loss [B] = w_k * CE_k, loss = their sum, weight = sum of the weights that count,
    grad [B, V] = d loss / d logits)."""
    z = _f64(logits)
    B, V = z.shape
    w = loss_weights(B, gamma)
    row_loss = np.zeros((B,), dtype=F64)
    grad = np.zeros((B, V), dtype=F64) if want_grad else None
    weight = 0.0
    for k in range(1, B):
        t = int(targets[k])
        if t < 0:
            continue
        m = np.max(z[k])
        e = np.exp(z[k] - m)
        lse = m + np.log(np.sum(e))
        row_loss[k] = w[k] * (lse - z[k, t])
        weight += w[k]
        if want_grad:
            grad[k] = w[k] * (e / np.sum(e))
            grad[k, t] -= w[k]
    return dict(row_loss=row_loss, loss=float(np.sum(row_loss)), weight=float(weight), grad=grad)


# --------------------------------------------------------------------------------------------
# toy causal target model (only for the losslessness check of the speculative cycle)
# --------------------------------------------------------------------------------------------
def toy_target_forward(tokens, tw, tcfg, tap_layers):
    """Plain causal transformer over the whole token list. Returns (logits [T, V], feats
    [T, k*D] = hidden states after the tapped layers, concatenated along features)."""
    T = len(tokens)
    x = _f64(tw["embed"][np.asarray(tokens, dtype=np.int64)])
    pos = np.arange(T)
    empty = np.zeros((0, tcfg.n_kv_heads, tcfg.head_dim), dtype=F64)
    taps = []
    for i, lw in enumerate(tw["layers"]):
        x = draft_layer(x, lw, empty, empty, pos, tcfg, causal=True)
        if i in tap_layers:
            taps.append(x)
    logits = lm_head(x, tw["g_f"], tw["W_lm"], tcfg.rms_eps)
    return logits, np.concatenate(taps, axis=-1)
