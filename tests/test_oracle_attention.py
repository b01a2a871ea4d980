"""Pins for the oracle's attention: special cases with known answers, brute-force loops, and a
library routine for the textbook causal case."""
import math

import numpy as np
import torch

from oracle import dflash_oracle as orc


def _rand(rng, *shape):
    return rng.standard_normal(shape)


def _attention_loops(q, k_ctx, v_ctx, k_blk, v_blk, scale, causal):
    """Scalar-loop definition: softmax over the visible keys of q.k*scale, weighted sum of values."""
    R, Hq, hd = q.shape
    Hkv = k_blk.shape[1]
    L = k_ctx.shape[0]
    out = np.zeros((R, Hq, hd))
    for r in range(R):
        for h in range(Hq):
            kv = h // (Hq // Hkv)
            keys = [k_ctx[j, kv] for j in range(L)]
            vals = [v_ctx[j, kv] for j in range(L)]
            for j in range(R):
                if causal and j > r:
                    continue
                keys.append(k_blk[j, kv])
                vals.append(v_blk[j, kv])
            s = [sum(q[r, h, d] * kk[d] for d in range(hd)) * scale for kk in keys]
            m = max(s)
            e = [math.exp(v - m) for v in s]
            z = sum(e)
            for d in range(hd):
                out[r, h, d] = sum(e[j] * vals[j][d] for j in range(len(vals))) / z
    return out


def test_matches_scalar_loops_full_and_causal():
    rng = np.random.default_rng(0)
    R, Hq, Hkv, hd, L = 3, 4, 2, 4, 5
    q, kc, vc = _rand(rng, R, Hq, hd), _rand(rng, L, Hkv, hd), _rand(rng, L, Hkv, hd)
    kb, vb = _rand(rng, R, Hkv, hd), _rand(rng, R, Hkv, hd)
    for causal in (False, True):
        got = orc.block_attention(q, kc, vc, kb, vb, 0.37, causal=causal)
        np.testing.assert_allclose(got, _attention_loops(q, kc, vc, kb, vb, 0.37, causal), atol=1e-13)


def test_uniform_keys_give_mean_of_values():
    rng = np.random.default_rng(1)
    R, Hq, Hkv, hd, L = 4, 2, 1, 8, 10
    key = _rand(rng, hd)
    kc = np.broadcast_to(key, (L, Hkv, hd)).copy()
    kb = np.broadcast_to(key, (R, Hkv, hd)).copy()
    vc, vb = _rand(rng, L, Hkv, hd), _rand(rng, R, Hkv, hd)
    out = orc.block_attention(_rand(rng, R, Hq, hd), kc, vc, kb, vb, 0.5)
    mean_v = np.concatenate((vc, vb))[:, 0].mean(axis=0)
    for r in range(R):
        for h in range(Hq):
            np.testing.assert_allclose(out[r, h], mean_v, atol=1e-13)


def test_dominant_key_selects_its_value():
    rng = np.random.default_rng(2)
    R, Hq, Hkv, hd, L = 2, 2, 2, 8, 6
    q = np.ones((R, Hq, hd))
    kc, vc = 0.01 * _rand(rng, L, Hkv, hd), _rand(rng, L, Hkv, hd)
    kb, vb = 0.01 * _rand(rng, R, Hkv, hd), _rand(rng, R, Hkv, hd)
    kc[3, 1] = 100.0          # kv head 1, context entry 3
    kb[1, 0] = 100.0          # kv head 0, block row 1
    out = orc.block_attention(q, kc, vc, kb, vb, 1.0)
    np.testing.assert_allclose(out[0, 1], vc[3, 1], atol=1e-12)   # q head 1 -> kv head 1
    np.testing.assert_allclose(out[0, 0], vb[1, 0], atol=1e-12)   # q head 0 -> kv head 0, sees a LATER block row
    # in causal mode row 0 must not see block row 1
    outc = orc.block_attention(q, kc, vc, kb, vb, 1.0, causal=True)
    assert np.max(np.abs(outc[0, 0] - vb[1, 0])) > 1e-3
    np.testing.assert_allclose(outc[1, 0], vb[1, 0], atol=1e-12)


def test_context_permutation_invariance_and_last_row_modes_agree():
    rng = np.random.default_rng(3)
    R, Hq, Hkv, hd, L = 4, 4, 2, 8, 9
    q, kc, vc = _rand(rng, R, Hq, hd), _rand(rng, L, Hkv, hd), _rand(rng, L, Hkv, hd)
    kb, vb = _rand(rng, R, Hkv, hd), _rand(rng, R, Hkv, hd)
    base = orc.block_attention(q, kc, vc, kb, vb, 0.3)
    perm = rng.permutation(L)
    np.testing.assert_allclose(orc.block_attention(q, kc[perm], vc[perm], kb, vb, 0.3), base, atol=1e-13)
    causal = orc.block_attention(q, kc, vc, kb, vb, 0.3, causal=True)
    np.testing.assert_allclose(causal[-1], base[-1], atol=1e-13)
    assert np.max(np.abs(causal[0] - base[0])) > 1e-4


def test_gqa_equals_replicated_mha():
    rng = np.random.default_rng(4)
    R, Hq, Hkv, hd, L = 3, 6, 2, 4, 7
    q, kc, vc = _rand(rng, R, Hq, hd), _rand(rng, L, Hkv, hd), _rand(rng, L, Hkv, hd)
    kb, vb = _rand(rng, R, Hkv, hd), _rand(rng, R, Hkv, hd)
    g = Hq // Hkv
    rep = lambda a: np.repeat(a, g, axis=1)
    np.testing.assert_allclose(orc.block_attention(q, kc, vc, kb, vb, 0.5),
                               orc.block_attention(q, rep(kc), rep(vc), rep(kb), rep(vb), 0.5), atol=1e-13)


def test_causal_without_context_is_textbook_causal_attention():
    rng = np.random.default_rng(5)
    R, H, hd = 6, 3, 8
    q, k, v = _rand(rng, R, H, hd), _rand(rng, R, H, hd), _rand(rng, R, H, hd)
    empty = np.zeros((0, H, hd))
    got = orc.block_attention(q, empty, empty, k, v, 1.0 / math.sqrt(hd), causal=True)
    tq, tk, tv = (torch.from_numpy(a).permute(1, 0, 2)[None] for a in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0].permute(1, 0, 2)
    np.testing.assert_allclose(got, ref.numpy(), atol=1e-12)


def test_single_query_decode_and_split_merge_identity():
    rng = np.random.default_rng(6)
    Hq, Hkv, hd, L = 2, 1, 8, 12
    q, kc, vc = _rand(rng, 1, Hq, hd), _rand(rng, L, Hkv, hd), _rand(rng, L, Hkv, hd)
    kb, vb = _rand(rng, 1, Hkv, hd), _rand(rng, 1, Hkv, hd)
    out = orc.block_attention(q, kc, vc, kb, vb, 0.4)
    # merge of two partial softmaxes over a split of the keys (log-sum-exp identity)
    keys = np.concatenate((kc, kb))[:, 0]
    vals = np.concatenate((vc, vb))[:, 0]
    for h in range(Hq):
        s = keys @ q[0, h] * 0.4
        parts = []
        for sl in (slice(0, 5), slice(5, None)):
            m = s[sl].max()
            e = np.exp(s[sl] - m)
            parts.append((m, e.sum(), e @ vals[sl]))
        M = max(p[0] for p in parts)
        den = sum(p[1] * math.exp(p[0] - M) for p in parts)
        num = sum(p[2] * math.exp(p[0] - M) for p in parts)
        np.testing.assert_allclose(out[0, h], num / den, atol=1e-13)


def test_large_scores_do_not_overflow():
    q = np.full((1, 1, 4), 50.0)
    kb = np.full((1, 1, 4), 50.0)
    kc = np.zeros((2, 1, 4))
    vc = np.array([[[1.0, 0, 0, 0]], [[0, 1.0, 0, 0]]])
    vb = np.array([[[0, 0, 1.0, 0]]])
    out = orc.block_attention(q, kc, vc, kb, vb, 1.0)
    assert np.all(np.isfinite(out))
    np.testing.assert_allclose(out[0, 0], [0, 0, 1.0, 0], atol=1e-12)
