"""Structure checks on the oracle's composed draft forward (its parts are pinned elsewhere)."""
import dataclasses

import numpy as np

from oracle import dflash_oracle as orc
from paper_2602_06036_b200 import synth


def _setup(cfg, L, seed=0):
    w = synth.weights_to_numpy(synth.make_weights(cfg, seed))
    feats = synth.to_numpy_f32(synth.make_features(cfg, L, seed))
    K, V = orc.ctx_project(feats, np.arange(L), w, cfg)
    return w, [K[i] for i in range(cfg.n_layers)], [V[i] for i in range(cfg.n_layers)]


def test_without_positions_mask_rows_are_interchangeable():
    # Bidirectional attention inside the block + identical mask embeddings: with no positional
    # signal every mask row must produce the same hidden state. (A causal mask would break this.)
    cfg = dataclasses.replace(synth.TINY, use_rope=0)
    w, K, V = _setup(cfg, 20)
    out = orc.draft_block(5, 20, K, V, w, cfg)
    h = out["hidden"]
    for r in range(2, cfg.block_size):
        np.testing.assert_allclose(h[r], h[1], atol=1e-12)
    assert np.max(np.abs(h[0] - h[1])) > 1e-3
    # with rotary positions they differ
    w, K, V = _setup(synth.TINY, 20)
    h = orc.draft_block(5, 20, K, V, w, synth.TINY)["hidden"]
    assert np.max(np.abs(h[2] - h[1])) > 1e-4


def test_identity_layers_reduce_to_lm_head_of_embeddings():
    cfg = synth.TINY
    w, K, V = _setup(cfg, 8)
    for lw in w["layers"]:
        lw["W_o"] = np.zeros_like(lw["W_o"])
        lw["W_down"] = np.zeros_like(lw["W_down"])
    out = orc.draft_block(11, 8, K, V, w, cfg, return_logits=True)
    E = w["embed"].astype(np.float64)
    ids = [11] + [cfg.mask_token_id] * (cfg.block_size - 1)
    np.testing.assert_array_equal(out["hidden"], E[ids])
    x = E[ids]
    z = w["g_f"].astype(np.float64) * x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + cfg.rms_eps)
    ref = z @ w["W_lm"].astype(np.float64).T
    np.testing.assert_allclose(out["logits"], ref, atol=1e-11)
    assert out["ids"].tolist() == np.argmax(ref, axis=-1).tolist()


def test_context_enters_only_as_keys_and_values():
    # Replacing the context by a permutation of itself (K with V) leaves the block untouched; a
    # different context changes it; position offset L matters through the rotary encoding.
    cfg = synth.TINY
    w, K, V = _setup(cfg, 30)
    base = orc.draft_block(3, 30, K, V, w, cfg)["hidden"]
    perm = np.random.default_rng(0).permutation(30)
    same = orc.draft_block(3, 30, [k[perm] for k in K], [v[perm] for v in V], w, cfg)["hidden"]
    np.testing.assert_allclose(same, base, atol=1e-11)
    other = orc.draft_block(3, 30, [k[::-1] * 1.5 for k in K], V, w, cfg)["hidden"]
    assert np.max(np.abs(other - base)) > 1e-4
    shifted = orc.draft_block(3, 31, K, V, w, cfg)["hidden"]
    assert np.max(np.abs(shifted - base)) > 1e-6


def test_empty_context_is_allowed():
    cfg = synth.TINY
    w, _, _ = _setup(cfg, 1)
    empty = [np.zeros((0, cfg.n_kv_heads, cfg.head_dim))] * cfg.n_layers
    out = orc.draft_block(0, 0, empty, empty, w, cfg)
    assert out["ids"].shape == (cfg.block_size,) and np.all(np.isfinite(out["hidden"]))
