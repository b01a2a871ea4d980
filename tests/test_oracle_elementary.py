"""Pins for the oracle's elementary steps: closed forms, invariants and brute-force loops that do
not re-use the oracle's own expressions."""
import math
import os

import numpy as np
import pytest

from oracle import dflash_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_linear_matches_triple_loop():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((3, 7))
    W = rng.standard_normal((5, 7)).astype(np.float32)
    y = orc.linear(x, W)
    for m in range(3):
        for n in range(5):
            acc = 0.0
            for k in range(7):
                acc += x[m, k] * float(W[n, k])
            assert abs(y[m, n] - acc) < 1e-12
    # orientation: a weight with a single 1 at [out=2, in=4] copies input 4 to output 2
    W1 = np.zeros((5, 7), dtype=np.float32)
    W1[2, 4] = 1.0
    y1 = orc.linear(x, W1)
    assert np.array_equal(y1[:, 2], x[:, 4]) and np.count_nonzero(y1) == 3


def test_linear_chunking_is_invisible():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((2, 16))
    W = rng.standard_normal((orc._CHUNK_ROWS + 37, 16)).astype(np.float32)
    y = orc.linear(x, W)
    assert y.shape == (2, orc._CHUNK_ROWS + 37)
    sel = [0, orc._CHUNK_ROWS - 1, orc._CHUNK_ROWS, orc._CHUNK_ROWS + 36]
    for n in sel:
        assert abs(y[1, n] - float(np.dot(x[1], W[n].astype(np.float64)))) < 1e-12


def test_rmsnorm_closed_forms():
    eps = 1e-6
    # constant vector c -> g * c / sqrt(c^2 + eps)
    c = 3.0
    g = np.array([1.0, 2.0, -0.5, 0.25])
    out = orc.rmsnorm(np.full((4,), c), g, eps)
    np.testing.assert_allclose(out, g * c / math.sqrt(c * c + eps), rtol=1e-14)
    # hand-computed: y = (3, 4): mean square 12.5
    out = orc.rmsnorm(np.array([3.0, 4.0]), np.ones(2), 0.0)
    np.testing.assert_allclose(out, np.array([3.0, 4.0]) / math.sqrt(12.5), rtol=1e-15)
    rng = np.random.default_rng(3)
    y = rng.standard_normal((5, 64))
    o = orc.rmsnorm(y, np.ones(64), 0.0)
    np.testing.assert_allclose(np.sqrt(np.mean(o * o, axis=-1)), 1.0, rtol=1e-13)   # unit rms
    np.testing.assert_allclose(orc.rmsnorm(7.5 * y, np.ones(64), 0.0), o, rtol=1e-13)  # scale-free
    # eps really sits inside the square root, added to the MEAN (not the sum) of squares
    out = orc.rmsnorm(np.array([0.0, 0.0, 2.0, 0.0]), np.ones(4), 3.0)
    np.testing.assert_allclose(out[2], 2.0 / math.sqrt(1.0 + 3.0), rtol=1e-15)
    # rows are normalised independently
    o2 = orc.rmsnorm(np.stack((y[0], 100 * y[1])), np.ones(64), 0.0)
    np.testing.assert_allclose(o2[0], o[0], rtol=1e-13)


def test_silu_points():
    assert orc.silu(np.array([0.0]))[0] == 0.0
    np.testing.assert_allclose(orc.silu(np.array([40.0]))[0], 40.0, rtol=1e-15)
    np.testing.assert_allclose(orc.silu(np.array([-40.0]))[0], 0.0, atol=1e-15)
    np.testing.assert_allclose(orc.silu(np.array([1.0]))[0], 1.0 / (1.0 + math.exp(-1.0)), rtol=1e-15)
    # silu(x) - silu(-x) = x
    x = np.linspace(-5, 5, 41)
    np.testing.assert_allclose(orc.silu(x) - orc.silu(-x), x, atol=1e-14)


def _rope_pair_loop(x, pos, theta):
    T, H, hd = x.shape
    out = np.zeros_like(x)
    for t in range(T):
        for h in range(H):
            for i in range(hd // 2):
                ang = pos[t] * theta ** (-2.0 * i / hd)
                a, b = x[t, h, i], x[t, h, i + hd // 2]
                out[t, h, i] = a * math.cos(ang) - b * math.sin(ang)
                out[t, h, i + hd // 2] = a * math.sin(ang) + b * math.cos(ang)
    return out


def test_rope_properties():
    rng = np.random.default_rng(4)
    theta = 1.0e6
    x = rng.standard_normal((6, 3, 16))
    pos = np.array([0, 1, 5, 17, 300, 32767])
    y = orc.rope(x, pos, theta)
    # a plain 2-D rotation of each (i, i+hd/2) pair, written as loops
    np.testing.assert_allclose(y, _rope_pair_loop(x, pos, theta), atol=1e-12)
    # position 0 is the identity; rotations preserve pair norms
    np.testing.assert_array_equal(y[0], x[0])
    half = 8
    np.testing.assert_allclose(y[..., :half] ** 2 + y[..., half:] ** 2,
                               x[..., :half] ** 2 + x[..., half:] ** 2, rtol=1e-12)
    # <RoPE(q, m), RoPE(k, n)> depends on m - n only
    q = rng.standard_normal((1, 1, 16))
    k = rng.standard_normal((1, 1, 16))

    def dot(m, n):
        return float(np.sum(orc.rope(q, np.array([m]), theta) * orc.rope(k, np.array([n]), theta)))

    assert abs(dot(10, 3) - dot(1007, 1000)) < 1e-9
    assert abs(dot(10, 3) - dot(3, 10)) > 1e-6      # and it does depend on the sign of m - n
    # first pair rotates by exactly `pos` radians (frequency index 0 has inverse frequency 1)
    e = np.zeros((1, 1, 16))
    e[0, 0, 0] = 1.0
    r = orc.rope(e, np.array([2]), theta)
    np.testing.assert_allclose([r[0, 0, 0], r[0, 0, 8]], [math.cos(2.0), math.sin(2.0)], rtol=1e-14)


def test_rope_matches_fp32_table_generator():
    # The library is handed fp32 cos/sin tables built by the input module; the oracle evaluates its
    # own angles. The two must describe the same rotation.
    from paper_2602_06036_b200 import synth
    cfg = synth.TINY
    cos, sin = synth.rope_tables(cfg, 4100)
    rng = np.random.default_rng(5)
    x = rng.standard_normal((3, 2, cfg.head_dim))
    pos = np.array([0, 129, 4099])
    y = orc.rope(x, pos, cfg.rope_theta)
    half = cfg.head_dim // 2
    c = cos.numpy().astype(np.float64)[pos][:, None, :]
    s = sin.numpy().astype(np.float64)[pos][:, None, :]
    ref = np.concatenate((x[..., :half] * c - x[..., half:] * s,
                          x[..., half:] * c + x[..., :half] * s), axis=-1)
    np.testing.assert_allclose(y, ref, atol=5e-7)


def test_argmax_top2():
    rng = np.random.default_rng(6)
    z = rng.standard_normal((4, 1000))
    z[0, 777] = 9.0
    z[1, [5, 400, 999]] = 8.0            # three-way tie -> lowest index, margin 0
    z[2, 0] = np.nan                      # NaN never wins
    z[2, 123] = 7.0
    z[3, :] = np.nan                      # all-NaN row -> 0
    idx, top1, margin = orc.argmax_top2(z)
    assert idx.tolist() == [777, 5, 123, 0]
    assert top1[0] == 9.0 and top1[1] == 8.0 and margin[1] == 0.0
    second = np.sort(z[0])[-2]
    assert margin[0] == 9.0 - second
    # brute force on a small random matrix
    y = rng.integers(-3, 4, size=(50, 9)).astype(np.float64)
    idx, top1, margin = orc.argmax_top2(y)
    for r in range(50):
        best, bi = -math.inf, 0
        for j in range(9):
            if y[r, j] > best:
                best, bi = y[r, j], j
        others = [y[r, j] for j in range(9) if j != bi]
        assert idx[r] == bi and top1[r] == best and margin[r] == best - max(others)


def _golden():
    vals = {}
    with open(os.path.join(GOLDEN, "appendix_a3_memory.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            parts = line.split()
            vals[parts[0]] = (int(parts[1]), parts[2])
    return vals


def test_layouts_reproduce_appendix_a3_memory_figures():
    """The paper's worked numbers (App. A.3) fix the layouts: W_c is D x kD, the projection input
    is [tokens, k*D], its output [tokens, D], 2 bytes per element."""
    gold = _golden()
    D, k, bpe = 2048, 5, 2
    rng = np.random.default_rng(7)
    # use the oracle's own shape conventions at a scaled-down D and scale the byte counts
    d, T = 8, 4
    feats = rng.standard_normal((T, k * d))
    W_c = rng.standard_normal((d, k * d)).astype(np.float32)
    H_t = orc.ctx_fuse(feats, W_c, np.ones(d), 1e-6)
    assert H_t.shape == (T, d)
    s = D // d
    w_bytes = W_c.size * s * s * bpe
    in_bytes = feats.size // T * s * 2048 * bpe
    out_bytes = H_t.size // T * s * 2048 * bpe
    tmp_bytes = (feats.size // T + H_t.size // T) * s * 16 * bpe
    assert w_bytes == gold["W_c_bytes"][0]
    assert abs(in_bytes - gold["proj_input_bytes_seq2048"][0]) <= 0.06 * gold["proj_input_bytes_seq2048"][0]
    assert abs(out_bytes - gold["proj_output_bytes_seq2048"][0]) <= 0.06 * gold["proj_output_bytes_seq2048"][0]
    assert tmp_bytes < gold["decode_temp_bytes_B16_max"][0]


def test_ctx_fuse_concat_order_and_value():
    rng = np.random.default_rng(8)
    d, k, T = 6, 3, 5
    hs = [rng.standard_normal((T, d)) for _ in range(k)]
    Wb = [rng.standard_normal((d, d)).astype(np.float32) for _ in range(k)]
    g = rng.standard_normal(d)
    H = orc.ctx_fuse(np.concatenate(hs, axis=1), np.concatenate(Wb, axis=1), g, 1e-6)
    # W_c [h1; h2; h3] = sum_j W_j h_j, then the closed-form norm, token by token
    for t in range(T):
        y = sum(Wb[j].astype(np.float64) @ hs[j][t] for j in range(k))
        ref = g * y / math.sqrt(float(np.mean(y ** 2)) + 1e-6)
        np.testing.assert_allclose(H[t], ref, rtol=1e-12)
    # permuting the feature blocks together with the matching column blocks changes nothing
    perm = [2, 0, 1]
    H2 = orc.ctx_fuse(np.concatenate([hs[j] for j in perm], axis=1),
                      np.concatenate([Wb[j] for j in perm], axis=1), g, 1e-6)
    np.testing.assert_allclose(H2, H, rtol=1e-12)


def test_ctx_kv_heads_positions_and_v_unrotated():
    from paper_2602_06036_b200 import synth
    cfg = synth.TINY
    rng = np.random.default_rng(9)
    T = 4
    H_t = rng.standard_normal((T, cfg.d_model))
    W_k = rng.standard_normal((cfg.kv_dim, cfg.d_model)).astype(np.float32)
    W_v = rng.standard_normal((cfg.kv_dim, cfg.d_model)).astype(np.float32)
    pos = np.array([0, 3, 64, 1000])
    K, V = orc.ctx_kv(H_t, W_k, W_v, pos, cfg)
    assert K.shape == (T, cfg.n_kv_heads, cfg.head_dim)
    # V is the plain projection; head h takes rows h*hd .. (h+1)*hd of the weight
    ref_v = H_t @ W_v.astype(np.float64).T
    np.testing.assert_allclose(V[:, 1, :], ref_v[:, cfg.head_dim:2 * cfg.head_dim], rtol=1e-12)
    # K at position 0 is unrotated, elsewhere it is rotated (norm-preserving)
    ref_k = (H_t @ W_k.astype(np.float64).T).reshape(T, cfg.n_kv_heads, cfg.head_dim)
    np.testing.assert_allclose(K[0], ref_k[0], rtol=1e-12)
    assert np.max(np.abs(K[2] - ref_k[2])) > 1e-3
    np.testing.assert_allclose(np.linalg.norm(K, axis=-1), np.linalg.norm(ref_k, axis=-1), rtol=1e-12)


def test_pool_roundtrip_and_page_scatter():
    from paper_2602_06036_b200 import synth
    cfg = synth.TINY
    rng = np.random.default_rng(10)
    L = 150
    K = rng.standard_normal((cfg.n_layers, L, cfg.n_kv_heads, cfg.head_dim))
    V = rng.standard_normal((cfg.n_layers, L, cfg.n_kv_heads, cfg.head_dim))
    for table in ([0, 1, 2], [5, 2, 7]):
        pool = np.zeros(synth.kv_pool_shape(cfg, 8))
        orc.pool_write(pool, table, list(range(L)), K, V, cfg.page_size)
        k, v = orc.pool_read(pool, table, L, 0, cfg.page_size)
        np.testing.assert_array_equal(k, K[0])
        np.testing.assert_array_equal(v, V[0])
        # position p lives in page table[p // 64], slot p % 64, as [K|V][head][slot][hd]
        p = 131
        assert pool[0, table[p // 64], 0, 1, p % 64, 3] == K[0, p, 1, 3]
        assert pool[0, table[p // 64], 1, 0, p % 64, 5] == V[0, p, 0, 5]


def test_qk_norm_is_a_per_head_rmsnorm_before_the_rotation():
    # the optional attention variant (cfg.qk_norm): checked against explicit loops over heads, and through
    # two properties: the layer's output does not change when W_q (or W_k) is scaled by a positive constant,
    # and with it off the same scaling does change the output
    import dataclasses
    from paper_2602_06036_b200 import synth
    cfg = dataclasses.replace(synth.TINY, qk_norm=1, block_size=4)
    w = synth.weights_to_numpy(synth.make_weights(cfg, 21))
    lw = w["layers"][0]
    rng = np.random.default_rng(2)
    x = rng.normal(size=(4, cfg.d_model))
    kc = rng.normal(size=(9, cfg.n_kv_heads, cfg.head_dim))
    vc = rng.normal(size=(9, cfg.n_kv_heads, cfg.head_dim))
    pos = np.arange(9, 13)
    base = orc.draft_layer(x, lw, kc, vc, pos, cfg)
    scaled = dict(lw, W_q=lw["W_q"] * 3.7, W_k=lw["W_k"] * 0.21)
    np.testing.assert_allclose(orc.draft_layer(x, scaled, kc, vc, pos, cfg), base, rtol=0, atol=1e-4)      # exact up to eps / mean square
    off = dataclasses.replace(cfg, qk_norm=0)
    assert np.abs(orc.draft_layer(x, scaled, kc, vc, pos, off) - orc.draft_layer(x, lw, kc, vc, pos, off)).max() > 1e-2
    # context keys: loops over tokens and heads
    H_t = rng.normal(size=(5, cfg.d_model))
    K, V = orc.ctx_kv(H_t, lw["W_k"], lw["W_v"], np.arange(5), cfg, lw["g_k"])
    raw = (H_t @ lw["W_k"].T).reshape(5, cfg.n_kv_heads, cfg.head_dim)
    for t in range(5):
        for h in range(cfg.n_kv_heads):
            r = raw[t, h]
            n = lw["g_k"] * r / np.sqrt(np.mean(r * r) + cfg.rms_eps)
            np.testing.assert_allclose(K[t, h], orc.rope(n[None, None, :], np.array([t]), cfg.rope_theta)[0, 0], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(V, (H_t @ lw["W_v"].T).reshape(5, cfg.n_kv_heads, cfg.head_dim), rtol=1e-12)


def test_target_verify_continues_a_full_causal_forward():
    # the verify pass over the last rows, on top of the K/V its own earlier pass cached, must equal
    # the plain causal transformer run over the whole token list at once (logits and tapped features)
    import dataclasses
    from paper_2602_06036_b200 import synth
    tcfg = dataclasses.replace(synth.TINY, n_layers=3, block_size=4)
    tw = synth.weights_to_numpy(synth.make_weights(tcfg, 31))
    rng = np.random.default_rng(4)
    tokens = rng.integers(0, tcfg.vocab - 1, size=13).tolist()
    taps = (0, 2)
    full_logits, full_feats = orc.toy_target_forward(tokens, tw, tcfg, taps)
    empty = [np.zeros((0, tcfg.n_kv_heads, tcfg.head_dim))] * tcfg.n_layers
    Lp = 8
    pre = orc.target_verify(tokens[:Lp], 0, empty, empty, tw, tcfg, taps)
    np.testing.assert_allclose(pre["logits"], full_logits[:Lp], rtol=1e-9, atol=1e-9)
    inc = orc.target_verify(tokens[Lp:], Lp, pre["K"], pre["V"], tw, tcfg, taps)
    np.testing.assert_allclose(inc["logits"], full_logits[Lp:], rtol=1e-9, atol=1e-9)
    np.testing.assert_allclose(inc["feats"], full_feats[Lp:], rtol=1e-9, atol=1e-9)
    assert inc["feats"].shape == (5, 2 * tcfg.d_model) and len(inc["K"]) == 3 and inc["K"][0].shape == (5, tcfg.n_kv_heads, tcfg.head_dim)
    # a later row never influences an earlier one: dropping the last token leaves the other rows unchanged
    short = orc.target_verify(tokens[Lp:-1], Lp, pre["K"], pre["V"], tw, tcfg, taps)
    np.testing.assert_allclose(short["logits"], inc["logits"][:-1], rtol=1e-12, atol=1e-12)
