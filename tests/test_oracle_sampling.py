"""Pins of the oracle's sampling verification (speculative sampling; the paper's T = 1 setting,
Sec. 5.1) against what the mathematics fixes: exactness of the emitted distribution, a hand-worked
case, and the limits that reduce to other rules."""
import itertools

import numpy as np
import pytest

from oracle import dflash_oracle as orc


def _cells(edges):
    """Midpoints and lengths of the cells that `edges` (values in [0, 1]) cut the unit interval into."""
    e = np.unique(np.clip(np.concatenate([[0.0, 1.0], np.asarray(edges, dtype=np.float64)]), 0.0, 1.0))
    return [((a + b) / 2, b - a) for a, b in zip(e[:-1], e[1:]) if b - a > 1e-15]


@pytest.mark.parametrize("seed,V,T", [(0, 3, 1.0), (1, 5, 1.0), (2, 4, 0.7), (3, 6, 1.6)])
def test_first_emitted_token_is_distributed_as_the_target(seed, V, T):
    # One draft (gamma = 1). The draft token comes from sample_cdf(q, u_d); the cycle then emits either
    # it, or a residual draw. The map (u_d, u_a, u_f) -> first emitted token is piecewise constant: the
    # measure of each outcome is summed cell by cell and must equal p_0 (losslessness of speculative
    # sampling), whatever q is.
    rng = np.random.default_rng(seed)
    zq, zp = rng.normal(size=(1, V)) * 2, rng.normal(size=(2, V)) * 2
    q, p = orc.softmax_t(zq, T)[0], orc.softmax_t(zp, T)
    res = np.maximum(p[0] - q, 0)
    mass = np.zeros(V)
    d_cells = _cells(np.cumsum(q))
    f_edges = np.concatenate([np.cumsum(res) / res.sum() if res.sum() > 0 else [], np.cumsum(p[0]), np.cumsum(p[1])])
    for ud, wd in d_cells:
        d, _ = orc.sample_cdf(q, ud)
        for ua, wa in _cells([p[0, d] / q[d]]):
            for uf, wf in _cells(f_edges):
                tau, out, tok, _, _ = orc.verify_accept_sample([d], zq, zp, T, [ua], uf, 10)
                mass[out[0]] += wd * wa * wf
    np.testing.assert_allclose(mass.sum(), 1.0, atol=1e-12)
    np.testing.assert_allclose(mass, p[0], atol=1e-12)


def test_two_drafts_joint_distribution_of_the_first_two_tokens():
    # gamma = 2 with position-wise independent drafts (the block-diffusion case): the pair of tokens at
    # positions 0, 1 must follow p_0(x0) * p_1(x1) whenever the cycle emits two or more tokens, and the
    # marginal of position 0 is p_0 in every case. Position 1's target row here does not depend on x0
    # (a fixed table), which is all the rule needs to see.
    V, T = 3, 1.0
    rng = np.random.default_rng(7)
    zq, zp = rng.normal(size=(2, V)), rng.normal(size=(3, V))
    q, p = orc.softmax_t(zq, T), orc.softmax_t(zp, T)
    first = np.zeros(V)
    pair = np.zeros((V, V))
    edges_f = []
    for j in range(2):
        r = np.maximum(p[j] - q[j], 0)
        if r.sum() > 0:
            edges_f.append(np.cumsum(r) / r.sum())
    edges_f += [np.cumsum(p[j]) for j in range(3)]
    f_cells = _cells(np.concatenate(edges_f))
    for (u0, w0), (u1, w1) in itertools.product(_cells(np.cumsum(q[0])), _cells(np.cumsum(q[1]))):
        d0, _ = orc.sample_cdf(q[0], u0)
        d1, _ = orc.sample_cdf(q[1], u1)
        for (a0, wa0), (a1, wa1) in itertools.product(_cells([p[0, d0] / q[0, d0]]), _cells([p[1, d1] / q[1, d1]])):
            for uf, wf in f_cells:
                tau, out, _, _, _ = orc.verify_accept_sample([d0, d1], zq, zp, T, [a0, a1], uf, 0)
                w = w0 * w1 * wa0 * wa1 * wf
                first[out[0]] += w
                if tau >= 2:
                    pair[out[0], out[1]] += w
    np.testing.assert_allclose(first, p[0], atol=1e-12)
    # P(tau >= 2, x0, x1) = P(x0 kept) * p_1(x1), and P(x0 kept) = min(p_0, q_0)(x0)
    kept = np.minimum(p[0], q[0])
    np.testing.assert_allclose(pair, kept[:, None] * p[1][None, :], atol=1e-12)


def test_hand_worked_two_token_vocabulary():
    # q = (1/2, 1/2), p = (4/5, 1/5) at T = 1 (logits = log probabilities).
    # draft token 1: kept iff u < p/q = 0.4; on rejection the residual is (0.3, 0) / 0.3 -> token 0.
    # draft token 0: p/q = 1.6 > 1 -> always kept.
    zq = np.log(np.array([[0.5, 0.5]]))
    zp = np.log(np.array([[0.8, 0.2], [0.25, 0.75]]))
    tau, out, tok, new_len, info = orc.verify_accept_sample([1], zq, zp, 1.0, [0.39], 0.5, 7)
    assert (tau, list(out), tok, new_len) == (2, [1, 1], 1, 9)          # kept; bonus from p_1: cdf (0.25, 1.0), u = 0.5 -> 1
    tau, out, tok, new_len, info = orc.verify_accept_sample([1], zq, zp, 1.0, [0.41], 0.99, 7)
    assert (tau, list(out), tok, new_len) == (1, [0, -1], 0, 8) and info["residual"]
    tau, out, tok, _, _ = orc.verify_accept_sample([0], zq, zp, 1.0, [0.999999], 0.1, 7)
    assert (tau, list(out), tok) == (2, [0, 0], 0)                       # bonus: u = 0.1 < 0.25 -> 0


def test_identical_distributions_keep_every_draft():
    rng = np.random.default_rng(3)
    z = rng.normal(size=(6, 50)) * 3
    for trial in range(20):
        u = rng.random(5)
        ids = [orc.sample_cdf(orc.softmax_t(z[j], 0.9), rng.random())[0] for j in range(5)]
        tau, out, tok, _, info = orc.verify_accept_sample(ids, z[:5], z, 0.9, u, rng.random(), 0)
        assert tau == 6 and list(out[:5]) == ids and not info["residual"]


def test_low_temperature_limit_is_the_greedy_rule():
    rng = np.random.default_rng(11)
    V, gamma = 40, 6
    for trial in range(30):
        zp = rng.normal(size=(gamma + 1, V)) * 4
        zq = zp[:gamma] + rng.normal(size=(gamma, V)) * (2.0 if trial % 2 else 0.2)
        ids = [int(np.argmax(zq[j])) for j in range(gamma)]       # T -> 0 drafting
        g_tau, g_out, g_bonus, g_len = orc.verify_accept_logits(ids, zp, 5)
        tau, out, tok, new_len, _ = orc.verify_accept_sample(ids, zq, zp, 1e-3, rng.random(gamma) * 0.98 + 0.01,
                                                             rng.random(), 5)
        assert (tau, list(out), tok, new_len) == (g_tau, list(g_out), g_bonus, g_len)


def test_rejection_only_emits_tokens_the_target_prefers():
    rng = np.random.default_rng(5)
    V = 30
    n_rej = 0
    for trial in range(200):
        zq, zp = rng.normal(size=(1, V)) * 2, rng.normal(size=(2, V)) * 2
        q, p = orc.softmax_t(zq, 1.0)[0], orc.softmax_t(zp, 1.0)
        d, _ = orc.sample_cdf(q, rng.random())
        tau, out, tok, _, info = orc.verify_accept_sample([d], zq, zp, 1.0, [rng.random()], rng.random(), 0)
        if info["residual"]:
            n_rej += 1
            assert p[0, tok] > q[tok] and tok != d
    assert n_rej > 20


def test_sample_cdf_edges_and_margin():
    w = np.array([0.0, 2.0, 0.0, 1.0, 1.0])
    assert orc.sample_cdf(w, 0.0)[0] == 1                # never an empty entry
    assert orc.sample_cdf(w, 0.49)[0] == 1
    assert orc.sample_cdf(w, 0.51)[0] == 3
    assert orc.sample_cdf(w, 0.999999)[0] == 4
    i, m = orc.sample_cdf(w, 0.25)
    assert i == 1 and abs(m - 0.25) < 1e-12              # interval [0, 0.5): 0.25 from either edge
    counts = np.zeros(5)
    for u in (np.arange(4000) + 0.5) / 4000:
        counts[orc.sample_cdf(w, u)[0]] += 1
    np.testing.assert_allclose(counts / 4000, w / w.sum(), atol=1e-3)
