"""Pins for the oracle's training loss of a block (Sec. 4.2 "Loss weighting", Eq. 4; App. A.1)."""
import numpy as np
import pytest

from oracle import dflash_oracle as orc


@pytest.mark.parametrize("B,gamma", [(16, 7.0), (10, 5.0), (8, 4.0)])      # the settings of App. A.1
def test_weights_start_at_one_and_decay_by_a_constant_ratio(B, gamma):
    w = orc.loss_weights(B, gamma)
    assert w[0] == 0.0 and w[1] == 1.0
    ratios = w[2:] / w[1:-1]
    np.testing.assert_allclose(ratios, np.exp(-1.0 / gamma), rtol=1e-14)
    # closed form of the geometric sum
    r = np.exp(-1.0 / gamma)
    np.testing.assert_allclose(w.sum(), (1 - r ** (B - 1)) / (1 - r), rtol=1e-13)
    # Eq. 4 at the last position of a block of 16 with gamma = 7: exp(-14/7)
    if B == 16:
        np.testing.assert_allclose(w[15], np.exp(-2.0), rtol=1e-15)


def test_uniform_logits_cost_ln_v_per_unit_weight():
    B, V, gamma = 8, 37, 4.0
    z = np.full((B, V), 3.25)
    t = np.arange(B) % V
    r = orc.block_loss(z, t, gamma)
    w = orc.loss_weights(B, gamma)
    np.testing.assert_allclose(r["row_loss"], w * np.log(V), rtol=1e-13)
    np.testing.assert_allclose(r["loss"], w.sum() * np.log(V), rtol=1e-13)
    np.testing.assert_allclose(r["weight"], w.sum(), rtol=1e-15)


def test_dominant_logit_costs_nothing_and_the_wrong_one_costs_the_gap():
    B, V, gamma = 4, 11, 5.0
    z = np.zeros((B, V))
    z[:, 3] = 80.0
    right = orc.block_loss(z, np.full(B, 3), gamma)
    assert 0.0 <= right["loss"] < 1e-12
    wrong = orc.block_loss(z, np.full(B, 5), gamma)
    np.testing.assert_allclose(wrong["row_loss"][1:], orc.loss_weights(B, gamma)[1:] * 80.0, rtol=1e-12)


def test_gradient_rows_sum_to_zero_and_match_finite_differences():
    rng = np.random.default_rng(5)
    B, V, gamma = 6, 9, 3.0
    z = rng.normal(size=(B, V)) * 2.0
    t = rng.integers(0, V, size=B)
    t[4] = -1                                   # an ignored position
    r = orc.block_loss(z, t, gamma)
    np.testing.assert_allclose(r["grad"].sum(axis=1), 0.0, atol=1e-14)
    assert np.all(r["grad"][0] == 0.0) and np.all(r["grad"][4] == 0.0) and r["row_loss"][4] == 0.0
    h = 1e-6
    num = np.zeros_like(z)
    for i in range(B):
        for j in range(V):
            zp = z.copy(); zp[i, j] += h
            zm = z.copy(); zm[i, j] -= h
            num[i, j] = (orc.block_loss(zp, t, gamma, want_grad=False)["loss"] -
                         orc.block_loss(zm, t, gamma, want_grad=False)["loss"]) / (2 * h)
    np.testing.assert_allclose(r["grad"], num, atol=1e-8)


def test_infinite_gamma_is_the_unweighted_sum_of_cross_entropies():
    rng = np.random.default_rng(6)
    B, V = 5, 13
    z = rng.normal(size=(B, V))
    t = rng.integers(0, V, size=B)
    r = orc.block_loss(z, t, 1e300)
    # cross entropy written independently: -log of the softmax probability of the target
    p = np.exp(z) / np.exp(z).sum(axis=1, keepdims=True)
    ce = -np.log(p[np.arange(B), t])
    np.testing.assert_allclose(r["loss"], ce[1:].sum(), rtol=1e-13)
    np.testing.assert_allclose(r["weight"], B - 1, rtol=1e-15)


def test_shifting_a_row_changes_nothing():
    rng = np.random.default_rng(7)
    B, V, gamma = 4, 7, 7.0
    z = rng.normal(size=(B, V))
    t = rng.integers(0, V, size=B)
    a = orc.block_loss(z, t, gamma)
    b = orc.block_loss(z + 1000.0, t, gamma)
    np.testing.assert_allclose(a["row_loss"], b["row_loss"], rtol=1e-9)
    np.testing.assert_allclose(a["grad"], b["grad"], atol=1e-12)
