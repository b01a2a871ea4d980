"""Pins for the greedy verify/accept rule (Sec. 3.1: tau in [1, gamma+1] including the bonus token;
lossless under greedy decoding)."""
import itertools

import numpy as np
import pytest

from oracle import dflash_oracle as orc
from paper_2602_06036_b200 import synth


def _literal_definition(d, p):
    """Largest a such that every one of the first a drafts equals the target's choice one step
    earlier, found by testing every a from gamma downwards."""
    gamma = len(d)
    for a in range(gamma, -1, -1):
        if all(d[i] == p[i] for i in range(a)):
            return a
    raise AssertionError


@pytest.mark.parametrize("gamma", [1, 2, 5, 8])
def test_all_match_patterns(gamma):
    V = 5
    p = [(3 * j + 1) % V for j in range(gamma + 1)]
    for pattern in itertools.product((0, 1), repeat=gamma):
        d = [p[i] if pattern[i] else (p[i] + 2) % V for i in range(gamma)]
        tau, out, bonus, new_len = orc.verify_accept(d, p, 100)
        a = _literal_definition(d, p)
        assert tau == a + 1 and 1 <= tau <= gamma + 1
        assert out[:a].tolist() == d[:a] and out[a] == p[a] and np.all(out[a + 1:] == -1)
        assert bonus == p[a] and new_len == 100 + tau
        # the first mismatch ends acceptance even if later drafts agree again
        first_bad = pattern.index(0) if 0 in pattern else gamma
        assert a == first_bad


def test_invariants():
    p = [7, 8, 9, 10]
    assert orc.verify_accept([7, 8, 9], p, 0)[0] == 4                 # draft == target argmax: all accepted
    tau, out, bonus, new_len = orc.verify_accept([1, 8, 9], p, 5)      # first draft wrong
    assert (tau, bonus, new_len) == (1, 7, 6) and out.tolist() == [7, -1, -1, -1]
    tau, out, bonus, _ = orc.verify_accept([7, 8, 0], p, 5)
    assert tau == 3 and out.tolist() == [7, 8, 9, -1] and bonus == 9


def test_planted_prefixes_over_many_seeds():
    gamma, V = 8, 1024
    taus = []
    for seed in range(200):
        logits, drafts, a = synth.make_verify_case(1, gamma, V, 0.3, seed)
        tau, out, bonus, new_len = orc.verify_accept_logits(drafts[0].numpy(), logits[0].numpy(), 128)
        assert tau == int(a[0]) + 1
        assert 1 <= tau <= gamma + 1 and new_len == 128 + tau
        assert bonus == int(np.argmax(logits[0, tau - 1].numpy()))
        taus.append(tau)
    # planted lengths follow min(Geometric(0.3), gamma): mean a = (1-p)/p * (1 - (1-p)^gamma) = 2.199
    assert abs(np.mean(taus) - 1 - 2.199) < 0.45
    assert max(taus) == gamma + 1 or max(taus) >= 7


def test_paper_mode_gamma_is_block_minus_one():
    # gamma = B-1: the same rule on one fewer draft; tau ranges over [1, B]
    B = 8
    logits, drafts, a = synth.make_verify_case(3, B - 1, 50, 0.2, 1)
    for b in range(3):
        tau = orc.verify_accept_logits(drafts[b].numpy(), logits[b].numpy(), 0)[0]
        assert tau == int(a[b]) + 1 <= B


def test_bf16_ties_take_lowest_index():
    z = np.zeros((2, 16))
    z[0, [4, 9]] = 2.5
    z[1, 3] = 1.0
    tau, out, bonus, _ = orc.verify_accept_logits([4], z, 0)
    assert tau == 2 and bonus == 3
    tau, out, bonus, _ = orc.verify_accept_logits([9], z, 0)
    assert tau == 1 and bonus == 4
