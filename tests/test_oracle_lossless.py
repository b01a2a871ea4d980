"""Speculative decoding with the oracle's draft forward and accept rule reproduces plain greedy
decoding of the same toy target exactly (the paper's "lossless" property), whatever the drafter
proposes. Brute force on tiny random models."""
import numpy as np
import pytest

from oracle import dflash_oracle as orc
from paper_2602_06036_b200 import synth

TARGET = synth.DFlashConfig(n_layers=3, d_model=64, n_q_heads=4, n_kv_heads=2, head_dim=16, d_ffn=96,
                            vocab=97, n_feat_layers=2, d_target=64, block_size=8, dtype="fp32")
DRAFT = synth.DFlashConfig(n_layers=2, d_model=64, n_q_heads=4, n_kv_heads=2, head_dim=16, d_ffn=96,
                           vocab=97, n_feat_layers=2, d_target=64, block_size=8, dtype="fp32")
TAPS = (0, 2)


def _greedy(tw, prompt, n_new):
    toks = list(prompt)
    for _ in range(n_new):
        logits, _ = orc.toy_target_forward(toks, tw, TARGET, TAPS)
        toks.append(int(orc.argmax_top2(logits[-1])[0]))
    return toks[len(prompt):]


def _speculative(tw, dw, prompt, n_new, gamma_mode, cheat_rng=None, truth=None):
    """Full cycle: prefill -> ctx K/V -> [draft block -> causal verify -> accept -> ctx K/V of the
    committed positions] ... Returns (tokens, list of tau, final ctx_len)."""
    B = DRAFT.block_size
    seq = list(prompt)
    logits, feats = orc.toy_target_forward(seq, tw, TARGET, TAPS)
    anchor = int(orc.argmax_top2(logits[-1])[0])          # first token = first anchor
    produced = [anchor]
    L = len(seq)
    K, V = orc.ctx_project(feats, np.arange(L), dw, DRAFT)
    ctx_K = [K[i] for i in range(DRAFT.n_layers)]
    ctx_V = [V[i] for i in range(DRAFT.n_layers)]
    taus = []
    while len(produced) < n_new:
        d = orc.draft_block(anchor, L, ctx_K, ctx_V, dw, DRAFT)["ids"]
        drafts = list(d) if gamma_mode == "B" else list(d[1:])
        if cheat_rng is not None:
            # a drafter that knows part of the true continuation: first n drafts are right
            n = int(cheat_rng.integers(0, len(drafts) + 1))
            nxt = truth[len(produced):len(produced) + n]
            drafts[:len(nxt)] = nxt
        gamma = len(drafts)
        block = seq + [anchor] + [int(t) for t in drafts]
        logits, feats = orc.toy_target_forward(block, tw, TARGET, TAPS)
        tau, out, bonus, new_len = orc.verify_accept_logits(drafts, logits[L:L + gamma + 1], L)
        assert 1 <= tau <= gamma + 1 and new_len == L + tau
        taus.append(tau)
        # committed positions: the anchor and the accepted drafts (rows 0..tau-1 of the verify pass)
        Kn, Vn = orc.ctx_project(feats[L:L + tau], np.arange(L, L + tau), dw, DRAFT)
        for i in range(DRAFT.n_layers):
            ctx_K[i] = np.concatenate((ctx_K[i], Kn[i]))
            ctx_V[i] = np.concatenate((ctx_V[i], Vn[i]))
        seq = block[:L + tau]
        produced.extend(int(t) for t in out[:tau])
        anchor, L = bonus, new_len
    return produced, taus, L


@pytest.mark.parametrize("seed", [0, 1, 2])
@pytest.mark.parametrize("gamma_mode", ["B", "B-1"])
def test_speculative_equals_greedy(seed, gamma_mode):
    tw = synth.weights_to_numpy(synth.make_weights(TARGET, seed=100 + seed))
    dw = synth.weights_to_numpy(synth.make_weights(DRAFT, seed=200 + seed))
    prompt = [int(t) for t in np.random.default_rng(seed).integers(0, 96, size=5)]
    n_new = 64
    truth = _greedy(tw, prompt, n_new + DRAFT.block_size + 2)

    # (a) the random drafter (almost never right): tau stays 1, output still exact
    got, taus, L = _speculative(tw, dw, prompt, n_new, gamma_mode)
    assert got[:n_new] == truth[:n_new]
    assert sum(taus) + 1 == len(got) and L == len(prompt) + len(got) - 1

    # (b) a drafter that is right for a random prefix: long accepts, output still exact
    got, taus, L = _speculative(tw, dw, prompt, n_new, gamma_mode,
                                cheat_rng=np.random.default_rng(seed + 7), truth=truth)
    assert got[:n_new] == truth[:n_new]
    assert sum(taus) + 1 == len(got) and L == len(prompt) + len(got) - 1
    assert max(taus) > 3 and min(taus) <= 2
    gamma = DRAFT.block_size if gamma_mode == "B" else DRAFT.block_size - 1
    assert max(taus) <= gamma + 1
