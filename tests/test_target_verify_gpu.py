"""Parity of the target's verify pass (causal stack over given tokens on a paged cache, tapped features,
block K/V written behind the committed context) against the CPU oracle, and one whole speculative
cycle on the GPU: target verify -> accept -> context projection from the tapped rows -> draft."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import dflash_oracle as orc
from paper_2602_06036_b200 import binding, synth
from tests.harness import Case, assert_close, assert_ids_match

pytestmark = pytest.mark.gpu


def _run_verify(case, tokens, taps):
    cfg, dev = case.cfg, case.device
    S, R = tokens.shape
    ids = torch.full((S, R), -3, dtype=torch.int32, device=dev)
    logits = torch.zeros((S * R, cfg.vocab), dtype=torch.float32, device=dev)
    feats = torch.zeros((S, R, len(taps) * cfg.d_model), dtype=cfg.torch_dtype, device=dev)
    case.lib.status.zero_()
    case.lib.dflash_target_verify(tokens.to(dev), case.ctx_len, max(case.ctx_lens + [0]), case.page_table, case.pool, list(taps), ids,
                                  feats_out=feats if taps else None, logits_out=logits)
    torch.cuda.synchronize()
    assert int(case.lib.status.item()) == 0
    return ids.cpu().numpy(), logits.cpu().numpy().reshape(S, R, -1), feats.float().cpu().numpy()


@pytest.mark.parametrize("name,layers,rows,taps,lens", [
    ("tiny", 3, 5, (0, 2), (0, 61, 130)),
    ("mid", 3, 17, (0, 1, 2), (0, 70, 200)),       # gamma + 1 = 17 rows: 68 query rows per kv head
    ("mid", 2, 9, (1,), (63,)),                    # the block crosses a page edge
    ("mid", 4, 16, (), (5, 300)),                  # no taps
])
def test_target_verify_matches_oracle(name, layers, rows, taps, lens):
    base = synth.TINY if name == "tiny" else synth.MID
    cfg = dataclasses.replace(base, n_layers=layers, block_size=min(rows, 16))
    case = Case(cfg, lens, seed=41, headroom=rows + 4)
    case.fill_pool_synthetic()
    before = case.pool.clone()
    tokens = torch.randint(0, cfg.vocab - 1, (case.S, rows), generator=synth.substream(41, "verify.tokens"), dtype=torch.int32)
    ids, logits, feats = _run_verify(case, tokens, taps)
    got_pool = case.pool.float().cpu().numpy()
    n_sure = 0
    for b, L in enumerate(case.ctx_lens):
        Ks, Vs = case.oracle_ctx(b)
        ref = orc.target_verify(tokens[b].tolist(), L, Ks, Vs, case.w_np, cfg, taps)
        assert_close(logits[b], ref["logits"], cfg.dtype, f"logits seq {b}")
        n_sure += assert_ids_match(ids[b], ref["ids"], ref["margin"], cfg.dtype, f"ids seq {b}")
        if taps:
            assert_close(feats[b], ref["feats"], cfg.dtype, f"tapped rows seq {b}")
        # the block's K/V landed at positions L .. L + rows - 1 of every layer, nothing else changed
        for i in range(cfg.n_layers):
            gk, gv = orc.pool_read(got_pool, case.page_table_cpu[b].numpy(), L + rows, i, cfg.page_size)
            assert_close(gk[L:], ref["K"][i], cfg.dtype, f"committed K seq {b} layer {i}")
            assert_close(gv[L:], ref["V"][i], cfg.dtype, f"committed V seq {b} layer {i}")
            bk, bv = orc.pool_read(before.float().cpu().numpy(), case.page_table_cpu[b].numpy(), L, i, cfg.page_size)
            assert np.array_equal(gk[:L], bk) and np.array_equal(gv[:L], bv)
    assert n_sure >= case.S * rows // 2


def test_a_later_row_never_changes_an_earlier_one():
    cfg = dataclasses.replace(synth.MID, n_layers=2)
    case = Case(cfg, (90,), seed=43, headroom=40)
    case.fill_pool_synthetic()
    tokens = torch.randint(0, cfg.vocab - 1, (1, 12), generator=synth.substream(43, "t"), dtype=torch.int32)
    _, full, _ = _run_verify(case, tokens, ())
    _, part, _ = _run_verify(case, tokens[:, :7].contiguous(), ())
    np.testing.assert_allclose(part[0], full[0, :7], rtol=0, atol=2e-2)


def test_one_speculative_cycle_on_the_gpu():
    # target (3 layers, taps 0 and 2) and drafter (2 layers, k = 2) with random weights of the same width:
    # verify [anchor, drafts] -> accept -> project the tapped rows of the kept tokens -> draft the next block.
    # Every step is compared with the oracle run from the same inputs.
    tcfg = dataclasses.replace(synth.MID, n_layers=3)
    dcfg = dataclasses.replace(synth.MID, n_layers=2, n_feat_layers=2, d_target=tcfg.d_model)
    taps = (0, 2)
    gamma = dcfg.block_size
    lens = (70, 131)
    tgt = Case(tcfg, lens, seed=51, headroom=2 * gamma + 4)
    drf = Case(dcfg, lens, seed=52, headroom=2 * gamma + 4)
    tgt.fill_pool_synthetic()
    drf.fill_pool_synthetic()
    dev = tgt.device
    S = len(lens)
    anchors = synth.make_anchors(dcfg, S, 52)
    drafts = drf.run_draft(anchors)["ids"]                                  # [S, gamma]
    tokens = torch.cat([anchors.view(S, 1), torch.from_numpy(drafts[:, :gamma].astype(np.int32))], dim=1).to(torch.int32)
    ids, logits, feats = _run_verify(tgt, tokens, taps)
    # accept on the GPU from the verify logits
    acc = torch.zeros(S, dtype=torch.int32, device=dev)
    out = torch.zeros((S, gamma + 1), dtype=torch.int32, device=dev)
    bonus = torch.zeros(S, dtype=torch.int32, device=dev)
    new_len = torch.zeros(S, dtype=torch.int32, device=dev)
    d_ids = torch.from_numpy(drafts.astype(np.int32)).to(dev)
    tgt.lib.dflash_verify_accept(d_ids, gamma, gamma, tgt.ctx_len, acc, out, bonus, new_len,
                                 logits=torch.from_numpy(logits).to(dev))
    torch.cuda.synchronize()
    for b, L in enumerate(lens):
        Ks, Vs = tgt.oracle_ctx(b)
        ref = orc.target_verify(tokens[b].tolist(), L, Ks, Vs, tgt.w_np, tcfg, taps)
        tau, o, bon, nl = orc.verify_accept_logits(drafts[b, :gamma], logits[b], L)      # integer work on the GPU's own logits
        assert (int(acc[b]), out[b].tolist(), int(bonus[b]), int(new_len[b])) == (tau, list(o), bon, nl)
        assert_close(feats[b], ref["feats"], tcfg.dtype, f"tapped rows seq {b}")
    # the kept tokens' tapped rows go straight into the drafter's context projection
    n_new = acc.clone()
    feats_dev = torch.from_numpy(feats).to(dcfg.torch_dtype).to(dev)
    drf.lib.dflash_ctx_project(feats_dev, n_new, drf.ctx_len, drf.page_table, drf.pool)
    torch.cuda.synchronize()
    got_pool = drf.pool.float().cpu().numpy()
    for b, L in enumerate(lens):
        n = int(acc[b])
        K, V = orc.ctx_project(feats[b, :n], np.arange(L, L + n), drf.w_np, dcfg)
        for i in range(dcfg.n_layers):
            gk, gv = orc.pool_read(got_pool, drf.page_table_cpu[b].numpy(), L + n, i, dcfg.page_size)
            assert_close(gk[L:], K[i], dcfg.dtype, f"injected K seq {b} layer {i}")
            assert_close(gv[L:], V[i], dcfg.dtype, f"injected V seq {b} layer {i}")


def test_speculative_decoding_on_the_gpu_equals_greedy_decoding():
    # fp32 target (2 layers) and drafter (1 layer); every kernel of the cycle runs on the GPU:
    #   verify [anchor, drafts] -> accept -> commit length -> project the kept rows' taps -> draft.
    # The emitted tokens must equal the target's own greedy decoding (one row per step through the same
    # call), whatever the drafter proposes; planted correct drafts make some cycles keep several tokens.
    tcfg = dataclasses.replace(synth.TINY, n_layers=2, block_size=8)
    dcfg = dataclasses.replace(synth.TINY, n_layers=1, block_size=8, n_feat_layers=2, d_target=tcfg.d_model)
    taps, gamma, P, n_out = (0, 1), 8, 11, 40
    S = 2
    room = P + n_out + 3 * gamma
    dev = torch.device("cuda:0")
    prompt = torch.randint(0, tcfg.vocab - 1, (S, P), generator=synth.substream(61, "prompt"), dtype=torch.int32)

    def fresh(cfg, seed):
        c = Case(cfg, (0,) * S, seed=seed, headroom=room)
        return c

    def prefill(tgt):
        ids = torch.zeros((S, P), dtype=torch.int32, device=dev)
        feats = torch.zeros((S, P, len(taps) * tcfg.d_model), dtype=tcfg.torch_dtype, device=dev)
        tgt.lib.dflash_target_verify(prompt.to(dev), tgt.ctx_len, 0, tgt.page_table, tgt.pool, list(taps), ids, feats_out=feats)
        tgt.ctx_len += P
        return ids[:, -1].clone(), feats

    # ---- plain greedy decoding with the target alone
    tgt = fresh(tcfg, 61)
    tok, _ = prefill(tgt)
    greedy = [tok.cpu()]
    one = torch.zeros((S, 1), dtype=torch.int32, device=dev)
    for _ in range(n_out + gamma):
        tgt.lib.dflash_target_verify(greedy[-1].view(S, 1).to(dev), tgt.ctx_len, P + n_out + gamma, tgt.page_table, tgt.pool, [], one)
        tgt.ctx_len += 1
        greedy.append(one[:, 0].cpu().clone())
    greedy = torch.stack(greedy, dim=1)                    # [S, n_out + gamma + 1]: greedy[:, 0] follows the prompt

    # ---- speculative decoding
    tgt, drf = fresh(tcfg, 61), fresh(dcfg, 62)
    anchor, feats = prefill(tgt)
    drf.lib.dflash_ctx_project(feats, torch.full((S,), P, dtype=torch.int32, device=dev), drf.ctx_len, drf.page_table, drf.pool)
    drf.ctx_len += P
    emitted = [[int(anchor[b])] for b in range(S)]
    acc = torch.zeros(S, dtype=torch.int32, device=dev)
    out = torch.zeros((S, gamma + 1), dtype=torch.int32, device=dev)
    bonus = torch.zeros(S, dtype=torch.int32, device=dev)
    new_len = torch.zeros(S, dtype=torch.int32, device=dev)
    drafts = torch.zeros((S, gamma), dtype=torch.int32, device=dev)
    logits = torch.zeros((S * (gamma + 1), tcfg.vocab), dtype=torch.float32, device=dev)
    vfeats = torch.zeros((S, gamma + 1, len(taps) * tcfg.d_model), dtype=tcfg.torch_dtype, device=dev)
    vids = torch.zeros((S, gamma + 1), dtype=torch.int32, device=dev)
    taus = []
    cycle = 0
    while min(len(e) for e in emitted) < n_out:
        drf.lib.dflash_draft_block(anchor, drf.ctx_len, P + n_out + gamma, drf.page_table, drf.pool, drafts)
        for b in range(S):                                  # plant a few correct drafts (known greedy continuation)
            k = (cycle + b) % 5
            n = len(emitted[b])
            drafts[b, :k] = greedy[b, n:n + k].to(dev)
        tokens = torch.cat([anchor.view(S, 1), drafts], dim=1).contiguous()
        tgt.lib.dflash_target_verify(tokens, tgt.ctx_len, P + n_out + gamma, tgt.page_table, tgt.pool, list(taps), vids,
                                     feats_out=vfeats, logits_out=logits)
        tgt.lib.dflash_verify_accept(drafts, gamma, gamma, tgt.ctx_len, acc, out, bonus, new_len, logits=logits.view(S, gamma + 1, -1))
        drf.lib.dflash_ctx_project(vfeats, acc, drf.ctx_len, drf.page_table, drf.pool)
        torch.cuda.synchronize()
        assert int(tgt.lib.status.item()) == 0 and int(drf.lib.status.item()) == 0
        for b in range(S):
            t = int(acc[b])
            emitted[b] += out[b, :t].tolist()
            taus.append(t)
        tgt.ctx_len.copy_(new_len)
        drf.ctx_len.copy_(new_len)
        anchor = bonus.clone()
        cycle += 1
    for b in range(S):
        assert emitted[b][:n_out] == greedy[b, :n_out].tolist(), b
    assert max(taus) >= 4 and min(taus) == 1
