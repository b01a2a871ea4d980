"""Parity at the benchmark's full sizes (Qwen3-8B-shaped drafter, bf16), in the launch
configuration bench.py times: cfg1 end to end (context projection -> draft block) against the
oracle, cfg2/cfg3/cfg4 on sampled sequences, rows and tokens the oracle can compute one by one."""
import numpy as np
import pytest
import torch

from oracle import dflash_oracle as orc
from paper_2602_06036_b200 import synth
from tests.harness import Case, assert_close, assert_ids_match, TOL

pytestmark = pytest.mark.gpu

CFG = synth.QWEN3_8B
MAX_POS = 32768 + 64


@pytest.fixture(scope="module")
def model():
    from paper_2602_06036_b200 import binding
    w = synth.make_weights(CFG, 0)
    w_np = synth.weights_to_numpy(w)
    lib = binding.DFlash(CFG)
    cos, sin = synth.rope_tables(CFG, MAX_POS)
    lib.set_weights(synth.pack_device_weights(CFG, w), cos, sin)
    return w, w_np, lib


def _case(model, ctx_lens, seed=0):
    w, w_np, lib = model
    return Case(CFG, ctx_lens, seed=seed, weights=w, w_np=w_np, lib=lib)


def test_cfg1_end_to_end(model):
    wl = synth.workload("cfg1")
    case = _case(model, wl.ctx_lens)
    case.project_prefill(oracle=True)          # both sides project all 2048 context tokens
    cfg = CFG
    got_pool = case.pool.float().cpu().numpy()
    for i in range(cfg.n_layers):
        gk, gv = orc.pool_read(got_pool, case.page_table_cpu[0].numpy(), 2048, i, cfg.page_size)
        rk, rv = orc.pool_read(case.pool_np, case.page_table_cpu[0].numpy(), 2048, i, cfg.page_size)
        assert_close(gk, rk, "bf16", f"ctx K layer {i}")
        assert_close(gv, rv, "bf16", f"ctx V layer {i}")
    got = case.run_draft(want_logits=True)
    n_sure = case.check_draft(got)
    assert n_sure >= 4

def test_cfg1_step_as_benchmarked(model):
    # The step bench.py times: the rows the previous cycle committed (the last 17 of the 2048 the block attends
    # over) are projected INSIDE the draft call (one chained launch with the first QKV), then the block is drafted.
    wl = synth.workload("cfg1")
    cfg = CFG
    case = _case(model, wl.ctx_lens, seed=3)
    case.project_prefill(oracle=True)
    dev = case.device
    B, n = cfg.block_size, cfg.block_size + 1
    L = wl.ctx_lens[0]
    feats = synth.make_features(cfg, n, 3, "step.feats").reshape(1, n, cfg.feat_dim)
    anchors = synth.make_anchors(cfg, 1, 3)
    ids = torch.zeros((1, B), dtype=torch.int32, device=dev)
    hidden = torch.zeros((B, cfg.d_model), dtype=torch.float32, device=dev)
    logits = torch.zeros((B, cfg.vocab), dtype=torch.float32, device=dev)
    before = torch.tensor([L - n], dtype=torch.int32, device=dev)
    case.lib.status.zero_()
    case.lib.dflash_draft_block(anchors.to(dev), case.ctx_len, L, case.page_table, case.pool, ids, hidden_out=hidden,
                                logits_out=logits, ctx=(feats.to(dev), torch.tensor([n], dtype=torch.int32, device=dev), before))
    torch.cuda.synchronize()
    assert int(case.lib.status.item()) == 0
    pos = np.arange(L - n, L)
    K, V = orc.ctx_project(synth.to_numpy_f32(feats[0]), pos, case.w_np, cfg)
    orc.pool_write(case.pool_np, case.page_table_cpu[0].numpy(), list(pos), K, V, cfg.page_size)
    got_pool = case.pool.float().cpu().numpy()
    for i in range(cfg.n_layers):
        gk, gv = orc.pool_read(got_pool, case.page_table_cpu[0].numpy(), L, i, cfg.page_size)
        rk, rv = orc.pool_read(case.pool_np, case.page_table_cpu[0].numpy(), L, i, cfg.page_size)
        assert_close(gk[L - n:], rk[L - n:], "bf16", f"new ctx K layer {i}")
        assert_close(gv[L - n:], rv[L - n:], "bf16", f"new ctx V layer {i}")
    case.anchors_cpu = anchors
    ref = case.oracle_draft(0)
    assert_close(hidden.cpu().numpy(), ref["hidden"], "bf16", "hidden")
    assert_close(logits.cpu().numpy(), ref["logits"], "bf16", "logits")
    assert_ids_match(ids.cpu().numpy()[0], ref["ids"], ref["margin"], "bf16", "draft ids")


def test_cfg1_step_replayed_as_a_cuda_graph_equals_eager_launches(model):
    # bench.py times a CUDA-graph replay of the cfg1 step (token tiles of 16 / 32 rows, two K slabs per stage,
    # cluster launches): the replay must give, bit for bit, what the same calls give launched one by one.
    wl = synth.workload("cfg1")
    cfg = CFG
    case = _case(model, wl.ctx_lens, seed=5)
    case.project_prefill(oracle=False)
    dev = case.device
    S, B, L = 1, cfg.block_size, wl.ctx_lens[0]
    n = B + 1
    feats = synth.make_features(cfg, n, 5, "graph.feats").reshape(1, n, cfg.feat_dim).to(dev)
    anchors = synth.make_anchors(cfg, 1, 5).to(dev)
    n_new = torch.tensor([n], dtype=torch.int32, device=dev)
    before = torch.tensor([L - n], dtype=torch.int32, device=dev)
    tlog, _, _ = synth.make_verify_case(S, B, cfg.vocab, 0.25, 5, cfg.torch_dtype)
    tlog = tlog.to(dev)
    ids = torch.zeros((S, B), dtype=torch.int32, device=dev)
    hidden = torch.zeros((S * B, cfg.d_model), dtype=torch.float32, device=dev)
    top1 = torch.zeros((S, B), dtype=torch.float32, device=dev)
    tau = torch.zeros(S, dtype=torch.int32, device=dev)
    out = torch.zeros((S, B + 1), dtype=torch.int32, device=dev)
    bonus = torch.zeros(S, dtype=torch.int32, device=dev)
    new_len = torch.zeros(S, dtype=torch.int32, device=dev)
    pool0 = case.pool.clone()

    def step():
        case.lib.dflash_draft_block(anchors, case.ctx_len, L, case.page_table, case.pool, ids, top1=top1, hidden_out=hidden,
                                    ctx=(feats, n_new, before))
        case.lib.dflash_verify_accept(ids, B, B, case.ctx_len, tau, out, bonus, new_len, logits=tlog)

    def snapshot():
        torch.cuda.synchronize()
        assert int(case.lib.status.item()) == 0
        return [t.clone() for t in (case.pool, ids, hidden, top1, tau, out, bonus, new_len)]

    case.lib.status.zero_()
    step()
    eager = snapshot()
    step()
    again = snapshot()
    for a, b in zip(eager, again):                 # launch-to-launch: fixed reduction orders everywhere
        assert torch.equal(a, b)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            step()
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(3):
        case.pool.copy_(pool0)
        for t in (ids, hidden, top1, tau, out, bonus, new_len):
            t.zero_()
        g.replay()
        got = snapshot()
        for a, b in zip(eager, got):
            assert torch.equal(a, b)


def test_cfg2_ragged_batch_and_accept_from_logits(model):
    wl = synth.workload("cfg2")
    case = _case(model, wl.ctx_lens)
    case.fill_pool_synthetic()
    got = case.run_draft(want_logits=True)
    order = np.argsort(wl.ctx_lens)
    case.check_draft(got)                      # all 8 sequences, element by element
    # every sequence inside the batch equals the same sequence run alone
    b = int(order[-1])
    solo = _case(model, (wl.ctx_lens[b],))
    solo.page_table.copy_(case.page_table[b:b + 1, :solo.page_table.shape[1]])
    solo.pool = case.pool
    solo.n_pages = case.n_pages
    alone = solo.run_draft(anchors=case.anchors_cpu[b:b + 1], want_logits=False)
    B = CFG.block_size
    assert_close(alone["hidden"], got["hidden"][b * B:(b + 1) * B], "bf16", "batched vs alone")
    # verify / accept from bf16 logits [8, 17, V] with planted prefixes: bit exact
    S, g = wl.batch, B
    logits, drafts, planted = synth.make_verify_case(S, g, CFG.vocab, wl.accept_p, 0, torch.bfloat16)
    dev = case.device
    tau = torch.zeros(S, dtype=torch.int32, device=dev)
    toks = torch.zeros((S, g + 1), dtype=torch.int32, device=dev)
    bonus = torch.zeros(S, dtype=torch.int32, device=dev)
    new_len = torch.zeros(S, dtype=torch.int32, device=dev)
    case.lib.dflash_verify_accept(drafts.to(dev), g, g, case.ctx_len, tau, toks, bonus, new_len, logits=logits.to(dev))
    torch.cuda.synchronize()
    for s in range(S):
        t, out, bn, nl = orc.verify_accept_logits(drafts[s].numpy(), synth.to_numpy_f32(logits[s]), wl.ctx_lens[s])
        assert int(tau[s]) == t == int(planted[s]) + 1
        assert toks[s].tolist() == out.tolist() and int(bonus[s]) == bn and int(new_len[s]) == nl


def test_cfg3_long_context(model):
    wl = synth.workload("cfg3")
    case = _case(model, wl.ctx_lens)
    case.fill_pool_synthetic()
    got = case.run_draft(want_logits=True)
    case.check_draft(got)
    # context projection at large positions: sampled rows of a decode step appended at 32768
    cfg = CFG
    n = 17
    feats = synth.make_features(cfg, n, 3, "cfg3.decode").reshape(1, n, cfg.feat_dim)
    case.lib.dflash_ctx_project(feats.to(case.device), None, case.ctx_len, case.page_table, case.pool)
    torch.cuda.synchronize()
    assert int(case.lib.status.item()) == 0
    pos = np.arange(32768, 32768 + n)
    K, V = orc.ctx_project(synth.to_numpy_f32(feats[0]), pos, case.w_np, cfg)
    got_pool = case.pool
    for t, p in enumerate(pos):
        page = int(case.page_table_cpu[0, p // 64])
        gk = got_pool[:, page, 0, :, p % 64, :].float().cpu().numpy()
        gv = got_pool[:, page, 1, :, p % 64, :].float().cpu().numpy()
        assert_close(gk, K[:, t], "bf16", f"ctx K at position {p}")
        assert_close(gv, V[:, t], "bf16", f"ctx V at position {p}")


def test_cfg4_serving_mix_step(model):
    from paper_2602_06036_b200 import binding
    wl = synth.workload("cfg4")
    case = _case(model, wl.ctx_lens)
    case.fill_pool_synthetic()
    cfg, S, B = CFG, wl.batch, CFG.block_size
    g = B
    dev = case.device
    lens = np.array(wl.ctx_lens)
    # the shortest and the longest sequence plus six seeded picks: eight of the 32 sequences against the oracle
    rest = [b for b in range(S) if b not in (int(np.argmin(lens)), int(np.argmax(lens)))]
    picks = [int(np.argmin(lens)), int(np.argmax(lens))] + sorted(int(x) for x in np.random.default_rng(4).choice(rest, 6, replace=False))
    # (1) context projection of the rows committed by the previous cycle (n_new = tau, ragged)
    logits_unused, drafts, planted = synth.make_verify_case(S, g, 1000, wl.accept_p, 1)
    n_new = (planted + 1).to(torch.int32)
    feats = synth.make_features(cfg, S * (g + 1), 4, "cfg4.feats").reshape(S, g + 1, cfg.feat_dim)
    before = case.pool.clone()
    case.lib.status.zero_()
    case.lib.dflash_ctx_project(feats.to(dev), n_new.to(dev), case.ctx_len, case.page_table, case.pool)
    torch.cuda.synchronize()
    assert int(case.lib.status.item()) == 0
    for b in picks:
        n = int(n_new[b])
        pos = np.arange(lens[b], lens[b] + n)
        K, V = orc.ctx_project(synth.to_numpy_f32(feats[b, :n]), pos, case.w_np, cfg)
        for t, p in enumerate(pos):
            page = int(case.page_table_cpu[b, p // 64])
            assert_close(case.pool[:, page, 0, :, p % 64, :].float().cpu().numpy(), K[:, t], "bf16", "ctx K")
            assert_close(case.pool[:, page, 1, :, p % 64, :].float().cpu().numpy(), V[:, t], "bf16", "ctx V")
        p = int(lens[b] + n)                     # the slot after the last valid row is untouched
        page = int(case.page_table_cpu[b, p // 64])
        assert torch.equal(case.pool[:, page, :, :, p % 64], before[:, page, :, :, p % 64])
    case.pool.copy_(before)
    # (2) draft block for the whole batch, oracle on the eight picked sequences
    got = case.run_draft(want_logits=False)
    for b in picks:
        ref = case.oracle_draft(b, return_logits=False)
        assert_close(got["hidden"][b * B:(b + 1) * B], ref["hidden"], "bf16", f"hidden seq {b}")
        assert_ids_match(got["ids"][b], ref["ids"], ref["margin"], "bf16", f"ids seq {b}")
    # (3) target-shaped causal verify attention over (gamma+1) rows, one layer
    R = g + 1
    q = synth.normal((S, R, cfg.n_q_heads, cfg.head_dim), 1.0, 5, "v.q", torch.bfloat16)
    k = synth.normal((S, R, cfg.n_kv_heads, cfg.head_dim), 1.0, 5, "v.k", torch.bfloat16)
    v = synth.normal((S, R, cfg.n_kv_heads, cfg.head_dim), 1.0, 5, "v.v", torch.bfloat16)
    out = torch.zeros_like(q, device=dev)
    case.lib.dflash_block_attention(binding.ATTN_CAUSAL, q.to(dev), k.to(dev), v.to(dev), case.ctx_len, int(lens.max()),
                                    case.page_table, case.pool, 2, out)
    torch.cuda.synchronize()
    for b in picks[:4]:
        kc, vc = orc.pool_read(case.pool_np, case.page_table_cpu[b].numpy(), int(lens[b]), 2, cfg.page_size)
        ref = orc.block_attention(synth.to_numpy_f32(q[b]), kc, vc, synth.to_numpy_f32(k[b]), synth.to_numpy_f32(v[b]),
                                  cfg.softmax_scale, causal=True)
        assert_close(out[b].float().cpu().numpy(), ref, "bf16", f"verify attention seq {b}")
    # (4) LM head + argmax on a target-shaped hidden [S*(gamma+1), D], then accept in IDS mode
    M = S * R
    hid = synth.normal((M, cfg.d_model), 1.0, 6, "v.hidden", torch.bfloat16)
    tids = torch.zeros(M, dtype=torch.int32, device=dev)
    top1 = torch.zeros(M, dtype=torch.float32, device=dev)
    margin = torch.zeros(M, dtype=torch.float32, device=dev)
    case.lib.dflash_lmhead_argmax(hid.to(dev), 1, tids, top1, margin)
    torch.cuda.synchronize()
    rows = list(range(0, M, 23))
    z = orc.rmsnorm(synth.to_numpy_f32(hid[rows]), case.w_np["g_f"], cfg.rms_eps)
    ref_logits = orc.linear(z, case.w_np["W_lm"])
    rid, rtop, rmargin = orc.argmax_top2(ref_logits)
    got_ids = tids.cpu().numpy()[rows]
    sure = rmargin > TOL["bf16"]["margin"]
    assert sure.sum() >= 5 and np.array_equal(got_ids[sure], rid[sure])
    assert np.max(np.abs(top1.cpu().numpy()[rows] - ref_logits[np.arange(len(rows)), got_ids])) <= TOL["bf16"]["max_abs"]
    # planted drafts against the ids the kernel produced: accept is bit exact given the ids
    tids2 = tids.reshape(S, R).cpu()
    d = torch.randint(0, cfg.vocab, (S, g), generator=synth.substream(7, "cfg4.d"), dtype=torch.int32)
    for b in range(S):
        a = int(planted[b])
        d[b, :a] = tids2[b, :a]
        if a < g and d[b, a] == tids2[b, a]:
            d[b, a] = (d[b, a] + 1) % cfg.vocab
    tau = torch.zeros(S, dtype=torch.int32, device=dev)
    toks = torch.zeros((S, R), dtype=torch.int32, device=dev)
    bonus = torch.zeros(S, dtype=torch.int32, device=dev)
    new_len = torch.zeros(S, dtype=torch.int32, device=dev)
    case.lib.dflash_verify_accept(d.to(dev), g, g, case.ctx_len, tau, toks, bonus, new_len, target_ids=tids.reshape(S, R))
    torch.cuda.synchronize()
    for b in range(S):
        t, o, bn, nl = orc.verify_accept(d[b].numpy(), tids2[b].numpy(), int(lens[b]))
        assert int(tau[b]) == t == int(planted[b]) + 1 and toks[b].tolist() == o.tolist()
        assert int(bonus[b]) == bn and int(new_len[b]) == nl
