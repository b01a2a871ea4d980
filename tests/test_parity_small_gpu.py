"""Element-by-element parity of the CUDA path against the CPU oracle on the tiny fp32 configuration
and on a reduced bf16 shape (several weight tiles, ragged vocabulary tail, ragged batch, empty
context), through the C ABI."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import dflash_oracle as orc
from paper_2602_06036_b200 import synth
from tests.harness import Case, assert_close, assert_ids_match, TOL

pytestmark = pytest.mark.gpu


def _check_pool(case):
    cfg = case.cfg
    got = case.pool.float().cpu().numpy()
    for b, L in enumerate(case.ctx_lens):
        for i in range(cfg.n_layers):
            gk, gv = orc.pool_read(got, case.page_table_cpu[b].numpy(), L, i, cfg.page_size)
            rk, rv = orc.pool_read(case.pool_np, case.page_table_cpu[b].numpy(), L, i, cfg.page_size)
            if L:
                assert_close(gk, rk, cfg.dtype, f"ctx K seq {b} layer {i}")
                assert_close(gv, rv, cfg.dtype, f"ctx V seq {b} layer {i}")
    # pages nobody owns stay untouched (zero)
    owned = set(int(p) for p in case.page_table_cpu.reshape(-1).tolist() if p >= 0)
    free = [p for p in range(case.n_pages) if p not in owned]
    assert free and float(np.abs(got[:, free]).max()) == 0.0


@pytest.mark.parametrize("name", ["cfg0", "mid"])
def test_full_cycle_matches_oracle(name):
    wl = synth.workload(name)
    case = Case(wl.cfg, wl.ctx_lens, seed=wl.seed)
    case.project_prefill()
    _check_pool(case)
    got = case.run_draft()
    n_sure = case.check_draft(got)
    assert n_sure >= case.S * wl.cfg.block_size // 2       # the id check is not vacuous


def test_tiny_without_rope_and_paper_block_sizes():
    for B, use_rope in ((8, 0), (1, 1), (10, 1)):
        cfg = dataclasses.replace(synth.TINY, block_size=B, use_rope=use_rope)
        case = Case(cfg, (65,), seed=3)
        case.project_prefill()
        got = case.run_draft()
        case.check_draft(got)


@pytest.mark.parametrize("B,k,layers,lens", [(8, 3, 2, (33, 150)), (10, 5, 3, (0, 64, 129)), (16, 5, 1, (257,)),
                                             (16, 3, 8, (40, 100))])     # 8 layers: the context K/V of layer 8 takes a second launch
def test_bf16_block_sizes_and_feature_counts(B, k, layers, lens):
    # tensor-core path at the block sizes the paper runs (8, 10, 16: Sec. 5.3 and the LLaMA setting),
    # with k = 5 tapped layers (App. A.1) and other layer counts; contexts end inside, at and past a page edge
    cfg = dataclasses.replace(synth.MID, block_size=B, n_feat_layers=k, n_layers=layers)
    case = Case(cfg, lens, seed=11)
    case.project_prefill()
    _check_pool(case)
    got = case.run_draft()
    n_sure = case.check_draft(got)
    assert n_sure >= case.S * B // 2


@pytest.mark.parametrize("name", ["cfg0", "mid"])
def test_block_size_chosen_per_call(name):
    # one handle (block size 8 or 16), blocks of fewer rows per call (Sec. 5.3: a drafter trained with a
    # large block also drafts smaller ones); the oracle runs the same weights at that block size
    wl = synth.workload(name)
    case = Case(wl.cfg, wl.ctx_lens, seed=wl.seed)
    case.project_prefill()
    full = wl.cfg.block_size
    for rows in sorted({1, full // 2, min(10, full), full}):
        cfg_r = dataclasses.replace(wl.cfg, block_size=rows)
        S, dev = case.S, case.device
        ids = torch.full((S, rows), -7, dtype=torch.int32, device=dev)
        margin = torch.zeros((S, rows), dtype=torch.float32, device=dev)
        logits = torch.zeros((S * rows, wl.cfg.vocab), dtype=torch.float32, device=dev)
        anchors = synth.make_anchors(wl.cfg, S, wl.seed)
        case.lib.status.zero_()
        case.lib.dflash_draft_block(anchors.to(dev), case.ctx_len, max(case.ctx_lens + [0]), case.page_table, case.pool, ids,
                                    margin=margin, logits_out=logits, block_rows=rows)
        torch.cuda.synchronize()
        assert int(case.lib.status.item()) == 0
        got_logits = logits.cpu().numpy().reshape(S, rows, -1)
        for b in range(S):
            Ks, Vs = case.oracle_ctx(b)
            ref = orc.draft_block(int(anchors[b]), case.ctx_lens[b], Ks, Vs, case.w_np, cfg_r, return_logits=True)
            assert_close(got_logits[b], ref["logits"], wl.cfg.dtype, f"logits rows={rows} seq {b}")
            sure = ref["margin"] > (0.1 if wl.cfg.dtype == "bf16" else 1e-3)
            assert (ids[b].cpu().numpy()[sure] == ref["ids"][sure]).all()
    with pytest.raises(Exception):
        case.lib.dflash_draft_block(anchors.to(dev), case.ctx_len, 0, case.page_table, case.pool, ids, block_rows=full + 1)


@pytest.mark.parametrize("base,over", [("tiny", {}), ("mid", {}), ("mid", dict(head_dim=64, n_q_heads=8, n_kv_heads=2)),
                                       ("mid", dict(block_size=10, n_layers=3)), ("mid12", {})])
def test_per_head_qk_norm(base, over):
    # the optional attention variant: q and k heads RMS-normalised (own gains) before the rotation, for
    # block rows and for the injected context keys; CUDA-core path (tiny), tensor-core path with one head
    # per 128-row weight tile (hd = 128) and with two (hd = 64); 12 sequences: 192 block rows, the contraction
    # kernel's CTA-pair form with the head norms in its epilogues
    cfg = dataclasses.replace(synth.TINY if base == "tiny" else synth.MID, qk_norm=1, **over)
    lens = {"tiny": (65,), "mid": (0, 70, 131), "mid12": (0, 70, 131, 5, 64, 65, 200, 17, 33, 128, 90, 1)}[base]
    case = Case(cfg, lens, seed=23)
    case.project_prefill()
    _check_pool(case)
    got = case.run_draft()
    n_sure = case.check_draft(got)
    assert n_sure >= case.S * cfg.block_size // 2
    # and it is not a no-op: the same inputs without the norm give other logits
    off = Case(dataclasses.replace(cfg, qk_norm=0), case.ctx_lens, seed=23)
    off.project_prefill()
    assert np.abs(off.run_draft()["logits"] - got["logits"]).max() > 0.05


@pytest.mark.parametrize("seed", range(8))
def test_bf16_random_shapes(seed):
    # seeded draws of widths, head counts, layer counts, block sizes and batch sizes: every token-tile size of
    # the contraction kernel (16 ... 256 rows), shared and whole-tile schedules, chained and single launches
    rng = np.random.default_rng(1000 + seed)
    hq, hkv = [(2, 1), (4, 2), (8, 2), (8, 8), (4, 4)][rng.integers(5)]
    cfg = dataclasses.replace(
        synth.MID, d_model=int(rng.choice([256, 384, 512, 640, 1024])), d_ffn=int(rng.choice([512, 1024, 1536, 2048])),
        n_q_heads=hq, n_kv_heads=hkv, vocab=int(rng.choice([1000, 3001, 8192, 20011])), n_layers=int(rng.integers(1, 5)),
        block_size=int(rng.choice([4, 8, 10, 16])), n_feat_layers=int(rng.choice([1, 3, 5])), d_target=int(rng.choice([256, 512])),
        qk_norm=int(rng.integers(2)))
    S = int(rng.choice([1, 2, 3, 5, 9, 16]))
    lens = tuple(int(x) for x in rng.integers(0, 260, size=S))
    case = Case(cfg, lens, seed=seed)
    case.project_prefill()
    _check_pool(case)
    got = case.run_draft()
    case.check_draft(got)


@pytest.mark.parametrize("name,layers", [("mid", 2), ("mid", 6), ("mid", 7), ("cfg0", 1)])
def test_context_projection_inside_the_draft_call(name, layers):
    # draft_block with `ctx`: the projection of the newly committed rows runs inside the call (one chained
    # launch with the first QKV on the tensor-core path when the layer count allows, separate launches
    # otherwise). The pool must end up exactly as the separate call leaves it (same kernels, same split of
    # the same sums) and the block must match the oracle run on the oracle's own updated cache.
    wl = synth.workload(name)
    cfg = dataclasses.replace(wl.cfg, n_layers=layers)
    lens = (5, 70, 190) if name == "mid" else (100,)
    S, B = len(lens), cfg.block_size
    max_new = B + 1
    n_new = torch.tensor([3, max_new, 1][:S], dtype=torch.int32)
    feats = synth.make_features(cfg, S * max_new, 77, "fused.feats").reshape(S, max_new, cfg.feat_dim)
    anchors = synth.make_anchors(cfg, S, 77)
    results = []
    for fused in (False, True):
        case = Case(cfg, lens, seed=77)
        case.project_prefill(oracle=fused)
        dev = case.device
        after = (case.ctx_len + n_new.to(dev)).to(torch.int32)
        ids = torch.zeros((S, B), dtype=torch.int32, device=dev)
        hidden = torch.zeros((S * B, cfg.d_model), dtype=torch.float32, device=dev)
        logits = torch.zeros((S * B, cfg.vocab), dtype=torch.float32, device=dev)
        case.lib.status.zero_()
        if fused:
            case.lib.dflash_draft_block(anchors.to(dev), after, max(lens) + max_new, case.page_table, case.pool, ids,
                                        hidden_out=hidden, logits_out=logits, ctx=(feats.to(dev), n_new.to(dev), case.ctx_len))
        else:
            case.lib.dflash_ctx_project(feats.to(dev), n_new.to(dev), case.ctx_len, case.page_table, case.pool)
            case.lib.dflash_draft_block(anchors.to(dev), after, max(lens) + max_new, case.page_table, case.pool, ids,
                                        hidden_out=hidden, logits_out=logits)
        torch.cuda.synchronize()
        assert int(case.lib.status.item()) == 0
        results.append((case.pool.float().cpu().numpy(), logits.cpu().numpy(), ids.cpu().numpy(), hidden.cpu().numpy()))
    (pool_a, log_a, ids_a, hid_a), (pool_b, log_b, ids_b, hid_b) = results
    assert np.array_equal(pool_a, pool_b)
    # `case` is the fused one: bring the oracle's cache up to date and draft from it
    for b in range(S):
        n = int(n_new[b])
        pos = np.arange(lens[b], lens[b] + n)
        K, V = orc.ctx_project(synth.to_numpy_f32(feats[b, :n]), pos, case.w_np, cfg)
        orc.pool_write(case.pool_np, case.page_table_cpu[b].numpy(), list(pos), K, V, cfg.page_size)
        case.ctx_lens[b] += n
    case.anchors_cpu = anchors
    for b in range(S):
        ref = case.oracle_draft(b)
        sl = slice(b * B, (b + 1) * B)
        for got_h, got_l, got_i, what in ((hid_b, log_b, ids_b, "inside the call"), (hid_a, log_a, ids_a, "separate calls")):
            assert_close(got_h[sl], ref["hidden"], cfg.dtype, f"hidden seq {b}, {what}")
            assert_close(got_l[sl], ref["logits"], cfg.dtype, f"logits seq {b}, {what}")
            assert_ids_match(got_i[b], ref["ids"], ref["margin"], cfg.dtype, f"ids seq {b}, {what}")


@pytest.mark.parametrize("S", [9, 33])
def test_context_projection_inside_the_draft_call_for_batches(S):
    # 9 sequences: 153 projected rows and 144 block rows in one 256-column token tile; 33 sequences: 561 and 528
    # rows over three and two token tiles. Pool against the separate call (bit-equal), sampled blocks against the oracle.
    cfg = synth.MID
    B = cfg.block_size
    g = synth.substream(53, "fusedbatch.lens")
    lens = [int(v) for v in torch.randint(0, 200, (S,), generator=g)]
    n_new = torch.randint(0, B + 2, (S,), generator=g, dtype=torch.int32)
    n_new[0], n_new[1] = B + 1, 0
    feats = synth.make_features(cfg, S * (B + 1), 53, "fusedbatch.feats").reshape(S, B + 1, cfg.feat_dim)
    anchors = synth.make_anchors(cfg, S, 53)
    results = []
    for fused in (False, True):
        case = Case(cfg, lens, seed=53)
        case.project_prefill(oracle=fused)
        dev = case.device
        after = (case.ctx_len + n_new.to(dev)).to(torch.int32)
        ids = torch.zeros((S, B), dtype=torch.int32, device=dev)
        hidden = torch.zeros((S * B, cfg.d_model), dtype=torch.float32, device=dev)
        case.lib.status.zero_()
        if fused:
            case.lib.dflash_draft_block(anchors.to(dev), after, max(lens) + B + 1, case.page_table, case.pool, ids, hidden_out=hidden,
                                        ctx=(feats.to(dev), n_new.to(dev), case.ctx_len))
        else:
            case.lib.dflash_ctx_project(feats.to(dev), n_new.to(dev), case.ctx_len, case.page_table, case.pool)
            case.lib.dflash_draft_block(anchors.to(dev), after, max(lens) + B + 1, case.page_table, case.pool, ids, hidden_out=hidden)
        torch.cuda.synchronize()
        assert int(case.lib.status.item()) == 0
        results.append((case.pool.float().cpu().numpy(), ids.cpu().numpy(), hidden.cpu().numpy()))
    (pool_a, ids_a, hid_a), (pool_b, ids_b, hid_b) = results
    assert np.array_equal(pool_a, pool_b)
    for b in range(S):
        n = int(n_new[b])
        pos = np.arange(lens[b], lens[b] + n)
        if n:
            K, V = orc.ctx_project(synth.to_numpy_f32(feats[b, :n]), pos, case.w_np, cfg)
            orc.pool_write(case.pool_np, case.page_table_cpu[b].numpy(), list(pos), K, V, cfg.page_size)
        case.ctx_lens[b] += n
    case.anchors_cpu = anchors
    for b in (0, 1, S // 2, S - 1):
        ref = case.oracle_draft(b)
        sl = slice(b * B, (b + 1) * B)
        assert_close(hid_b[sl], ref["hidden"], cfg.dtype, f"hidden seq {b}, inside the call")
        assert_close(hid_a[sl], ref["hidden"], cfg.dtype, f"hidden seq {b}, separate calls")
        assert_ids_match(ids_b[b], ref["ids"], ref["margin"], cfg.dtype, f"ids seq {b}")


def test_step_replayed_as_a_cuda_graph():
    # The benchmark replays one captured step: context projection inside the draft call, then verification from
    # logits. A replay must give, bit for bit, what the same calls give when launched one by one.
    cfg = synth.MID
    lens = (5, 70, 190)
    S, B = len(lens), cfg.block_size
    case = Case(cfg, lens, seed=41)
    case.project_prefill(oracle=False)
    dev = case.device
    n_new = torch.tensor([3, B + 1, 1], dtype=torch.int32, device=dev)
    feats = synth.make_features(cfg, S * (B + 1), 41, "graph.feats").reshape(S, B + 1, cfg.feat_dim).to(dev)
    anchors = synth.make_anchors(cfg, S, 41).to(dev)
    after = (case.ctx_len + n_new).to(torch.int32)
    tlog, _, _ = synth.make_verify_case(S, B, cfg.vocab, 0.5, 41, cfg.torch_dtype)
    tlog = tlog.to(dev)
    ids = torch.zeros((S, B), dtype=torch.int32, device=dev)
    logits = torch.zeros((S * B, cfg.vocab), dtype=torch.float32, device=dev)
    tau = torch.zeros(S, dtype=torch.int32, device=dev)
    out = torch.zeros((S, B + 1), dtype=torch.int32, device=dev)
    bonus = torch.zeros(S, dtype=torch.int32, device=dev)
    new_len = torch.zeros(S, dtype=torch.int32, device=dev)
    pool0 = case.pool.clone()

    def step():
        case.lib.dflash_draft_block(anchors, after, max(lens) + B + 1, case.page_table, case.pool, ids, logits_out=logits,
                                    ctx=(feats, n_new, case.ctx_len))
        case.lib.dflash_verify_accept(ids, B, B, after, tau, out, bonus, new_len, logits=tlog)

    def snapshot():
        torch.cuda.synchronize()
        assert int(case.lib.status.item()) == 0
        return [t.clone() for t in (case.pool, ids, logits, tau, out, bonus, new_len)]

    case.lib.status.zero_()
    step()
    eager = snapshot()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):          # capture on a side stream, after the eager run has sized every buffer
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            step()
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(3):
        case.pool.copy_(pool0)
        for t in (ids, logits, tau, out, bonus, new_len):
            t.zero_()
        g.replay()
        got = snapshot()
        for a, b in zip(eager, got):
            assert torch.equal(a, b)


def test_largest_block_and_empty_calls():
    # block size 32 (the largest the library takes): 32 rows x 4 q heads fill the 128-row attention operand
    cfg = dataclasses.replace(synth.MID, block_size=32)
    case = Case(cfg, (0, 63, 64, 200), seed=29)
    case.project_prefill()
    _check_pool(case)
    got = case.run_draft()
    assert case.check_draft(got) >= case.S * 16
    # nothing to do: empty batch, zero new rows; the pool and the outputs stay as they were
    dev = case.device
    before = case.pool.clone()
    none_i = torch.zeros((0,), dtype=torch.int32, device=dev)
    case.lib.dflash_draft_block(none_i, none_i, 0, case.page_table[:0], case.pool, torch.zeros((0, 32), dtype=torch.int32, device=dev))
    case.lib.dflash_ctx_project(torch.zeros((0, 4, cfg.feat_dim), dtype=cfg.torch_dtype, device=dev), none_i, none_i,
                                case.page_table[:0], case.pool)
    feats = synth.make_features(cfg, case.S * 3, 29, "none").reshape(case.S, 3, cfg.feat_dim).to(dev)
    case.lib.dflash_ctx_project(feats, torch.zeros(case.S, dtype=torch.int32, device=dev), case.ctx_len, case.page_table, case.pool)
    torch.cuda.synchronize()
    assert int(case.lib.status.item()) == 0 and torch.equal(case.pool, before)


def test_bf16_feature_dims_that_are_not_multiples_of_64():
    # contraction lengths of 520 / 1544 / 1560 (multiples of 8 only): the one-slab ring stages with a
    # zero-filled K tail, ragged 128-feature tiles in the folded norms, a ragged last weight tile
    cfg = dataclasses.replace(synth.MID, d_model=520, d_ffn=1544, d_target=520, vocab=3001)
    case = Case(cfg, (5, 140), seed=13)
    case.project_prefill()
    _check_pool(case)
    got = case.run_draft()
    n_sure = case.check_draft(got)
    assert n_sure >= case.S * cfg.block_size // 2


def test_decode_step_appends_at_ctx_len():
    # second projection call with n_new < max_new appends rows at positions L..L+n-1 only
    cfg = synth.MID
    case = Case(cfg, (60, 130), seed=5)
    case.project_prefill()
    max_new = 17
    n_new = [3, 17]
    feats = synth.make_features(cfg, 2 * max_new, 5, "decode.feats").reshape(2, max_new, cfg.feat_dim)
    before = case.pool.clone()
    case.lib.dflash_ctx_project(feats.to(case.device), torch.tensor(n_new, dtype=torch.int32, device=case.device),
                                case.ctx_len, case.page_table, case.pool)
    torch.cuda.synchronize()
    assert int(case.lib.status.item()) == 0
    for b in range(2):
        L, n = case.ctx_lens[b], n_new[b]
        K, V = orc.ctx_project(synth.to_numpy_f32(feats[b, :n]), np.arange(L, L + n), case.w_np, cfg)
        orc.pool_write(case.pool_np, case.page_table_cpu[b].numpy(), list(range(L, L + n)), K, V, cfg.page_size)
    case.ctx_lens = [case.ctx_lens[b] + n_new[b] for b in range(2)]
    _check_pool(case)
    # rows beyond n_new were not written: slot L+3 of sequence 0 is still what it was
    p = 60 + 3
    page = int(case.page_table_cpu[0, p // cfg.page_size])
    assert torch.equal(case.pool[:, page, :, :, p % cfg.page_size], before[:, page, :, :, p % cfg.page_size])


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("mode", ["full", "causal"])
@pytest.mark.parametrize("n_seq", [8, 260])
def test_block_attention_building_block(dtype, mode, n_seq):
    # 8 sequences: lengths around the tile edges, with ties (the kernel takes the sequences longest first, equal
    # lengths by index); 260 sequences: more than the kernel ranks by length, taken in index order
    from paper_2602_06036_b200 import binding
    cfg = synth.TINY if dtype == "fp32" else synth.MID
    lens = (0, 1, 63, 64, 65, 300, 64, 300)
    if n_seq > len(lens):
        lens = tuple((37 * i) % 131 for i in range(n_seq))
    case = Case(cfg, lens, seed=7)
    case.fill_pool_synthetic()
    R = 9 if mode == "causal" else cfg.block_size
    S = len(lens)
    q = synth.normal((S, R, cfg.n_q_heads, cfg.head_dim), 1.0, 7, "attn.q", cfg.torch_dtype)
    k = synth.normal((S, R, cfg.n_kv_heads, cfg.head_dim), 1.0, 7, "attn.k", cfg.torch_dtype)
    v = synth.normal((S, R, cfg.n_kv_heads, cfg.head_dim), 1.0, 7, "attn.v", cfg.torch_dtype)
    out = torch.zeros_like(q, device=case.device)
    layer = cfg.n_layers - 1
    case.lib.dflash_block_attention(binding.ATTN_CAUSAL if mode == "causal" else binding.ATTN_FULL,
                                    q.to(case.device), k.to(case.device), v.to(case.device), case.ctx_len,
                                    max(lens), case.page_table, case.pool, layer, out)
    torch.cuda.synchronize()
    assert int(case.lib.status.item()) == 0
    for b, L in enumerate(lens):
        kc, vc = orc.pool_read(case.pool_np, case.page_table_cpu[b].numpy(), L, layer, cfg.page_size)
        ref = orc.block_attention(synth.to_numpy_f32(q[b]), kc, vc, synth.to_numpy_f32(k[b]),
                                  synth.to_numpy_f32(v[b]), cfg.softmax_scale, causal=(mode == "causal"))
        assert_close(out[b].float().cpu().numpy(), ref, dtype, f"attention seq {b} L={L}")


def test_many_anchor_blocks_over_one_cached_sequence():
    # the training-side layout (Sec. 4.2: many anchor blocks drawn from one sequence, each bidirectional
    # inside and seeing only the injected features before its anchor) is, for the forward pass, a batch of
    # blocks that share ONE page-table row and differ in ctx_len = anchor position
    from paper_2602_06036_b200 import binding
    cfg = synth.MID
    one = Case(cfg, (330,), seed=17)
    one.fill_pool_synthetic()
    anchors = (0, 16, 64, 65, 200, 313)
    S, R = len(anchors), cfg.block_size
    table = one.page_table.repeat(S, 1).contiguous()
    ctx = torch.tensor(anchors, dtype=torch.int32, device=one.device)
    q = synth.normal((S, R, cfg.n_q_heads, cfg.head_dim), 1.0, 17, "tr.q", cfg.torch_dtype)
    k = synth.normal((S, R, cfg.n_kv_heads, cfg.head_dim), 1.0, 17, "tr.k", cfg.torch_dtype)
    v = synth.normal((S, R, cfg.n_kv_heads, cfg.head_dim), 1.0, 17, "tr.v", cfg.torch_dtype)
    out = torch.zeros_like(q, device=one.device)
    one.lib.dflash_block_attention(binding.ATTN_FULL, q.to(one.device), k.to(one.device), v.to(one.device), ctx, max(anchors),
                                   table, one.pool, 1, out)
    torch.cuda.synchronize()
    assert int(one.lib.status.item()) == 0
    for b, a in enumerate(anchors):
        kc, vc = orc.pool_read(one.pool_np, one.page_table_cpu[0].numpy(), a, 1, cfg.page_size)
        ref = orc.block_attention(synth.to_numpy_f32(q[b]), kc, vc, synth.to_numpy_f32(k[b]), synth.to_numpy_f32(v[b]),
                                  cfg.softmax_scale, causal=False)
        assert_close(out[b].float().cpu().numpy(), ref, cfg.dtype, f"block anchored at {a}")


@pytest.mark.parametrize("dtype,M", [("fp32", 70), ("bf16", 70), ("bf16", 136), ("bf16", 330), ("bf16", 512)])
def test_lmhead_argmax_building_block(dtype, M):
    # 70 rows: more than one logits staging chunk. 136 / 330 / 512 rows: token tiles of 160 / 192 / 256 columns, which
    # run as CTA pairs (two CTAs per MMA); the vocabulary's odd number of 128-row tiles leaves the last pair half empty
    cfg = synth.TINY if dtype == "fp32" else synth.MID
    if M == 330:
        cfg = dataclasses.replace(cfg, vocab=4900)       # 39 tiles
    case = Case(cfg, (0,), seed=9)
    hid = synth.normal((M, cfg.d_model), 1.0, 9, "lm.hidden", cfg.torch_dtype)
    dev = case.device
    ids = torch.zeros(M, dtype=torch.int32, device=dev)
    top1 = torch.zeros(M, dtype=torch.float32, device=dev)
    margin = torch.zeros(M, dtype=torch.float32, device=dev)
    logits = torch.zeros((M, cfg.vocab), dtype=torch.float32, device=dev)
    for apply_norm in (0, 1):
        case.lib.dflash_lmhead_argmax(hid.to(dev), apply_norm, ids, top1, margin, logits)
        torch.cuda.synchronize()
        x = synth.to_numpy_f32(hid)
        z = orc.rmsnorm(x, case.w_np["g_f"], cfg.rms_eps) if apply_norm else x
        ref = orc.linear(z, case.w_np["W_lm"])
        rid, rtop, rmargin = orc.argmax_top2(ref)
        assert_close(logits.cpu().numpy(), ref, dtype, "lm-head logits")
        sure = rmargin > TOL[dtype]["margin"]
        assert sure.sum() > M // 3
        assert np.array_equal(ids.cpu().numpy()[sure], rid[sure])
        assert np.max(np.abs(top1.cpu().numpy() - ref[np.arange(M), ids.cpu().numpy()])) <= TOL[dtype]["max_abs"]
        # the fused argmax agrees exactly with an argmax over the logits the same kernel wrote
        # wherever those logits have a unique maximum
        lg = logits.cpu().numpy()
        srt = np.sort(lg, axis=-1)
        uniq = srt[:, -1] > srt[:, -2]
        assert np.array_equal(ids.cpu().numpy()[uniq], np.argmax(lg, axis=-1)[uniq])


def test_bad_token_and_bad_page_are_flagged_not_fatal():
    from paper_2602_06036_b200 import binding
    cfg = synth.TINY
    case = Case(cfg, (70,), seed=11)
    case.fill_pool_synthetic()
    dev = case.device
    ids = torch.zeros((1, cfg.block_size), dtype=torch.int32, device=dev)
    case.lib.status.zero_()
    case.lib.dflash_draft_block(torch.tensor([cfg.vocab + 5], dtype=torch.int32, device=dev), case.ctx_len, 70,
                                case.page_table, case.pool, ids)
    torch.cuda.synchronize()
    assert int(case.lib.status.item()) & binding.DEV_BAD_TOKEN
    bad_table = case.page_table.clone()
    bad_table[0, 1] = case.n_pages + 100
    case.lib.status.zero_()
    case.lib.dflash_draft_block(torch.tensor([3], dtype=torch.int32, device=dev), case.ctx_len, 70, bad_table,
                                case.pool, ids)
    torch.cuda.synchronize()
    assert int(case.lib.status.item()) & binding.DEV_BAD_PAGE
    # the context stays usable
    case.lib.status.zero_()
    got = case.run_draft()
    case.check_draft(got)


def test_empty_batch_is_a_no_op():
    cfg = synth.TINY
    case = Case(cfg, (5,), seed=1)
    dev = case.device
    e = torch.zeros(0, dtype=torch.int32, device=dev)
    n0 = __import__("paper_2602_06036_b200.binding", fromlist=["x"]).launch_count()
    case.lib.dflash_draft_block(e, e, 0, case.page_table[:0].contiguous().reshape(0, case.page_table.shape[1]),
                                case.pool, e.reshape(0, cfg.block_size))
    assert __import__("paper_2602_06036_b200.binding", fromlist=["x"]).launch_count() == n0
