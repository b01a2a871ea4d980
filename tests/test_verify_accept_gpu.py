"""Bit-exact parity of the verify/accept kernels with the oracle's accept rule."""
import numpy as np
import pytest
import torch

from oracle import dflash_oracle as orc
from paper_2602_06036_b200 import synth

pytestmark = pytest.mark.gpu


def _run(lib, drafts, gamma, ctx_len, logits=None, target_ids=None, draft_stride=None, draft_offset=0):
    dev = lib.device
    S = ctx_len.shape[0]
    out = dict(tau=torch.zeros(S, dtype=torch.int32, device=dev),
               toks=torch.zeros((S, gamma + 1), dtype=torch.int32, device=dev),
               bonus=torch.zeros(S, dtype=torch.int32, device=dev),
               new_len=torch.zeros(S, dtype=torch.int32, device=dev),
               tids=torch.zeros((S, gamma + 1), dtype=torch.int32, device=dev))
    lib.dflash_verify_accept(drafts.to(dev), draft_stride or drafts.shape[1], gamma, ctx_len.to(dev), out["tau"],
                             out["toks"], out["bonus"], out["new_len"],
                             logits=None if logits is None else logits.to(dev),
                             target_ids=None if target_ids is None else target_ids.to(dev),
                             target_ids_out=out["tids"], draft_offset=draft_offset)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


def _lib(cfg=synth.TINY):
    from paper_2602_06036_b200 import binding
    return binding.DFlash(cfg)


@pytest.mark.parametrize("ldtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("gamma", [8, 7, 16])
def test_logits_mode_many_seeds(ldtype, gamma):
    lib = _lib()
    V = 1024
    S = 40
    for seed in range(5):
        logits, drafts, a = synth.make_verify_case(S, gamma, V, 0.3, seed, ldtype)
        ctx = torch.arange(S, dtype=torch.int32) * 3 + 100
        got = _run(lib, drafts, gamma, ctx, logits=logits)
        for b in range(S):
            tau, out, bonus, new_len = orc.verify_accept_logits(drafts[b].numpy(), synth.to_numpy_f32(logits[b]), int(ctx[b]))
            assert got["tau"][b] == tau == int(a[b]) + 1
            assert got["toks"][b].tolist() == out.tolist()
            assert got["bonus"][b] == bonus and got["new_len"][b] == new_len
            assert got["tids"][b].tolist() == orc.argmax_top2(synth.to_numpy_f32(logits[b]))[0].tolist()


def test_ids_mode_and_strided_drafts_paper_mode():
    # gamma = B-1: the drafts are rows 1..B-1 of a [S, B] draft array (stride B, offset 1)
    lib = _lib()
    B, S, V = 16, 9, 500
    g = torch.Generator().manual_seed(3)
    block = torch.randint(0, V, (S, B), generator=g, dtype=torch.int32)
    tids = torch.randint(0, V, (S, B), generator=g, dtype=torch.int32)
    for b in range(S):
        tids[b, :b] = block[b, 1:1 + b]          # sequence b accepts exactly min(b, B-1) drafts
    ctx = torch.full((S,), 77, dtype=torch.int32)
    got = _run(lib, block, B - 1, ctx, target_ids=tids, draft_stride=B, draft_offset=1)
    for b in range(S):
        tau, out, bonus, new_len = orc.verify_accept(block[b, 1:].numpy(), tids[b].numpy(), 77)
        assert got["tau"][b] == tau
        assert got["toks"][b].tolist() == out.tolist() and got["bonus"][b] == bonus and got["new_len"][b] == new_len


def test_ties_nan_and_ragged_vocab():
    lib = _lib()
    V = 1003
    z = torch.zeros((2, 3, V))
    z[0, 0, [17, 900]] = 5.0            # tie -> 17
    z[0, 1, 0] = float("nan")
    z[0, 1, 1002] = 1.0                 # last element of a ragged row
    z[0, 2, :] = float("nan")           # all NaN -> 0
    z[1, 0, 5] = 2.0
    z[1, 1, 6] = 2.0
    z[1, 2, 7] = 2.0
    drafts = torch.tensor([[17, 1002], [5, 9]], dtype=torch.int32)
    got = _run(lib, drafts, 2, torch.tensor([0, 10], dtype=torch.int32), logits=z)
    assert got["tids"].tolist() == [[17, 1002, 0], [5, 6, 7]]
    assert got["tau"].tolist() == [3, 2] and got["bonus"].tolist() == [0, 6]
    assert got["toks"].tolist() == [[17, 1002, 0], [5, 6, -1]] and got["new_len"].tolist() == [3, 12]
    for b in range(2):
        tau, out, bonus, new_len = orc.verify_accept_logits(drafts[b].numpy(), z[b].numpy(), [0, 10][b])
        assert (tau, bonus, new_len) == (got["tau"][b], got["bonus"][b], got["new_len"][b])


def test_new_len_may_alias_ctx_len():
    lib = _lib()
    dev = lib.device
    S, gamma = 4, 3
    tids = torch.tensor([[1, 2, 3, 4]] * S, dtype=torch.int32, device=dev)
    drafts = torch.tensor([[1, 2, 3], [1, 2, 0], [1, 0, 3], [0, 2, 3]], dtype=torch.int32, device=dev)
    ctx = torch.tensor([10, 20, 30, 40], dtype=torch.int32, device=dev)
    tau = torch.zeros(S, dtype=torch.int32, device=dev)
    toks = torch.zeros((S, gamma + 1), dtype=torch.int32, device=dev)
    bonus = torch.zeros(S, dtype=torch.int32, device=dev)
    lib.dflash_verify_accept(drafts, gamma, gamma, ctx, tau, toks, bonus, ctx, target_ids=tids)
    torch.cuda.synchronize()
    assert tau.tolist() == [4, 3, 2, 1] and ctx.tolist() == [14, 23, 32, 41]


def test_more_sequences_than_tickets_take_two_launches_with_the_same_result():
    # the one-launch form keeps one ticket per sequence for up to 4096 sequences; a larger batch runs the segment
    # scan and the per-sequence merge as two launches. Both forms against numpy's first-occurrence argmax + the
    # oracle's accept rule, and the one-launch form twice in a row (its tickets must be back at zero).
    lib = _lib()
    gamma, V = 2, 4099
    for S in (4096, 4100):
        logits, drafts, a = synth.make_verify_case(S, gamma, V, 0.5, 11, torch.bfloat16)
        ctx = torch.arange(S, dtype=torch.int32) + 7
        ref_ids = np.argmax(synth.to_numpy_f32(logits), axis=-1)
        for _ in range(2):
            got = _run(lib, drafts, gamma, ctx, logits=logits)
            assert np.array_equal(got["tids"], ref_ids)
            assert np.array_equal(got["tau"], a.numpy() + 1)
            for b in (0, 1, S // 2, S - 1):
                tau, out, bonus, new_len = orc.verify_accept(drafts[b].numpy(), ref_ids[b], int(ctx[b]))
                assert got["toks"][b].tolist() == out.tolist() and got["bonus"][b] == bonus and got["new_len"][b] == new_len
