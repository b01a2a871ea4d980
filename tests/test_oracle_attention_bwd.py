"""Pins for the oracle's training-side attention gradient (block_attention_backward, block_attention_lse):
finite differences of the forward, torch autograd of an independently written attention, and closed forms."""
import numpy as np
import torch

from oracle import dflash_oracle as orc


def _case(seed, R=5, Hq=4, Hkv=2, hd=6, L=7):
    rng = np.random.default_rng(seed)
    g = lambda *s: rng.standard_normal(s)
    return g(R, Hq, hd), g(L, Hkv, hd), g(L, Hkv, hd), g(R, Hkv, hd), g(R, Hkv, hd), g(R, Hq, hd)


def test_matches_central_finite_differences_of_the_forward():
    scale = 0.37
    for causal in (False, True):
        q, kc, vc, kb, vb, dout = _case(1 + causal)
        grads = orc.block_attention_backward(q, kc, vc, kb, vb, dout, scale, causal=causal)
        args = [q, kc, vc, kb, vb]
        order = [0, 1, 2, 3, 4]                     # dq, dk_ctx, dv_ctx, dk_blk, dv_blk follow the argument order
        loss = lambda a: float(np.sum(orc.block_attention(a[0], a[1], a[2], a[3], a[4], scale, causal=causal) * dout))
        eps = 1e-6
        rng = np.random.default_rng(9)
        for gi, ai in enumerate(order):
            flat_idx = rng.choice(args[ai].size, size=min(12, args[ai].size), replace=False)
            for f in flat_idx:
                idx = np.unravel_index(f, args[ai].shape)
                plus = [a.copy() for a in args]
                minus = [a.copy() for a in args]
                plus[ai][idx] += eps
                minus[ai][idx] -= eps
                num = (loss(plus) - loss(minus)) / (2 * eps)
                assert abs(num - grads[gi][idx]) < 1e-7 * max(1.0, abs(num)), (causal, gi, idx, num, grads[gi][idx])


def test_matches_torch_autograd_of_an_attention_written_independently():
    scale = 0.25
    for causal in (False, True):
        q, kc, vc, kb, vb, dout = _case(5 + causal, R=6, Hq=6, Hkv=2, hd=8, L=11)
        t = [torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in (q, kc, vc, kb, vb)]
        tq, tkc, tvc, tkb, tvb = t
        R, Hq, L = q.shape[0], q.shape[1], kc.shape[0]
        group = Hq // kb.shape[1]
        keys = torch.cat((tkc, tkb), 0).repeat_interleave(group, dim=1)      # kv head h // group serves q head h
        vals = torch.cat((tvc, tvb), 0).repeat_interleave(group, dim=1)
        mask = torch.ones(R, L + R, dtype=torch.bool)
        if causal:
            mask[:, L:] = torch.tril(torch.ones(R, R, dtype=torch.bool))
        out = torch.nn.functional.scaled_dot_product_attention(tq.transpose(0, 1), keys.transpose(0, 1), vals.transpose(0, 1),
                                                               attn_mask=mask, scale=scale).transpose(0, 1)
        np.testing.assert_allclose(out.detach().numpy(), orc.block_attention(q, kc, vc, kb, vb, scale, causal=causal), atol=1e-12)
        out.backward(torch.tensor(dout))
        got = orc.block_attention_backward(q, kc, vc, kb, vb, dout, scale, causal=causal)
        for g, ref in zip(got, t):
            np.testing.assert_allclose(g, ref.grad.numpy(), atol=1e-12)


def test_closed_forms():
    scale = 0.5
    q, kc, vc, kb, vb, dout = _case(11)
    dq, dkc, dvc, dkb, dvb = orc.block_attention_backward(q, kc, vc, kb, vb, dout, scale)
    group = q.shape[1] // kb.shape[1]
    # every probability row sums to one, so the value gradients of a kv head add up to the sum of dout over rows and its q heads
    for kv in range(kb.shape[1]):
        total = dvc[:, kv].sum(0) + dvb[:, kv].sum(0)
        np.testing.assert_allclose(total, dout[:, kv * group:(kv + 1) * group].sum((0, 1)), atol=1e-12)
    # moving every key of a kv head by the same vector shifts all scores of a row by one constant, which softmax
    # does not see: the output stays, and the key gradients of a kv head therefore add up to zero
    shift = np.random.default_rng(3).standard_normal(kc.shape[-1])
    out0 = orc.block_attention(q, kc, vc, kb, vb, scale)
    out1 = orc.block_attention(q, kc + shift, vc, kb + shift, vb, scale)
    np.testing.assert_allclose(out1, out0, atol=1e-12)
    for kv in range(kb.shape[1]):
        np.testing.assert_allclose(dkc[:, kv].sum(0) + dkb[:, kv].sum(0), 0.0, atol=1e-12)
    # a block of one row without context: the only key has probability 1: dv = dout summed over the group, dq = dk = 0
    q1, kb1, vb1, do1 = q[:1], kb[:1], vb[:1], dout[:1]
    empty = np.zeros((0,) + kc.shape[1:])
    dq1, _, _, dk1, dv1 = orc.block_attention_backward(q1, empty, empty, kb1, vb1, do1, scale)
    assert np.all(dq1 == 0) and np.all(dk1 == 0)
    for kv in range(kb.shape[1]):
        np.testing.assert_allclose(dv1[0, kv], do1[0, kv * group:(kv + 1) * group].sum(0), atol=1e-15)
    # causal: the last block row's keys get no gradient from earlier rows
    dqc, _, _, dkbc, dvbc = orc.block_attention_backward(q, kc, vc, kb, vb, dout, scale, causal=True)
    d2 = dout.copy()
    d2[:-1] = 0.0                                     # only the last row carries gradient
    _, _, _, dk_last, dv_last = orc.block_attention_backward(q, kc, vc, kb, vb, d2, scale, causal=True)
    d3 = dout.copy()
    d3[-1] = 0.0                                      # every row but the last
    _, _, _, dk_rest, dv_rest = orc.block_attention_backward(q, kc, vc, kb, vb, d3, scale, causal=True)
    assert np.all(dk_rest[-1] == 0) and np.all(dv_rest[-1] == 0)
    np.testing.assert_allclose(dk_last + dk_rest, dkbc, atol=1e-12)           # linear in dout


def test_lse_is_the_log_of_the_normaliser():
    scale = 0.3
    q, kc, vc, kb, vb, _ = _case(21)
    for causal in (False, True):
        lse = orc.block_attention_lse(q, kc, vc, kb, vb, scale, causal=causal)
        R, Hq, L = q.shape[0], q.shape[1], kc.shape[0]
        group = Hq // kb.shape[1]
        for r in range(R):
            for h in range(Hq):
                tot = 0.0
                for t in range(L):
                    tot += np.exp(scale * float(np.dot(q[r, h], kc[t, h // group])))
                for t in range(R):
                    if causal and t > r:
                        continue
                    tot += np.exp(scale * float(np.dot(q[r, h], kb[t, h // group])))
                assert abs(lse[r, h] - np.log(tot)) < 1e-12


def test_context_gradients_of_blocks_over_one_sequence_add_up_by_position():
    # two anchor blocks over one cached sequence: the loss is the sum of the blocks' losses, so the gradient of a
    # context position is the sum of what each block that sees it sends back (finite differences of the joint loss)
    scale = 0.4
    rng = np.random.default_rng(31)
    Lseq, R, Hq, Hkv, hd = 9, 3, 2, 1, 4
    kc, vc = rng.standard_normal((Lseq, Hkv, hd)), rng.standard_normal((Lseq, Hkv, hd))
    anchors = (4, 9)
    blocks = [tuple(rng.standard_normal(s) for s in ((R, Hq, hd), (R, Hkv, hd), (R, Hkv, hd), (R, Hq, hd))) for _ in anchors]
    dk_tot, dv_tot = np.zeros_like(kc), np.zeros_like(vc)
    for a, (q, kb, vb, do) in zip(anchors, blocks):
        _, dkc, dvc, _, _ = orc.block_attention_backward(q, kc[:a], vc[:a], kb, vb, do, scale)
        dk_tot[:a] += dkc
        dv_tot[:a] += dvc

    def joint(kc_, vc_):
        return sum(float(np.sum(orc.block_attention(q, kc_[:a], vc_[:a], kb, vb, scale) * do)) for a, (q, kb, vb, do) in zip(anchors, blocks))
    eps = 1e-6
    for pos in (0, 3, 4, 8):
        for d in range(hd):
            kp, km = kc.copy(), kc.copy()
            kp[pos, 0, d] += eps
            km[pos, 0, d] -= eps
            assert abs((joint(kp, vc) - joint(km, vc)) / (2 * eps) - dk_tot[pos, 0, d]) < 1e-7
            vp, vm = vc.copy(), vc.copy()
            vp[pos, 0, d] += eps
            vm[pos, 0, d] -= eps
            assert abs((joint(kc, vp) - joint(kc, vm)) / (2 * eps) - dv_tot[pos, 0, d]) < 1e-7
