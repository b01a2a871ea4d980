"""Parity of the sampling (temperature > 0) calls against the CPU oracle, through the C ABI.
An index decided by a running sum may legitimately differ when the uniform lies next to an interval
edge: indices are compared where the oracle's margin is clear, and checked for validity (inside the
interval the oracle's float64 sums allow) otherwise. Accept decisions likewise."""
import numpy as np
import pytest
import torch

from oracle import dflash_oracle as orc
from paper_2602_06036_b200 import binding, synth

pytestmark = pytest.mark.gpu

MARGIN = 1e-5      # relative to the total weight; the kernel's sums are fp32 weights added in double


def _lib():
    return binding.DFlash(synth.TINY)


def _logits(shape, seed, name, scale, dtype):
    return (synth.normal(shape, scale, seed, name, torch.float32)).to(dtype)


def _valid_draw(w, u, tok, slack):
    c = np.cumsum(np.asarray(w, dtype=np.float64))
    x = u * c[-1]
    return w[tok] > 0 and c[tok] - w[tok] - slack * c[-1] <= x <= c[tok] + slack * c[-1]


@pytest.mark.parametrize("V,dtype,T", [(1024, torch.float32, 1.0), (5003, torch.bfloat16, 0.7), (151936, torch.bfloat16, 1.0),
                                       (151936, torch.float32, 1.3)])
def test_sample_rows_matches_oracle(V, dtype, T):
    lib = _lib()
    dev = lib.device
    n = 24 if V < 100000 else 12
    z = _logits((n, V), 3, f"samp.z.{V}", 2.5, dtype)
    u = torch.rand(n, generator=synth.substream(3, f"samp.u.{V}"), dtype=torch.float32)
    u[0], u[1] = 0.0, 0.99999994          # both ends of the unit interval
    ids = torch.full((n,), -7, dtype=torch.int32, device=dev)
    prob = torch.zeros(n, dtype=torch.float32, device=dev)
    lib.dflash_sample_rows(z.to(dev), T, u.to(dev), ids, prob)
    torch.cuda.synchronize()
    assert int(lib.status.item()) == 0
    zn = z.float().numpy().astype(np.float64)
    n_exact = 0
    for m in range(n):
        p = orc.softmax_t(zn[m], T)
        tok, margin = orc.sample_cdf(p, float(u[m]))
        got = int(ids[m])
        if margin > MARGIN:
            assert got == tok, (m, got, tok, margin)
            n_exact += 1
        else:
            assert _valid_draw(p, float(u[m]), got, MARGIN), (m, got, tok)
        np.testing.assert_allclose(float(prob[m]), p[got], rtol=2e-3 if dtype == torch.float32 else 2e-2)
    assert n_exact >= n // 2


def _verify_case(S, gamma, V, T, seed, t_dtype, d_dtype, rows_per_seq, closeness):
    """Seeded target / draft logits; the draft is the target plus noise (closeness sets how often drafts are kept)."""
    zt = synth.normal((S, gamma + 1, V), 2.5, seed, "vs.target", torch.float32)
    zd_used = zt[:, :gamma] + synth.normal((S, gamma, V), closeness, seed, "vs.noise", torch.float32)
    zd = synth.normal((S, rows_per_seq, V), 2.5, seed, "vs.draft.pad", torch.float32)
    zd[:, :gamma] = zd_used
    zt, zd = zt.to(t_dtype), zd.to(d_dtype)
    g = synth.substream(seed, "vs.u")
    u_draft = torch.rand((S, gamma), generator=g, dtype=torch.float32)
    u_acc = torch.rand((S, gamma), generator=g, dtype=torch.float32)
    u_fin = torch.rand((S,), generator=g, dtype=torch.float32)
    ctx = torch.randint(0, 5000, (S,), generator=g, dtype=torch.int32)
    # drafts drawn from the draft distribution by the oracle (the GPU draw is tested separately)
    ids = torch.zeros((S, gamma), dtype=torch.int32)
    zdn = zd.float().numpy().astype(np.float64)
    for b in range(S):
        for j in range(gamma):
            ids[b, j] = orc.sample_cdf(orc.softmax_t(zdn[b, j], T), float(u_draft[b, j]))[0]
    return zt, zd, ids, u_acc, u_fin, ctx


@pytest.mark.parametrize("S,gamma,V,T,t_dtype,d_dtype,rows_per_seq,closeness", [
    (5, 7, 1024, 1.0, torch.float32, torch.float32, 8, 0.5),
    (6, 16, 5003, 1.0, torch.bfloat16, torch.float32, 16, 0.3),
    (3, 15, 151936, 1.0, torch.bfloat16, torch.float32, 16, 0.4),     # paper mode: gamma = B - 1, rows stored per block = B
    (4, 16, 151936, 0.8, torch.bfloat16, torch.bfloat16, 16, 1.0),
    (2, 0, 1024, 1.0, torch.float32, torch.float32, 1, 0.5),          # no drafts: the cycle only emits a token from p_0
])
def test_verify_accept_sample_matches_oracle(S, gamma, V, T, t_dtype, d_dtype, rows_per_seq, closeness):
    lib = _lib()
    dev = lib.device
    zt, zd, ids, u_acc, u_fin, ctx = _verify_case(S, gamma, V, T, 17, t_dtype, d_dtype, rows_per_seq, closeness)
    acc = torch.full((S,), -1, dtype=torch.int32, device=dev)
    out = torch.full((S, gamma + 1), -9, dtype=torch.int32, device=dev)
    bonus = torch.full((S,), -1, dtype=torch.int32, device=dev)
    new_len = torch.full((S,), -1, dtype=torch.int32, device=dev)
    lib.dflash_verify_accept_sample(zt.to(dev), zd.to(dev) if gamma else None, rows_per_seq, ids.to(dev) if gamma else None,
                                    max(gamma, 1), gamma, T, u_acc.to(dev) if gamma else None, u_fin.to(dev), ctx.to(dev),
                                    acc, out, bonus, new_len)
    torch.cuda.synchronize()
    assert int(lib.status.item()) == 0
    ztn, zdn = zt.float().numpy().astype(np.float64), zd.float().numpy().astype(np.float64)
    taus, n_checked = [], 0
    for b in range(S):
        tau, o, tok, nl, info = orc.verify_accept_sample(ids[b].numpy(), zdn[b, :gamma], ztn[b], T, u_acc[b].numpy(),
                                                         float(u_fin[b]), int(ctx[b]))
        taus.append(tau)
        if any(m < 1e-3 for m in info["accept_margin"]):
            # an accept test too close to call: the result must still be a prefix of the drafts plus one token
            g_tau = int(acc[b])
            assert 1 <= g_tau <= gamma + 1 and out[b, :g_tau - 1].tolist() == ids[b, :g_tau - 1].tolist()
            continue
        assert int(acc[b]) == tau and int(new_len[b]) == nl
        assert out[b, :tau - 1].tolist() == list(o[:tau - 1]) and out[b, tau:].tolist() == [-1] * (gamma + 1 - tau)
        got = int(out[b, tau - 1])
        assert int(bonus[b]) == got
        a = info["a"]
        p = orc.softmax_t(ztn[b, a], T)
        w = p
        if info["residual"]:
            w = np.maximum(p - orc.softmax_t(zdn[b, a], T), 0)
        if info["final_margin"] > MARGIN:
            assert got == tok, (b, got, tok, info)
        else:
            assert _valid_draw(w, float(u_fin[b]), got, MARGIN)
        n_checked += 1
    assert n_checked >= (S + 1) // 2
    if gamma >= 7 and S >= 4:
        assert min(taus) < max(taus)          # the case exercises both rejections and kept drafts


def test_identical_logits_keep_all_and_greedy_limit():
    lib = _lib()
    dev = lib.device
    S, gamma, V = 4, 8, 5003
    z = synth.normal((S, gamma + 1, V), 3.0, 5, "same.z", torch.float32)
    ids = z[:, :gamma].argmax(-1).to(torch.int32)
    u_acc = torch.rand((S, gamma), generator=synth.substream(5, "same.u")) * 0.98 + 0.01
    u_fin = torch.rand((S,), generator=synth.substream(5, "same.uf"))
    ctx = torch.tensor([0, 10, 20, 30], dtype=torch.int32)
    bufs = [torch.zeros((S,), dtype=torch.int32, device=dev), torch.zeros((S, gamma + 1), dtype=torch.int32, device=dev),
            torch.zeros((S,), dtype=torch.int32, device=dev), torch.zeros((S,), dtype=torch.int32, device=dev)]
    # p = q: every draft is kept whatever the uniforms
    lib.dflash_verify_accept_sample(z.to(dev), z[:, :gamma].contiguous().to(dev), gamma, ids.to(dev), gamma, gamma, 1.0,
                                    u_acc.to(dev), u_fin.to(dev), ctx.to(dev), *bufs)
    torch.cuda.synchronize()
    assert bufs[0].tolist() == [gamma + 1] * S and bufs[3].tolist() == [int(c) + gamma + 1 for c in ctx]
    # T -> 0: the greedy rule (drafts = argmax of a perturbed draft model)
    zd = z[:, :gamma] + synth.normal((S, gamma, V), 1.5, 5, "same.noise", torch.float32)
    ids = zd.argmax(-1).to(torch.int32)
    lib.dflash_verify_accept_sample(z.to(dev), zd.contiguous().to(dev), gamma, ids.to(dev), gamma, gamma, 1e-3,
                                    u_acc.to(dev), u_fin.to(dev), ctx.to(dev), *bufs)
    torch.cuda.synchronize()
    for b in range(S):
        tau, o, bon, nl = orc.verify_accept_logits(ids[b].numpy(), z[b].numpy(), int(ctx[b]))
        assert int(bufs[0][b]) == tau and bufs[1][b].tolist() == list(o) and int(bufs[2][b]) == bon


def test_host_validation_and_bad_draft_id():
    lib = _lib()
    dev = lib.device
    z = torch.zeros((1, 2, 1024), device=dev)
    zd = torch.zeros((1, 1, 1024), device=dev)
    one = torch.zeros((1,), dtype=torch.int32, device=dev)
    out = torch.zeros((1, 2), dtype=torch.int32, device=dev)
    u = torch.full((1, 1), 0.5, device=dev)
    with pytest.raises(binding.DFlashError):
        lib.dflash_verify_accept_sample(z, zd, 1, one.clone(), 1, 1, 0.0, u, u[0], one, one.clone(), out, one.clone(), one.clone())
    with pytest.raises(binding.DFlashError):
        lib.dflash_sample_rows(z[0], -1.0, u[0].repeat(2), torch.zeros(2, dtype=torch.int32, device=dev))
    # a draft id outside the vocabulary is rejected and reported
    bad = torch.tensor([5000], dtype=torch.int32, device=dev)
    acc = one.clone()
    lib.dflash_verify_accept_sample(z, zd, 1, bad, 1, 1, 1.0, u, u[0], one, acc, out, one.clone(), one.clone())
    torch.cuda.synchronize()
    assert int(acc[0]) == 1 and int(lib.status.item()) & binding.DEV_BAD_TOKEN
