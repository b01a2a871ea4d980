"""GPU parity of the position-weighted block loss (Sec. 4.2 Eq. 4) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import dflash_oracle as orc
from paper_2602_06036_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _case(nb, B, V, seed, dtype, scale=3.0):
    z = synth.normal((nb, B, V), scale, seed, "loss.logits", torch.float32).to(dtype)
    g = synth.substream(seed, "loss.targets")
    t = torch.randint(0, V, (nb, B), generator=g, dtype=torch.int32)
    t[torch.rand((nb, B), generator=g) < 0.1] = -1          # positions past the end of a sequence
    return z, t


@pytest.mark.parametrize("nb,B,V,gamma,in_dtype,out_dtype", [
    (3, 16, 151936, 7.0, torch.bfloat16, torch.bfloat16),      # the drafter's vocabulary, bf16 logits and gradient
    (2, 10, 151936, 5.0, torch.float32, torch.float32),
    (5, 8, 5003, 4.0, torch.bfloat16, torch.float32),          # odd vocabulary: rows lose 16-byte alignment
    (4, 16, 32000, 7.0, torch.float32, torch.bfloat16),
    (1, 1, 300, 7.0, torch.float32, torch.float32),            # a block of the anchor alone: no loss at all
    (3, 4, 16, 4.0, torch.bfloat16, torch.float32),            # one 16-byte vector per CTA of the cluster
    (2, 8, 8, 4.0, torch.bfloat16, torch.bfloat16),            # the second CTA of the cluster holds nothing
    (200, 2, 4096, 4.0, torch.float32, torch.float32),         # more rows than clusters, every other row an anchor
])
def test_block_loss_matches_oracle(nb, B, V, gamma, in_dtype, out_dtype):
    dev = torch.device("cuda:0")
    lib = binding.DFlash(synth.TINY, "cuda:0")
    z, t = _case(nb, B, V, 23, in_dtype)
    row_loss = torch.full((nb * B,), -5.0, dtype=torch.float32, device=dev)
    sums = torch.zeros(2, dtype=torch.float32, device=dev)
    dz = torch.full((nb, B, V), 9.0, dtype=out_dtype, device=dev)
    scale = 0.37
    lib.dflash_block_loss(z.to(dev), t.to(dev), gamma, row_loss, sums, dz, grad_scale=scale)
    torch.cuda.synchronize()
    assert int(lib.status.item()) == 0
    zn = synth.to_numpy_f32(z).astype(np.float64)
    got_loss = row_loss.cpu().numpy().reshape(nb, B)
    got_dz = dz.float().cpu().numpy()
    tot, wsum = 0.0, 0.0
    for b in range(nb):
        ref = orc.block_loss(zn[b], t[b].numpy(), gamma)
        np.testing.assert_allclose(got_loss[b], ref["row_loss"], rtol=2e-5, atol=2e-5)
        tol = 1e-6 if out_dtype == torch.float32 else 2.0 ** -8
        err = np.abs(got_dz[b] - scale * ref["grad"])
        assert np.all(err <= tol * np.abs(scale * ref["grad"]) + 1e-7), float(err.max())
        tot += ref["loss"]
        wsum += ref["weight"]
    np.testing.assert_allclose(sums.cpu().numpy(), [tot, wsum], rtol=2e-5, atol=1e-6)


def test_block_loss_without_gradient_in_place_and_many_rows():
    dev = torch.device("cuda:0")
    lib = binding.DFlash(synth.TINY, "cuda:0")
    nb, B, V, gamma = 40, 16, 151936, 7.0          # 640 rows of bf16: several L2-sized groups
    z, t = _case(nb, B, V, 29, torch.bfloat16)
    zd = z.to(dev)
    loss_a = torch.zeros(nb * B, dtype=torch.float32, device=dev)
    lib.dflash_block_loss(zd, t.to(dev), gamma, loss_a)
    # in place: the gradient replaces the logits
    loss_b = torch.zeros(nb * B, dtype=torch.float32, device=dev)
    sums = torch.zeros(2, dtype=torch.float32, device=dev)
    buf = zd.clone()
    lib.dflash_block_loss(buf, t.to(dev), gamma, loss_b, sums, buf)
    torch.cuda.synchronize()
    assert torch.equal(loss_a, loss_b)
    zn = synth.to_numpy_f32(z).astype(np.float64)
    for b in (0, 17, 39):
        ref = orc.block_loss(zn[b], t[b].numpy(), gamma)
        np.testing.assert_allclose(loss_a.cpu().numpy().reshape(nb, B)[b], ref["row_loss"], rtol=2e-5, atol=2e-5)
        err = np.abs(buf[b].float().cpu().numpy() - ref["grad"])
        assert np.all(err <= 2.0 ** -8 * np.abs(ref["grad"]) + 1e-7)
    # every gradient row sums to (almost) zero, anchor and ignored rows are exactly zero
    g = buf.float()
    assert float(g.sum(dim=-1).abs().max()) < 2e-2
    off = (t.to(dev) < 0) | (torch.arange(B, device=dev)[None, :] == 0)
    assert float(g[off].abs().max()) == 0.0
    np.testing.assert_allclose(float(sums[0]), float(loss_a.double().sum()), rtol=1e-6)


def test_block_loss_flags_a_target_outside_the_vocabulary():
    dev = torch.device("cuda:0")
    lib = binding.DFlash(synth.TINY, "cuda:0")
    z, t = _case(2, 8, 4096, 31, torch.float32)
    t[1, 3] = 4096
    loss = torch.zeros(16, dtype=torch.float32, device=dev)
    lib.status.zero_()
    lib.dflash_block_loss(z.to(dev), t.to(dev), 4.0, loss)
    torch.cuda.synchronize()
    assert int(lib.status.item()) & 1 and float(loss[8 + 3]) == 0.0
