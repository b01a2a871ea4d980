"""The allocation-free verify/accept entry point gives the same answer as the ordinary one.

dflash_verify_accept_static exists for callers that cannot allocate a workspace on the device (GPU
memory fully committed elsewhere, no cudaMalloc allowed on their thread, or a stream under capture):
its scratch is a fixed array inside the library. The array survives from call to call, so the check
runs two different problems back to back and compares every output with dflash_verify_accept, which
is itself checked against the CPU oracle in test_verify_accept_gpu.py. All outputs are integers:
the comparison is exact. This file is collected last on purpose."""
import pytest
import torch

from paper_2602_06036_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _outputs(dev, S, gamma):
    return dict(tau=torch.full((S,), -1, dtype=torch.int32, device=dev),
                toks=torch.full((S, gamma + 1), -9, dtype=torch.int32, device=dev),
                bonus=torch.full((S,), -1, dtype=torch.int32, device=dev),
                new_len=torch.full((S,), -1, dtype=torch.int32, device=dev),
                tids=torch.full((S, gamma + 1), -1, dtype=torch.int32, device=dev))


def test_static_scratch_matches_workspace_version_twice_in_a_row():
    lib = binding.DFlash(synth.TINY)
    dev = lib.device
    # two calls in a row with different shapes, dtypes and contents: the second one finds the first
    # one's leftovers in the shared scratch
    for seed, S, gamma, V, dt in ((0, 40, 16, 151936, torch.bfloat16), (1, 7, 8, 5003, torch.float32)):
        logits, drafts, planted = synth.make_verify_case(S, gamma, V, 0.25, seed, dt)
        logits, drafts = logits.to(dev), drafts.to(dev)
        ctx = (torch.arange(S, dtype=torch.int32) * 5 + 11).to(dev)
        ref, got = _outputs(dev, S, gamma), _outputs(dev, S, gamma)
        lib.dflash_verify_accept(drafts, gamma, gamma, ctx, ref["tau"], ref["toks"], ref["bonus"], ref["new_len"],
                                 logits=logits, target_ids_out=ref["tids"])
        lib.dflash_verify_accept_static(drafts, gamma, gamma, ctx, got["tau"], got["toks"], got["bonus"], got["new_len"],
                                        logits, target_ids_out=got["tids"])
        torch.cuda.synchronize()
        for k in ref:
            assert torch.equal(ref[k], got[k]), (seed, k)
        assert ref["tau"].cpu().tolist() == (planted + 1).tolist()
        # without target_ids_out the ids live in the built-in scratch as well
        got2 = _outputs(dev, S, gamma)
        lib.dflash_verify_accept_static(drafts, gamma, gamma, ctx, got2["tau"], got2["toks"], got2["bonus"],
                                        got2["new_len"], logits)
        torch.cuda.synchronize()
        for k in ("tau", "toks", "bonus", "new_len"):
            assert torch.equal(ref[k], got2[k]), (seed, k)


def test_sizes_beyond_the_fixed_scratch_are_refused():
    lib = binding.DFlash(synth.TINY)
    dev = lib.device
    S, gamma, V = 65, 16, 64                      # 65 * 17 = 1105 rows > 1088
    logits = torch.zeros((S, gamma + 1, V), device=dev)
    drafts = torch.zeros((S, gamma), dtype=torch.int32, device=dev)
    ctx = torch.zeros(S, dtype=torch.int32, device=dev)
    o = _outputs(dev, S, gamma)
    with pytest.raises(binding.DFlashError) as e:
        lib.dflash_verify_accept_static(drafts, gamma, gamma, ctx, o["tau"], o["toks"], o["bonus"], o["new_len"], logits)
    assert e.value.code == -2
    torch.cuda.synchronize()
    assert o["tau"].cpu().tolist() == [-1] * S    # nothing was launched
