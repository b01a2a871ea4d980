"""Shared scaffolding of the GPU parity tests: builds one seeded case, hands the identical numbers
to the CUDA library (through the C ABI binding) and to the CPU oracle, and compares."""
from __future__ import annotations

import numpy as np
import torch

from oracle import dflash_oracle as orc
from paper_2602_06036_b200 import synth

# Tolerances. bf16: the benchmark definition's (relative L2 <= 1e-2, max abs <= 5e-2, argmax ids
# equal where the oracle's top-1/top-2 margin exceeds 0.1). fp32: rounding-order differences of an
# fp32 FMA path against the float64 oracle over K <= 768 terms.
TOL = {
    "bf16": dict(rel_l2=1e-2, max_abs=5e-2, margin=0.1),
    "fp32": dict(rel_l2=1e-5, max_abs=1e-4, margin=1e-3),
}


def assert_close(got, ref, dtype, what=""):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    t = TOL[dtype]
    assert np.all(np.isfinite(got)), what
    rel = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)
    mx = float(np.max(np.abs(got - ref))) if got.size else 0.0
    assert rel <= t["rel_l2"] and mx <= t["max_abs"], f"{what}: rel_l2={rel:.3e} max_abs={mx:.3e}"
    return rel, mx


def assert_ids_match(got_ids, ref_ids, ref_margin, dtype, what=""):
    got_ids = np.asarray(got_ids).reshape(-1)
    ref_ids = np.asarray(ref_ids).reshape(-1)
    sure = np.asarray(ref_margin).reshape(-1) > TOL[dtype]["margin"]
    bad = np.nonzero(sure & (got_ids != ref_ids))[0]
    assert bad.size == 0, f"{what}: rows {bad.tolist()} differ where the oracle margin is decisive"
    return int(sure.sum())


class Case:
    """One model + batch of sequences with paged context, on both sides."""

    def __init__(self, cfg, ctx_lens, seed=0, weights=None, headroom=None, device="cuda:0", w_np=None, lib=None):
        from paper_2602_06036_b200 import binding
        self.cfg = cfg
        self.dtype = cfg.dtype
        self.ctx_lens = [int(v) for v in ctx_lens]
        self.S = len(self.ctx_lens)
        self.device = torch.device(device)
        self.seed = seed
        B = cfg.block_size
        self.headroom = headroom if headroom is not None else 2 * B + 2
        if weights is None:
            weights = synth.make_weights(cfg, seed)
        self.w_cpu = weights
        self.w_np = w_np if w_np is not None else synth.weights_to_numpy(weights)
        self.max_pos = max(self.ctx_lens + [0]) + self.headroom + 1
        cos, sin = synth.rope_tables(cfg, self.max_pos)
        if lib is None:
            self.lib = binding.DFlash(cfg, device)
            self.lib.set_weights(synth.pack_device_weights(cfg, weights), cos, sin)
        else:                      # a handle that already holds these weights (rope tables long enough)
            self.lib = lib
        caps = [L + self.headroom for L in self.ctx_lens]
        self.page_table_cpu, self.n_pages = synth.make_page_table(cfg, caps, seed)
        self.page_table = self.page_table_cpu.to(self.device)
        self.ctx_len = torch.tensor(self.ctx_lens, dtype=torch.int32, device=self.device)
        self.pool = torch.zeros(synth.kv_pool_shape(cfg, self.n_pages), dtype=cfg.torch_dtype, device=self.device)
        self.pool_np = None      # oracle-side pool (float32 holding the same values)

    # ---- context --------------------------------------------------------------------------
    def fill_pool_synthetic(self):
        """Fill both pools with the same N(0,1) entries (no projection involved)."""
        cpu = synth.make_kv_pool(self.cfg, self.n_pages, self.seed)
        self.pool.copy_(cpu)
        self.pool_np = synth.to_numpy_f32(cpu)

    def project_prefill(self, oracle=True):
        """Run the context projection for positions 0..L_b-1 of every sequence on the GPU and, if
        asked, with the oracle into its own pool."""
        cfg = self.cfg
        max_new = max(self.ctx_lens + [1])
        feats = torch.zeros((self.S, max_new, cfg.feat_dim), dtype=cfg.torch_dtype)
        for b, L in enumerate(self.ctx_lens):
            if L:
                feats[b, :L] = synth.make_features(cfg, L, self.seed, f"feats.seq{b}")
        self.feats_cpu = feats
        n_new = torch.tensor(self.ctx_lens, dtype=torch.int32, device=self.device)
        zero = torch.zeros(self.S, dtype=torch.int32, device=self.device)
        self.lib.dflash_ctx_project(feats.to(self.device), n_new, zero, self.page_table, self.pool)
        torch.cuda.synchronize()
        if oracle:
            self.pool_np = np.zeros(synth.kv_pool_shape(cfg, self.n_pages), dtype=np.float64)
            for b, L in enumerate(self.ctx_lens):
                if L == 0:
                    continue
                K, V = orc.ctx_project(synth.to_numpy_f32(feats[b, :L]), np.arange(L), self.w_np, cfg)
                orc.pool_write(self.pool_np, self.page_table_cpu[b].numpy(), list(range(L)), K, V, cfg.page_size)

    def oracle_ctx(self, b):
        cfg = self.cfg
        L = self.ctx_lens[b]
        Ks, Vs = [], []
        for i in range(cfg.n_layers):
            K, V = orc.pool_read(self.pool_np, self.page_table_cpu[b].numpy(), L, i, cfg.page_size)
            Ks.append(K)
            Vs.append(V)
        return Ks, Vs

    # ---- draft ----------------------------------------------------------------------------
    def run_draft(self, anchors=None, want_logits=True):
        cfg = self.cfg
        B, S = cfg.block_size, self.S
        if anchors is None:
            anchors = synth.make_anchors(cfg, S, self.seed)
        self.anchors_cpu = anchors
        dev = self.device
        out = {
            "ids": torch.full((S, B), -7, dtype=torch.int32, device=dev),
            "top1": torch.zeros((S, B), dtype=torch.float32, device=dev),
            "margin": torch.zeros((S, B), dtype=torch.float32, device=dev),
            "hidden": torch.zeros((S * B, cfg.d_model), dtype=torch.float32, device=dev),
            "logits": torch.zeros((S * B, cfg.vocab), dtype=torch.float32, device=dev) if want_logits else None,
        }
        self.lib.status.zero_()
        self.lib.dflash_draft_block(anchors.to(dev), self.ctx_len, max(self.ctx_lens + [0]), self.page_table,
                                    self.pool, out["ids"], out["top1"], out["margin"], out["hidden"], out["logits"])
        torch.cuda.synchronize()
        assert int(self.lib.status.item()) == 0
        return {k: (v.cpu().numpy() if v is not None else None) for k, v in out.items()}

    def oracle_draft(self, b, return_logits=True):
        Ks, Vs = self.oracle_ctx(b)
        return orc.draft_block(int(self.anchors_cpu[b]), self.ctx_lens[b], Ks, Vs, self.w_np, self.cfg,
                               return_logits=return_logits)

    def check_draft(self, got, seqs=None, logit_cols=None):
        """Compare the GPU block with the oracle for the listed sequences (default: all)."""
        cfg = self.cfg
        B = cfg.block_size
        n_sure = 0
        for b in (range(self.S) if seqs is None else seqs):
            ref = self.oracle_draft(b, return_logits=True)
            sl = slice(b * B, (b + 1) * B)
            assert_close(got["hidden"][sl], ref["hidden"], self.dtype, f"hidden seq {b}")
            if got["logits"] is not None:
                assert_close(got["logits"][sl], ref["logits"], self.dtype, f"logits seq {b}")
            n_sure += assert_ids_match(got["ids"][b], ref["ids"], ref["margin"], self.dtype, f"draft ids seq {b}")
            # the winning logit agrees with the oracle's value at the index the GPU chose
            picked = ref["logits"][np.arange(B), got["ids"][b]]
            assert np.max(np.abs(got["top1"][b] - picked)) <= TOL[self.dtype]["max_abs"]
            assert np.all(got["margin"][b] >= 0)
        return n_sure
