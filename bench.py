#!/usr/bin/env python
"""Benchmark of the DFlash hot path on B200: one step = context projection of the rows committed by
the previous cycle + one single-pass draft block + greedy verify/accept, for one batch.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg1] [--impl reference]

Prints ONE JSON line (rank 0). `value` = draft tokens/s with all inputs resident in HBM; `e2e` = the
same metric through the C ABI with host buffers (H2D of the step's inputs and D2H of its results
inside the timed region). `roofline` describes the dominant kernel (LM head + argmax) against the
measured HBM peak; `kernels` lists every kernel family. `cpu_baseline` is the CPU oracle timed on
this machine's host cores (a reported baseline, not the target).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2602_06036_b200 import synth  # noqa: E402

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


# ------------------------------------------------------------------------------------------------
# algorithmic bytes (what the method must move): weights once per block, KV once per sequence/layer
# ------------------------------------------------------------------------------------------------
def algorithmic_bytes(cfg, ctx_lens, n_new_rows):
    es = 4 if cfg.dtype == "fp32" else 2
    D, F, V = cfg.d_model, cfg.d_ffn, cfg.vocab
    qkv = (cfg.q_dim + 2 * cfg.kv_dim) * D * es
    o = D * cfg.q_dim * es
    gateup = 2 * F * D * es
    down = D * F * es
    lm = V * D * es
    kv_layer = 2 * cfg.kv_dim * es * sum(ctx_lens)
    ctx = (D * cfg.feat_dim + cfg.n_layers * 2 * cfg.kv_dim * D) * es + \
        n_new_rows * (cfg.feat_dim * es + cfg.n_layers * 2 * cfg.kv_dim * es)
    return {
        "gemm_qkv": qkv, "gemm_o": o, "gemm_gateup": gateup, "gemm_down": down, "lmhead_argmax": lm,
        "attention": kv_layer, "ctx_fuse": D * cfg.feat_dim * es + n_new_rows * cfg.feat_dim * es,
        "ctx_kv": cfg.n_layers * 2 * cfg.kv_dim * D * es + n_new_rows * cfg.n_layers * 2 * cfg.kv_dim * es,
        "draft_block_total": cfg.n_layers * (qkv + o + gateup + down + kv_layer) + lm,
        "ctx_project_total": ctx,
    }


class ClockSampler:
    """nvidia-smi polling during the timed region."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.idx = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.idx), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx = float(f[2])
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# the step
# ------------------------------------------------------------------------------------------------
def make_lib(cfg, device, max_ctx, seed=0):
    """A library handle holding the seeded random-init weights, with rotary tables long enough for max_ctx."""
    from paper_2602_06036_b200 import binding
    lib = binding.DFlash(cfg, str(device))
    w = synth.make_weights(cfg, seed)
    cos, sin = synth.rope_tables(cfg, max_ctx + 4 * cfg.block_size + 8)
    lib.set_weights(synth.pack_device_weights(cfg, w), cos, sin)
    return lib


class Step:
    """One workload's buffers and its step. `full_verify` (the serving-mix workload): the verify side of the step is
    the target-shaped (B+1)-row causal verify attention of one layer over a paged target cache + the LM head with
    row argmax on the [S * (B+1), D] target-shaped hidden + the accept rule on those ids, as the benchmark
    definition words it; otherwise (and as a separately timed figure) verify/accept starts from given target logits."""

    def __init__(self, wl, device, seed=0, temperature=0.0, fuse_ctx=True, lib=None, full_verify=None):
        from paper_2602_06036_b200 import binding
        cfg = wl.cfg
        self.T = float(temperature)
        self.fuse_ctx = bool(fuse_ctx)
        self.wl, self.cfg, self.dev = wl, cfg, device
        B, S = cfg.block_size, wl.batch
        self.gamma = B
        self.full_verify = (wl.name == "cfg4" and self.T <= 0) if full_verify is None else bool(full_verify)
        self.lib = lib if lib is not None else make_lib(cfg, device, max(wl.ctx_lens), seed)
        caps = [L + 2 * B + 2 for L in wl.ctx_lens]
        table, n_pages = synth.make_page_table(cfg, caps, seed)
        self.page_table = table.to(device)
        self.n_pages = n_pages
        self.ctx_len = torch.tensor(wl.ctx_lens, dtype=torch.int32, device=device)
        # context K/V: produced by the library's own context projection from N(0,1) features
        self.pool = torch.zeros(synth.kv_pool_shape(cfg, n_pages), dtype=cfg.torch_dtype, device=device)
        zero = torch.zeros(S, dtype=torch.int32, device=device)
        chunk = 4096
        for b, L in enumerate(wl.ctx_lens):
            for p0 in range(0, L, chunk):
                n = min(chunk, L - p0)
                f = synth.make_features(cfg, n, seed, f"feats.seq{b}.{p0}").to(device).reshape(1, n, cfg.feat_dim)
                self.lib.dflash_ctx_project(f, None, torch.tensor([p0], dtype=torch.int32, device=device),
                                            self.page_table[b:b + 1].contiguous(), self.pool)
        torch.cuda.synchronize()
        # per-step inputs (host masters, pinned; device copies for the resident run)
        g = self.gamma
        self.h_feats = synth.make_features(cfg, S * (g + 1), seed, "step.feats").reshape(S, g + 1, cfg.feat_dim).pin_memory()
        self.h_anchor = synth.make_anchors(cfg, S, seed).pin_memory()
        logits, drafts, planted = synth.make_verify_case(S, g, cfg.vocab, wl.accept_p, seed, cfg.torch_dtype)
        self.h_logits = logits.pin_memory()
        self.planted = planted
        self.d_feats = self.h_feats.to(device)
        self.d_anchor = self.h_anchor.to(device)
        self.d_logits = self.h_logits.to(device)
        # end-to-end staging: features and anchors share one pinned host buffer and one device buffer (one copy)
        nf = self.h_feats.numel() * self.h_feats.element_size()
        nf_pad = (nf + 255) // 256 * 256
        self.h_in = torch.zeros(nf_pad + 4 * S, dtype=torch.uint8).pin_memory()
        self.h_in[:nf].copy_(self.h_feats.view(torch.uint8).reshape(-1))
        self.h_in[nf_pad:].copy_(self.h_anchor.view(torch.uint8).reshape(-1))
        self.e_in = torch.empty(nf_pad + 4 * S, dtype=torch.uint8, device=device)
        self.e_feats = self.e_in[:nf].view(cfg.torch_dtype).view(S, g + 1, cfg.feat_dim)
        self.e_anchor = self.e_in[nf_pad:].view(torch.int32)
        self.e_logits = torch.empty_like(self.d_logits)
        self.n_new = (planted + 1).to(torch.int32).to(device)      # rows committed by the previous cycle
        # those rows are the last n_new of the context the block attends over: the step projects them, then drafts
        self.ctx_before = (self.ctx_len - self.n_new).clamp_(min=0).to(torch.int32)
        self.n_new = (self.ctx_len - self.ctx_before).to(torch.int32)
        # every result of a step lives in one flat int32 buffer, so the end-to-end run reads it back in one copy
        n_out = S * B + S * (g + 1) + 3 * S
        self.d_out = torch.zeros(n_out, dtype=torch.int32, device=device)
        self.h_out = torch.zeros(n_out, dtype=torch.int32).pin_memory()
        o = 0
        self.draft_ids = self.d_out[o:o + S * B].view(S, B); o += S * B
        self.out_tokens = self.d_out[o:o + S * (g + 1)].view(S, g + 1); o += S * (g + 1)
        self.tau = self.d_out[o:o + S]; o += S
        self.bonus = self.d_out[o:o + S]; o += S
        self.new_len = self.d_out[o:o + S]
        self.max_ctx = max(wl.ctx_lens)
        self.rows_new = int(self.n_new.sum().item())
        self.side = None
        self.vlib = None
        if self.full_verify:
            # the target's side of the cycle, one target-shaped layer (same head geometry as the drafter's layers):
            # its own paged cache over the same page table, the rotated queries and tail keys/values of the gamma+1
            # verify rows, and the hidden rows its LM head reads; all N(0,1), seeded
            import dataclasses
            tcfg = dataclasses.replace(cfg, n_layers=1)
            self.vlib = binding.DFlash(tcfg, str(device))
            R = g + 1
            self.t_pool = torch.empty(synth.kv_pool_shape(tcfg, n_pages), dtype=cfg.torch_dtype, device=device)
            gen = torch.Generator(device=device)
            gen.manual_seed(1234 + seed)
            self.t_pool.normal_(0.0, 1.0, generator=gen)
            mk = lambda *shape: torch.empty(shape, dtype=torch.float32, device=device).normal_(0.0, 1.0, generator=gen).to(cfg.torch_dtype)
            self.t_q = mk(S, R, cfg.n_q_heads, cfg.head_dim)
            self.t_k = mk(S, R, cfg.n_kv_heads, cfg.head_dim)
            self.t_v = mk(S, R, cfg.n_kv_heads, cfg.head_dim)
            self.t_attn = torch.zeros_like(self.t_q)
            self.t_hidden = mk(S * R, cfg.d_model)
            self.t_ids = torch.zeros(S * R, dtype=torch.int32, device=device)
        if self.T > 0:
            # sampling: the draft's logits are kept (fp32), drafts are drawn from them, and verification
            # is speculative sampling; the uniforms are seeded inputs
            gu = synth.substream(seed, "step.uniforms")
            self.draft_logits = torch.empty((S * B, cfg.vocab), dtype=torch.float32, device=device)
            self.u_draft = torch.rand((S * B,), generator=gu, dtype=torch.float32).to(device)
            self.u_acc = torch.rand((S, g), generator=gu, dtype=torch.float32).to(device)
            self.u_fin = torch.rand((S,), generator=gu, dtype=torch.float32).to(device)

    def run_draft(self, feats, anchor):
        lib = self.lib
        ctx = None
        if self.fuse_ctx:       # the projection rides in the draft call (one chained launch with the first QKV)
            ctx = (feats, self.n_new, self.ctx_before)
        else:
            lib.dflash_ctx_project(feats, self.n_new, self.ctx_before, self.page_table, self.pool)
        if self.T > 0:
            lib.dflash_draft_block(anchor, self.ctx_len, self.max_ctx, self.page_table, self.pool, self.draft_ids,
                                   logits_out=self.draft_logits, ctx=ctx)
            lib.dflash_sample_rows(self.draft_logits, self.T, self.u_draft, self.draft_ids.view(-1))
        else:
            lib.dflash_draft_block(anchor, self.ctx_len, self.max_ctx, self.page_table, self.pool, self.draft_ids, ctx=ctx)

    def run_verify_full(self):
        # causal verify attention of one target-shaped layer, LM head + row argmax over the gamma+1 rows of every
        # sequence, accept rule on the resulting ids (the drafter's own block is what gets verified)
        from paper_2602_06036_b200 import binding
        self.vlib.dflash_block_attention(binding.ATTN_CAUSAL, self.t_q, self.t_k, self.t_v, self.ctx_len, self.max_ctx,
                                         self.page_table, self.t_pool, 0, self.t_attn)
        self.lib.dflash_lmhead_argmax(self.t_hidden, 1, self.t_ids)
        self.lib.dflash_verify_accept(self.draft_ids, self.cfg.block_size, self.gamma, self.ctx_len, self.tau,
                                      self.out_tokens, self.bonus, self.new_len,
                                      target_ids=self.t_ids.view(self.wl.batch, self.gamma + 1))

    def run_verify(self, logits):
        # The target's forward is outside this step: its logits are an input. What is verified is the drafter's own
        # block of this step (random-init weights, so tau = 1 nearly always; the kernels' cost does not depend on
        # tau). The planted-prefix drafts of the synthetic verify case are exercised by the parity tests.
        if self.full_verify:
            return self.run_verify_full()
        if self.T > 0:
            self.lib.dflash_verify_accept_sample(logits, self.draft_logits, self.cfg.block_size, self.draft_ids,
                                                 self.cfg.block_size, self.gamma, self.T, self.u_acc, self.u_fin,
                                                 self.ctx_len, self.tau, self.out_tokens, self.bonus, self.new_len)
            return
        self.lib.dflash_verify_accept(self.draft_ids, self.cfg.block_size, self.gamma, self.ctx_len, self.tau,
                                      self.out_tokens, self.bonus, self.new_len, logits=logits)

    def step_resident(self):
        self.run_draft(self.d_feats, self.d_anchor)
        self.run_verify(self.d_logits)

    def verify_from_logits(self):
        self.lib.dflash_verify_accept(self.draft_ids, self.cfg.block_size, self.gamma, self.ctx_len, self.tau,
                                      self.out_tokens, self.bonus, self.new_len, logits=self.d_logits)

    def dev_status(self):
        st = int(self.lib.status.item())
        if self.vlib is not None:
            st |= int(self.vlib.status.item())
        return st

    def step_e2e(self):
        # The verify logits are only needed at the end of the step: their host-to-device copy runs on a
        # side stream next to the context projection and the draft (a fork/join inside the captured graph).
        # The small inputs the draft starts from go first; the logits follow on the side stream only after them, so
        # the 5 MB copy cannot sit in front of the features on the host-to-device path.
        cur = torch.cuda.current_stream()
        if self.side is None:
            self.side = torch.cuda.Stream()
        self.e_in.copy_(self.h_in, non_blocking=True)
        if self.full_verify:       # the verify side's inputs are produced on the device by the target: nothing to copy
            self.run_draft(self.e_feats, self.e_anchor)
            self.run_verify_full()
            self.h_out.copy_(self.d_out, non_blocking=True)
            return
        self.side.wait_stream(cur)
        with torch.cuda.stream(self.side):
            self.e_logits.copy_(self.h_logits, non_blocking=True)
        self.run_draft(self.e_feats, self.e_anchor)
        cur.wait_stream(self.side)
        self.run_verify(self.e_logits)
        self.h_out.copy_(self.d_out, non_blocking=True)

    def e2e_bytes(self):
        h2d = self.h_in.numel()
        if not self.full_verify:
            h2d += self.h_logits.numel() * self.h_logits.element_size()
        return h2d, self.h_out.numel() * 4


def capture(fn):
    """Capture one step into a CUDA graph (after the eager warm-up has sized every buffer)."""
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        fn()
    return g.replay


def max_over_ranks(ms, device):
    """The slowest rank's time (replicas run independently; the job is as slow as its slowest rank)."""
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return float(t.item())


def timed(fn, steps, warmup, dist_on, repeats=1):
    """`repeats` timed regions of exactly `steps` calls each, every region bracketed by a barrier (N > 1) and a
    device synchronisation on both sides and timed with a CUDA event pair on the launching stream; per region the
    maximum over ranks. Returns the list of region times in ms."""
    for _ in range(warmup):
        fn()
    out = []
    for _ in range(max(repeats, 1)):
        torch.cuda.synchronize()
        if dist_on:
            torch.distributed.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        if dist_on:
            ms = max_over_ranks(ms, "cuda")
        out.append(ms)
    return out


# ------------------------------------------------------------------------------------------------
# CPU oracle arm
# ------------------------------------------------------------------------------------------------
def oracle_sample(wl, seed=0, layers=1, vocab_frac=8):
    """A bounded sample of one step for the CPU oracle, one sequence: the context projection of the
    step's rows, `layers` of the N draft layers over the full context, the LM head over
    V/vocab_frac rows, and the accept rule on full-vocabulary logits.
    Returns (seconds, fraction of the step's algorithmic bytes covered)."""
    from oracle import dflash_oracle as orc
    import dataclasses
    cfg = wl.cfg
    layers = min(layers, cfg.n_layers)
    B = cfg.block_size
    Vs = max(cfg.vocab // vocab_frac, 2)
    sub_v = dataclasses.replace(cfg, n_layers=layers, vocab=Vs)
    w = synth.weights_to_numpy(synth.make_weights(sub_v, seed))
    L = wl.ctx_lens[0]
    ctxK = [synth.to_numpy_f32(synth.normal((L, cfg.n_kv_heads, cfg.head_dim), 1.0, seed, f"o.K{i}", cfg.torch_dtype))
            for i in range(layers)]
    ctxV = [synth.to_numpy_f32(synth.normal((L, cfg.n_kv_heads, cfg.head_dim), 1.0, seed, f"o.V{i}", cfg.torch_dtype))
            for i in range(layers)]
    feats = synth.to_numpy_f32(synth.make_features(cfg, B + 1, seed, "o.feats"))
    logits, drafts, _ = synth.make_verify_case(1, B, cfg.vocab, wl.accept_p, seed, cfg.torch_dtype)
    lg = synth.to_numpy_f32(logits[0])
    t0 = time.perf_counter()
    orc.ctx_project(feats, L + np.arange(B + 1), w, sub_v)
    orc.draft_block(3, L, ctxK, ctxV, w, sub_v)
    orc.verify_accept_logits(drafts[0].numpy(), lg, L)
    dt = time.perf_counter() - t0
    full = algorithmic_bytes(cfg, [L], B + 1)
    es = 2 if cfg.dtype == "bf16" else 4
    per_layer = (full["draft_block_total"] - full["lmhead_argmax"]) / cfg.n_layers
    covered = layers * per_layer + full["lmhead_argmax"] / cfg.vocab * Vs + \
        (cfg.d_model * cfg.feat_dim + layers * 2 * cfg.kv_dim * cfg.d_model) * es
    total = full["draft_block_total"] + full["ctx_project_total"]
    return dt, min(covered / total, 1.0)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = synth.workload(args.workload)
    cores = len(os.sched_getaffinity(0))
    B = wl.cfg.block_size
    times = []
    frac = 1.0
    for i in range(args.warmup + args.steps):
        dt, frac = oracle_sample(wl)
        if i >= args.warmup:
            times.append(dt)
    per_step = statistics.mean(times) / frac            # extrapolated to the whole step, one sequence
    value = B / per_step
    sample = (f"per step: ctx projection of {B + 1} rows + 1 of {wl.cfg.n_layers} draft layers over the full "
              f"context + LM head over V/8 + accept, one sequence; {frac:.3f} of the step's algorithmic bytes, "
              f"time scaled by 1/{frac:.3f}")
    line = {
        "impl": "reference", "metric": "draft_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "batch": 1, "block_size": B, "ctx_len": wl.ctx_lens[0]},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


class _LibOnly:
    """What the single-kernel runs that need no cached context take in place of a Step."""

    def __init__(self, wl, lib, device):
        self.wl, self.cfg, self.lib = wl, wl.cfg, lib
        self.ctx_len = torch.tensor(wl.ctx_lens, dtype=torch.int32, device=device)
        self.max_ctx = max(wl.ctx_lens)


def run_kernel_only(args, step, device):
    """One building block alone, launched eagerly `steps` times after `warmup` (profiler captures)."""
    from paper_2602_06036_b200 import binding
    cfg, wl = step.cfg, step.wl
    S, B = wl.batch, cfg.block_size
    if args.kernel == "verify":
        # greedy verify/accept from bf16 target logits [S, B+1, V] (each logit crosses HBM once)
        logits, drafts, planted = synth.make_verify_case(S, B, cfg.vocab, wl.accept_p, 0, cfg.torch_dtype)
        logits, drafts = logits.to(device), drafts.to(device)
        tau = torch.zeros(S, dtype=torch.int32, device=device)
        toks = torch.zeros((S, B + 1), dtype=torch.int32, device=device)
        bonus, new_len = torch.zeros_like(tau), torch.zeros_like(tau)
        fn = lambda: step.lib.dflash_verify_accept(drafts, B, B, step.ctx_len, tau, toks, bonus, new_len, logits=logits)
        nbytes = logits.numel() * 2
        ms = timed(fn, args.steps, args.warmup, False)[0]
        assert torch.equal(tau.cpu(), (planted + 1).to(torch.int32))
        us = ms / args.steps * 1e3
        print(json.dumps({"kernel": "verify", "workload": wl.name, "us_per_call": us, "alg_bytes": nbytes, "gbs": nbytes / (us * 1e-6) / 1e9}))
        return
    if args.kernel == "target_verify":
        # The target's verify pass over gamma + 1 rows with a target-sized stack (36 layers of the same
        # shape; the weight tensors of the drafter's layers are reused round-robin: 1.9 GB of distinct
        # weights per cycle of 5 layers, far beyond L2, so every layer streams from HBM).
        import dataclasses
        n_layers, rows = 36, B + 1
        tcfg = dataclasses.replace(cfg, n_layers=n_layers)
        tlib = binding.DFlash(tcfg, str(device))
        w = synth.pack_device_weights(cfg, synth.make_weights(cfg, 1))
        w["layers"] = [{k: v.to(device) for k, v in lw.items()} for lw in w["layers"]]
        w["layers"] = [w["layers"][i % cfg.n_layers] for i in range(n_layers)]
        cos, sin = synth.rope_tables(tcfg, max(wl.ctx_lens) + 4 * B + 8)
        tlib.set_weights(w, cos, sin)
        table, n_pages = synth.make_page_table(tcfg, [L + 2 * B + 2 for L in wl.ctx_lens], 1)
        table = table.to(device)
        pool = torch.randn(synth.kv_pool_shape(tcfg, n_pages), device=device).to(tcfg.torch_dtype)
        tokens = torch.randint(0, cfg.vocab - 1, (S, rows), dtype=torch.int32, device=device)
        taps = [1, 9, 17, 25, 33]
        ids = torch.zeros((S, rows), dtype=torch.int32, device=device)
        feats = torch.zeros((S, rows, len(taps) * cfg.d_model), dtype=cfg.torch_dtype, device=device)
        logits = torch.zeros((S * rows, cfg.vocab), dtype=torch.float32, device=device)
        fn = lambda: tlib.dflash_target_verify(tokens, step.ctx_len, step.max_ctx, table, pool, taps, ids, feats_out=feats,
                                               logits_out=logits)
        alg = algorithmic_bytes(cfg, wl.ctx_lens, 0)
        nbytes = n_layers * (alg["gemm_qkv"] + alg["gemm_o"] + alg["gemm_gateup"] + alg["gemm_down"] + alg["attention"]) + \
            alg["lmhead_argmax"]
    elif args.kernel == "block_loss":
        # Training side: the position-weighted cross entropy with its gradient over the blocks of one training
        # sequence (512 anchors per sequence, App. A.1; --loss-blocks for a smaller capture), bf16 logits of the
        # drafter's vocabulary in, bf16 gradient out. Algorithmic bytes: logits read once + gradient written once.
        nb = args.loss_blocks
        gamma = {16: 7.0, 10: 5.0, 8: 4.0}.get(B, 7.0)
        z = torch.empty((nb, B, cfg.vocab), dtype=torch.bfloat16, device=device).normal_(0.0, 3.0)
        t = torch.randint(0, cfg.vocab, (nb, B), dtype=torch.int32, device=device)
        dz = torch.empty_like(z)
        row_loss = torch.zeros(nb * B, dtype=torch.float32, device=device)
        sums = torch.zeros(2, dtype=torch.float32, device=device)
        fn = lambda: step.lib.dflash_block_loss(z, t, gamma, row_loss, sums, dz, grad_scale=1.0 / (nb * (B - 1)))
        nbytes = 2 * z.numel() * 2
    elif args.kernel == "attention_bwd":
        # Training side: backward of the block attention over one training sequence (App. A.1: 3072 tokens, 512
        # anchor blocks of 16 rows; --loss-blocks for a smaller capture), one layer of the drafter's head geometry.
        # Bound: the five contractions of the softmax-attention gradient, 2 flops per multiply-add, over the keys
        # each block sees (context before its anchor + itself) against the sustained bf16 tensor figure; the
        # operands stay in L2 (the sequence's K/V of one layer is 12.6 MB), so HBM only sees q, k, v, out, dout
        # and the gradients once.
        nb, Lseq = args.loss_blocks, 3072
        table, n_pages = synth.make_page_table(cfg, [Lseq], 2)
        table = table.to(device).repeat(nb, 1).contiguous()
        pool = torch.randn(synth.kv_pool_shape(cfg, n_pages), device=device).to(cfg.torch_dtype)
        gen = torch.Generator().manual_seed(5)
        anchors = torch.randint(1, Lseq - B, (nb,), generator=gen, dtype=torch.int32).to(device)
        mk = lambda *shape: torch.randn(*shape, device=device).to(cfg.torch_dtype)
        q, k, v = mk(nb, B, cfg.n_q_heads, cfg.head_dim), mk(nb, B, cfg.n_kv_heads, cfg.head_dim), mk(nb, B, cfg.n_kv_heads, cfg.head_dim)
        dout, out = mk(nb, B, cfg.n_q_heads, cfg.head_dim), torch.zeros(nb, B, cfg.n_q_heads, cfg.head_dim, device=device, dtype=cfg.torch_dtype)
        lse = torch.zeros(nb, B, cfg.n_q_heads, dtype=torch.float32, device=device)
        max_a = int(anchors.max().item())
        step.lib.dflash_block_attention(binding.ATTN_FULL, q, k, v, anchors, max_a, table, pool, 0, out, lse_out=lse)
        dq, dk, dv = torch.zeros_like(q), torch.zeros_like(k), torch.zeros_like(v)
        dkv = torch.zeros((n_pages, 2, cfg.n_kv_heads, cfg.page_size, cfg.head_dim), dtype=torch.float32, device=device)
        fn = lambda: step.lib.dflash_block_attention_bwd(binding.ATTN_FULL, q, k, v, out, lse, dout, anchors, max_a, table, pool, 0,
                                                         dq, dk, dv, dkv, shared_page_row=True)
        keys = float((anchors.float() + B).sum().item())
        flops = 5 * 2.0 * (B * cfg.n_q_heads) * cfg.head_dim * keys
        nbytes = (3 * q.numel() + 2 * q.numel() + 4 * k.numel()) * 2 + 2 * cfg.kv_dim * 2 * Lseq + dkv.numel() * 4 * Lseq // (n_pages * cfg.page_size)
        ms = timed(fn, args.steps, args.warmup, False)[0]
        us = ms / args.steps * 1e3
        peaks = load_peaks()
        tf = flops / (us * 1e-6) / 1e12
        peak = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
        print(json.dumps({"kernel": "attention_bwd", "blocks": nb, "seq_len": Lseq, "us_per_call": us, "flops": flops, "tflops": tf,
                          "bound": "tensor", "peak_tflops": peak, "frac": tf / peak, "hbm_bytes": nbytes,
                          "us_at_tensor_peak": flops / (peak * 1e12) * 1e6, "us_at_hbm_peak": nbytes / (peaks["hbm_gbs"] * 1e9) * 1e6}))
        return
    elif args.kernel == "lmhead":
        hid = torch.randn(S * B, cfg.d_model, device=device).to(cfg.torch_dtype)
        ids = torch.zeros(S * B, dtype=torch.int32, device=device)
        fn = lambda: step.lib.dflash_lmhead_argmax(hid, 1, ids)
        nbytes = algorithmic_bytes(cfg, wl.ctx_lens, 0)["lmhead_argmax"]
    else:
        q = torch.randn(S, B, cfg.n_q_heads, cfg.head_dim, device=device).to(cfg.torch_dtype)
        k = torch.randn(S, B, cfg.n_kv_heads, cfg.head_dim, device=device).to(cfg.torch_dtype)
        v = torch.randn(S, B, cfg.n_kv_heads, cfg.head_dim, device=device).to(cfg.torch_dtype)
        out = torch.zeros_like(q)
        fn = lambda: step.lib.dflash_block_attention(binding.ATTN_FULL, q, k, v, step.ctx_len, step.max_ctx,
                                                     step.page_table, step.pool, 0, out)
        nbytes = algorithmic_bytes(cfg, wl.ctx_lens, 0)["attention"]
    ms = timed(fn, args.steps, args.warmup, False)[0]
    us = ms / args.steps * 1e3
    print(json.dumps({"kernel": args.kernel, "workload": wl.name, "us_per_call": us, "alg_bytes": nbytes,
                      "gbs": nbytes / (us * 1e-6) / 1e9}))


# ------------------------------------------------------------------------------------------------
def phase_table(trace_rows, cfg, alg, hbm, prefix=""):
    """Per kernel family: microseconds per launch from a device-side timeline (a phase's interval runs from
    max(its inputs ready, previous record's end) to the moment its last CTA signalled completion)."""
    kernels = {}
    prev_end = None
    for fam, t_start, t_dep, t_loop, t_end in trace_rows:
        if t_end is None:
            continue
        cands = [v for v in (t_dep, prev_end) if v is not None]
        begin = max(cands) if cands else t_start
        dur = max(t_end - begin, 0) / 1e3
        prev_end = t_end if prev_end is None else max(prev_end, t_end)
        e = kernels.setdefault(prefix + fam, {"us_total": 0.0, "launches_per_step": 0})
        e["us_total"] += dur
        e["launches_per_step"] += 1
    for fam, e in kernels.items():
        n = e["launches_per_step"]
        if fam == "attention":               # one or two records (main kernel, merge kernel) make one attention per layer
            n = cfg.n_layers
            e["launches_per_step"] = n
        if fam == "verify_attention":
            n = 1
            e["launches_per_step"] = n
        e["us_per_launch"] = e.pop("us_total") / n
        if fam in alg and e["us_per_launch"] > 0:
            e["alg_bytes"] = alg[fam]
            e["gbs"] = alg[fam] / (e["us_per_launch"] * 1e-6) / 1e9
            e["frac_hbm"] = e["gbs"] / hbm
    return kernels


def measure(step, args, peaks, dist_on, rank, sampler=None, repeats=7, e2e_repeats=3):
    """Times one workload's step (resident: CUDA-graph replay unless --no-graph; end to end: host buffers through
    the C ABI), checks the timed step's outputs, and reads the device-side timeline of one eager step."""
    from paper_2602_06036_b200 import binding
    wl, cfg = step.wl, step.cfg
    S, B = wl.batch, cfg.block_size
    run_resident, run_e2e = step.step_resident, step.step_e2e
    for _ in range(2):           # eager warm-up: sizes the workspace, sets kernel attributes
        run_resident()
        run_e2e()
    torch.cuda.synchronize()
    if step.dev_status() != 0:       # e.g. a bounded wait that ran out: do not go on to time a broken step
        raise RuntimeError(f"bench: device status {step.dev_status()} after the warm-up steps of {wl.name}")
    n0 = binding.launch_count()
    run_resident()
    launches_per_step = binding.launch_count() - n0
    if not args.no_graph:
        run_resident = capture(step.step_resident)
        run_e2e = capture(step.step_e2e)
    step.lib.status.zero_()
    if step.vlib is not None:
        step.vlib.status.zero_()
    if sampler is not None:
        sampler.start()
    regions = timed(run_resident, args.steps, args.warmup, dist_on, repeats)
    clocks = sampler.stop() if sampler is not None else None
    out_resident = step.d_out.clone()
    regions_e2e = timed(run_e2e, args.steps, args.warmup, dist_on, e2e_repeats)
    torch.cuda.synchronize()
    # the timed steps' results: no device-detected problem (bad id / page, expired wait), the end-to-end run's
    # outputs equal the resident run's (same inputs), and what came back to the host is what the device holds
    status = step.dev_status()
    same = bool(torch.equal(step.d_out, out_resident)) and bool(torch.equal(step.h_out, step.d_out.cpu()))
    in_range = bool(((step.draft_ids >= 0) & (step.draft_ids < cfg.vocab)).all().item()) and \
        bool(((step.tau >= 1) & (step.tau <= step.gamma + 1)).all().item())
    checked = status == 0 and same and in_range
    if not checked:
        raise RuntimeError(f"bench self-check failed on {wl.name}: dev_status={status} outputs_equal={same} in_range={in_range}")

    per = sorted(ms / args.steps for ms in regions)
    per_step_ms = statistics.median(per)
    per_e2e = statistics.median(ms / args.steps for ms in regions_e2e)
    res = {"ms_per_step": per_step_ms, "ms_per_step_min": per[0], "ms_per_step_max": per[-1], "regions": len(per),
           "ms_per_step_e2e": per_e2e, "launches_per_step": int(launches_per_step), "clocks": clocks, "checked": True}
    if rank != 0:
        return res
    alg = algorithmic_bytes(cfg, wl.ctx_lens, step.rows_new)
    hbm = peaks["hbm_gbs"]
    es = 4 if cfg.dtype == "fp32" else 2
    if not step.full_verify:      # greedy verify from the target's logits: one launch, every logit read once
        alg["row_argmax"] = step.d_logits.numel() * step.d_logits.element_size()
    # device-side timeline of one extra eager step; the verify side of the serving-mix step runs on a second
    # handle (the target-shaped layer) and on the LM head of this one: traced separately and prefixed
    if step.full_verify:
        kernels = phase_table(step.lib.trace(lambda: step.run_draft(step.d_feats, step.d_anchor)), cfg, alg, hbm)
        alg_v = {"verify_attention": 2 * cfg.kv_dim * es * sum(wl.ctx_lens), "verify_lmhead_argmax": alg["lmhead_argmax"]}
        from paper_2602_06036_b200 import binding as bnd
        tr_a = step.vlib.trace(lambda: step.vlib.dflash_block_attention(bnd.ATTN_CAUSAL, step.t_q, step.t_k, step.t_v, step.ctx_len,
                                                                         step.max_ctx, step.page_table, step.t_pool, 0, step.t_attn))
        kernels.update(phase_table(tr_a, cfg, alg_v, hbm, prefix="verify_"))
        tr_l = step.lib.trace(lambda: step.lib.dflash_lmhead_argmax(step.t_hidden, 1, step.t_ids))
        kernels.update(phase_table(tr_l, cfg, alg_v, hbm, prefix="verify_"))
        res["trace_rows"] = []
    else:
        rows = step.lib.trace(step.step_resident)
        kernels = phase_table(rows, cfg, alg, hbm)
        res["trace_rows"] = rows
    # lower bound of the step: its phases run one after the other, each bound by the slower of its
    # HBM traffic and its dense bf16 contraction (2 x rows x weights; sustained tensor figure)
    tensor = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]) * 1e12
    bound_s, tensor_phases = 0.0, []
    phases = [("ctx_fuse", 1, step.rows_new, alg["ctx_fuse"]), ("ctx_kv", 1, step.rows_new, alg["ctx_kv"]),
              ("gemm_qkv", cfg.n_layers, S * B, alg["gemm_qkv"]), ("gemm_o", cfg.n_layers, S * B, alg["gemm_o"]),
              ("gemm_gateup", cfg.n_layers, S * B, alg["gemm_gateup"]), ("gemm_down", cfg.n_layers, S * B, alg["gemm_down"]),
              ("lmhead_argmax", 1, S * B, alg["lmhead_argmax"]), ("attention", cfg.n_layers, 0, alg["attention"])]
    step_bytes = alg["draft_block_total"] + alg["ctx_project_total"]
    if step.full_verify:
        phases += [("verify_attention", 1, 0, alg_v["verify_attention"]),
                   ("verify_lmhead_argmax", 1, S * (B + 1), alg_v["verify_lmhead_argmax"])]
        step_bytes += alg_v["verify_attention"] + alg_v["verify_lmhead_argmax"]
    else:
        step_bytes += S * (B + 1) * cfg.vocab * 2
        bound_s += S * (B + 1) * cfg.vocab * 2 / (hbm * 1e9)      # verify reads the target logits once
    for fam, n_launch, rows_, nbytes in phases:
        t_hbm = nbytes / (hbm * 1e9)
        t_tc = 2.0 * rows_ * (nbytes / es) / tensor if cfg.dtype != "fp32" else 0.0
        if t_tc > t_hbm:
            tensor_phases.append(fam)
        bound_s += n_launch * max(t_hbm, t_tc)
        if fam in kernels:
            kernels[fam]["us_at_peak"] = max(t_hbm, t_tc) * 1e6
            kernels[fam]["bound"] = "tensor" if t_tc > t_hbm else "hbm"
            kernels[fam]["frac_of_bound"] = kernels[fam]["us_at_peak"] / kernels[fam]["us_per_launch"]
    res.update({"alg": alg, "kernels": kernels, "step_bytes": step_bytes,
                "step_roofline": {"alg_bytes": step_bytes, "us_at_hbm_peak": step_bytes / (hbm * 1e9) * 1e6,
                                  "us_at_peak": bound_s * 1e6, "frac": bound_s / (per_step_ms * 1e-3),
                                  "tensor_bound_phases": tensor_phases,
                                  "note": "sum over the step's phases of max(bytes / measured HBM, flops / measured sustained bf16)"}})
    if step.full_verify:
        # the same step's verify side from given target logits instead (the logits cross HBM once), timed alone
        fn = step.verify_from_logits
        fn()
        fn = fn if args.no_graph else capture(fn)
        ms = statistics.median(timed(fn, args.steps, 3, False, 3)) / args.steps
        nb = S * (B + 1) * cfg.vocab * 2
        res["accept_from_logits"] = {"us_per_call": ms * 1e3, "alg_bytes": nb, "gbs": nb / (ms * 1e-3) / 1e9,
                                     "frac_hbm": nb / (ms * 1e-3) / 1e9 / hbm}
    return res


def step_text(step, args):
    if args.temperature > 0:
        return f"ctx_project(n_new=tau) + draft_block(logits kept) + sample_rows + verify_accept_sample, T={args.temperature}"
    if step.full_verify:
        return ("ctx_project(n_new=tau) + draft_block + causal verify attention of one target-shaped layer over (B+1) rows + "
                "LM head with row argmax on [S*(B+1), D] + verify_accept(ids)")
    return "ctx_project(n_new=tau) + draft_block + verify_accept(logits)"


def spawn_ranks(n):
    """`python bench.py --gpus N` started without a launcher: start the N ranks ourselves (one process per GPU,
    the same command line torch.distributed.run would be given) and pass their output through."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    sys.exit(subprocess.call(cmd))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="cfg1")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--kernel", default=None, choices=["lmhead", "attention", "target_verify", "block_loss", "attention_bwd", "verify"],
                    help="run one building block alone (for profiler captures) instead of the step")
    ap.add_argument("--loss-blocks", type=int, default=512, help="--kernel block_loss: blocks (of block_size rows) per call")
    ap.add_argument("--trace", default=None, help="write a device-side timeline of one step to this file")
    ap.add_argument("--temperature", type=float, default=0.0,
                    help="> 0: drafts are drawn from the draft's logits and verified by speculative sampling (default: greedy)")
    ap.add_argument("--separate-ctx", action="store_true",
                    help="run the context projection as its own call before the draft call instead of inside it")
    ap.add_argument("--no-graph", action="store_true", help="launch every step eagerly instead of replaying a CUDA graph")
    ap.add_argument("--ctx-len", type=int, default=0,
                    help="> 0: every sequence of the workload gets this context length (a small case of the same launches for profiler captures)")
    ap.add_argument("--repeats", type=int, default=7, help="timed regions of --steps steps each; ms_per_step is their median")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="skip the extra key with the other benchmark configurations (cfg2, cfg3, cfg4) measured in the same run")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "b200" else max(args.warmup, 0)

    if args.impl == "reference":
        run_reference(args)
        return

    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus > 1 and world == 1 and "RANK" not in os.environ:
        spawn_ranks(args.gpus)
    if world != args.gpus:
        sys.exit(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s); start one rank per GPU "
                 f"(python -m torch.distributed.run --nproc-per-node {args.gpus} ...) or run plain `python bench.py --gpus {args.gpus}`")
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist_on = world > 1
    torch.cuda.set_device(local)
    device = torch.device(f"cuda:{local}")
    if dist_on:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.distributed.init_process_group("nccl", device_id=device)

    from paper_2602_06036_b200 import build
    build.build()
    wl = synth.workload(args.workload)
    if args.ctx_len > 0:
        import dataclasses
        wl = dataclasses.replace(wl, ctx_lens=tuple(args.ctx_len for _ in wl.ctx_lens))
        args.no_other_workloads = True
    cfg = wl.cfg
    peaks = load_peaks()
    hbm = peaks["hbm_gbs"]
    others = [] if (args.no_other_workloads or args.kernel or args.temperature > 0 or cfg.dtype == "fp32") else \
        [n for n in ("cfg1", "cfg2", "cfg3", "cfg4") if n != wl.name]
    if not others or args.workload == "cfg0":
        others = []
    # replicas: every rank runs the same batch on its own GPU; there is no data-path collective.
    # One handle (one copy of the weights) serves every workload of the run.
    max_ctx = max([max(wl.ctx_lens)] + [max(synth.workload(n).ctx_lens) for n in others])
    lib = make_lib(cfg, device, max_ctx, seed=0)
    if args.kernel in ("verify", "lmhead", "block_loss", "attention_bwd"):      # no cached context needed
        run_kernel_only(args, _LibOnly(wl, lib, device), device)
        return
    step = Step(wl, device, seed=0, temperature=args.temperature, fuse_ctx=not args.separate_ctx, lib=lib)
    S, B = wl.batch, cfg.block_size

    if args.kernel:
        run_kernel_only(args, step, device)
        return

    sampler = ClockSampler(local) if rank == 0 else None
    m = measure(step, args, peaks, dist_on, rank, sampler, repeats=args.repeats)
    # The dominant kernel alone, timed with CUDA event pairs around each of its launches.
    lm_us = None
    if rank == 0:
        hid = torch.randn(S * B, cfg.d_model, device=device).to(cfg.torch_dtype)
        ids = torch.zeros(S * B, dtype=torch.int32, device=device)
        lm_call = lambda: step.lib.dflash_lmhead_argmax(hid, 1, ids)
        for _ in range(3):
            lm_call()
        prof_lm = step.lib.profile(lm_call, max(args.steps, 10))
        lm_us = prof_lm.get("lmhead_argmax", (None, 0))[0]
    if args.trace and rank == 0:
        with open(args.trace, "w") as f:
            f.write("# kernel family, first CTA start, dependency resolved, main loop end, last CTA exit (us since first start)\n")
            for fam, a, b, c, d in m.get("trace_rows", []):
                us = lambda v: "      -" if v is None else f"{v / 1e3:8.2f}"
                f.write(f"{fam:16s} {us(a)} {us(b)} {us(c)} {us(d)}\n")

    h2d, d2h = step.e2e_bytes()
    main_step_text = step_text(step, args)
    # the other benchmark configurations, same process and weights (every rank runs them: the regions hold barriers)
    extra = {}
    del step
    for name in others:
        torch.cuda.empty_cache()
        st2 = Step(synth.workload(name), device, seed=0, fuse_ctx=not args.separate_ctx, lib=lib)
        r = measure(st2, args, peaks, dist_on, rank, None, repeats=3, e2e_repeats=1)
        if rank == 0:
            S2 = st2.wl.batch
            e = {"ms_per_step": r["ms_per_step"], "ms_per_step_min": r["ms_per_step_min"], "ms_per_step_max": r["ms_per_step_max"],
                 "us_per_draft_block": r["ms_per_step"] * 1e3, "draft_tokens_per_s": S2 * B * world / (r["ms_per_step"] * 1e-3),
                 "ms_per_step_e2e": r["ms_per_step_e2e"], "batch": S2, "ctx_tokens": int(sum(st2.wl.ctx_lens)),
                 "step": step_text(st2, args), "step_roofline": r["step_roofline"], "kernels": r["kernels"],
                 "gpu_launches_per_step": r["launches_per_step"], "checked": r["checked"]}
            if "accept_from_logits" in r:
                e["accept_from_logits"] = r["accept_from_logits"]
            extra[name] = e
        del st2

    if rank != 0:
        if dist_on:
            torch.distributed.destroy_process_group()
        return

    per_step_ms = m["ms_per_step"]
    tokens = S * B * world
    value = tokens / (per_step_ms * 1e-3)
    e2e_value = tokens / (m["ms_per_step_e2e"] * 1e-3)
    alg, kernels = m["alg"], m["kernels"]
    roofline = None
    if lm_us:
        traffic = None
        prof_file = os.path.join(ROOT, "profiles", "lmhead_argmax_cfg1.md")
        if os.path.exists(prof_file):
            for line in open(prof_file):
                if line.startswith("dram_bytes_per_launch:"):
                    traffic = int(line.split(":")[1].strip().split()[0])
        gbs = alg["lmhead_argmax"] / (lm_us * 1e-6) / 1e9
        roofline = {"kernel": "gemm_tc_kernel<16, 2> as LM head + argmax (V x D weights, 16 rows)", "bound": "hbm",
                    "achieved": gbs, "peak": hbm, "unit": "GB/s", "frac": gbs / hbm, "traffic": traffic,
                    "peak_source": peaks["_source"] + " (copy bandwidth)", "us_per_launch": lm_us,
                    "timing": "CUDA event pair around each launch of the kernel run alone (dflash_lmhead_argmax), "
                              "same weights and row count as in the step",
                    "in_step_us": kernels.get("lmhead_argmax", {}).get("us_per_launch")}
    line = {
        "metric": "draft_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": per_step_ms, "us_per_draft_block": per_step_ms * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "config": {"workload": wl.name, "batch": S, "block_size": B, "ctx_lens": list(wl.ctx_lens)[:8],
                   "step": main_step_text,
                   "l2": "per-step weight traffic (3.2 GB) exceeds the 126 MB L2; no flush",
                   "launch": "eager" if args.no_graph else "cuda graph replay of one step",
                   "parallelism": "replicas" if world > 1 else "single"},
        "timing": {"regions": m["regions"], "steps_per_region": args.steps, "ms_per_step_median": per_step_ms,
                   "ms_per_step_min": m["ms_per_step_min"], "ms_per_step_max": m["ms_per_step_max"],
                   "note": "ms_per_step is the median over the timed regions; each region is exactly `steps` steps between "
                           "synchronisations, timed by a CUDA event pair, maximum over ranks"},
        "checked": m["checked"],
        "checked_note": "after timing: device status word 0, the end-to-end run's outputs equal the resident run's and the host copy, ids and accept lengths in range",
        "step_roofline": m["step_roofline"],
        "roofline": roofline, "kernels": kernels,
        "kernels_note": "device-side timeline of one eager step: per phase, from inputs ready to last CTA done",
        "clocks": m["clocks"], "gpu_launches": int(m["launches_per_step"] * args.steps * m["regions"]),
        "e2e": {"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": m["ms_per_step_e2e"]},
    }
    if extra:
        line["workloads"] = extra
    if not args.no_cpu_baseline:
        # the whole step (all layers, full vocabulary) for one sequence: about 10-30 s of host work
        reps, spent = [], 0.0
        while spent < 10.0 and len(reps) < 8:
            dt, frac = oracle_sample(wl, layers=cfg.n_layers, vocab_frac=1)
            reps.append(dt)
            spent += dt
        dt = statistics.mean(reps)
        cores = len(os.sched_getaffinity(0))
        line["cpu_baseline"] = {
            "value": B / (dt / frac), "unit": "tokens/s", "cores": cores, "kind": "oracle",
            "sample": f"one sequence of the batch, whole step (ctx projection of {B + 1} rows, all {cfg.n_layers} draft layers "
                      f"over its full context, full-vocabulary LM head, accept): mean of {len(reps)} runs, {dt:.1f} s each, float64 numpy"}
    print(json.dumps(line))
    if dist_on:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
