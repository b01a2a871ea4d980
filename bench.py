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
class Step:
    def __init__(self, wl, device, seed=0, temperature=0.0, fuse_ctx=True):
        from paper_2602_06036_b200 import binding
        cfg = wl.cfg
        self.T = float(temperature)
        self.fuse_ctx = bool(fuse_ctx)
        self.wl, self.cfg, self.dev = wl, cfg, device
        B, S = cfg.block_size, wl.batch
        self.gamma = B
        self.lib = binding.DFlash(cfg, str(device))
        w = synth.make_weights(cfg, seed)
        cos, sin = synth.rope_tables(cfg, max(wl.ctx_lens) + 4 * B + 8)
        self.lib.set_weights(synth.pack_device_weights(cfg, w), cos, sin)
        del w
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

    def run_verify(self, logits):
        # The target's verify pass is outside this library; its logits are an input. The drafts
        # verified are synthetic ones with a planted agreeing prefix (the random-init drafter would
        # never be accepted), so the accept kernel sees realistic accept lengths.
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

    def step_e2e(self):
        # The verify logits are only needed at the end of the step: their host-to-device copy runs on a
        # side stream next to the context projection and the draft (a fork/join inside the captured graph).
        # The small inputs the draft starts from go first; the logits follow on the side stream only after them, so
        # the 5 MB copy cannot sit in front of the features on the host-to-device path.
        cur = torch.cuda.current_stream()
        if self.side is None:
            self.side = torch.cuda.Stream()
        self.e_in.copy_(self.h_in, non_blocking=True)
        self.side.wait_stream(cur)
        with torch.cuda.stream(self.side):
            self.e_logits.copy_(self.h_logits, non_blocking=True)
        self.run_draft(self.e_feats, self.e_anchor)
        cur.wait_stream(self.side)
        self.run_verify(self.e_logits)
        self.h_out.copy_(self.d_out, non_blocking=True)

    def e2e_bytes(self):
        h2d = self.h_in.numel() + \
            self.h_logits.numel() * self.h_logits.element_size()
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


def timed(fn, steps, warmup, dist_on):
    for _ in range(warmup):
        fn()
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
    return ms


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


def run_kernel_only(args, step, device):
    """One building block alone, launched eagerly `steps` times after `warmup` (profiler captures)."""
    from paper_2602_06036_b200 import binding
    cfg, wl = step.cfg, step.wl
    S, B = wl.batch, cfg.block_size
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
    ms = timed(fn, args.steps, args.warmup, False)
    us = ms / args.steps * 1e3
    print(json.dumps({"kernel": args.kernel, "workload": wl.name, "us_per_call": us, "alg_bytes": nbytes,
                      "gbs": nbytes / (us * 1e-6) / 1e9}))


# ------------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="cfg1")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--kernel", default=None, choices=["lmhead", "attention", "target_verify", "block_loss"],
                    help="run one building block alone (for profiler captures) instead of the step")
    ap.add_argument("--loss-blocks", type=int, default=512, help="--kernel block_loss: blocks (of block_size rows) per call")
    ap.add_argument("--trace", default=None, help="write a device-side timeline of one step to this file")
    ap.add_argument("--temperature", type=float, default=0.0,
                    help="> 0: drafts are drawn from the draft's logits and verified by speculative sampling (default: greedy)")
    ap.add_argument("--separate-ctx", action="store_true",
                    help="run the context projection as its own call before the draft call instead of inside it")
    ap.add_argument("--no-graph", action="store_true", help="launch every step eagerly instead of replaying a CUDA graph")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "b200" else max(args.warmup, 0)

    if args.impl == "reference":
        run_reference(args)
        return

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist_on = world > 1
    torch.cuda.set_device(local)
    device = torch.device(f"cuda:{local}")
    if dist_on:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.distributed.init_process_group("nccl", device_id=device)

    from paper_2602_06036_b200 import binding, build
    build.build()
    wl = synth.workload(args.workload)
    cfg = wl.cfg
    peaks = load_peaks()
    # replicas: every rank runs the same batch on its own GPU; there is no data-path collective
    step = Step(wl, device, seed=0, temperature=args.temperature, fuse_ctx=not args.separate_ctx)
    S, B = wl.batch, cfg.block_size

    if args.kernel:
        run_kernel_only(args, step, device)
        return

    sampler = ClockSampler(local)
    run_resident, run_e2e = step.step_resident, step.step_e2e
    for _ in range(2):           # eager warm-up: sizes the workspace, sets kernel attributes
        run_resident()
        run_e2e()
    torch.cuda.synchronize()
    n0 = binding.launch_count()
    run_resident()
    launches_per_step = binding.launch_count() - n0
    if not args.no_graph:
        run_resident = capture(step.step_resident)
        run_e2e = capture(step.step_e2e)
    if rank == 0:
        sampler.start()
    ms = timed(run_resident, args.steps, args.warmup, dist_on)
    launches = launches_per_step * args.steps
    clocks = sampler.stop() if rank == 0 else None
    ms_e2e = timed(run_e2e, args.steps, args.warmup, dist_on)

    # Per-kernel figures. Chained launches hide their phases from CUDA events, so the library's
    # device-side timeline (global-timer stamps written by the kernels themselves) is read for one
    # extra, eager step: a phase's interval runs from max(its inputs ready, previous record's end) to
    # the moment its last CTA signalled completion.
    trace_rows = step.lib.trace(step.step_resident) if rank == 0 else []
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
        rows = trace_rows
        with open(args.trace, "w") as f:
            f.write("# kernel family, first CTA start, dependency resolved, main loop end, last CTA exit (us since first start)\n")
            for fam, a, b, c, d in rows:
                us = lambda v: "      -" if v is None else f"{v / 1e3:8.2f}"
                f.write(f"{fam:16s} {us(a)} {us(b)} {us(c)} {us(d)}\n")

    if rank != 0:
        if dist_on:
            torch.distributed.destroy_process_group()
        return

    per_step_ms = ms / args.steps
    tokens = S * B * world
    value = tokens / (per_step_ms * 1e-3)
    e2e_value = tokens / (ms_e2e / args.steps * 1e-3)
    h2d, d2h = step.e2e_bytes()
    alg = algorithmic_bytes(cfg, wl.ctx_lens, step.rows_new)
    hbm = peaks["hbm_gbs"]
    kernels = {}
    prev_end = None
    for fam, t_start, t_dep, t_loop, t_end in trace_rows:
        if t_end is None:
            continue
        cands = [v for v in (t_dep, prev_end) if v is not None]
        begin = max(cands) if cands else t_start
        dur = max(t_end - begin, 0) / 1e3
        prev_end = t_end if prev_end is None else max(prev_end, t_end)
        e = kernels.setdefault(fam, {"us_total": 0.0, "launches_per_step": 0})
        e["us_total"] += dur
        e["launches_per_step"] += 1
    for fam, e in kernels.items():
        n = e["launches_per_step"]
        if fam == "attention":               # one or two records (main kernel, merge kernel) make one attention per layer
            n = cfg.n_layers
            e["launches_per_step"] = n
        e["us_per_launch"] = e.pop("us_total") / n
        if fam in alg and e["us_per_launch"] > 0:
            e["alg_bytes"] = alg[fam]
            e["gbs"] = alg[fam] / (e["us_per_launch"] * 1e-6) / 1e9
            e["frac_hbm"] = e["gbs"] / hbm
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
    step_bytes = alg["draft_block_total"] + alg["ctx_project_total"] + S * (B + 1) * cfg.vocab * 2
    # lower bound of the step: its phases run one after the other, each bound by the slower of its
    # HBM traffic and its dense bf16 contraction (2 x rows x weights; sustained tensor figure)
    tensor = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]) * 1e12
    es = 4 if cfg.dtype == "fp32" else 2
    bound_s, tensor_phases = 0.0, []
    for fam, n_launch, rows in (("ctx_fuse", 1, step.rows_new), ("ctx_kv", 1, step.rows_new),
                                ("gemm_qkv", cfg.n_layers, S * B), ("gemm_o", cfg.n_layers, S * B),
                                ("gemm_gateup", cfg.n_layers, S * B), ("gemm_down", cfg.n_layers, S * B),
                                ("lmhead_argmax", 1, S * B), ("attention", cfg.n_layers, 0)):
        t_hbm = alg[fam] / (hbm * 1e9)
        t_tc = 2.0 * rows * (alg[fam] / es) / tensor if cfg.dtype != "fp32" else 0.0
        if t_tc > t_hbm:
            tensor_phases.append(fam)
        bound_s += n_launch * max(t_hbm, t_tc)
        if fam in kernels:
            kernels[fam]["us_at_peak"] = max(t_hbm, t_tc) * 1e6
            kernels[fam]["bound"] = "tensor" if t_tc > t_hbm else "hbm"
    bound_s += S * (B + 1) * cfg.vocab * 2 / (hbm * 1e9)      # verify reads the target logits once
    line = {
        "metric": "draft_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": per_step_ms, "us_per_draft_block": per_step_ms * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "config": {"workload": wl.name, "batch": S, "block_size": B, "ctx_lens": list(wl.ctx_lens)[:8],
                   "step": "ctx_project(n_new=tau) + draft_block + verify_accept(logits)" if args.temperature <= 0 else
                           f"ctx_project(n_new=tau) + draft_block(logits kept) + sample_rows + verify_accept_sample, T={args.temperature}",
                   "l2": "per-step weight traffic (3.2 GB) exceeds the 126 MB L2; no flush",
                   "launch": "eager" if args.no_graph else "cuda graph replay of one step",
                   "parallelism": "replicas" if world > 1 else "single"},
        "step_roofline": {"alg_bytes": step_bytes, "us_at_hbm_peak": step_bytes / (hbm * 1e9) * 1e6,
                          "us_at_peak": bound_s * 1e6, "frac": bound_s / (per_step_ms * 1e-3),
                          "tensor_bound_phases": tensor_phases,
                          "note": "sum over the step's phases of max(bytes / measured HBM, flops / measured sustained bf16)"},
        "roofline": roofline, "kernels": kernels,
        "kernels_note": "device-side timeline of one eager step: per phase, from inputs ready to last CTA done",
        "clocks": clocks, "gpu_launches": int(launches),
        "e2e": {"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": ms_e2e / args.steps},
    }
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
