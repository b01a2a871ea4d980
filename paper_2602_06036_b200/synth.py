"""Seeded synthetic inputs for the DFlash draft-block / verify-accept path.

This module only *draws* inputs (weights, target features, paged-KV contents, page tables,
verify logits with planted accept prefixes) and lays them out. It holds none of the method's
arithmetic: no norm, projection, attention, RoPE rotation or accept rule lives here. Both the
CUDA path and the CPU oracle receive the tensors produced here, so the two are compared on
identical numbers.

Recipe (one named sub-stream per tensor, so adding a tensor never shifts the others):
  * projection / attention / FFN / LM-head weights  ~ N(0,1) * fan_in**-0.5
  * embedding rows ~ N(0,1); norm gains = 1 + 0.1*N(0,1)
  * target features ~ N(0,1)
  * everything is rounded (RNE) to the config dtype before either side sees it
  * mask_token_id = V-1; anchors uniform in [0, V-1)
  * physical KV pages are a random permutation of the pool (non-contiguous, unordered)
  * verify logits ~ N(0,1); an accepted-prefix length a ~ min(Geometric(p), gamma) is planted by
    setting the first a drafts to the row-wise first-occurrence maximum of the logits and the
    (a+1)-th draft to a different id.
"""
from __future__ import annotations

import dataclasses
import math
import zlib
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch


@dataclasses.dataclass(frozen=True)
class DFlashConfig:
    """Shape of a DFlash drafter (notation of the paper's App. A.3: D, k, W_c; B = block size)."""

    n_layers: int          # N draft transformer layers
    d_model: int           # D
    n_q_heads: int         # Hq
    n_kv_heads: int        # Hkv
    head_dim: int          # hd
    d_ffn: int             # F (SwiGLU)
    vocab: int             # V
    n_feat_layers: int     # k tapped target layers
    d_target: int          # D_t, hidden size of the target model
    block_size: int        # B
    dtype: str = "bf16"    # "fp32" | "bf16"
    page_size: int = 64
    use_rope: int = 1
    rms_eps: float = 1e-6
    rope_theta: float = 1.0e6
    qk_norm: int = 0       # 1: per-head RMSNorm of q and k (gains g_q, g_k of length hd) before the rotation

    @property
    def mask_token_id(self) -> int:
        return self.vocab - 1

    @property
    def softmax_scale(self) -> float:
        return 1.0 / math.sqrt(self.head_dim)

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    @property
    def feat_dim(self) -> int:
        return self.n_feat_layers * self.d_target

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "fp32" else torch.bfloat16


TINY = DFlashConfig(n_layers=1, d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=64, d_ffn=768,
                    vocab=1024, n_feat_layers=3, d_target=256, block_size=8, dtype="fp32")
QWEN3_8B = DFlashConfig(n_layers=5, d_model=4096, n_q_heads=32, n_kv_heads=8, head_dim=128,
                        d_ffn=12288, vocab=151936, n_feat_layers=3, d_target=4096, block_size=16,
                        dtype="bf16")
# A reduced bf16 shape for element-by-element parity: spans several 128-row weight tiles, a ragged
# vocabulary tail (5003 is prime) and the same head geometry as the full shape.
MID = DFlashConfig(n_layers=2, d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=128, d_ffn=1536,
                   vocab=5003, n_feat_layers=3, d_target=512, block_size=16, dtype="bf16")


@dataclasses.dataclass(frozen=True)
class Workload:
    """One of the five benchmark configurations: a model shape plus a batch of context lengths."""

    name: str
    cfg: DFlashConfig
    ctx_lens: tuple
    accept_p: float = 0.25
    seed: int = 0

    @property
    def batch(self) -> int:
        return len(self.ctx_lens)


def _uniform_lens(n: int, lo: int, hi: int, seed: int, name: str) -> tuple:
    g = substream(seed, name)
    return tuple(int(v) for v in torch.randint(lo, hi + 1, (n,), generator=g).tolist())


def workload(name: str) -> Workload:
    """cfg0..cfg4 as named by the benchmark definition (cfg0 tiny fp32 ... cfg4 serving mix)."""
    if name == "cfg0":
        return Workload("cfg0", TINY, (128,), accept_p=0.3)
    if name == "cfg1":
        return Workload("cfg1", QWEN3_8B, (2048,))
    if name == "cfg2":
        return Workload("cfg2", QWEN3_8B, _uniform_lens(8, 512, 4096, 0, "cfg2.ctx_lens"))
    if name == "cfg3":
        return Workload("cfg3", QWEN3_8B, (32768,))
    if name == "cfg4":
        return Workload("cfg4", QWEN3_8B, _uniform_lens(32, 1024, 8192, 0, "cfg4.ctx_lens"))
    if name == "mid":
        return Workload("mid", MID, (0, 70, 200))
    raise KeyError(name)


def substream(seed: int, name: str) -> torch.Generator:
    """Independent, reproducible CPU generator for (seed, tensor name)."""
    g = torch.Generator(device="cpu")
    g.manual_seed((int(seed) * 0x9E3779B1 + zlib.crc32(name.encode())) % (2 ** 63 - 1))
    return g


def normal(shape: Sequence[int], std: float, seed: int, name: str, dtype: torch.dtype,
           mean: float = 0.0) -> torch.Tensor:
    """N(mean, std^2) drawn in fp32 on the CPU, then rounded to `dtype`."""
    g = substream(seed, name)
    t = torch.empty(tuple(shape), dtype=torch.float32)
    t.normal_(0.0, 1.0, generator=g)
    if std != 1.0:
        t.mul_(std)
    if mean != 0.0:
        t.add_(mean)
    return t.to(dtype)


def make_weights(cfg: DFlashConfig, seed: int = 0) -> Dict:
    """Random-init weights in the paper's notation. All matrices are row-major [out, in]."""
    dt = cfg.torch_dtype
    D, F = cfg.d_model, cfg.d_ffn

    def lin(name, out_f, in_f):
        return normal((out_f, in_f), in_f ** -0.5, seed, name, dt)

    def gain(name):
        return normal((D,), 0.1, seed, name, dt, mean=1.0)

    w = {
        "embed": normal((cfg.vocab, D), 1.0, seed, "embed", dt),
        "W_c": lin("W_c", D, cfg.feat_dim),
        "g_c": gain("g_c"),
        "layers": [],
        "g_f": gain("g_f"),
        "W_lm": lin("W_lm", cfg.vocab, D),
    }
    for i in range(cfg.n_layers):
        p = f"layer{i}."
        w["layers"].append({
            "g1": gain(p + "g1"),
            "W_q": lin(p + "W_q", cfg.q_dim, D),
            "W_k": lin(p + "W_k", cfg.kv_dim, D),
            "W_v": lin(p + "W_v", cfg.kv_dim, D),
            "W_o": lin(p + "W_o", D, cfg.q_dim),
            "g2": gain(p + "g2"),
            "W_gate": lin(p + "W_gate", F, D),
            "W_up": lin(p + "W_up", F, D),
            "W_down": lin(p + "W_down", D, F),
        })
        if cfg.qk_norm:
            w["layers"][-1]["g_q"] = normal((cfg.head_dim,), 0.1, seed, p + "g_q", dt, mean=1.0)
            w["layers"][-1]["g_k"] = normal((cfg.head_dim,), 0.1, seed, p + "g_k", dt, mean=1.0)
    return w


def pack_device_weights(cfg: DFlashConfig, w: Dict) -> Dict:
    """Re-lay the weights the way the C-ABI wants them (pure concatenation / row interleave).

    W_qkv    = [W_q ; W_k ; W_v]            rows: q heads, then k heads, then v heads
    W_gateup = rows alternate gate_j, up_j  (row 2j = W_gate[j], row 2j+1 = W_up[j])
    """
    out = {k: w[k] for k in ("embed", "W_c", "g_c", "g_f", "W_lm")}
    out["layers"] = []
    for lw in w["layers"]:
        gu = torch.stack((lw["W_gate"], lw["W_up"]), dim=1).reshape(2 * cfg.d_ffn, cfg.d_model)
        out["layers"].append({
            "g1": lw["g1"],
            "W_qkv": torch.cat((lw["W_q"], lw["W_k"], lw["W_v"]), dim=0).contiguous(),
            "W_o": lw["W_o"],
            "g2": lw["g2"],
            "W_gateup": gu.contiguous(),
            "W_down": lw["W_down"],
        })
        if cfg.qk_norm:
            out["layers"][-1]["g_q"] = lw["g_q"]
            out["layers"][-1]["g_k"] = lw["g_k"]
    return out


def rope_tables(cfg: DFlashConfig, max_pos: int):
    """cos/sin tables [max_pos, hd/2] handed to the library as an input buffer.

    Angles are evaluated in float64 and rounded once to fp32. (The oracle does not read these
    tables; it evaluates its own angles.)
    """
    half = cfg.head_dim // 2
    inv = torch.pow(torch.tensor(cfg.rope_theta, dtype=torch.float64),
                    -torch.arange(half, dtype=torch.float64) * 2.0 / cfg.head_dim)
    ang = torch.arange(max_pos, dtype=torch.float64)[:, None] * inv[None, :]
    return torch.cos(ang).float().contiguous(), torch.sin(ang).float().contiguous()


def make_features(cfg: DFlashConfig, n_tokens: int, seed: int, name: str = "feats") -> torch.Tensor:
    """Concatenated hidden states of the k tapped target layers: [n_tokens, k*D_t], N(0,1)."""
    return normal((n_tokens, cfg.feat_dim), 1.0, seed, name, cfg.torch_dtype)


def make_anchors(cfg: DFlashConfig, batch: int, seed: int) -> torch.Tensor:
    g = substream(seed, "anchors")
    return torch.randint(0, cfg.vocab - 1, (batch,), generator=g, dtype=torch.int32)


def pages_needed(cfg: DFlashConfig, n_tokens: int) -> int:
    return (n_tokens + cfg.page_size - 1) // cfg.page_size


def make_page_table(cfg: DFlashConfig, capacities: Sequence[int], seed: int,
                    spare_pages: int = 3):
    """Random, non-contiguous page assignment.

    capacities[b] = number of token slots sequence b may ever use. Returns (page_table int32
    [S, max_pages] with -1 in unused entries, n_pool_pages).
    """
    need = [pages_needed(cfg, c) for c in capacities]
    total = sum(need) + spare_pages
    g = substream(seed, "page_perm")
    perm = torch.randperm(total, generator=g).to(torch.int32)
    max_pages = max(1, max(need))
    table = torch.full((len(capacities), max_pages), -1, dtype=torch.int32)
    o = 0
    for b, n in enumerate(need):
        table[b, :n] = perm[o:o + n]
        o += n
    return table, total


def kv_pool_shape(cfg: DFlashConfig, n_pages: int):
    """[layer][page][K|V][kv_head][slot][head_dim]."""
    return (cfg.n_layers, n_pages, 2, cfg.n_kv_heads, cfg.page_size, cfg.head_dim)


def make_kv_pool(cfg: DFlashConfig, n_pages: int, seed: int, name: str = "kv_pool") -> torch.Tensor:
    """A pool filled directly with N(0,1) entries (stand-in for projected context K/V when a test
    or benchmark wants a long context without running the context projection first)."""
    return normal(kv_pool_shape(cfg, n_pages), 1.0, seed, name, cfg.torch_dtype)


def make_verify_case(batch: int, gamma: int, vocab: int, p: float, seed: int,
                     dtype: torch.dtype = torch.float32, name: str = "verify"):
    """Target logits [S, gamma+1, V] ~ N(0,1) (rounded to dtype) and drafts [S, gamma] with a
    planted agreeing prefix of length a_b ~ min(Geometric(p), gamma), P(a = j) = (1-p)^j p.

    Returns (logits, drafts int32, planted_a int64[S]).
    """
    logits = normal((batch, gamma + 1, vocab), 1.0, seed, name + ".logits", dtype)
    g = substream(seed, name + ".plant")
    u = torch.rand((batch,), generator=g, dtype=torch.float64)
    a = torch.floor(torch.log1p(-u) / math.log1p(-p)).to(torch.int64).clamp_(0, gamma)
    drafts = torch.randint(0, vocab, (batch, gamma), generator=g, dtype=torch.int64)
    # first-occurrence row maximum of the values both sides will see
    top = torch.from_numpy(np.argmax(logits.float().numpy(), axis=-1))
    for b in range(batch):
        ab = int(a[b])
        drafts[b, :ab] = top[b, :ab]
        if ab < gamma:
            drafts[b, ab] = (top[b, ab] + 1) % vocab
    return logits, drafts.to(torch.int32), a


def to_numpy_f32(t: torch.Tensor) -> np.ndarray:
    """Exact widening of an fp32/bf16 tensor to a float32 numpy array."""
    return t.detach().cpu().float().numpy()


def weights_to_numpy(w: Dict) -> Dict:
    out = {}
    for k, v in w.items():
        if k == "layers":
            out[k] = [{kk: to_numpy_f32(vv) for kk, vv in lw.items()} for lw in v]
        else:
            out[k] = to_numpy_f32(v)
    return out
