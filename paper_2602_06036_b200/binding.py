"""ctypes binding of libdflash_b200.so: argument marshalling only.

Every step of the path runs in the library's CUDA kernels; this file turns torch tensors into the
plain pointers and sizes of `include/dflash.h`. There is no CPU fallback: if the library is missing
or fails to load, `load()` raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import torch

from .synth import DFlashConfig

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libdflash_b200.so")
_lib = None

F32, BF16 = 0, 1
ATTN_FULL, ATTN_CAUSAL = 0, 1
VERIFY_LOGITS, VERIFY_IDS = 0, 1
DEV_BAD_TOKEN, DEV_BAD_PAGE, DEV_CTX_OVERFLOW, DEV_TIMEOUT = 1, 2, 4, 8

EXPORTS = (
    "dflash_create", "dflash_destroy", "dflash_set_weights", "dflash_workspace_bytes",
    "dflash_ctx_project", "dflash_draft_block", "dflash_verify_accept", "dflash_block_attention",
    "dflash_lmhead_argmax", "dflash_status_string", "dflash_launch_count", "dflash_profile_enable",
    "dflash_profile_read", "dflash_family_name", "dflash_trace_enable", "dflash_trace_read",
    "dflash_verify_accept_static", "dflash_sample_rows", "dflash_verify_accept_sample",
    "dflash_sample_workspace_bytes", "dflash_target_verify", "dflash_block_loss", "dflash_attention_plan",
    "dflash_block_attention_bwd", "dflash_gemm_plan_check",
)
N_FAMILIES = 15


class Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab", "n_feat_layers",
        "d_target", "block_size", "page_size", "dtype", "mask_token_id", "use_rope")] + [
        ("rms_eps", C.c_float), ("softmax_scale", C.c_float), ("qk_norm", C.c_int32)]


class LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("g1", "W_qkv", "W_o", "g2", "W_gateup", "W_down", "g_q", "g_k")]


class Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("W_c", C.c_void_p), ("g_c", C.c_void_p),
                ("layers", C.POINTER(LayerWeights)), ("g_f", C.c_void_p), ("W_lm", C.c_void_p),
                ("rope_cos", C.c_void_p), ("rope_sin", C.c_void_p), ("rope_max_pos", C.c_int32)]


class CtxArgs(C.Structure):
    _fields_ = [("feats", C.c_void_p), ("batch", C.c_int32), ("max_new", C.c_int32), ("n_new", C.c_void_p),
                ("ctx_len", C.c_void_p), ("page_table", C.c_void_p), ("max_pages", C.c_int32),
                ("kv_pool", C.c_void_p), ("n_pool_pages", C.c_int32), ("workspace", C.c_void_p),
                ("workspace_bytes", C.c_int64), ("dev_status", C.c_void_p)]


class DraftArgs(C.Structure):
    _fields_ = [("anchor_ids", C.c_void_p), ("batch", C.c_int32), ("ctx_len", C.c_void_p),
                ("max_ctx_len", C.c_int32), ("page_table", C.c_void_p), ("max_pages", C.c_int32),
                ("kv_pool", C.c_void_p), ("n_pool_pages", C.c_int32), ("workspace", C.c_void_p),
                ("workspace_bytes", C.c_int64), ("draft_ids", C.c_void_p), ("top1", C.c_void_p),
                ("margin", C.c_void_p), ("hidden_out", C.c_void_p), ("logits_out", C.c_void_p),
                ("dev_status", C.c_void_p), ("block_rows", C.c_int32), ("ctx", C.POINTER(CtxArgs))]


class VerifyArgs(C.Structure):
    _fields_ = [("mode", C.c_int32), ("logits", C.c_void_p), ("logits_dtype", C.c_int32),
                ("logits_row_stride", C.c_int64), ("target_ids", C.c_void_p), ("draft_ids", C.c_void_p),
                ("draft_stride", C.c_int32), ("batch", C.c_int32), ("gamma", C.c_int32), ("vocab", C.c_int32),
                ("ctx_len", C.c_void_p), ("accept_len", C.c_void_p), ("out_tokens", C.c_void_p),
                ("bonus", C.c_void_p), ("new_ctx_len", C.c_void_p), ("target_ids_out", C.c_void_p),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_int64), ("dev_status", C.c_void_p)]


class TargetArgs(C.Structure):
    _fields_ = [("token_ids", C.c_void_p), ("batch", C.c_int32), ("rows", C.c_int32), ("ctx_len", C.c_void_p),
                ("max_ctx_len", C.c_int32), ("page_table", C.c_void_p), ("max_pages", C.c_int32),
                ("kv_pool", C.c_void_p), ("n_pool_pages", C.c_int32), ("tap_layers", C.POINTER(C.c_int32)),
                ("n_taps", C.c_int32), ("feats_out", C.c_void_p), ("logits_out", C.c_void_p),
                ("ids_out", C.c_void_p), ("workspace", C.c_void_p), ("workspace_bytes", C.c_int64),
                ("dev_status", C.c_void_p)]


class BlockLossArgs(C.Structure):
    _fields_ = [("logits", C.c_void_p), ("logits_dtype", C.c_int32), ("row_stride", C.c_int64),
                ("n_blocks", C.c_int32), ("block_rows", C.c_int32), ("vocab", C.c_int32), ("targets", C.c_void_p),
                ("gamma", C.c_float), ("row_loss", C.c_void_p), ("loss_sum", C.c_void_p), ("dlogits", C.c_void_p),
                ("dlogits_dtype", C.c_int32), ("dlogits_row_stride", C.c_int64), ("grad_scale", C.c_float),
                ("dev_status", C.c_void_p)]


class SampleArgs(C.Structure):
    _fields_ = [("logits", C.c_void_p), ("logits_dtype", C.c_int32), ("row_stride", C.c_int64),
                ("n_rows", C.c_int32), ("vocab", C.c_int32), ("temperature", C.c_float), ("u", C.c_void_p),
                ("ids", C.c_void_p), ("prob", C.c_void_p), ("workspace", C.c_void_p),
                ("workspace_bytes", C.c_int64), ("dev_status", C.c_void_p)]


class VerifySampleArgs(C.Structure):
    _fields_ = [("target_logits", C.c_void_p), ("target_dtype", C.c_int32), ("target_row_stride", C.c_int64),
                ("draft_logits", C.c_void_p), ("draft_dtype", C.c_int32), ("draft_row_stride", C.c_int64),
                ("draft_rows_per_seq", C.c_int32), ("draft_ids", C.c_void_p), ("draft_stride", C.c_int32),
                ("batch", C.c_int32), ("gamma", C.c_int32), ("vocab", C.c_int32), ("temperature", C.c_float),
                ("u_accept", C.c_void_p), ("u_final", C.c_void_p), ("ctx_len", C.c_void_p),
                ("accept_len", C.c_void_p), ("out_tokens", C.c_void_p), ("bonus", C.c_void_p),
                ("new_ctx_len", C.c_void_p), ("workspace", C.c_void_p), ("workspace_bytes", C.c_int64),
                ("dev_status", C.c_void_p)]


class AttnArgs(C.Structure):
    _fields_ = [("mode", C.c_int32), ("q", C.c_void_p), ("k_blk", C.c_void_p), ("v_blk", C.c_void_p),
                ("batch", C.c_int32), ("rows", C.c_int32), ("ctx_len", C.c_void_p), ("max_ctx_len", C.c_int32),
                ("page_table", C.c_void_p), ("max_pages", C.c_int32), ("kv_pool", C.c_void_p),
                ("n_pool_pages", C.c_int32), ("layer", C.c_int32), ("out", C.c_void_p),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_int64), ("dev_status", C.c_void_p),
                ("lse_out", C.c_void_p)]


class AttnBwdArgs(C.Structure):
    _fields_ = [("mode", C.c_int32), ("q", C.c_void_p), ("k_blk", C.c_void_p), ("v_blk", C.c_void_p), ("out", C.c_void_p),
                ("lse", C.c_void_p), ("dout", C.c_void_p), ("batch", C.c_int32), ("rows", C.c_int32), ("ctx_len", C.c_void_p),
                ("max_ctx_len", C.c_int32), ("page_table", C.c_void_p), ("max_pages", C.c_int32), ("kv_pool", C.c_void_p),
                ("n_pool_pages", C.c_int32), ("layer", C.c_int32), ("shared_page_row", C.c_int32), ("dq", C.c_void_p),
                ("dk_blk", C.c_void_p), ("dv_blk", C.c_void_p), ("dkv_ctx", C.c_void_p), ("workspace", C.c_void_p),
                ("workspace_bytes", C.c_int64), ("dev_status", C.c_void_p)]


class LmHeadArgs(C.Structure):
    _fields_ = [("hidden", C.c_void_p), ("hidden_is_f32", C.c_int32), ("n_rows", C.c_int32),
                ("apply_norm", C.c_int32), ("ids", C.c_void_p), ("top1", C.c_void_p), ("margin", C.c_void_p),
                ("logits_out", C.c_void_p), ("workspace", C.c_void_p), ("workspace_bytes", C.c_int64),
                ("dev_status", C.c_void_p)]


def load():
    """Load the shared library (once). Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} not found: build it with `python -m paper_2602_06036_b200.build`")
    lib = C.CDLL(_LIB_PATH)
    lib.dflash_create.argtypes = [C.POINTER(Config), C.POINTER(C.c_void_p)]
    lib.dflash_create.restype = C.c_int32
    lib.dflash_destroy.argtypes = [C.c_void_p]
    lib.dflash_destroy.restype = None
    lib.dflash_set_weights.argtypes = [C.c_void_p, C.POINTER(Weights)]
    lib.dflash_set_weights.restype = C.c_int32
    lib.dflash_workspace_bytes.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
    lib.dflash_workspace_bytes.restype = C.c_int64
    for name, st in (("dflash_ctx_project", CtxArgs), ("dflash_draft_block", DraftArgs),
                     ("dflash_verify_accept", VerifyArgs), ("dflash_verify_accept_static", VerifyArgs), ("dflash_block_attention", AttnArgs),
                     ("dflash_lmhead_argmax", LmHeadArgs), ("dflash_sample_rows", SampleArgs),
                     ("dflash_verify_accept_sample", VerifySampleArgs), ("dflash_target_verify", TargetArgs),
                     ("dflash_block_loss", BlockLossArgs), ("dflash_block_attention_bwd", AttnBwdArgs)):
        fn = getattr(lib, name)
        fn.argtypes = [C.c_void_p, C.POINTER(st), C.c_void_p]
        fn.restype = C.c_int32
    lib.dflash_sample_workspace_bytes.argtypes = [C.c_int32, C.c_int32]
    lib.dflash_sample_workspace_bytes.restype = C.c_int64
    lib.dflash_attention_plan.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.POINTER(C.c_int64)]
    lib.dflash_attention_plan.restype = C.c_int32
    lib.dflash_gemm_plan_check.argtypes = [C.c_int32] * 7 + [C.POINTER(C.c_int32)]
    lib.dflash_gemm_plan_check.restype = C.c_int32
    lib.dflash_status_string.argtypes = [C.c_int32]
    lib.dflash_status_string.restype = C.c_char_p
    lib.dflash_launch_count.argtypes = []
    lib.dflash_launch_count.restype = C.c_int64
    lib.dflash_profile_enable.argtypes = [C.c_void_p, C.c_int32]
    lib.dflash_profile_enable.restype = C.c_int32
    lib.dflash_profile_read.argtypes = [C.c_void_p, C.POINTER(C.c_float), C.POINTER(C.c_int32)]
    lib.dflash_profile_read.restype = C.c_int32
    lib.dflash_trace_enable.argtypes = [C.c_void_p, C.c_void_p, C.c_int32]
    lib.dflash_trace_enable.restype = C.c_int32
    lib.dflash_trace_read.argtypes = [C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    lib.dflash_trace_read.restype = C.c_int32
    lib.dflash_family_name.argtypes = [C.c_int32]
    lib.dflash_family_name.restype = C.c_char_p
    _lib = lib
    return lib


class DFlashError(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        super().__init__(f"dflash error {code}: {load().dflash_status_string(code).decode()}")


def _check(rc: int):
    if rc != 0:
        raise DFlashError(rc)


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device-contiguous tensor expected"
    return C.c_void_p(t.data_ptr())


def _stream(stream) -> C.c_void_p:
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def launch_count() -> int:
    return int(load().dflash_launch_count())


class DFlash:
    """Owns a library handle plus the torch tensors whose pointers it lent to the library."""

    def __init__(self, cfg: DFlashConfig, device: str = "cuda:0"):
        self.lib = load()
        self.cfg = cfg
        self.device = torch.device(device)
        self.ccfg = Config(cfg.n_layers, cfg.d_model, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.d_ffn,
                           cfg.vocab, cfg.n_feat_layers, cfg.d_target, cfg.block_size, cfg.page_size,
                           F32 if cfg.dtype == "fp32" else BF16, cfg.mask_token_id, cfg.use_rope,
                           cfg.rms_eps, cfg.softmax_scale, int(getattr(cfg, "qk_norm", 0)))
        hp = C.c_void_p()
        _check(self.lib.dflash_create(C.byref(self.ccfg), C.byref(hp)))
        self.h = hp
        self._keep = {}
        self._ws = None
        self.status = torch.zeros(1, dtype=torch.int32, device=self.device)

    def close(self):
        if getattr(self, "h", None):
            self.lib.dflash_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- set-up -------------------------------------------------------------------------
    def set_weights(self, packed: Dict, rope_cos: torch.Tensor, rope_sin: torch.Tensor):
        """`packed` = synth.pack_device_weights(...) moved to the device (any mapping with the same keys)."""
        dev = self.device
        keep = {k: packed[k].to(dev).contiguous() for k in ("embed", "W_c", "g_c", "g_f", "W_lm")}
        keep["layers"] = [{k: v.to(dev).contiguous() for k, v in lw.items()} for lw in packed["layers"]]
        keep["rope_cos"] = rope_cos.to(dev, torch.float32).contiguous()
        keep["rope_sin"] = rope_sin.to(dev, torch.float32).contiguous()
        arr = (LayerWeights * self.cfg.n_layers)()
        for i, lw in enumerate(keep["layers"]):
            arr[i] = LayerWeights(*(lw[k].data_ptr() for k in ("g1", "W_qkv", "W_o", "g2", "W_gateup", "W_down")),
                                  *((lw[k].data_ptr() if k in lw else None) for k in ("g_q", "g_k")))
        w = Weights(keep["embed"].data_ptr(), keep["W_c"].data_ptr(), keep["g_c"].data_ptr(), arr,
                    keep["g_f"].data_ptr(), keep["W_lm"].data_ptr(), keep["rope_cos"].data_ptr(),
                    keep["rope_sin"].data_ptr(), keep["rope_cos"].shape[0])
        _check(self.lib.dflash_set_weights(self.h, C.byref(w)))
        self._keep = keep

    def workspace_bytes(self, max_batch: int, max_rows: int) -> int:
        n = self.lib.dflash_workspace_bytes(self.h, max_batch, max_rows)
        if n < 0:
            raise DFlashError(int(n))
        return int(n)

    def workspace(self, max_batch: int, max_rows: int) -> torch.Tensor:
        need = self.workspace_bytes(max_batch, max_rows)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=self.device)
        return self._ws

    def profile(self, fn, steps: int):
        """Run `fn` `steps` times with an event pair around every launch of this handle.
        Returns {family: (microseconds per launch, launches per step)}."""
        _check(self.lib.dflash_profile_enable(self.h, 1))
        ms = (C.c_float * N_FAMILIES)()
        n = (C.c_int32 * N_FAMILIES)()
        try:
            for _ in range(steps):
                fn()
                _check(self.lib.dflash_profile_read(self.h, ms, n))
        finally:
            self.lib.dflash_profile_enable(self.h, 0)
        out = {}
        for f in range(N_FAMILIES):
            if n[f]:
                out[self.lib.dflash_family_name(f).decode()] = (1e3 * ms[f] / n[f], n[f] / steps)
        return out

    def trace(self, fn, capacity: int = 256):
        """Run `fn` once with the device-side timeline on. Returns a list of
        (family, start_ns, dependency_resolved_ns, main_loop_end_ns, end_ns) relative to the first start."""
        buf = torch.zeros(capacity * 4, dtype=torch.int64, device=self.device)
        _check(self.lib.dflash_trace_enable(self.h, C.c_void_p(buf.data_ptr()), capacity))
        try:
            fn()
            torch.cuda.synchronize()
            fam = (C.c_int32 * capacity)()
            n = C.c_int32()
            _check(self.lib.dflash_trace_read(self.h, fam, C.byref(n)))
        finally:
            self.lib.dflash_trace_enable(self.h, None, 0)
        rec = buf.cpu().view(capacity, 4).tolist()
        inv = lambda v: (~v) & 0xFFFFFFFFFFFFFFFF if v else 0
        fix = lambda v: v & 0xFFFFFFFFFFFFFFFF
        rows = []
        for i in range(n.value):
            r = rec[i]
            if r[3] == 0 and r[0] == 0:
                continue
            rows.append((self.lib.dflash_family_name(fam[i]).decode(), inv(fix(r[0])), inv(fix(r[1])), fix(r[2]), fix(r[3])))
        if not rows:
            return rows
        t0 = min(r[1] for r in rows if r[1])
        return [(f, a - t0 if a else None, b - t0 if b else None, c - t0 if c else None, d - t0 if d else None)
                for f, a, b, c, d in rows]

    # ---- the path -----------------------------------------------------------------------
    def dflash_ctx_project(self, feats, n_new, ctx_len, page_table, kv_pool, stream=None):
        """feats [S, max_new, k*D_t]; n_new (or None) and ctx_len int32 [S]; writes kv_pool in place."""
        S, max_new = feats.shape[0], feats.shape[1]
        ws = self.workspace(S, S * max_new)
        a = CtxArgs(_ptr(feats), S, max_new, _ptr(n_new), _ptr(ctx_len), _ptr(page_table), page_table.shape[1],
                    _ptr(kv_pool), kv_pool.shape[1], _ptr(ws), ws.numel(), _ptr(self.status))
        _check(self.lib.dflash_ctx_project(self.h, C.byref(a), _stream(stream)))

    def dflash_draft_block(self, anchor_ids, ctx_len, max_ctx_len, page_table, kv_pool, draft_ids,
                           top1=None, margin=None, hidden_out=None, logits_out=None, stream=None, block_rows=0, ctx=None):
        """block_rows: rows per sequence in this call (0 = the handle's block size).
        ctx = (feats [S, max_new, k*D_t], n_new or None, ctx_len_before): run that context projection inside
        this call, chained with the first layer's QKV contraction."""
        S = anchor_ids.shape[0]
        rows = S * self.cfg.block_size
        cptr = None
        if ctx is not None:
            feats, n_new, len_before = ctx
            rows = max(rows, S * feats.shape[1])
            self._ctx_keep = CtxArgs(_ptr(feats), S, feats.shape[1], _ptr(n_new), _ptr(len_before), _ptr(page_table),
                                     page_table.shape[1], _ptr(kv_pool), kv_pool.shape[1], None, 0, _ptr(self.status))
            cptr = C.pointer(self._ctx_keep)
        ws = self.workspace(S, rows)
        a = DraftArgs(_ptr(anchor_ids), S, _ptr(ctx_len), int(max_ctx_len), _ptr(page_table), page_table.shape[1],
                      _ptr(kv_pool), kv_pool.shape[1], _ptr(ws), ws.numel(), _ptr(draft_ids), _ptr(top1),
                      _ptr(margin), _ptr(hidden_out), _ptr(logits_out), _ptr(self.status), int(block_rows), cptr)
        _check(self.lib.dflash_draft_block(self.h, C.byref(a), _stream(stream)))

    def dflash_verify_accept(self, draft_ids, draft_stride, gamma, ctx_len, accept_len, out_tokens, bonus,
                             new_ctx_len, logits=None, target_ids=None, target_ids_out=None,
                             draft_offset=0, stream=None):
        """Mode LOGITS when `logits` [S, gamma+1, V] is given, else mode IDS with target_ids [S, gamma+1]."""
        S = ctx_len.shape[0]
        ws = self.workspace(S, S * (gamma + 1))
        dptr = C.c_void_p(draft_ids.data_ptr() + 4 * draft_offset)
        if logits is not None:
            mode, vocab = VERIFY_LOGITS, logits.shape[-1]
            ldt = F32 if logits.dtype == torch.float32 else BF16
        else:
            mode, vocab, ldt = VERIFY_IDS, self.cfg.vocab, F32
        a = VerifyArgs(mode, _ptr(logits), ldt, 0, _ptr(target_ids), dptr, draft_stride, S, gamma, vocab,
                       _ptr(ctx_len), _ptr(accept_len), _ptr(out_tokens), _ptr(bonus), _ptr(new_ctx_len),
                       _ptr(target_ids_out), _ptr(ws), ws.numel(), _ptr(self.status))
        _check(self.lib.dflash_verify_accept(self.h, C.byref(a), _stream(stream)))

    def dflash_verify_accept_static(self, draft_ids, draft_stride, gamma, ctx_len, accept_len, out_tokens, bonus,
                                    new_ctx_len, logits, target_ids_out=None, stream=None):
        """Logits-mode verify/accept on the library's built-in scratch: no workspace is passed, nothing is
        allocated. For callers that cannot allocate device memory; at most DFLASH_STATIC_MAX_ROWS rows, and
        calls must not overlap on the GPU (they share the scratch)."""
        S = ctx_len.shape[0]
        ldt = F32 if logits.dtype == torch.float32 else BF16
        a = VerifyArgs(VERIFY_LOGITS, _ptr(logits), ldt, 0, None, _ptr(draft_ids), draft_stride, S, gamma,
                       logits.shape[-1], _ptr(ctx_len), _ptr(accept_len), _ptr(out_tokens), _ptr(bonus),
                       _ptr(new_ctx_len), _ptr(target_ids_out), None, 0, _ptr(self.status))
        _check(self.lib.dflash_verify_accept_static(self.h, C.byref(a), _stream(stream)))

    def dflash_target_verify(self, token_ids, ctx_len, max_ctx_len, page_table, kv_pool, tap_layers, ids_out,
                             feats_out=None, logits_out=None, stream=None):
        """The target's verify pass: token_ids [S, rows]; writes the block's K/V into kv_pool at positions
        ctx_len .. ctx_len + rows - 1, the tapped hidden rows into feats_out [S, rows, len(tap_layers) * D]."""
        S, rows = token_ids.shape
        ws = self.workspace(S, S * rows)
        taps = (C.c_int32 * max(len(tap_layers), 1))(*tap_layers)
        a = TargetArgs(_ptr(token_ids), S, rows, _ptr(ctx_len), int(max_ctx_len), _ptr(page_table), page_table.shape[1],
                       _ptr(kv_pool), kv_pool.shape[1], taps, len(tap_layers), _ptr(feats_out), _ptr(logits_out),
                       _ptr(ids_out), _ptr(ws), ws.numel(), _ptr(self.status))
        _check(self.lib.dflash_target_verify(self.h, C.byref(a), _stream(stream)))

    def _sample_ws(self, n_rows, vocab):
        need = int(self.lib.dflash_sample_workspace_bytes(n_rows, vocab))
        if need < 0:
            raise DFlashError(-1)
        ws = getattr(self, "_samp_ws", None)
        if ws is None or ws.numel() < need:
            ws = torch.empty(max(need, 256), dtype=torch.uint8, device=self.device)
            self._samp_ws = ws
        return ws

    def dflash_block_loss(self, logits, targets, gamma, row_loss, loss_sum=None, dlogits=None, grad_scale=1.0, stream=None):
        """Position-weighted cross entropy of draft blocks. logits [n_blocks, B, V] (row 0 of a block = anchor, no
        loss), targets [n_blocks, B] int32 (< 0: ignored). row_loss [n_blocks * B] fp32; loss_sum [2] fp32;
        dlogits like logits (fp32 or bf16) = grad_scale * w_k * (softmax - onehot)."""
        nb, B, V = logits.shape
        a = BlockLossArgs(_ptr(logits), F32 if logits.dtype == torch.float32 else BF16, logits.stride(1), nb, B, V,
                          _ptr(targets), float(gamma), _ptr(row_loss), _ptr(loss_sum), _ptr(dlogits),
                          (F32 if dlogits.dtype == torch.float32 else BF16) if dlogits is not None else F32,
                          dlogits.stride(1) if dlogits is not None else 0, float(grad_scale), _ptr(self.status))
        _check(self.lib.dflash_block_loss(self.h, C.byref(a), _stream(stream)))

    def dflash_sample_rows(self, logits, temperature, u, ids, prob=None, stream=None):
        """ids[m] = inverse-CDF draw from softmax(logits[m] / T) with the uniform u[m]."""
        n, V = logits.shape[0], logits.shape[-1]
        ws = self._sample_ws(n, V)
        a = SampleArgs(_ptr(logits), F32 if logits.dtype == torch.float32 else BF16, logits.stride(0), n, V,
                       float(temperature), _ptr(u), _ptr(ids), _ptr(prob), _ptr(ws), ws.numel(), _ptr(self.status))
        _check(self.lib.dflash_sample_rows(self.h, C.byref(a), _stream(stream)))

    def dflash_verify_accept_sample(self, target_logits, draft_logits, draft_rows_per_seq, draft_ids, draft_stride,
                                    gamma, temperature, u_accept, u_final, ctx_len, accept_len, out_tokens, bonus,
                                    new_ctx_len, draft_row_offset=0, draft_offset=0, stream=None):
        """Speculative-sampling verification. target_logits [S, gamma+1, V]; draft_logits: 2-D [rows, V] with
        draft j of sequence b at row draft_row_offset + b * draft_rows_per_seq + j."""
        S, V = ctx_len.shape[0], target_logits.shape[-1]
        ws = self._sample_ws(S * (2 * gamma + 1), V)
        dl = draft_logits.reshape(-1, V) if draft_logits is not None else None
        dl_ptr = C.c_void_p(dl.data_ptr() + draft_row_offset * dl.stride(0) * dl.element_size()) if dl is not None else None
        a = VerifySampleArgs(_ptr(target_logits), F32 if target_logits.dtype == torch.float32 else BF16, 0, dl_ptr,
                             (F32 if dl.dtype == torch.float32 else BF16) if dl is not None else F32,
                             dl.stride(0) if dl is not None else 0, draft_rows_per_seq,
                             C.c_void_p(draft_ids.data_ptr() + 4 * draft_offset) if draft_ids is not None else None,
                             draft_stride, S, gamma, V, float(temperature), _ptr(u_accept), _ptr(u_final),
                             _ptr(ctx_len), _ptr(accept_len), _ptr(out_tokens), _ptr(bonus), _ptr(new_ctx_len),
                             _ptr(ws), ws.numel(), _ptr(self.status))
        _check(self.lib.dflash_verify_accept_sample(self.h, C.byref(a), _stream(stream)))

    def dflash_block_attention(self, mode, q, k_blk, v_blk, ctx_len, max_ctx_len, page_table, kv_pool, layer,
                               out, stream=None, lse_out=None):
        S, R = q.shape[0], q.shape[1]
        ws = self.workspace(S, S * R)
        a = AttnArgs(mode, _ptr(q), _ptr(k_blk), _ptr(v_blk), S, R, _ptr(ctx_len), int(max_ctx_len),
                     _ptr(page_table), page_table.shape[1], _ptr(kv_pool), kv_pool.shape[1], layer, _ptr(out),
                     _ptr(ws), ws.numel(), _ptr(self.status), _ptr(lse_out))
        _check(self.lib.dflash_block_attention(self.h, C.byref(a), _stream(stream)))

    def dflash_block_attention_bwd(self, mode, q, k_blk, v_blk, out, lse, dout, ctx_len, max_ctx_len, page_table, kv_pool, layer,
                                   dq, dk_blk, dv_blk, dkv_ctx=None, shared_page_row=False, stream=None):
        """Gradients of dflash_block_attention: dq / dk_blk / dv_blk like q / k_blk / v_blk; dkv_ctx fp32
        [n_pool_pages, 2, Hkv, page_size, hd] (one layer, the pool's layout) or None."""
        S, R = q.shape[0], q.shape[1]
        ws = self.workspace(S, S * R)
        a = AttnBwdArgs(mode, _ptr(q), _ptr(k_blk), _ptr(v_blk), _ptr(out), _ptr(lse), _ptr(dout), S, R, _ptr(ctx_len),
                        int(max_ctx_len), _ptr(page_table), page_table.shape[1], _ptr(kv_pool), kv_pool.shape[1], layer,
                        1 if shared_page_row else 0, _ptr(dq), _ptr(dk_blk), _ptr(dv_blk), _ptr(dkv_ctx), _ptr(ws), ws.numel(),
                        _ptr(self.status))
        _check(self.lib.dflash_block_attention_bwd(self.h, C.byref(a), _stream(stream)))

    def dflash_lmhead_argmax(self, hidden, apply_norm, ids, top1=None, margin=None, logits_out=None, stream=None):
        M = hidden.shape[0]
        ws = self.workspace(1, M)
        a = LmHeadArgs(_ptr(hidden), 1 if hidden.dtype == torch.float32 else 0, M, 1 if apply_norm else 0,
                       _ptr(ids), _ptr(top1), _ptr(margin), _ptr(logits_out), _ptr(ws), ws.numel(),
                       _ptr(self.status))
        _check(self.lib.dflash_lmhead_argmax(self.h, C.byref(a), _stream(stream)))
