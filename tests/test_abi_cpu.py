"""Host-side checks that need no GPU: the library builds, loads, exports every symbol the header
declares, its structs have the layout the binding assumes, and host-detectable errors come back as
return codes."""
import ctypes as C
import os
import re
import subprocess
import tempfile

import pytest

from paper_2602_06036_b200 import binding, build, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "dflash.h")


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def _declared():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dflash_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert set(binding.EXPORTS) <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_struct_layouts_match_the_header():
    structs = {"dflash_config": binding.Config, "dflash_layer_weights": binding.LayerWeights,
               "dflash_weights": binding.Weights, "dflash_ctx_args": binding.CtxArgs,
               "dflash_draft_args": binding.DraftArgs, "dflash_verify_args": binding.VerifyArgs,
               "dflash_attn_args": binding.AttnArgs, "dflash_lmhead_args": binding.LmHeadArgs,
               "dflash_sample_args": binding.SampleArgs, "dflash_verify_sample_args": binding.VerifySampleArgs,
               "dflash_target_args": binding.TargetArgs, "dflash_block_loss_args": binding.BlockLossArgs,
               "dflash_attn_bwd_args": binding.AttnBwdArgs}
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "dflash.h"', "int main(void){"]
    for cname, st in structs.items():
        lines.append(f'printf("{cname} %zu\\n", sizeof({cname}));')
        for f, _ in st._fields_:
            lines.append(f'printf("{cname}.{f} %zu\\n", offsetof({cname}, {f}));')
    lines.append("return 0;}")
    with tempfile.TemporaryDirectory() as d:
        src = os.path.join(d, "t.c")
        open(src, "w").write("\n".join(lines))
        exe = os.path.join(d, "t")
        subprocess.check_call(["gcc", "-std=c99", "-I", os.path.join(ROOT, "include"), src, "-o", exe])
        out = subprocess.check_output([exe], text=True)
    got = dict(line.split() for line in out.strip().splitlines())
    for cname, st in structs.items():
        assert int(got[cname]) == C.sizeof(st), cname
        for f, _ in st._fields_:
            assert int(got[f"{cname}.{f}"]) == getattr(st, f).offset, (cname, f)


def _cfg(**over):
    c = synth.TINY
    vals = dict(n_layers=c.n_layers, d_model=c.d_model, n_q_heads=c.n_q_heads, n_kv_heads=c.n_kv_heads,
                head_dim=c.head_dim, d_ffn=c.d_ffn, vocab=c.vocab, n_feat_layers=c.n_feat_layers,
                d_target=c.d_target, block_size=c.block_size, page_size=64, dtype=0, mask_token_id=c.vocab - 1,
                use_rope=1, rms_eps=1e-6, softmax_scale=0.125, qk_norm=0)
    vals.update(over)
    return binding.Config(**vals)


def test_create_validates_on_the_host(lib):
    h = C.c_void_p()
    assert lib.dflash_create(C.byref(_cfg()), C.byref(h)) == 0 and h.value
    # workspace grows with rows; invalid arguments are refused
    a = lib.dflash_workspace_bytes(h, 1, 8)
    b = lib.dflash_workspace_bytes(h, 4, 64)
    assert 0 < a < b and a % 256 == 0
    assert lib.dflash_workspace_bytes(h, -1, 8) < 0
    # calls before set_weights are refused without touching CUDA
    args = binding.DraftArgs()
    args.batch = 1
    assert lib.dflash_draft_block(h, C.byref(args), None) == -5
    assert lib.dflash_draft_block(None, C.byref(args), None) == -1
    lib.dflash_destroy(h)
    for bad in (dict(head_dim=48), dict(n_q_heads=3), dict(block_size=33), dict(dtype=2), dict(page_size=48),
                dict(n_layers=0), dict(mask_token_id=5000), dict(softmax_scale=0.0)):
        h2 = C.c_void_p()
        assert lib.dflash_create(C.byref(_cfg(**bad)), C.byref(h2)) < 0 and not h2.value, bad
    assert lib.dflash_create(None, C.byref(h)) == -1


def test_verify_args_validated_on_the_host(lib):
    h = C.c_void_p()
    assert lib.dflash_create(C.byref(_cfg()), C.byref(h)) == 0
    a = binding.VerifyArgs()
    a.batch, a.gamma, a.draft_stride = 1, 0, 8
    assert lib.dflash_verify_accept(h, C.byref(a), None) == -1      # gamma < 1
    a.gamma, a.draft_stride = 8, 4
    assert lib.dflash_verify_accept(h, C.byref(a), None) == -1      # stride < gamma
    a.draft_stride = 8
    assert lib.dflash_verify_accept(h, C.byref(a), None) == -1      # null pointers
    a.batch = 0
    assert lib.dflash_verify_accept(h, C.byref(a), None) == 0       # empty batch: nothing to do
    lib.dflash_destroy(h)


def test_sampling_and_loss_args_validated_on_the_host(lib):
    # every refusal below happens before the first CUDA call
    h = C.c_void_p()
    assert lib.dflash_create(C.byref(_cfg()), C.byref(h)) == 0
    s = binding.SampleArgs()
    s.n_rows, s.vocab, s.temperature = 4, 1000, 0.0
    assert lib.dflash_sample_rows(h, C.byref(s), None) == -1           # T must be > 0
    s.temperature, s.n_rows = 1.0, 0
    assert lib.dflash_sample_rows(h, C.byref(s), None) == 0            # nothing to do
    s.n_rows = 70000
    assert lib.dflash_sample_rows(h, C.byref(s), None) == -2           # more rows than one launch takes
    assert lib.dflash_sample_workspace_bytes(16, 151936) % 256 == 0 and lib.dflash_sample_workspace_bytes(-1, 10) < 0
    v = binding.VerifySampleArgs()
    v.batch, v.gamma, v.vocab, v.temperature = 1, 65, 1000, 1.0
    v.draft_rows_per_seq = v.draft_stride = 65
    for name in ("target_logits", "draft_logits", "draft_ids", "u_accept", "u_final", "ctx_len", "accept_len", "out_tokens",
                 "bonus", "new_ctx_len"):
        setattr(v, name, 256)                                          # non-null; never dereferenced on the host
    assert lib.dflash_verify_accept_sample(h, C.byref(v), None) == -2  # gamma above 64
    v.batch = 0
    assert lib.dflash_verify_accept_sample(h, C.byref(v), None) == 0
    b = binding.BlockLossArgs()
    b.n_blocks, b.block_rows, b.vocab, b.gamma = 2, 16, 1000, 0.0
    assert lib.dflash_block_loss(h, C.byref(b), None) == -1            # gamma must be > 0
    b.gamma, b.logits_dtype = 7.0, 5
    assert lib.dflash_block_loss(h, C.byref(b), None) == -1            # unknown dtype
    b.logits_dtype = 0
    assert lib.dflash_block_loss(h, C.byref(b), None) == -1            # null pointers
    b.n_blocks = 0
    assert lib.dflash_block_loss(h, C.byref(b), None) == 0             # nothing to do
    lib.dflash_destroy(h)


def _qwen_cfg():
    c = synth.QWEN3_8B
    return _cfg(n_layers=c.n_layers, d_model=c.d_model, n_q_heads=c.n_q_heads, n_kv_heads=c.n_kv_heads, head_dim=c.head_dim,
                d_ffn=c.d_ffn, vocab=c.vocab, n_feat_layers=c.n_feat_layers, d_target=c.d_target, block_size=c.block_size,
                dtype=1, mask_token_id=c.vocab - 1, softmax_scale=c.softmax_scale)


def test_attention_split_never_outgrows_its_partials_buffer(lib):
    # host arithmetic only: for every (batch, kv heads, context bound) the partial slots the kernels index
    # stay inside what the workspace provides, and every range covers the whole context
    for hkv, hq in ((8, 32), (1, 8), (2, 8), (32, 32)):
        h = C.c_void_p()
        cfg = _qwen_cfg()
        cfg.n_kv_heads, cfg.n_q_heads = hkv, hq
        assert lib.dflash_create(C.byref(cfg), C.byref(h)) == 0
        out = (C.c_int64 * 4)()
        for batch in (1, 2, 3, 8, 17, 18, 19, 32, 37, 64, 148, 149, 256, 1024):
            for L in (0, 1, 63, 64, 65, 2048, 8191, 8192, 32768, 40000, 65536, 131072, 1 << 20):
                assert lib.dflash_attention_plan(h, batch, L, out) == 0
                tiles_per_unit, n_chunks, units, capacity = out[0], out[1], out[2], out[3]
                T = (L + 63) // 64 + 1
                assert tiles_per_unit >= 1 and n_chunks >= 1
                assert n_chunks * tiles_per_unit >= T, (batch, hkv, L)
                assert (n_chunks - 1) * tiles_per_unit < T, (batch, hkv, L)       # no empty trailing range
                assert units == batch * hkv * n_chunks
                assert units <= capacity, (batch, hkv, L, units, capacity)
        assert lib.dflash_attention_plan(h, 0, 10, out) == -1 and lib.dflash_attention_plan(h, 1, -1, out) == -1
        lib.dflash_destroy(h)
    # the example that used to overflow: 32 sequences x 8 kv heads at 65536 tokens
    h = C.c_void_p()
    assert lib.dflash_create(C.byref(_qwen_cfg()), C.byref(h)) == 0
    out = (C.c_int64 * 4)()
    assert lib.dflash_attention_plan(h, 32, 65536, out) == 0 and out[2] <= out[3] and out[0] > 128
    lib.dflash_destroy(h)


def test_contraction_work_split_covers_every_chunk_once(lib):
    # host arithmetic only, the kernel's own walk: every (weight tile, K chunk) is taken by exactly one CTA, no CTA
    # holds more than two partial pieces, and the finishing code's idea of who contributed to a shared tile (and in
    # which partial slot) is what the walk produced - for the three forms of the launch (K-split clusters with up to
    # 32 token columns, plain CTAs, CTA pairs from 160 columns on) and for tile counts that are odd, ragged or tiny
    shapes = [(4096, 4096, 1), (6144, 4096, 1), (24576, 4096, 1), (4096, 12288, 1), (151936, 4096, 1), (4096, 20480, 1),
              (2048, 4096, 5), (1536, 512, 1), (5003, 512, 1), (4900, 512, 1), (512, 1536, 1), (128, 64, 1), (100, 200, 1),
              (129, 72, 2), (768, 256, 1)]
    rows = [1, 8, 16, 17, 32, 33, 64, 100, 128, 129, 136, 160, 161, 200, 256, 330, 512, 544, 1000]
    info = (C.c_int32 * 6)()
    forms = set()
    for N, K, groups in shapes:
        for M in rows:
            for sms, pair_cap, cluster_cap in ((148, 74, 33), (148, 0, 0), (132, 66, 20), (64, 3, 16), (7, 1, 1), (1, 0, 0)):
                rc = lib.dflash_gemm_plan_check(M, N, K, groups, sms, pair_cap, cluster_cap, info)
                assert rc == 0, (rc, M, N, K, groups, sms, pair_cap, cluster_cap, list(info))
                nt, pair, grid, cs = info[0], info[1], info[2], info[3]
                assert nt >= min(M, 256) or M > 256
                assert grid <= sms and (not pair or (grid % 2 == 0 and nt >= 160)) and (cs == 1 or (nt <= 32 and grid % cs == 0))
                forms.add((bool(pair), cs > 1, info[5] == 1))
    assert (True, False, False) in forms and (False, True, True) in forms and (False, True, False) in forms \
        and (False, False, False) in forms
    assert lib.dflash_gemm_plan_check(0, 128, 64, 1, 148, 74, 33, info) == -1


def test_workspace_grows_with_the_row_count(lib):
    # a workspace sized for R rows must serve every call with fewer rows (a draft of 512 rows inside a workspace
    # sized for the 544 rows of the projection that rides along): sizes never shrink as rows grow
    h = C.c_void_p()
    assert lib.dflash_create(C.byref(_qwen_cfg()), C.byref(h)) == 0
    prev = 0
    for rows in list(range(1, 300)) + list(range(300, 1200, 7)) + [2048, 4096]:
        n = lib.dflash_workspace_bytes(h, 32, rows)
        assert n >= prev, (rows, n, prev)
        prev = n
    lib.dflash_destroy(h)


def test_attention_and_fused_projection_arguments_validated_on_the_host(lib):
    h = C.c_void_p()
    assert lib.dflash_create(C.byref(_cfg()), C.byref(h)) == 0
    a = binding.AttnArgs()
    a.batch, a.rows, a.max_pages, a.n_pool_pages, a.max_ctx_len = 1, 8, 4, 4, 128
    for name in ("q", "k_blk", "v_blk", "ctx_len", "page_table", "kv_pool", "out"):
        setattr(a, name, 256)                                          # non-null; never dereferenced on the host
    a.layer = 1                                                        # the tiny shape has one layer
    assert lib.dflash_block_attention(h, C.byref(a), None) == -1
    a.layer = -1
    assert lib.dflash_block_attention(h, C.byref(a), None) == -1
    a.layer, a.batch = 0, 0
    assert lib.dflash_block_attention(h, C.byref(a), None) == 0        # nothing to do
    # a projection handed in with the draft call: a negative row count is refused like dflash_ctx_project refuses it
    lw = (binding.LayerWeights * 1)(binding.LayerWeights(*([256] * 8)))
    w = binding.Weights(256, 256, 256, lw, 256, 256, 256, 256, 1024)
    assert lib.dflash_set_weights(h, C.byref(w)) == 0                   # borrowed pointers only, nothing is read
    cx = binding.CtxArgs()
    cx.batch, cx.max_new, cx.max_pages, cx.n_pool_pages = 1, -1, 4, 4
    assert lib.dflash_ctx_project(h, C.byref(cx), None) == -1
    d = binding.DraftArgs()
    d.batch, d.max_pages, d.n_pool_pages, d.max_ctx_len = 1, 4, 4, 128
    for name in ("anchor_ids", "ctx_len", "page_table", "kv_pool", "draft_ids"):
        setattr(d, name, 256)
    d.ctx = C.pointer(cx)
    assert lib.dflash_draft_block(h, C.byref(d), None) == -1
    lib.dflash_destroy(h)


def test_status_strings(lib):
    seen = {lib.dflash_status_string(c).decode() for c in (0, -1, -2, -3, -4, -5)}
    assert len(seen) == 6 and lib.dflash_status_string(-99).decode() == "unknown status"
    assert lib.dflash_launch_count() >= 0


def test_binding_has_no_cpu_fallback():
    # the product path must not be able to reach the oracle
    for mod in ("binding.py", "build.py", "synth.py", "__init__.py"):
        text = open(os.path.join(ROOT, "paper_2602_06036_b200", mod)).read()
        assert "import oracle" not in text and "from oracle" not in text
