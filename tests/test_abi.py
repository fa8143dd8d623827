"""The C-ABI library without a GPU: it loads, exports every symbol the header
declares, and turns bad arguments into status codes before touching CUDA."""
import ctypes
import os
import re

import pytest

from paper_2509_18085_b200 import build as builder
from paper_2509_18085_b200 import spiffy

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    builder.build()
    return spiffy.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "spiffy.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(spiffy_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"spiffy_graph_attention", "spiffy_unmask_decide", "spiffy_accept_walk"} <= set(names)
    assert len(names) >= 20
    for name in names:
        assert getattr(lib, name) is not None
        # the binding gives every entry point a prototype: nothing is called through ctypes' defaults
        assert getattr(lib, name).argtypes is not None, name


def test_status_strings(lib):
    seen = {lib.spiffy_status_string(i) for i in range(6)}
    assert len(seen) == 6 and all(seen)
    assert lib.spiffy_status_string(99)


def test_attention_rejects_bad_arguments(lib):
    fake = ctypes.c_void_p(0x1000)
    good = spiffy.AttnDesc(1, 2, 8, 16, 4, 2, 64, spiffy.F32, 0.0, spiffy.ATTN_SIMT)
    call = lambda d, *ptrs: lib.spiffy_graph_attention(ctypes.byref(d), *ptrs, None, None, 0, None)
    assert call(good, None, fake, fake, fake, fake, fake) == spiffy.EINVAL
    assert call(good, fake, None, fake, fake, fake, fake) == spiffy.EINVAL  # P > 0 needs a prefix
    assert call(good, ctypes.c_void_p(0x1004), fake, fake, fake, fake, fake) == spiffy.EINVAL
    for field, value, want in [("n_kv_heads", 3, spiffy.EINVAL), ("head_dim", 96, spiffy.EUNSUPPORTED),
                               ("block_len", 65, spiffy.EUNSUPPORTED), ("dtype", 7, spiffy.EINVAL),
                               ("batch", 0, spiffy.EINVAL), ("prefix_len", -1, spiffy.EINVAL),
                               ("scale", float("nan"), spiffy.EINVAL), ("kernel", 9, spiffy.EINVAL)]:
        d = spiffy.AttnDesc(1, 2, 8, 16, 4, 2, 64, spiffy.F32, 0.0, spiffy.ATTN_SIMT)
        setattr(d, field, value)
        assert call(d, fake, fake, fake, fake, fake, fake) == want, field
    # fp32 has no tensor-core kernel
    d = spiffy.AttnDesc(1, 2, 8, 16, 4, 2, 64, spiffy.F32, 0.0, spiffy.ATTN_TCGEN05)
    assert call(d, fake, fake, fake, fake, fake, fake) == spiffy.EUNSUPPORTED
    assert lib.spiffy_graph_attention(None, fake, fake, fake, fake, fake, fake, None, None, 0, None) == spiffy.EINVAL


def test_decide_rejects_bad_arguments(lib):
    fake = ctypes.c_void_p(0x1000)

    def desc(**kw):
        d = spiffy.DecideDesc(1, 4, 8, 1024, spiffy.BF16, 1024, 1023, spiffy.RULE_TOPS, 1, 0.9)
        for k, v in kw.items():
            setattr(d, k, v)
        return d

    def call(d, ws=fake, ws_bytes=1 << 30, logits=fake):
        return lib.spiffy_unmask_decide(ctypes.byref(d), logits, fake, fake, fake, fake, fake, None,
                                        ws, ws_bytes, None)

    assert lib.spiffy_unmask_decide_workspace(ctypes.byref(desc())) > 0
    assert call(desc(), ws=None) == spiffy.EWORKSPACE
    assert call(desc(), ws_bytes=8) == spiffy.EWORKSPACE
    assert call(desc(), logits=None) == spiffy.EINVAL
    assert call(desc(row_stride=1000)) == spiffy.EINVAL     # shorter than a row
    assert call(desc(row_stride=1028)) == spiffy.EINVAL     # rows not 16-byte spaced
    assert call(desc(top_s=0)) == spiffy.EINVAL
    assert call(desc(rule=5)) == spiffy.EINVAL
    assert call(desc(block_len=65)) == spiffy.EUNSUPPORTED
    assert call(desc(vocab=0)) == spiffy.EINVAL
    assert call(desc(rule=spiffy.RULE_THRESHOLD, threshold=float("nan"))) == spiffy.EINVAL
    assert lib.spiffy_unmask_decide_workspace(ctypes.byref(desc(vocab=0))) == 0


def test_walk_rejects_bad_arguments(lib):
    fake = ctypes.c_void_p(0x1000)
    d = spiffy.DecideDesc(1, 4, 8, 0, 0, 0, 0, 0, 1, 0.0)
    args = [fake] * 3 + [4] + [fake] * 7 + [None]
    bad = list(args)
    bad[1] = None
    assert lib.spiffy_accept_walk(ctypes.byref(d), *bad) == spiffy.EINVAL
    neg = list(args)
    neg[3] = -1
    assert lib.spiffy_accept_walk(ctypes.byref(d), *neg) == spiffy.EINVAL


def test_decide_walk_rejects_bad_arguments(lib):
    """The one-call form checks what the two calls check, before any launch."""
    fake = ctypes.c_void_p(0x1000)

    def call(d, logits=fake, parent_off=fake, cap=4, next_block=fake, ws=fake, ws_bytes=1 << 30):
        # desc, logits, tokens, parent_off, parent_idx, cap, conf, top_tok, bits, n_unmask, decide_status,
        # accepted_node, n_accepted, path, next_block, walk_status, workspace, bytes, stream
        return lib.spiffy_decide_walk(ctypes.byref(d), logits, fake, parent_off, fake, cap, fake, fake, fake,
                                      fake, None, fake, fake, fake, next_block, None, ws, ws_bytes, None)

    good = spiffy.DecideDesc(1, 2, 4, 32, spiffy.F32, 32, 31, spiffy.RULE_TOPS, 1, 0.0)
    assert call(good, logits=None) == spiffy.EINVAL
    assert call(good, parent_off=None) == spiffy.EINVAL
    assert call(good, next_block=None) == spiffy.EINVAL
    assert call(good, cap=-1) == spiffy.EINVAL
    assert call(good, logits=ctypes.c_void_p(0x1004)) == spiffy.EINVAL
    assert call(good, ws=None) == spiffy.EWORKSPACE
    assert call(good, ws_bytes=8) == spiffy.EWORKSPACE
    assert call(spiffy.DecideDesc(1, 2, 65, 32, spiffy.F32, 32, 31, spiffy.RULE_TOPS, 1, 0.0)) == spiffy.EUNSUPPORTED
    assert call(spiffy.DecideDesc(1, 2, 4, 32, spiffy.F32, 32, 31, 7, 1, 0.0)) == spiffy.EINVAL
    assert call(spiffy.DecideDesc(1, 2, 4, 33, spiffy.F32, 33, 31, spiffy.RULE_TOPS, 1, 0.0)) == spiffy.EINVAL


def test_lazy_decide_walk_rejects_bad_arguments(lib):
    fake = ctypes.c_void_p(0x1000)
    good = spiffy.DecideDesc(2, 4, 8, 1024, spiffy.BF16, 1024, 1023, spiffy.RULE_THRESHOLD, 1, 0.9)
    need = lib.spiffy_decide_walk_lazy_workspace(ctypes.byref(good))
    # partial results of one node per sequence, plus the header and three words per sequence
    assert need >= 2 * 8 * 16 + 16 + 2 * 12
    assert need < lib.spiffy_unmask_decide_workspace(ctypes.byref(good)) + 64

    def call(d, logits=fake, parent_idx=fake, cap=4, ws=fake, ws_bytes=1 << 30):
        return lib.spiffy_decide_walk_lazy(ctypes.byref(d), logits, fake, fake, parent_idx, cap, fake, fake,
                                           fake, fake, None, fake, fake, fake, fake, None, ws, ws_bytes, None)

    assert call(good, logits=None) == spiffy.EINVAL
    assert call(good, parent_idx=None) == spiffy.EINVAL
    assert call(good, cap=-2) == spiffy.EINVAL
    assert call(good, ws=None) == spiffy.EWORKSPACE
    assert call(good, ws_bytes=need - 1) == spiffy.EWORKSPACE
    bad = spiffy.DecideDesc(2, 4, 8, 1024, spiffy.BF16, 1024, 1023, spiffy.RULE_TOPS, 0, 0.9)
    assert call(bad) == spiffy.EINVAL
    assert lib.spiffy_decide_walk_lazy_workspace(ctypes.byref(bad)) == 0


def test_stage_masked_rows_rejects_bad_arguments(lib):
    fake = ctypes.c_void_p(0x1000)
    call = lambda src=fake, dst=fake, row_bytes=256, tokens=fake, rows=4: lib.spiffy_stage_masked_rows(
        src, dst, row_bytes, tokens, 7, rows, None)
    assert call(src=None) == spiffy.EINVAL
    assert call(dst=None) == spiffy.EINVAL
    assert call(tokens=None) == spiffy.EINVAL
    assert call(row_bytes=0) == spiffy.EINVAL
    assert call(row_bytes=250) == spiffy.EINVAL            # rows must be whole 16-byte vectors
    assert call(src=ctypes.c_void_p(0x1008)) == spiffy.EINVAL
    assert call(rows=0) == spiffy.EINVAL
    assert call(rows=70000) == spiffy.EUNSUPPORTED


def test_sampled_decide_rejects_bad_arguments(lib):
    fake = ctypes.c_void_p(0x1000)
    good = spiffy.DecideDesc(1, 4, 8, 1024, spiffy.BF16, 1024, 1023, spiffy.RULE_TOPS, 1, 0.9)
    need = lib.spiffy_unmask_decide_sampled_workspace(ctypes.byref(good))
    # the greedy call's partial results (rounded up to 256 bytes) and one arrival counter per node
    greedy = lib.spiffy_unmask_decide_workspace(ctypes.byref(good))
    assert need == (greedy + 255) // 256 * 256 + 4 * 4
    # slice width: the fewest equal slices of at most 8192 bf16 / 4096 fp32 entries, whole 16-byte vectors
    width = lambda v, dt: lib.spiffy_sampled_slice_width(ctypes.byref(
        spiffy.DecideDesc(1, 4, 8, v, dt, v, v - 1, spiffy.RULE_TOPS, 1, 0.9)))
    assert width(1024, spiffy.BF16) == 1024 and width(8192, spiffy.BF16) == 8192
    assert width(126464, spiffy.BF16) == 7904 and width(8200, spiffy.BF16) == 4104
    assert width(4100, spiffy.F32) == 2052 and width(36, spiffy.F32) == 36
    assert width(0, spiffy.BF16) == 0

    def call(temperature=1.0, sample=True, logits=fake, ws=fake, ws_bytes=1 << 30, d=good):
        s = spiffy.SampleDesc(temperature, 0, 42)
        return lib.spiffy_unmask_decide_sampled(ctypes.byref(d), ctypes.byref(s) if sample else None, logits,
                                                fake, fake, fake, fake, fake, None, ws, ws_bytes, None)

    assert call(sample=False) == spiffy.EINVAL
    for t in (0.0, -0.5, float("nan"), float("inf")):
        assert call(temperature=t) == spiffy.EINVAL
    assert call(logits=None) == spiffy.EINVAL
    assert call(ws=None) == spiffy.EWORKSPACE
    assert call(ws_bytes=need - 1) == spiffy.EWORKSPACE
    assert call(d=spiffy.DecideDesc(1, 4, 65, 1024, spiffy.BF16, 1024, 1023, spiffy.RULE_TOPS, 1, 0.9)) == \
        spiffy.EUNSUPPORTED


def test_lmhead_decide_rejects_bad_arguments(lib):
    fake = ctypes.c_void_p(0x1000)
    good = spiffy.DecideDesc(1, 8, 32, 126464, 0, 0, 126463, spiffy.RULE_THRESHOLD, 1, 0.9)

    def call(d=good, hidden=4096, hs=fake, w=fake):
        return lib.spiffy_lmhead_decide(ctypes.byref(d), hidden, hs, w, fake, fake, fake, fake, fake, None,
                                        fake, 1 << 30, None)

    assert call(hidden=100) == spiffy.EUNSUPPORTED          # not a multiple of 128
    assert call(hidden=0) == spiffy.EUNSUPPORTED
    assert call(d=spiffy.DecideDesc(1, 9, 65, 1000, 0, 0, 999, spiffy.RULE_TOPS, 1, 0.0)) == spiffy.EUNSUPPORTED
    assert call(d=spiffy.DecideDesc(1, 8, 32, 0, 0, 0, 0, spiffy.RULE_TOPS, 1, 0.0)) == spiffy.EINVAL
    assert call(d=spiffy.DecideDesc(1, 8, 32, 1000, 0, 0, 999, 9, 1, 0.0)) == spiffy.EINVAL
    assert call(hs=None) == spiffy.EINVAL
    assert call(w=ctypes.c_void_p(0x1008)) == spiffy.EINVAL
    assert lib.spiffy_lmhead_decide_workspace(ctypes.byref(good), 100) == 0


def test_draft_rejects_bad_arguments(lib):
    fake = ctypes.c_void_p(0x1000)

    def desc(**kw):
        d = spiffy.DraftDesc(1, 8, 1024, spiffy.BF16, 1024, 1023, 10, 3, 3, 16)
        for k, v in kw.items():
            setattr(d, k, v)
        return d

    def call(d, ws=fake, ws_bytes=1 << 30, logits=fake):
        return lib.spiffy_draft_blocks(ctypes.byref(d), logits, *([fake] * 11), None, ws, ws_bytes, None)

    assert lib.spiffy_draft_blocks_workspace(ctypes.byref(desc())) > 0
    assert call(desc(), ws=None) == spiffy.EWORKSPACE
    assert call(desc(), ws_bytes=8) == spiffy.EWORKSPACE
    assert call(desc(), logits=None) == spiffy.EINVAL
    assert call(desc(budget=11)) == spiffy.EINVAL        # more drafts kept than formulas exist
    assert call(desc(budget=0)) == spiffy.EINVAL
    assert call(desc(top_k=5)) == spiffy.EUNSUPPORTED
    assert call(desc(top_k=0)) == spiffy.EINVAL
    assert call(desc(block_len=65)) == spiffy.EUNSUPPORTED
    assert call(desc(row_stride=1028)) == spiffy.EINVAL
    assert call(desc(parent_cap=0)) == spiffy.EINVAL
    assert lib.spiffy_draft_blocks_workspace(ctypes.byref(desc(vocab=0))) == 0


def test_binding_refuses_cpu_tensors():
    import torch
    t = torch.zeros(1, 1, 4, 8)
    tok = torch.zeros(1, 1, 4, dtype=torch.int32)
    with pytest.raises(ValueError):
        spiffy.spiffy_unmask_decide(t, tok, 7, spiffy.RULE_TOPS)


def test_full_sequence_attention_rejects_bad_arguments(lib):
    fake = ctypes.c_void_p(0x1000)
    good = spiffy.AttnDesc(1, 4, 32, 64, 8, 2, 128, spiffy.BF16, 0.0, spiffy.ATTN_TCGEN05)

    def call(d, S=32, q_suffix=fake, k_prefix=fake, out_suffix=fake, k_block=fake):
        return lib.spiffy_full_sequence_attention(ctypes.byref(d), S, fake, q_suffix, k_prefix, fake, fake, fake,
                                                  k_block, fake, fake, out_suffix, None, None, 0, None)

    assert call(good, q_suffix=None) == spiffy.EINVAL
    assert call(good, out_suffix=None) == spiffy.EINVAL
    assert call(good, k_prefix=None) == spiffy.EINVAL          # P > 0 needs a prefix
    assert call(good, k_block=ctypes.c_void_p(0x1008)) == spiffy.EINVAL
    assert call(good, S=-1) == spiffy.EINVAL
    assert call(good, S=1025) == spiffy.EUNSUPPORTED
    # the tensor-core kernel only: bf16, head dimension 128
    assert call(spiffy.AttnDesc(1, 4, 32, 64, 8, 2, 128, spiffy.F32, 0.0, spiffy.ATTN_AUTO)) == spiffy.EUNSUPPORTED
    assert call(spiffy.AttnDesc(1, 4, 32, 64, 8, 2, 64, spiffy.BF16, 0.0, spiffy.ATTN_AUTO)) == spiffy.EUNSUPPORTED
    assert lib.spiffy_full_sequence_attention_workspace(ctypes.byref(good), 2000) == 0


def test_host_step_rejects_bad_arguments(lib):
    fake = ctypes.c_void_p(0x1000)
    attn = spiffy.AttnDesc(1, 4, 8, 16, 4, 4, 64, spiffy.F32, 0.0, spiffy.ATTN_AUTO)
    dec = spiffy.DecideDesc(1, 4, 8, 1024, spiffy.F32, 1024, 1023, spiffy.RULE_TOPS, 1, 0.9)
    good = spiffy.StepDesc(attn, dec, 4)
    need = lib.spiffy_verify_step_host_workspace(ctypes.byref(good))
    # staging of every input, the attention output, the decision's results and scratch
    assert need > 2 * 1 * 4 * 8 * 4 * 64 * 4 + 4 * 8 * 1024 * 4

    def call(d, q=fake, out=fake, ws=ctypes.c_void_p(0x10000), ws_bytes=1 << 30):
        return lib.spiffy_verify_step_host(ctypes.byref(d), q, fake, fake, fake, fake, fake, fake, fake, fake,
                                           out, fake, fake, fake, fake, ws, ws_bytes, None)

    assert call(good, q=None) == spiffy.EINVAL
    assert call(good, out=None) == spiffy.EINVAL
    assert call(good, ws=None) == spiffy.EWORKSPACE
    assert call(good, ws_bytes=need - 1) == spiffy.EWORKSPACE
    assert call(good, ws=ctypes.c_void_p(0x10010)) == spiffy.EWORKSPACE   # 256-byte alignment
    mismatch = spiffy.StepDesc(attn, spiffy.DecideDesc(1, 5, 8, 1024, spiffy.F32, 1024, 1023, spiffy.RULE_TOPS, 1, 0.9), 4)
    assert call(mismatch) == spiffy.EINVAL
    assert lib.spiffy_verify_step_host_workspace(ctypes.byref(mismatch)) == 0
    assert call(spiffy.StepDesc(attn, dec, 0)) == spiffy.EINVAL
