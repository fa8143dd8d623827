"""spiffy_unmask_decide_static: the decision step for callers that cannot give
the library scratch memory (a plug-in inside an engine that owns all device
memory, a decode loop that must not hit cudaMalloc's device-wide sync).  Its
scratch is a fixed array inside the library, so the test checks what such a
caller relies on: same results as the regular entry point, call after call,
although every call reuses the same array with the previous call's leftovers.

Collected last on purpose (file name): a run that stops at the first failure
has then already run every other test."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2509_18085_b200 import spiffy
from paper_2509_18085_b200 import workloads as W

import gpu_util as G

pytestmark = pytest.mark.gpu


def empty_decision(B, N, L):
    dev = "cuda"
    return spiffy.Decision(torch.full((B, N, L), 7.0, dtype=torch.float32, device=dev),
                           torch.full((B, N, L), -3, dtype=torch.int32, device=dev),
                           torch.full((B, N), -1, dtype=torch.int64, device=dev),
                           torch.full((B, N), -1, dtype=torch.int32, device=dev),
                           torch.zeros((B,), dtype=torch.int32, device=dev))


def assert_same(a, b, tokens, mask_id):
    masked = (tokens == mask_id)
    ca, cb = a.conf.cpu().numpy(), b.conf.cpu().numpy()
    assert np.all(np.isneginf(ca[~masked])) and np.all(np.isneginf(cb[~masked]))
    # same reduction, same fixed merge order: the confidences agree bit for bit
    # (which is well inside the tolerance of the parity tests)
    assert np.max(np.abs(ca[masked] - cb[masked]), initial=0.0) <= G.TOL["bf16"]
    assert torch.equal(a.conf.view(torch.int32), b.conf.view(torch.int32))
    assert torch.equal(a.top_tok, b.top_tok)
    assert torch.equal(a.unmask_bits, b.unmask_bits)
    assert torch.equal(a.n_unmask, b.n_unmask)
    assert int(a.dev_status.abs().sum()) == 0 and int(b.dev_status.abs().sum()) == 0


def test_two_calls_in_a_row_match_the_regular_entry_point():
    cfg = W.config(2)
    B, N, L = cfg.batch, cfg.n_nodes, cfg.block_len
    for case in (0, 1):  # second call: other logits, other masks, same scratch array
        w = W.make(cfg, W.seed_for(2, 30 + case), attention=False)
        logits = G.to_dev(w.logits, torch.bfloat16)
        tokens = G.to_dev(w.block_tokens)
        want = spiffy.spiffy_unmask_decide(logits, tokens, cfg.mask_id, cfg.rule, cfg.top_s, cfg.threshold)
        got = spiffy.spiffy_unmask_decide_static(logits, tokens, cfg.mask_id, cfg.rule, empty_decision(B, N, L),
                                                 cfg.top_s, cfg.threshold)
        torch.cuda.synchronize()
        assert_same(got, want, w.block_tokens, cfg.mask_id)


def test_small_fp32_shape_then_repeat():
    cfg = W.config(1)
    w = W.make(cfg, W.seed_for(1, 3), attention=False)
    logits, tokens = G.to_dev(w.logits), G.to_dev(w.block_tokens)
    want = spiffy.spiffy_unmask_decide(logits, tokens, cfg.mask_id, cfg.rule, cfg.top_s)
    for _ in range(2):
        got = spiffy.spiffy_unmask_decide_static(logits, tokens, cfg.mask_id, cfg.rule,
                                                 empty_decision(cfg.batch, cfg.n_nodes, cfg.block_len), cfg.top_s)
        torch.cuda.synchronize()
        assert_same(got, want, w.block_tokens, cfg.mask_id)


def test_the_call_allocates_no_device_memory():
    """What the entry point promises its callers: after the first call on the
    device (which looks up the array's address), a call changes neither the
    driver's free-memory figure nor torch's allocation counters."""
    cfg = W.config(1)
    w = W.make(cfg, W.seed_for(1, 4), attention=False)
    logits, tokens = G.to_dev(w.logits), G.to_dev(w.block_tokens)
    out = empty_decision(cfg.batch, cfg.n_nodes, cfg.block_len)
    spiffy.spiffy_unmask_decide_static(logits, tokens, cfg.mask_id, cfg.rule, out, cfg.top_s)
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    count0 = torch.cuda.memory_stats()["allocation.all.allocated"]
    for _ in range(3):
        spiffy.spiffy_unmask_decide_static(logits, tokens, cfg.mask_id, cfg.rule, out, cfg.top_s)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    assert torch.cuda.memory_stats()["allocation.all.allocated"] == count0


def test_shapes_beyond_the_fixed_scratch_are_refused():
    # 65535 rows of a large vocabulary need more scratch than the library holds
    desc = spiffy.DecideDesc(1, 1023, 64, 126464, spiffy.BF16, 126464, 126463, spiffy.RULE_TOPS, 1, 0.9)
    assert spiffy.spiffy_unmask_decide_workspace(desc) > spiffy.DECIDE_STATIC_BYTES
    fake = ctypes.c_void_p(0x1000)
    st = spiffy.lib().spiffy_unmask_decide_static(ctypes.byref(desc), fake, fake, fake, fake, fake, fake,
                                                  None, None)
    assert st == spiffy.EUNSUPPORTED
