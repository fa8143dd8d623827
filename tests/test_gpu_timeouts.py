"""Failure detection on the device: every wait inside the kernels is bounded,
and a wait that runs out must end in SPIFFY_DEV_TIMEOUT in the caller's status
word, a normal return and a usable context.  The waits are made to run out from
the host (spiffy_set_wait_limits: fewer polls; one arrival that never comes);
nothing here faults, traps or hangs the GPU."""
import numpy as np
import pytest
import torch

from paper_2509_18085_b200 import spiffy
from paper_2509_18085_b200 import workloads as W

import gpu_util as G
import test_gpu_decide_walk as T

pytestmark = pytest.mark.gpu


@pytest.fixture
def limits():
    yield spiffy.set_wait_limits
    spiffy.set_wait_limits()  # back to the defaults, whatever the test did


def test_lazy_call_gives_up_on_an_arrival_that_never_comes(limits):
    logits, tokens, off, idx, mask = T.random_case(21, 3, 8, 16, 3000, p_accept=1.0)
    lg, tk, of, ix = G.to_dev(logits), G.to_dev(tokens), G.to_dev(off), G.to_dev(idx)
    want_dec, want_walk = spiffy.spiffy_decide_walk(lg, tk, of, ix, mask, spiffy.RULE_TOPS, lazy=True)
    torch.cuda.synchronize()
    assert int(want_walk.dev_status.sum()) == 0
    # sequence 0's tail now expects one arrival more than its reducers deliver,
    # and every wait gives up after 3000 polls (well under a second)
    limits(flag_polls=3000, lazy_extra_arrivals=1)
    dec, walk = spiffy.spiffy_decide_walk(lg, tk, of, ix, mask, spiffy.RULE_TOPS, lazy=True)
    torch.cuda.synchronize()  # the call returns: nothing waits for ever
    assert int(dec.dev_status[0]) & spiffy.DEV_TIMEOUT
    assert int(walk.dev_status[0]) & spiffy.DEV_TIMEOUT
    # the context is intact: the same call, limits restored, gives the earlier bits
    limits()
    dec2, walk2 = spiffy.spiffy_decide_walk(lg, tk, of, ix, mask, spiffy.RULE_TOPS, lazy=True)
    torch.cuda.synchronize()
    for f in ("accepted_node", "n_accepted", "path", "next_block", "dev_status"):
        assert torch.equal(getattr(walk2, f), getattr(want_walk, f)), f
    assert torch.equal(dec2.n_unmask, want_dec.n_unmask)


@pytest.mark.parametrize("index,n_nodes,over", [(5, 8, {}), (2, None, {}), (3, None, {}),
                                                (2, None, dict(batch=5, prefix_len=256))])
def test_attention_gives_up_when_its_mbarrier_waits_may_not_poll(limits, index, n_nodes, over):
    """The four routes of the tensor-core kernel: key tiles split through the
    workspace and the merge kernel (5, 8), the cluster pair (2), one M-tile per
    thread block over all key tiles (3), two M-tiles per block (2 with a batch of
    five).  With no poll allowed every role of the kernel gives up at its first
    wait, before any tensor-core product is issued."""
    cfg = W.config(index, n_nodes, **over)
    w = W.make(cfg, W.seed_for(index, 0), decision=False)
    dt = torch.bfloat16
    q, kp, vp, kb, vb = (G.to_dev(a, dt) for a in (w.q, w.k_prefix, w.v_prefix, w.k_block, w.v_block))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    want = spiffy.spiffy_graph_attention(q, kp, vp, kb, vb, kernel=spiffy.ATTN_TCGEN05, dev_status=status)
    torch.cuda.synchronize()
    assert int(status) == 0
    limits(mbarrier_polls=0)
    spiffy.spiffy_graph_attention(q, kp, vp, kb, vb, kernel=spiffy.ATTN_TCGEN05, dev_status=status)
    torch.cuda.synchronize()
    assert int(status) == spiffy.DEV_TIMEOUT
    limits()
    status.zero_()
    again = spiffy.spiffy_graph_attention(q, kp, vp, kb, vb, kernel=spiffy.ATTN_TCGEN05, dev_status=status)
    torch.cuda.synchronize()
    assert int(status) == 0 and torch.equal(again, want)


def test_fused_output_projection_gives_up_likewise(limits):
    g = torch.Generator().manual_seed(5)
    B, N, L, H, V = 1, 2, 32, 256, 3000
    hs = torch.randn((B, N, L, H), generator=g).to(torch.bfloat16).cuda()
    wt = (torch.randn((V, H), generator=g) * 0.2).to(torch.bfloat16).cuda()
    tokens = torch.full((B, N, L), V - 1, dtype=torch.int32, device="cuda")
    want = spiffy.spiffy_lmhead_decide(hs, wt, tokens, V - 1, spiffy.RULE_TOPS)
    torch.cuda.synchronize()
    assert int(want.dev_status.sum()) == 0
    limits(mbarrier_polls=0)
    got = spiffy.spiffy_lmhead_decide(hs, wt, tokens, V - 1, spiffy.RULE_TOPS)
    torch.cuda.synchronize()
    assert int(got.dev_status[0]) & spiffy.DEV_TIMEOUT
    limits()
    again = spiffy.spiffy_lmhead_decide(hs, wt, tokens, V - 1, spiffy.RULE_TOPS)
    torch.cuda.synchronize()
    assert int(again.dev_status.sum()) == 0 and torch.equal(again.top_tok, want.top_tok)
