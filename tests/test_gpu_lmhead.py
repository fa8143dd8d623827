"""spiffy_lmhead_decide: the decision reduced on the tensor cores from hidden
states and the output embedding, against the oracle's decision on the float64
product of the same (bf16-representable) operands."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2509_18085_b200 import spiffy
import gpu_util as G

pytestmark = pytest.mark.gpu

TOP_GAP = 1e-3   # the arg-max is compared where the two largest logits differ by more (fp32 accumulation)


def operands(seed, B, N, L, H, V, p_unmasked=0.3):
    g = torch.Generator().manual_seed(seed)
    hs = torch.randn((B, N, L, H), generator=g).to(torch.bfloat16)
    w = (torch.randn((V, H), generator=g) * (2.0 / H ** 0.5)).to(torch.bfloat16)  # logits of about N(0, 2)
    mask = V - 1
    w[mask] = 0
    w[mask, 0] = -30.0 / max(float(hs[..., 0].abs().max()), 1.0)  # the mask token is never the best one
    tokens = torch.where(torch.rand((B, N, L), generator=g) < p_unmasked, 3, mask).to(torch.int32)
    tokens[:, :, 0] = mask
    return hs, w, tokens, mask


def reference(hs, w, tokens, mask, rule, top_s, tau):
    B, N, L, H = hs.shape
    logits = (hs.double().reshape(-1, H) @ w.double().T).reshape(B, N, L, -1).numpy()
    o = oracle.unmask_decide(logits.astype(np.float32), tokens.numpy(), mask, rule, top_s, tau)
    srt = np.sort(logits, axis=-1)
    return o, srt[..., -1] - srt[..., -2]


@pytest.mark.parametrize("B,N,L,H,V", [(1, 2, 32, 128, 256), (1, 8, 32, 256, 5000), (1, 3, 32, 1024, 1000),
                                       (2, 3, 20, 384, 777), (1, 1, 1, 128, 64), (4, 2, 32, 128, 40000),
                                       (3, 5, 40, 256, 3000), (2, 8, 32, 128, 520)])
def test_decision_matches_the_oracle(B, N, L, H, V):
    """One or two M-tiles, row counts that fill neither, more than 256 rows (several
    passes, the last one ragged), vocabularies that end inside a tile, more tiles
    than SMs and fewer."""
    hs, w, tokens, mask = operands(V + H, B, N, L, H, V)
    for rule, S, tau in ((spiffy.RULE_TOPS, 2, 0.0), (spiffy.RULE_THRESHOLD, 1, 0.02)):
        dec = spiffy.spiffy_lmhead_decide(hs.cuda(), w.cuda(), tokens.cuda(), mask, rule, S, tau)
        torch.cuda.synchronize()
        o, gap = reference(hs, w, tokens, mask, rule, S, tau)
        m = tokens.numpy() == mask
        sure = m & (gap > TOP_GAP)
        assert sure.sum() >= 0.9 * m.sum()
        tok = dec.top_tok.cpu().numpy()
        assert np.array_equal(tok[sure], o.top_tok[sure])
        assert np.array_equal(tok[~m], tokens.numpy()[~m])
        np.testing.assert_allclose(dec.conf.cpu().numpy()[m], o.conf[m], atol=1e-4)
        node_ok = (sure | ~m).all(axis=2) & (o.margin > 1e-4)
        assert np.array_equal(G.bits_np(dec.unmask_bits)[node_ok], o.unmask_bits[node_ok])
        assert np.array_equal(dec.n_unmask.cpu().numpy()[node_ok], o.n_unmask[node_ok])
        assert int(dec.dev_status.sum()) == 0


def test_same_bits_as_the_decision_on_fp32_logits_and_on_every_call():
    """The fused call ends in the decision's own finalize kernel; repeated calls
    give identical bits (fixed merge order over the CTAs' partial results)."""
    hs, w, tokens, mask = operands(9, 1, 8, 32, 512, 20000)
    a = spiffy.spiffy_lmhead_decide(hs.cuda(), w.cuda(), tokens.cuda(), mask, spiffy.RULE_THRESHOLD, 1, 0.02)
    b = spiffy.spiffy_lmhead_decide(hs.cuda(), w.cuda(), tokens.cuda(), mask, spiffy.RULE_THRESHOLD, 1, 0.02)
    torch.cuda.synchronize()
    assert torch.equal(a.conf.view(torch.int32), b.conf.view(torch.int32))
    assert torch.equal(a.top_tok, b.top_tok) and torch.equal(a.unmask_bits, b.unmask_bits)
    # the two-step route: fp32 logits from the same fp32 accumulation order are not available, so
    # compare with the decision on float64 logits rounded to fp32 within the tolerance
    logits = (hs.double().reshape(-1, 512) @ w.double().T).reshape(1, 8, 32, -1).float().cuda()
    c = spiffy.spiffy_unmask_decide(logits, tokens.cuda(), mask, spiffy.RULE_THRESHOLD, 1, 0.02)
    m = (tokens == mask)
    assert float((a.conf.cpu()[m] - c.conf.cpu()[m]).abs().max()) < 1e-5


def test_benchmark_shape_on_sampled_rows():
    """hidden 4096, V = 126464, 256 rows: the shape of the LLaDA-8B output projection."""
    B, N, L, H, V = 1, 8, 32, 4096, 126464
    hs, w, tokens, mask = operands(5, B, N, L, H, V, p_unmasked=0.36)
    dec = spiffy.spiffy_lmhead_decide(hs.cuda(), w.cuda(), tokens.cuda(), mask, spiffy.RULE_THRESHOLD, 1, 0.9)
    torch.cuda.synchronize()
    rows = np.flatnonzero(tokens.numpy().reshape(-1) == mask)[::5][:32]
    lg = hs.double().reshape(-1, H)[rows] @ w.double().T
    p = torch.softmax(lg, -1)
    conf, tok = p.max(-1)
    srt = torch.sort(lg, -1).values
    sure = (srt[:, -1] - srt[:, -2]) > TOP_GAP
    assert int(sure.sum()) >= 28
    assert torch.equal(dec.top_tok.cpu().reshape(-1)[rows][sure].long(), tok[sure])
    assert float((dec.conf.cpu().reshape(-1)[rows].double() - conf).abs().max()) < 1e-5
    assert int(dec.dev_status.sum()) == 0


def test_nonfinite_rows_and_argument_checks():
    hs, w, tokens, mask = operands(2, 2, 2, 8, 128, 300)
    hs[1, 0, 0, 5] = float("nan")
    tokens[1, 0, 0] = mask
    dec = spiffy.spiffy_lmhead_decide(hs.cuda(), w.cuda(), tokens.cuda(), mask, spiffy.RULE_TOPS)
    assert dec.dev_status.cpu().tolist() == [0, spiffy.DEV_NONFINITE]
    good = operands(2, 2, 2, 8, 128, 300)
    with pytest.raises(spiffy.SpiffyError):   # hidden not a multiple of 128
        spiffy.spiffy_lmhead_decide(good[0][..., :64].contiguous().cuda(), good[1][:, :64].contiguous().cuda(),
                                    good[2].cuda(), good[3], spiffy.RULE_TOPS)
    with pytest.raises(spiffy.SpiffyError):
        spiffy.spiffy_lmhead_decide(good[0].cuda(), good[1].cuda(), good[2].cuda(), good[3], spiffy.RULE_TOPS,
                                    workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    with pytest.raises(ValueError):
        spiffy.spiffy_lmhead_decide(good[0].float().cuda(), good[1].cuda(), good[2].cuda(), good[3],
                                    spiffy.RULE_TOPS)
