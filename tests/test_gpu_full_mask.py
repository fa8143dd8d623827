"""The full-sequence verification mask (Fig. 3 caption, App. A.2) on the CUDA
path -- two calls of the tensor-core attention kernel -- against the
explicit-mask oracle; and the long blocks that make the second call possible."""
import numpy as np
import pytest
import torch

import oracle
from oracle import full_mask
from paper_2509_18085_b200 import spiffy
import gpu_util as G

pytestmark = pytest.mark.gpu


def bf16(r, *shape):
    return torch.from_numpy(r.standard_normal(shape).astype(np.float32)).to(torch.bfloat16)


@pytest.mark.parametrize("B,N,L,P,S,Hq,Hkv", [(1, 8, 32, 512, 96, 32, 32), (2, 4, 32, 100, 32, 8, 2),
                                              (1, 3, 16, 0, 200, 4, 4), (1, 1, 32, 64, 224, 4, 1)])
def test_full_sequence_mask(B, N, L, P, S, Hq, Hkv):
    r = np.random.default_rng(S + P)
    d = 128
    qn, qs = bf16(r, B, N, L, Hq, d), bf16(r, B, S, Hq, d)
    kp, vp = (bf16(r, B, P, Hkv, d), bf16(r, B, P, Hkv, d)) if P else (None, None)
    ks, vs, kb, vb = bf16(r, B, S, Hkv, d), bf16(r, B, S, Hkv, d), bf16(r, B, N, L, Hkv, d), bf16(r, B, N, L, Hkv, d)
    dev = lambda t: None if t is None else t.cuda()
    got_nodes, got_suffix = spiffy.spiffy_full_sequence_attention(dev(qn), dev(qs), dev(kp), dev(vp), dev(ks),
                                                                  dev(vs), dev(kb), dev(vb))
    torch.cuda.synchronize()
    f = lambda t: t.float().numpy()
    empty = np.zeros((B, 0, Hkv, d), dtype=np.float32)
    want_nodes, want_suffix = full_mask.full_sequence_attention(
        f(qn), f(qs), f(kp) if P else empty, f(vp) if P else empty, f(ks), f(vs), f(kb), f(vb))
    assert np.abs(got_nodes.float().cpu().numpy() - want_nodes).max() <= G.TOL["bf16"]
    assert np.abs(got_suffix.float().cpu().numpy() - want_suffix).max() <= G.TOL["bf16"]


@pytest.mark.parametrize("B,N,L,P,Hq,Hkv", [(1, 1, 96, 200, 4, 4), (1, 2, 128, 64, 8, 2), (2, 3, 200, 300, 4, 1),
                                            (1, 2, 65, 0, 2, 2), (1, 1, 1000, 128, 2, 1)])
def test_blocks_longer_than_a_key_tile(B, N, L, P, Hq, Hkv):
    """A node's block keys may span several key tiles; the CUDA-core kernel stays at 64."""
    r = np.random.default_rng(L)
    d = 128
    q, kb, vb = bf16(r, B, N, L, Hq, d), bf16(r, B, N, L, Hkv, d), bf16(r, B, N, L, Hkv, d)
    kp, vp = (bf16(r, B, P, Hkv, d), bf16(r, B, P, Hkv, d)) if P else (None, None)
    dev = lambda t: None if t is None else t.cuda()
    out = spiffy.spiffy_graph_attention(dev(q), dev(kp), dev(vp), dev(kb), dev(vb), kernel=spiffy.ATTN_TCGEN05)
    torch.cuda.synchronize()
    f = lambda t: t.float().numpy()
    empty = np.zeros((B, 0, Hkv, d), dtype=np.float32)
    want = oracle.graph_attention(f(q), f(kp) if P else empty, f(vp) if P else empty, f(kb), f(vb))
    assert np.abs(out.float().cpu().numpy() - want).max() <= G.TOL["bf16"]
    with pytest.raises(spiffy.SpiffyError):
        spiffy.spiffy_graph_attention(dev(q), dev(kp), dev(vp), dev(kb), dev(vb), kernel=spiffy.ATTN_SIMT)


@pytest.mark.parametrize("B,N,L,n_blocks,k,Hq,Hkv", [(1, 4, 32, 8, 5, 32, 32), (2, 8, 32, 6, 3, 8, 2),
                                                     (1, 3, 16, 4, 0, 4, 4), (1, 16, 32, 20, 19, 28, 4)])
def test_blockwise_causal_context(B, N, L, n_blocks, k, Hq, Hkv):
    """Block-causal models (last sentence of the caption of Fig. 3; App. A.2):
    the packed call for block k takes the cache of the blocks before it as its
    context -- a view of the sequence's cache, no copy -- and must equal the
    oracle that masks the whole sequence block-causally."""
    r = np.random.default_rng(n_blocks * 10 + k)
    d = 128
    T = n_blocks * L
    k_seq, v_seq = bf16(r, B, T, Hkv, d), bf16(r, B, T, Hkv, d)
    q, kb, vb = bf16(r, B, N, L, Hq, d), bf16(r, B, N, L, Hkv, d), bf16(r, B, N, L, Hkv, d)
    ks_dev, vs_dev = k_seq.cuda(), v_seq.cuda()
    if B == 1 and k > 0:  # a prefix of the cache is contiguous: pass the view itself
        kp, vp = ks_dev[:, :k * L], vs_dev[:, :k * L]
    else:
        kp, vp = (ks_dev[:, :k * L].contiguous(), vs_dev[:, :k * L].contiguous()) if k else (None, None)
    out = spiffy.spiffy_graph_attention(q.cuda(), kp, vp, kb.cuda(), vb.cuda(), kernel=spiffy.ATTN_TCGEN05)
    torch.cuda.synchronize()
    f = lambda t: t.float().numpy()
    want = full_mask.blockwise_causal_attention(f(q), f(k_seq), f(v_seq), f(kb), f(vb), k)
    assert np.abs(out.float().cpu().numpy() - want).max() <= G.TOL["bf16"]
