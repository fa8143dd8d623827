"""GPU parity of spiffy_graph_attention (Sec. 4.3, mask of Fig. 3) with the CPU
oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2509_18085_b200 import spiffy
from paper_2509_18085_b200 import workloads as W

import gpu_util as G

pytestmark = pytest.mark.gpu

KERNELS = [spiffy.ATTN_SIMT, spiffy.ATTN_AUTO, spiffy.ATTN_TCGEN05]


def tc_takes(cfg):
    """The tensor-core kernel takes bf16 inputs with head dimension 128."""
    return cfg.dtype == "bf16" and cfg.head_dim == 128 and cfg.n_q_heads // cfg.n_kv_heads <= 128


def run_or_expect_unsupported(w, kernel, **kw):
    """Forcing the tensor-core kernel on a shape it does not take must be
    refused with a status code, never silently served by another kernel."""
    if kernel == spiffy.ATTN_TCGEN05 and not tc_takes(w.cfg):
        with pytest.raises(spiffy.SpiffyError) as e:
            G.gpu_attention(w, kernel, **kw)
        assert e.value.status == spiffy.EUNSUPPORTED
        return None
    return G.gpu_attention(w, kernel, **kw)


def oracle_attention(w, scale=None):
    return oracle.graph_attention(w.q, w.k_prefix, w.v_prefix, w.k_block, w.v_block, scale=scale)


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("index,n_nodes", [(1, None), (2, None), (3, None), (5, 1), (5, 2), (5, 4), (5, 8),
                                           (5, 16), (5, 32), (5, 64)])
def test_configs(index, n_nodes, kernel):
    cfg = W.config(index, n_nodes)
    w = W.make(cfg, W.seed_for(index, 0), decision=False)
    got = run_or_expect_unsupported(w, kernel)
    if got is None:
        return
    want = oracle_attention(w)
    assert np.max(np.abs(got - want)) <= G.TOL[cfg.dtype]
    if cfg.dtype == "bf16":
        # the result is rounded once to bf16: the error is that rounding
        assert np.sqrt(np.mean((got - want) ** 2)) < 2e-3


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", [
    dict(batch=2, n_nodes=3, block_len=5, prefix_len=127, n_q_heads=6, n_kv_heads=2, head_dim=64),
    dict(batch=1, n_nodes=2, block_len=64, prefix_len=33, n_q_heads=2, n_kv_heads=1, head_dim=128),
    dict(batch=3, n_nodes=1, block_len=1, prefix_len=0, n_q_heads=1, n_kv_heads=1, head_dim=64),
    dict(batch=1, n_nodes=5, block_len=16, prefix_len=0, n_q_heads=4, n_kv_heads=4, head_dim=128),
    dict(batch=2, n_nodes=7, block_len=32, prefix_len=300, n_q_heads=8, n_kv_heads=2, head_dim=128),
    dict(batch=1, n_nodes=9, block_len=8, prefix_len=1000, n_q_heads=3, n_kv_heads=3, head_dim=128),
    # query-head groups of 16, 128 and 3 per kv head: 8, 1 and 42 (node, position) pairs per M-tile
    dict(batch=1, n_nodes=3, block_len=10, prefix_len=50, n_q_heads=16, n_kv_heads=1, head_dim=128),
    dict(batch=1, n_nodes=2, block_len=3, prefix_len=20, n_q_heads=128, n_kv_heads=1, head_dim=128),
    dict(batch=2, n_nodes=4, block_len=12, prefix_len=129, n_q_heads=6, n_kv_heads=2, head_dim=128),
    # 26 nodes of 5 positions under one M-tile: their block keys need two key tiles
    dict(batch=1, n_nodes=30, block_len=5, prefix_len=70, n_q_heads=2, n_kv_heads=2, head_dim=128),
    # enough M-tiles for the two-tiles-per-CTA variant; an odd tile count leaves one CTA half empty
    dict(batch=3, n_nodes=9, block_len=32, prefix_len=300, n_q_heads=32, n_kv_heads=32, head_dim=128),
    dict(batch=10, n_nodes=6, block_len=16, prefix_len=130, n_q_heads=32, n_kv_heads=16, head_dim=128),
])
def test_odd_shapes(shape, dtype, kernel):
    cfg = W.Config("odd", dtype=dtype, vocab=16, rule=0, **shape)
    w = W.make(cfg, 77, decision=False)
    got = run_or_expect_unsupported(w, kernel)
    if got is None:
        return
    want = oracle_attention(w)
    assert np.max(np.abs(got - want)) <= G.TOL[dtype]


@pytest.mark.parametrize("prefix_len,n_nodes,block_len", [
    (384, 8, 32),   # 3 context tiles + 1 block tile: even, the two CTAs of a pair each finish half the columns
    (512, 8, 32),   # 5 key tiles: odd, one CTA of the pair has a tile more
    (640, 8, 32),   # 6
    (300, 4, 32),   # 4, ragged context tile, one M-tile per head
    (400, 6, 48),   # nodes of 48 positions: M-tiles with one and with two block-key tiles (odd and even in one launch)
    (257, 3, 7),    # 4 tiles, a nearly empty M-tile
])
def test_cluster_pairs_with_even_and_odd_tile_counts(prefix_len, n_nodes, block_len):
    """Few M-tiles (at most 74): the key tiles of each M-tile are split over the
    two CTAs of a cluster, which merge through each other's shared memory."""
    cfg = W.Config("pairs", dtype="bf16", vocab=16, rule=0, batch=1, n_nodes=n_nodes, block_len=block_len,
                   prefix_len=prefix_len, n_q_heads=16, n_kv_heads=16, head_dim=128)
    w = W.make(cfg, 31 + prefix_len, decision=False)
    got = G.gpu_attention(w, spiffy.ATTN_TCGEN05)
    want = oracle_attention(w)
    assert np.max(np.abs(got - want)) <= G.TOL["bf16"]
    assert np.sqrt(np.mean((got - want) ** 2)) < 2e-3


@pytest.mark.parametrize("kernel", KERNELS)
def test_custom_scale(kernel):
    cfg = W.config(2, n_nodes=2, prefix_len=200)
    w = W.make(cfg, 5, decision=False)
    got = G.gpu_attention(w, kernel, scale=0.05)
    assert np.max(np.abs(got - oracle_attention(w, scale=0.05))) <= G.TOL["bf16"]


@pytest.mark.parametrize("kernel", KERNELS)
def test_packing_invariance_on_the_gpu(kernel):
    """A draft block's rows must not depend on which other blocks are packed
    with it (App. A.2): compare the packed call with one call per node."""
    cfg = W.config(2, n_nodes=5, prefix_len=256)
    w = W.make(cfg, 9, decision=False)
    dt = torch.bfloat16
    q, kp, vp, kb, vb = (G.to_dev(a, dt) for a in (w.q, w.k_prefix, w.v_prefix, w.k_block, w.v_block))
    packed = spiffy.spiffy_graph_attention(q, kp, vp, kb, vb, kernel=kernel)
    for n in range(5):
        alone = spiffy.spiffy_graph_attention(q[:, n:n + 1].contiguous(), kp, vp,
                                              kb[:, n:n + 1].contiguous(),
                                              vb[:, n:n + 1].contiguous(), kernel=kernel)
        diff = (alone[:, 0].float() - packed[:, n].float()).abs().max().item()
        assert diff <= 2e-2
    # another node's block must not leak: change node 3's keys, others unchanged bit for bit
    kb2 = kb.clone()
    kb2[:, 3] += 1.0
    again = spiffy.spiffy_graph_attention(q, kp, vp, kb2, vb, kernel=kernel)
    keep = [0, 1, 2, 4]
    assert torch.equal(again[:, keep], packed[:, keep])
    assert not torch.equal(again[:, 3], packed[:, 3])


def test_full_size_long_batched_sampled_nodes():
    """Configuration 4 at full size (B=4, P=4096, N=32): the oracle checks a
    sample of (sequence, node) pairs one by one, using the fact that a node's
    output depends only on the context and its own block."""
    cfg = W.config(4)
    w = W.make(cfg, W.seed_for(4, 0), decision=False)
    got = G.gpu_attention(w)
    rng = np.random.default_rng(0)
    for _ in range(6):
        b, n = int(rng.integers(0, cfg.batch)), int(rng.integers(0, cfg.n_nodes))
        want = oracle.graph_attention(w.q[b:b + 1, n:n + 1], w.k_prefix[b:b + 1], w.v_prefix[b:b + 1],
                                      w.k_block[b:b + 1, n:n + 1], w.v_block[b:b + 1, n:n + 1])
        assert np.max(np.abs(got[b, n] - want[0, 0])) <= G.TOL["bf16"]
    assert np.all(np.isfinite(got))


@pytest.mark.parametrize("kernel", [spiffy.ATTN_SIMT, spiffy.ATTN_TCGEN05])
def test_peaked_scores_and_a_late_maximum(kernel):
    """Scores far from zero, and a row maximum that only shows up in the last key
    tiles: the accumulator is rescaled late (the reference maximum moves by far
    more than its slack) and probabilities are nearly one-hot."""
    cfg = W.config(2, n_nodes=3, prefix_len=700)
    w = W.make(cfg, 21, decision=False)
    w.q *= 6.0                       # scores of standard deviation 6 before the softmax
    w.k_prefix[:, 600:650] *= 3.0    # the largest scores sit late in the context ...
    w.k_block[:, 1] *= 4.0           # ... or in one node's own block
    for a in ("q", "k_prefix", "k_block"):
        setattr(w, a, W.round_to(getattr(w, a), "bf16"))
    got = G.gpu_attention(w, kernel)
    want = oracle_attention(w)
    assert np.all(np.isfinite(got))
    assert np.max(np.abs(got - want)) <= G.TOL["bf16"]
