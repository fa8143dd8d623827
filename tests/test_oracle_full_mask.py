"""Pins of the full-sequence mask oracle (Fig. 3 caption, App. A.2)."""
import numpy as np
import torch

import oracle
from oracle import full_mask


def case(seed, B=2, N=3, L=4, P=5, S=6, Hq=4, Hkv=2, d=8):
    r = np.random.default_rng(seed)
    f = lambda *s: r.standard_normal(s).astype(np.float32).astype(np.float64)  # float32-representable
    return dict(q_nodes=f(B, N, L, Hq, d), q_suffix=f(B, S, Hq, d), k_prefix=f(B, P, Hkv, d),
                v_prefix=f(B, P, Hkv, d), k_suffix=f(B, S, Hkv, d), v_suffix=f(B, S, Hkv, d),
                k_block=f(B, N, L, Hkv, d), v_block=f(B, N, L, Hkv, d))


def test_node_rows_are_packed_attention_with_the_suffix_as_context():
    """For the nodes the suffix is one more piece of shared context (R2): the
    C++ packed-attention oracle on [prefix ; suffix] must give the same rows."""
    for seed, kw in ((0, {}), (1, dict(N=5, L=3, P=0, S=7, Hq=6, Hkv=3)), (2, dict(N=1, S=2))):
        c = case(seed, **kw)
        nodes, _ = full_mask.full_sequence_attention(**c)
        ctx_k = np.concatenate([c["k_prefix"], c["k_suffix"]], 1)
        ctx_v = np.concatenate([c["v_prefix"], c["v_suffix"]], 1)
        want = oracle.graph_attention(c["q_nodes"], ctx_k, ctx_v, c["k_block"], c["v_block"])
        np.testing.assert_allclose(nodes, want, atol=1e-12)


def test_suffix_rows_are_plain_attention_over_the_true_sequence():
    c = case(3, Hq=4, Hkv=4)
    _, suffix = full_mask.full_sequence_attention(**c)
    keys = np.concatenate([c["k_prefix"], c["k_block"][:, 0], c["k_suffix"]], 1)
    vals = np.concatenate([c["v_prefix"], c["v_block"][:, 0], c["v_suffix"]], 1)
    t = lambda a: torch.from_numpy(a).permute(0, 2, 1, 3)  # [B,H,rows,d]
    want = torch.nn.functional.scaled_dot_product_attention(t(c["q_suffix"]), t(keys), t(vals))
    np.testing.assert_allclose(suffix, want.permute(0, 2, 1, 3).numpy(), atol=1e-12)


def test_drafts_do_not_see_the_true_block_and_the_true_rows_see_no_draft():
    c = case(4)
    nodes, suffix = full_mask.full_sequence_attention(**c)
    c2 = {k: v.copy() for k, v in c.items()}
    c2["k_block"][:, 0] += 3.0       # change the true block's keys and values
    c2["v_block"][:, 0] -= 2.0
    nodes2, suffix2 = full_mask.full_sequence_attention(**c2)
    np.testing.assert_allclose(nodes2[:, 1:], nodes[:, 1:], atol=1e-12)   # drafts unchanged
    assert np.abs(nodes2[:, 0] - nodes[:, 0]).max() > 1e-3                 # true rows changed
    assert np.abs(suffix2 - suffix).max() > 1e-3
    c3 = {k: v.copy() for k, v in c.items()}
    c3["k_block"][:, 1:] += 3.0      # change the drafts
    nodes3, suffix3 = full_mask.full_sequence_attention(**c3)
    np.testing.assert_allclose(nodes3[:, 0], nodes[:, 0], atol=1e-12)
    np.testing.assert_allclose(suffix3, suffix, atol=1e-12)


def test_blockwise_causal_rows_equal_library_attention_on_the_sequence_with_that_node_in_place():
    """Block-causal models (last sentence of the caption of Fig. 3; App. A.2):
    what a node gets in the packed call is what its block would get if it stood
    in the sequence in place of the block being decoded and the model ran with
    its ordinary block-causal mask -- computed here by torch's attention."""
    r = np.random.default_rng(9)
    B, N, L, Hq, Hkv, d, n_blocks, k = 2, 3, 4, 4, 2, 8, 5, 2
    f = lambda *s: r.standard_normal(s).astype(np.float32).astype(np.float64)
    T = n_blocks * L
    q_seq, k_seq, v_seq = f(B, T, Hq, d), f(B, T, Hkv, d), f(B, T, Hkv, d)
    q_nodes, k_block, v_block = f(B, N, L, Hq, d), f(B, N, L, Hkv, d), f(B, N, L, Hkv, d)
    got = full_mask.blockwise_causal_attention(q_nodes, k_seq, v_seq, k_block, v_block, k)
    blk = np.arange(T) // L
    causal = torch.from_numpy(blk[:, None] >= blk[None, :])  # row block >= key block
    t = lambda a: torch.from_numpy(a).permute(0, 2, 1, 3)
    for n in range(N):
        qs, ks, vs = q_seq.copy(), k_seq.copy(), v_seq.copy()
        qs[:, k * L:(k + 1) * L] = q_nodes[:, n]
        ks[:, k * L:(k + 1) * L] = k_block[:, n]
        vs[:, k * L:(k + 1) * L] = v_block[:, n]
        rep = Hq // Hkv
        want = torch.nn.functional.scaled_dot_product_attention(
            t(qs), t(ks).repeat_interleave(rep, 1), t(vs).repeat_interleave(rep, 1), attn_mask=causal)
        want = want.permute(0, 2, 1, 3).numpy()[:, k * L:(k + 1) * L]
        np.testing.assert_allclose(got[:, n], want, atol=1e-12)
    # later blocks are invisible: changing them changes nothing
    k2, v2 = k_seq.copy(), v_seq.copy()
    k2[:, k * L:] += 5.0
    v2[:, k * L:] -= 5.0
    np.testing.assert_allclose(full_mask.blockwise_causal_attention(q_nodes, k2, v2, k_block, v_block, k), got,
                               atol=1e-12)
    # and it is the packed-attention oracle with the earlier blocks as context
    want = oracle.graph_attention(q_nodes, k_seq[:, :k * L], v_seq[:, :k * L], k_block, v_block)
    np.testing.assert_allclose(got, want, atol=1e-12)
