"""Pins of the attention oracle (Sec. 4.3, mask of Fig. 3) against things the
paper and the mathematics fix: probability rows, an explicit-mask formulation
of the packed sequence, closed forms, symmetries and a library SDPA."""
import numpy as np
import pytest
import torch

import oracle


def rand_case(seed, B=2, N=3, L=4, P=5, Hq=4, Hkv=2, d=8):
    r = np.random.default_rng(seed)
    f = lambda *s: r.standard_normal(s).astype(np.float32)
    return dict(q=f(B, N, L, Hq, d), kp=f(B, P, Hkv, d), vp=f(B, P, Hkv, d),
                kb=f(B, N, L, Hkv, d), vb=f(B, N, L, Hkv, d))


def run(c, **kw):
    return oracle.graph_attention(c["q"], c["kp"], c["vp"], c["kb"], c["vb"], **kw)


def explicit_mask_attention(c, scale=None):
    """The packed sequence as the paper's model call sees it: one key axis
    [context ; block of node 0 ; ... ; block of node N-1] and a boolean mask
    built from the rule in Fig. 3's caption (a block sees the context and
    itself).  Generic masked attention through torch's library softmax/matmul
    in float64, heads expanded for GQA."""
    q, kp, vp, kb, vb = (torch.from_numpy(np.asarray(c[k], dtype=np.float64))
                         for k in ("q", "kp", "vp", "kb", "vb"))
    B, N, L, Hq, d = q.shape
    P, Hkv = kp.shape[1], kp.shape[2]
    rep = Hq // Hkv
    keys = torch.cat([kp, kb.reshape(B, N * L, Hkv, d)], 1).repeat_interleave(rep, dim=2)
    vals = torch.cat([vp, vb.reshape(B, N * L, Hkv, d)], 1).repeat_interleave(rep, dim=2)
    qq = q.reshape(B, N * L, Hq, d)
    mask = torch.zeros(N * L, P + N * L, dtype=torch.bool)
    mask[:, :P] = True
    for n in range(N):
        mask[n * L:(n + 1) * L, P + n * L:P + (n + 1) * L] = True
    s = torch.einsum("bqhd,bkhd->bhqk", qq, keys) * (scale or 1.0 / np.sqrt(d))
    s = s.masked_fill(~mask, float("-inf"))
    p = torch.softmax(s, dim=-1)
    o = torch.einsum("bhqk,bkhd->bqhd", p, vals)
    return o.reshape(B, N, L, Hq, d).numpy()


@pytest.mark.parametrize("seed", range(3))
def test_probability_rows(seed):
    c = rand_case(seed)
    _, probs = run(c, return_probs=True)
    assert np.all(probs >= 0)
    np.testing.assert_allclose(probs.sum(-1), 1.0, atol=1e-12)


@pytest.mark.parametrize("shape", [dict(), dict(Hq=6, Hkv=2, N=5, L=3, P=7),
                                   dict(Hq=3, Hkv=3, N=2, L=5, P=1),
                                   dict(Hq=8, Hkv=1, N=4, L=2, P=9, d=16)])
def test_matches_explicit_mask_formulation(shape):
    c = rand_case(11, **shape)
    np.testing.assert_allclose(run(c), explicit_mask_attention(c), atol=1e-12, rtol=0)


def test_custom_scale_is_applied_to_scores():
    c = rand_case(12)
    np.testing.assert_allclose(run(c, scale=0.37), explicit_mask_attention(c, scale=0.37),
                               atol=1e-12, rtol=0)


def test_packing_invariance_each_node_alone():
    """A draft block's output must be what the same block gets when it is the
    only block in the call (the exactness condition of App. A.2)."""
    c = rand_case(5, N=4)
    packed = run(c)
    for n in range(4):
        alone = oracle.graph_attention(c["q"][:, n:n + 1], c["kp"], c["vp"],
                                       c["kb"][:, n:n + 1], c["vb"][:, n:n + 1])
        assert np.array_equal(alone[:, 0], packed[:, n])


def test_other_nodes_blocks_do_not_leak():
    c = rand_case(6, N=3)
    base = run(c)
    c2 = {k: v.copy() for k, v in c.items()}
    c2["kb"][:, 1] += 3.0
    c2["vb"][:, 1] -= 2.0
    out = run(c2)
    assert np.array_equal(out[:, 0], base[:, 0]) and np.array_equal(out[:, 2], base[:, 2])
    assert not np.allclose(out[:, 1], base[:, 1])


def test_sdpa_library_p0_single_node():
    """N = 1, P = 0 is textbook bidirectional attention."""
    c = rand_case(7, B=2, N=1, L=6, P=0, Hq=3, Hkv=3, d=16)
    q = torch.from_numpy(c["q"][:, 0].astype(np.float64)).permute(0, 2, 1, 3)
    k = torch.from_numpy(c["kb"][:, 0].astype(np.float64)).permute(0, 2, 1, 3)
    v = torch.from_numpy(c["vb"][:, 0].astype(np.float64)).permute(0, 2, 1, 3)
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v).permute(0, 2, 1, 3)
    np.testing.assert_allclose(run(c)[:, 0], ref.numpy(), atol=1e-12, rtol=0)


def test_sdpa_library_context_plus_block_gqa():
    c = rand_case(8, B=1, N=2, L=3, P=10, Hq=4, Hkv=2, d=8)
    out = run(c)
    for n in range(2):
        q = torch.from_numpy(c["q"][:, n].astype(np.float64)).permute(0, 2, 1, 3)
        k = torch.from_numpy(np.concatenate([c["kp"], c["kb"][:, n]], 1).astype(np.float64))
        v = torch.from_numpy(np.concatenate([c["vp"], c["vb"][:, n]], 1).astype(np.float64))
        k = k.repeat_interleave(2, dim=2).permute(0, 2, 1, 3)
        v = v.repeat_interleave(2, dim=2).permute(0, 2, 1, 3)
        ref = torch.nn.functional.scaled_dot_product_attention(q, k, v).permute(0, 2, 1, 3)
        np.testing.assert_allclose(out[:, n], ref.numpy(), atol=1e-12, rtol=0)


def test_equal_values_give_that_value():
    c = rand_case(1)
    row = np.arange(8, dtype=np.float32) - 3.0
    c["vp"][:] = row
    c["vb"][:] = row
    np.testing.assert_allclose(run(c), np.broadcast_to(row, run(c).shape), atol=1e-13)


def test_equal_keys_give_mean_of_values():
    c = rand_case(2, Hq=2, Hkv=2)
    c["kp"][:] = 0.25
    c["kb"][:] = 0.25
    out = run(c)
    B, N, L, Hq, d = c["q"].shape
    for n in range(N):
        mean = np.concatenate([c["vp"], c["vb"][:, n]], 1).astype(np.float64).mean(1)
        np.testing.assert_allclose(out[:, n], np.broadcast_to(mean[:, None], (B, L, Hq, d)),
                                   atol=1e-13)


def test_dominant_key_selects_its_value():
    c = rand_case(3, B=1, Hq=2, Hkv=2, d=8)
    c["q"][:] = 0.0
    c["q"][..., 0] = 1.0
    c["kp"][:] = 0.0
    c["kb"][:] = 0.0
    c["kb"][0, 1, 2, :, 0] = 400.0  # node 1's own key r=2 wins for node 1 only
    out = run(c)
    np.testing.assert_allclose(out[0, 1], np.broadcast_to(c["vb"][0, 1, 2], out[0, 1].shape),
                               atol=1e-12)
    assert not np.allclose(out[0, 0], np.broadcast_to(c["vb"][0, 1, 2], out[0, 0].shape))


def test_context_permutation_and_node_permutation():
    c = rand_case(4, N=4, P=9)
    base = run(c)
    perm = np.random.default_rng(0).permutation(9)
    c2 = dict(c, kp=c["kp"][:, perm], vp=c["vp"][:, perm])
    np.testing.assert_allclose(run(c2), base, atol=1e-13)
    nperm = np.array([2, 0, 3, 1])
    c3 = dict(c, q=c["q"][:, nperm], kb=c["kb"][:, nperm], vb=c["vb"][:, nperm])
    assert np.array_equal(run(c3), base[:, nperm])


def test_value_linearity_and_key_shift():
    """Linear in V; adding a constant vector to all keys of one query's key set
    shifts every score of that query equally, so nothing changes."""
    c = rand_case(9, Hq=2, Hkv=2)
    base = run(c)
    c2 = dict(c, vp=c["vp"] * 2, vb=c["vb"] * 2)
    np.testing.assert_allclose(run(c2), 2 * base, atol=1e-12)
    shift = np.float32(0.5)
    c3 = dict(c, kp=c["kp"] + shift, kb=c["kb"] + shift)
    np.testing.assert_allclose(run(c3), base, atol=1e-5)
