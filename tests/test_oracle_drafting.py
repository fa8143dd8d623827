"""Pins of the drafting/pruning oracle (Sec. 4.4.2, Sec. 4.4.4): it must agree
with what the paper and the mathematics fix, not with itself."""
import itertools

import numpy as np
import pytest

import oracle
from oracle import drafting

MASK = 15


def case(seed, B=2, L=6, V=16, p_unmasked=0.3):
    r = np.random.default_rng(seed)
    logits = (r.standard_normal((B, L, V)) * 2).astype(np.float32)
    logits[..., MASK] = -30.0  # the mask token is never a candidate
    state = np.where(r.random((B, L)) < p_unmasked, r.integers(0, V - 1, (B, L)), MASK).astype(np.int32)
    state[:, 0] = MASK
    return logits, state


def test_first_rank_formulas_reproduce_the_next_step_of_verification():
    """The draft {(0,0)} is the block after one top-1 step, {(0,0),(1,0)} after one
    top-2 step (Sec. 4.4.2: drafts are built from the target distribution that
    Algorithm 1 unmasks from)."""
    for seed in range(20):
        logits, state = case(seed)
        B, L, V = logits.shape
        d = drafting.draft_blocks(logits, state, MASK, [[(0, 0)], [(0, 0), (1, 0)]], [[1], []], 2, 1)
        for S, node in ((1, 1), (2, 2)):
            dec = oracle.unmask_decide(logits[:, None], state[:, None], MASK, oracle.RULE_TOPS, top_s=S)
            for b in range(B):
                if (state[b] == MASK).sum() >= S:
                    assert np.array_equal(d.tokens[b, node], dec.next_tokens[b, 0]), (seed, S)
        assert np.array_equal(d.tokens[:, 0], state)


def test_ranks_and_candidates_by_brute_force():
    for seed in range(10):
        logits, state = case(100 + seed, L=5, V=8 + 8)
        d = drafting.draft_blocks(logits, state, MASK, [[(0, 0)]], [[]], 1, 3)
        for b in range(logits.shape[0]):
            x = logits[b].astype(np.float64)
            p = np.exp(x) / np.exp(x).sum(axis=1, keepdims=True)  # naive softmax, small values
            masked = [l for l in range(x.shape[0]) if state[b, l] == MASK]
            # every (probability, position) pair, sorted: the first occurrence of each position ranks it
            seen = []
            for pr, l in sorted(((-p[l].max(), l) for l in masked)):
                seen.append(l)
            assert [int(d.position_rank[b, l]) for l in seen] == list(range(len(seen)))
            assert all(d.position_rank[b, l] == -1 for l in range(x.shape[0]) if l not in masked)
            for l in masked:
                top = np.argsort(-p[l], kind="stable")[:3]
                assert d.cand_tok[b, l].tolist() == top.tolist()
                np.testing.assert_allclose(d.cand_prob[b, l], p[l][top], rtol=1e-12)


def test_geometric_mean_scores_closed_forms():
    # every masked row has the same two-peak shape: probabilities are known in closed form
    L, V = 4, 16
    logits = np.full((1, L, V), -40.0, dtype=np.float32)
    state = np.full((1, L), MASK, dtype=np.int32)
    pa = [0.9, 0.8, 0.6, 0.5]
    for l in range(L):
        logits[0, l, 3] = np.log(pa[l])
        logits[0, l, 7] = np.log(1.0 - pa[l])
    formulas = [[(0, 0)], [(0, 0), (1, 0)], [(0, 0), (1, 1)], [(0, 0), (1, 0), (2, 0)]]
    children = [[1, 2], [3], [], []]
    d = drafting.draft_blocks(logits, state, MASK, formulas, children, 4, 2)
    loc = [0.9, (0.9 * 0.8) ** 0.5, (0.9 * 0.2) ** 0.5, (0.9 * 0.8 * 0.6) ** (1 / 3)]
    np.testing.assert_allclose(d.local[0], loc, rtol=1e-6)
    want = [(loc[0] * (loc[1] * loc[2]) ** 0.5) ** 0.5, (loc[1] * loc[3]) ** 0.5, loc[2], loc[3]]
    np.testing.assert_allclose(d.score[0], want, rtol=1e-6)
    # tokens: rank-0 position is 0 (p = 0.9), rank 1 is position 1; vocabulary rank 1 there is token 7
    assert d.tokens[0, 3].tolist() == [3, 7, MASK, MASK]
    assert d.tokens[0, 4].tolist() == [3, 3, 3, MASK]
    # parents: node 0 = current block; formula sets by strict inclusion
    off, idx = d.parent_off[0], d.parent_idx[0]
    parents = [idx[off[c]:off[c + 1]].tolist() for c in range(5)]
    assert parents == [[], [0], [0, 1], [0, 1], [0, 1, 2]]


def test_relabelling_the_vocabulary_relabels_the_drafts():
    logits, state = case(7, B=1, L=6, V=16, p_unmasked=0.0)
    perm = np.random.default_rng(1).permutation(MASK)  # the mask id stays
    perm = np.concatenate([perm, [MASK]])
    formulas = [[(0, 0)], [(1, 1)], [(0, 0), (2, 2)]]
    a = drafting.draft_blocks(logits, state, MASK, formulas, [[2], [], []], 3, 3)
    b = drafting.draft_blocks(logits[..., np.argsort(perm)], state, MASK, formulas, [[2], [], []], 3, 3)
    m = a.tokens != MASK
    assert np.array_equal(perm[a.tokens[m]], b.tokens[m]) and np.array_equal(a.tokens == MASK, b.tokens == MASK)
    np.testing.assert_allclose(a.score, b.score, rtol=1e-12)


def test_pruning_keeps_the_best_by_brute_force_and_skips_unbuildable_formulas():
    for seed in range(10):
        logits, state = case(200 + seed, B=1, L=5, V=16, p_unmasked=0.4)
        n_masked = int((state == MASK).sum())
        formulas = [[(i, j)] for i in range(4) for j in range(2)] + [[(0, 0), (1, 0)], [(0, 0), (1, 0), (4, 1)]]
        children = [[] for _ in formulas]
        children[0] = [8]
        children[8] = [9]
        for budget in (1, 3, 6):
            d = drafting.draft_blocks(logits, state, MASK, formulas, children, budget, 2)
            ok = [q for q, f in enumerate(formulas) if all(i < n_masked for i, _ in f)]
            assert all(np.isneginf(d.score[0, q]) for q in range(len(formulas)) if q not in ok)
            # brute force: the subset of size min(budget, |ok|) with the largest score sum, ties to low indices
            size = min(budget, len(ok))
            best = max(itertools.combinations(ok, size),
                       key=lambda c: (sorted((d.score[0, q] for q in c), reverse=True), [-q for q in c]))
            assert d.kept[0, :size].tolist() == sorted(best)
            assert all(d.kept[0, size:] == -1)
