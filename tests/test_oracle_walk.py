"""Pins of the acceptance-walk oracle (Algorithm 1 step 5; graph of Sec. 4.4.1)
against brute-force searches on tiny random graphs."""
import numpy as np

import oracle
from oracle import toy

MASK = 7


def random_graph(rng, N, L, vocab=4, p_follow=0.6):
    """Tiny random draft graph plus a random 'decision' (top_tok, bits) per
    node.  With probability p_follow a new node is made equal to next(a) of an
    earlier node a, so that acceptances do happen."""
    states = [np.where(rng.random(L) < 0.3, rng.integers(0, vocab, L), MASK).astype(np.int32)]
    top, bits = [], []

    def decision(s):
        t = np.where(s == MASK, rng.integers(0, vocab, L), s).astype(np.int32)
        masked = np.flatnonzero(s == MASK)
        b = 0
        if len(masked):
            k = rng.integers(1, min(3, len(masked)) + 1)
            for l in rng.choice(masked, size=k, replace=False):
                b |= 1 << int(l)
        return t, b

    t, b = decision(states[0])
    top.append(t)
    bits.append(b)
    while len(states) < N:
        a = int(rng.integers(0, len(states)))
        sel = ((bits[a] >> np.arange(L)) & 1).astype(bool)
        s = np.where(sel, top[a], states[a]).astype(np.int32)
        if rng.random() > p_follow:
            free = np.flatnonzero(s != MASK)
            if len(free):
                s[rng.choice(free)] = rng.integers(0, vocab)
        states.append(s)
        t, b = decision(s)
        top.append(t)
        bits.append(b)
    # topological order: by number of unmasked tokens (stable)
    order = np.argsort([np.sum(s != MASK) for s in states], kind="stable")
    if order[0] != 0:  # keep the true block first
        order = np.concatenate([[0], order[order != 0]])
    states = np.asarray(states)[order]
    top = np.asarray(top)[order]
    bits = np.asarray(bits, dtype=np.uint64)[order]
    return states, top, bits


def next_states(states, top, bits):
    L = states.shape[1]
    sel = ((bits[:, None] >> np.arange(L, dtype=np.uint64)) & np.uint64(1)).astype(bool)
    return np.where(sel, top, states).astype(np.int32)


def brute_force_paths(states, nxt, bits, children):
    """Every root-started path whose hops all satisfy state(m) == next(cur)."""
    paths = []

    def dfs(path):
        cur = path[-1]
        ext = []
        if bits[cur] != 0:
            ext = [m for m in children(cur) if np.array_equal(states[m], nxt[cur])]
        if not ext:
            paths.append(list(path))
        for m in ext:
            dfs(path + [m])

    dfs([0])
    return paths


def run_oracle(states, off, idx, nxt, bits):
    o, i = toy.pad_parent_lists(off, idx)
    return oracle.accept_walk(states[None], o, i, nxt[None], bits[None])


def test_walk_equals_brute_force_over_all_paths():
    rng = np.random.default_rng(0)
    deep = 0
    for trial in range(1500):
        N = int(rng.integers(1, 9))
        L = int(rng.integers(1, 7))
        states, top, bits = random_graph(rng, N, L)
        off, idx = toy.parent_lists(states, MASK)
        nxt = next_states(states, top, bits)
        w = run_oracle(states, off, idx, nxt, bits)
        kids = lambda a: [m for m in range(N) if a in idx[off[m]:off[m + 1]]]
        paths = brute_force_paths(states, nxt, bits, kids)
        # greedy walk = lexicographically first maximal path
        first = min(paths)
        got = [int(v) for v in w.path[0] if v >= 0]
        assert got == first
        assert w.accepted_node[0] == first[-1] and w.n_accepted[0] == len(first) - 1
        assert np.array_equal(w.next_block[0], nxt[first[-1]])
        # with unique states the maximal path is unique, hence the deepest
        if len({tuple(s) for s in states}) == N:
            assert len(paths) == 1
        deep += len(first) > 2
    assert deep > 50  # the generator does exercise multi-hop accepts


def test_complete_parent_lists_make_the_lists_redundant():
    """A state equal to next(cur) is by definition a structural child of cur
    (Eqs. draft-graph-1..3), so with complete lists a scan over all nodes gives
    the same walk; with an incomplete list it does not."""
    rng = np.random.default_rng(1)
    differ = 0
    for trial in range(600):
        N = int(rng.integers(2, 9))
        L = int(rng.integers(2, 7))
        states, top, bits = random_graph(rng, N, L)
        if len({tuple(s) for s in states}) != N:
            continue
        off, idx = toy.parent_lists(states, MASK)
        nxt = next_states(states, top, bits)
        w = run_oracle(states, off, idx, nxt, bits)
        free = brute_force_paths(states, nxt, bits, lambda a: range(N))
        # next(cur) has strictly more unmasked tokens unless top_tok == MASK,
        # which random_graph never draws
        assert [int(v) for v in w.path[0] if v >= 0] == min(free)
        if w.n_accepted[0] > 0:
            # drop the edge that carried the first hop
            m = int(w.path[0, 1])
            keep = [(c, a) for c in range(N) for a in idx[off[c]:off[c + 1]] if (c, a) != (m, 0)]
            off2 = np.zeros(N + 1, dtype=np.int32)
            idx2 = []
            for c in range(N):
                idx2 += [a for (cc, a) in keep if cc == c]
                off2[c + 1] = len(idx2)
            w2 = run_oracle(states, off2, np.asarray(idx2, dtype=np.int32), nxt, bits)
            assert w2.n_accepted[0] == 0 and w2.accepted_node[0] == 0
            differ += 1
    assert differ > 50


def test_hand_built_diamond():
    """Root R, A = R+{a}, B = R+{b}, C = R+{a,b} with parents A and B (and R):
    the multiple-parent shape of Sec. 4.4.1."""
    M = MASK
    R = [M, M, M, 5]
    A = [1, M, M, 5]
    Bn = [M, 2, M, 5]
    C = [1, 2, M, 5]
    states = np.asarray([R, A, Bn, C], dtype=np.int32)
    off, idx = toy.parent_lists(states, M)
    assert [list(idx[off[m]:off[m + 1]]) for m in range(4)] == [[], [0], [0], [0, 1, 2]]
    top = np.asarray([[1, 2, 9, 5], [1, 2, 9, 5], [1, 2, 9, 5], [1, 2, 3, 5]], dtype=np.int32)

    def walk(bits):
        b = np.asarray(bits, dtype=np.uint64)
        return run_oracle(states, off, idx, next_states(states, top, b), b)

    w = walk([0b001, 0b010, 0b001, 0b100])        # R->A->C, then C has no child
    assert list(w.path[0]) == [0, 1, 3, -1] and w.n_accepted[0] == 2
    assert list(w.next_block[0]) == [1, 2, 3, 5]
    w = walk([0b011, 0b010, 0b001, 0b100])        # R unmasks two at once: R->C
    assert list(w.path[0]) == [0, 3, -1, -1] and w.accepted_node[0] == 3
    w = walk([0b100, 0b010, 0b001, 0b100])        # next(R) matches no draft
    assert list(w.path[0]) == [0, -1, -1, -1] and list(w.next_block[0]) == [M, M, 9, 5]
    w = walk([0b010, 0b010, 0b001, 0b100])        # R->B->C
    assert list(w.path[0]) == [0, 2, 3, -1]


def test_structural_validator():
    M = MASK
    assert toy.is_structural_parent([M, M, 1], [M, 2, 1], M)
    assert not toy.is_structural_parent([M, M, 1], [M, 2, 3], M)   # disagrees on a token
    assert not toy.is_structural_parent([M, 2, 1], [M, 2, 1], M)   # not a strict superset
    assert not toy.is_structural_parent([M, 2, 1], [M, M, 1], M)   # wrong direction
    assert not toy.is_structural_parent([4, M, M], [M, 2, 1], M)   # not a subset
