"""CPU oracle of Spiffy's offline draft-graph calibration -- TEST INFRASTRUCTURE ONLY.

Plain Python written from Algorithm 2 and App. D.1 in the paper's order, brute
force where the paper says brute force.  Nothing in the product package imports
this module and it imports nothing from the product.

  Part 1  rewind a recorded plain-decoding run: for every timestep t and every
          look-ahead level k = 1..lookahead, the tokens that plain decoding
          unmasks k steps after t, each named by its (token position rank i,
          vocabulary rank j) under the distribution at t (Eqs. i-select,
          j-select; ranks start at 0 here).
  Part 2  per level k, a node is the union of the (i, j) sets of levels <= k;
          the three most frequent nodes of every level form the candidate
          graph G, with an edge from p to q whenever p is a strict subset of q.
  Part 3  among all D-node subsets of G that are connected (App. D.1: a node is
          connected if its level is 1 or 2 or one of its parents is in the
          subset), the one with the largest sum of node frequencies.

Readings: ties in frequency go to the lower level, then to the lexicographically
smaller sorted (i, j) list; the "top in-edges" of Part 2 add no edge beyond the
subset edges and are not modelled; a token whose rank cannot be named (its
position was already unmasked at t, or its vocabulary rank is beyond max_rank)
ends the look-ahead of that timestep.

Pins (tests/test_oracle_calibration.py): a three-position run worked by hand
(ranks, sequences, counts, ties); a nine-node graph whose most frequent node has
no parent (App. D.1) for D = 1..9; under top-S decoding the level-1 node is the
S most confident positions with their best tokens; the closed loop on the toy
model (the calibrated graph is accepted, a graph of deep ranks is not).
"""
from __future__ import annotations

import itertools
from collections import Counter

import numpy as np


def ranks_at(logits, state, mask_id):
    """Token position rank of every masked position and the vocabulary order of
    every position under one distribution (Sec. 4.4.2)."""
    logits = np.asarray(logits, dtype=np.float64)
    L, V = logits.shape
    masked = [l for l in range(L) if state[l] == mask_id]
    conf = {l: 1.0 / np.exp(logits[l] - logits[l].max()).sum() for l in masked}
    order = sorted(masked, key=lambda l: (-conf[l], l))
    pos_rank = {l: i for i, l in enumerate(order)}
    vocab_order = {l: sorted(range(V), key=lambda v: (-logits[l, v], v)) for l in masked}
    return pos_rank, vocab_order


def rewind(states, logits, mask_id, lookahead, max_rank):
    """Part 1 for one run.  states: the T+1 blocks visited by plain decoding,
    logits[t]: the distribution [L, V] plain decoding unmasked from at step t.
    Returns one sequence per timestep: [(k, frozenset{(i, j)})], k = 1.."""
    out = []
    T = len(states) - 1
    for t in range(T):
        pos_rank, vocab_order = ranks_at(logits[t], states[t], mask_id)
        seq = []
        for k in range(1, lookahead + 1):
            if t + k > T:
                break
            new = [l for l in range(len(states[t])) if states[t + k][l] != states[t + k - 1][l]]
            pairs = set()
            for l in new:
                if l not in pos_rank:
                    pairs = None
                    break
                j = vocab_order[l].index(int(states[t + k][l]))
                if j >= max_rank:
                    pairs = None
                    break
                pairs.add((pos_rank[l], j))
            if pairs is None:
                break
            seq.append((k, frozenset(pairs)))
        out.append(seq)
    return out


def _key(node):
    return sorted(node)


def candidate_graph(sequences, lookahead, top=3):
    """Part 2.  Returns a list of (level, node, count), level by level, the
    `top` most frequent nodes of each level."""
    graph = []
    for k in range(1, lookahead + 1):
        count = Counter()
        for seq in sequences:
            if any(level == k for level, _ in seq):
                node = frozenset().union(*[s for level, s in seq if level <= k])
                count[node] += 1
        best = sorted(count.items(), key=lambda kv: (-kv[1], _key(kv[0])))[:top]
        graph += [(k, node, c) for node, c in best]
    return graph


def is_connected(graph, subset):
    """App. D.1: every node of the subset has level 1 or 2 or a parent (a
    strict subset) inside the subset."""
    for a in subset:
        level, node, _ = graph[a]
        if level <= 2:
            continue
        if not any(graph[b][1] < node for b in subset if b != a):
            return False
    return True


def best_subgraph(graph, D):
    """Part 3 by brute force over every D-subset (indices into graph, ascending)."""
    best, best_score = None, -1
    for subset in itertools.combinations(range(len(graph)), min(D, len(graph))):
        if not is_connected(graph, subset):
            continue
        score = sum(graph[a][2] for a in subset)
        if score > best_score:  # combinations come in lexicographic order: the first maximum stays
            best, best_score = subset, score
    return list(best) if best is not None else [], best_score


def formulas_of(graph, subset):
    """The chosen nodes as draft formulas (sorted (i, j) lists) with each
    formula's children (the chosen strict supersets), parents first."""
    nodes = [graph[a][1] for a in subset]
    order = sorted(range(len(nodes)), key=lambda a: (len(nodes[a]), _key(nodes[a])))
    nodes = [nodes[a] for a in order]
    formulas = [_key(n) for n in nodes]
    children = [[c for c in range(len(nodes)) if nodes[q] < nodes[c]] for q in range(len(nodes))]
    return formulas, children
