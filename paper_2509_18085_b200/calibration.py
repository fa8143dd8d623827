"""Offline draft-graph calibration (Algorithm 2, App. D.1) -- host code.

Calibration runs once per model, offline, on recorded plain-decoding runs; the
paper does it on the CPU and so does this module.  Its result, D draft formulas
{(i, j)} with their children, is what ``spiffy.draft_graph`` uploads for
``spiffy_draft_blocks``.

    sequences = []
    for run in runs:                       # one run = states visited + the logits used at every step
        sequences += record(run.states, run.logits, mask_id, lookahead=3, max_rank=3)
    graph = build_graph(sequences, lookahead=3)
    formulas, children, score = calibrate(graph, n_drafts=10)

Ranks are zero-based: i = 0 is the most confident still-masked position, j = 0
the most probable token.  Ties: lower position, lower token id; among equally
frequent nodes the lower level, then the smaller sorted (i, j) list.
"""
from __future__ import annotations

from collections import defaultdict

import numpy as np


def record(states, logits, mask_id, lookahead, max_rank):
    """Part 1 of Algorithm 2 for one plain-decoding run.  ``states``: T+1 blocks
    [L] (int), ``logits[t]``: [L, V] the distribution unmasked from at step t.
    Returns, per timestep, the list [(k, frozenset{(i, j)})] for k = 1, 2, ...:
    the tokens unmasked k steps later, named by their ranks at step t.  The list
    of a timestep stops at the first level that cannot be named (a position
    already unmasked at t, or a vocabulary rank >= max_rank)."""
    states = [np.asarray(s) for s in states]
    T = len(states) - 1
    out = []
    for t in range(T):
        x = np.asarray(logits[t], dtype=np.float64)
        masked = states[t] == mask_id
        conf = np.where(masked, 1.0 / np.exp(x - x.max(axis=1, keepdims=True)).sum(axis=1), -np.inf)
        # position rank: confidence descending, position ascending
        order = np.lexsort((np.arange(len(conf)), -conf))
        rank = np.empty(len(conf), dtype=np.int64)
        rank[order] = np.arange(len(conf))
        seq = []
        for k in range(1, lookahead + 1):
            if t + k > T:
                break
            new = np.flatnonzero(states[t + k] != states[t + k - 1])
            if not np.all(masked[new]):
                break
            pairs = []
            for l in new:
                tok = int(states[t + k][l])
                # vocabulary rank without sorting: tokens strictly ahead, then equal ones with a lower id
                j = int((x[l] > x[l, tok]).sum() + (x[l, :tok] == x[l, tok]).sum())
                pairs.append((int(rank[l]), j))
            if any(j >= max_rank for _, j in pairs):
                break
            seq.append((k, frozenset(pairs)))
        out.append(seq)
    return out


def build_graph(sequences, lookahead, top=3):
    """Part 2: per level k the ``top`` most frequent nodes, a node being the
    union of a sequence's (i, j) sets up to level k.  Returns
    [(level, node, count)] level by level."""
    counts = [defaultdict(int) for _ in range(lookahead + 1)]
    for seq in sequences:
        node = frozenset()
        expect = 1
        for k, pairs in seq:  # levels come in order 1, 2, ...
            if k != expect or k > lookahead:
                break
            node = node | pairs
            counts[k][node] += 1
            expect += 1
    graph = []
    for k in range(1, lookahead + 1):
        ranked = sorted(counts[k].items(), key=lambda kv: (-kv[1], sorted(kv[0])))
        graph += [(k, node, c) for node, c in ranked[:top]]
    return graph


def calibrate(graph, n_drafts):
    """Part 3: the connected n_drafts-node subset of the candidate graph with the
    largest sum of frequencies (App. D.1: a node is connected if its level is 1
    or 2, or one of its strict subsets is chosen too).  Branch and bound over
    the subsets in lexicographic order; the first maximum wins.  Returns
    (formulas, children, score): formulas as sorted (i, j) lists, parents
    first; children[q] = the chosen strict supersets of formula q."""
    n = len(graph)
    D = min(n_drafts, n)
    counts = [c for _, _, c in graph]
    parents = [[b for b in range(n) if graph[b][1] < graph[a][1]] for a in range(n)]
    # best[i][r]: the largest sum of r counts among nodes i.. (an optimistic bound)
    tail = [[0] * (D + 1) for _ in range(n + 1)]
    for i in range(n - 1, -1, -1):
        rest = sorted(counts[i:], reverse=True)
        for r in range(1, D + 1):
            tail[i][r] = sum(rest[:r]) if len(rest) >= r else -1
    best = {"score": -1, "subset": None}
    chosen = []

    def connected():
        inside = set(chosen)
        return all(graph[a][0] <= 2 or any(b in inside for b in parents[a]) for a in chosen)

    def search(i, score):
        left = D - len(chosen)
        if left == 0:
            if score > best["score"] and connected():
                best["score"], best["subset"] = score, list(chosen)
            return
        if i >= n or tail[i][left] < 0 or score + tail[i][left] <= best["score"]:
            return
        chosen.append(i)
        search(i + 1, score + counts[i])
        chosen.pop()
        search(i + 1, score)

    search(0, 0)
    subset = best["subset"] or []
    nodes = sorted((graph[a][1] for a in subset), key=lambda s: (len(s), sorted(s)))
    formulas = [sorted(s) for s in nodes]
    children = [[c for c in range(len(nodes)) if nodes[q] < nodes[c]] for q in range(len(nodes))]
    return formulas, children, best["score"]
