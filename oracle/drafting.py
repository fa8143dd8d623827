"""CPU oracle of Spiffy's drafting and pruning step -- TEST INFRASTRUCTURE ONLY.

Plain numpy in float64, written from the paper's definitions in the paper's
order; nothing in the product package may import this module and it imports
nothing from the CUDA package.

  Sec. 4.4.2 "Drafting Source": from the marginals p_1..p_L of the current
      target distribution, sort the positions by their maximum probability
      (token position rank i) and, per position, the vocabulary by probability
      (vocabulary rank j); the candidate c_ij is the token of vocabulary rank j
      at the position of rank i.  A draft block is the current block plus a set
      of candidates {c_ij}; which (i, j) a draft uses is fixed offline by the
      calibration (a "draft formula").
  Sec. 4.4.4 "Draft Graph Pruning": localScore = geometric mean of the
      probabilities of a draft's candidates, childScore = geometric mean of the
      children's local scores, score = geometric mean of the two; the D* best
      drafts are kept.

Readings where the paper is silent (listed with the others in the design notes):
  - only still-masked positions are ranked (an unmasked position has no
    marginal to draft from); rank 0 is the most confident one;
  - ties: lower position first, lower token id first, lower formula index first;
  - a formula that asks for a position rank beyond the number of masked
    positions cannot be built: its score is -inf and it is never kept;
  - a draft without (buildable) children has score = localScore;
  - kept drafts keep the order of their formulas (parents before children), the
    current block is node 0, and the parent lists hold every kept node (the
    current block included) whose candidate set is a strict subset.

Pins (tests/test_oracle_drafting.py): agreement with the verification oracle's
Next() on the formulas {(0,0)}, {(0,0),(1,0)}; closed forms of the geometric
means; brute-force ranking on tiny vocabularies; relabelling the vocabulary
relabels the drafts; brute-force selection of the D* best.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass
class Drafts:
    tokens: np.ndarray      # [B, D*+1, L] int32: node 0 = current block, then the kept drafts
    kept: np.ndarray        # [B, D*] int32 formula index of each kept draft, -1 padding
    score: np.ndarray       # [B, D] float64, -inf for formulas that cannot be built
    local: np.ndarray       # [B, D] float64 local scores
    parent_off: np.ndarray  # [B, D*+2] int32 CSR over the D*+1 nodes
    parent_idx: np.ndarray  # [B, cap] int32
    position_rank: np.ndarray  # [B, L] int32: rank i of each position, -1 when unmasked
    cand_tok: np.ndarray    # [B, L, K] int32: token of vocabulary rank j at each position
    cand_prob: np.ndarray   # [B, L, K] float64


def _gm(values):
    """Geometric mean (Sec. 4.4.4), through logarithms; 0 if any value is 0."""
    v = np.asarray(values, dtype=np.float64)
    if np.any(v <= 0.0):
        return 0.0
    return float(np.exp(np.mean(np.log(v))))


def draft_blocks(logits, state, mask_id, formulas, children, budget, top_k):
    """logits [B,L,V] (float32-representable), state [B,L] int32;
    formulas: list of D lists of (i, j) pairs; children: list of D lists of
    formula indices; budget = D*; top_k = number of vocabulary ranks."""
    logits = np.asarray(logits, dtype=np.float64)
    state = np.asarray(state, dtype=np.int32)
    B, L, V = logits.shape
    D = len(formulas)
    K = int(top_k)
    assert all(0 <= j < K and i >= 0 for f in formulas for i, j in f)
    tokens = np.zeros((B, budget + 1, L), dtype=np.int32)
    kept = np.full((B, budget), -1, dtype=np.int32)
    score = np.full((B, D), -np.inf)
    local = np.full((B, D), -np.inf)
    pos_rank = np.full((B, L), -1, dtype=np.int32)
    cand_tok = np.zeros((B, L, K), dtype=np.int32)
    cand_prob = np.zeros((B, L, K))
    lists = []
    for b in range(B):
        masked = [l for l in range(L) if state[b, l] == mask_id]
        # marginals p_n of the masked positions (softmax over the vocabulary)
        top_p = {}
        for l in masked:
            x = logits[b, l]
            p = np.exp(x - x.max())
            p /= p.sum()
            # Eq. (vocab-sort): vocabulary sorted by probability, ties to the lower id
            order = sorted(range(V), key=lambda v: (-p[v], v))[:K]
            cand_tok[b, l, :len(order)] = order
            cand_prob[b, l, :len(order)] = p[order]
            top_p[l] = p[order[0]]
        # Eq. (token-position-sort): positions sorted by their maximum probability
        n = sorted(masked, key=lambda l: (-top_p[l], l))
        for i, l in enumerate(n):
            pos_rank[b, l] = i
        # candidates and local scores of every formula
        built = []
        for f in formulas:
            if any(i >= len(n) for i, _ in f) or len(f) == 0:
                built.append(None)
                continue
            built.append([(n[i], int(cand_tok[b, n[i], j]), float(cand_prob[b, n[i], j])) for i, j in f])
        for q, c in enumerate(built):
            if c is not None:
                local[b, q] = _gm([p for _, _, p in c])
        for q, c in enumerate(built):
            if c is None:
                continue
            kids = [local[b, x] for x in children[q] if built[x] is not None]
            score[b, q] = _gm([local[b, q], _gm(kids)]) if kids else local[b, q]
        # the D* best; they keep the order of their formulas
        best = sorted((q for q in range(D) if built[q] is not None), key=lambda q: (-score[b, q], q))[:budget]
        best.sort()
        tokens[b, :] = state[b]
        for slot, q in enumerate(best):
            kept[b, slot] = q
            for l, tok, _ in built[q]:
                tokens[b, slot + 1, l] = tok
        # parent lists: every kept node (node 0 = the current block, the empty
        # candidate set) whose candidate set is a strict subset
        sets = [frozenset()] + [frozenset(formulas[q]) for q in best]
        off, idx = [0], []
        for c in range(budget + 1):
            if c < len(sets):
                idx += [a for a in range(c) if sets[a] < sets[c]]
            off.append(len(idx))
        lists.append((off, idx))
    cap = max(4, (max(len(i) for _, i in lists) + 3) // 4 * 4)
    parent_off = np.zeros((B, budget + 2), dtype=np.int32)
    parent_idx = np.zeros((B, cap), dtype=np.int32)
    for b, (off, idx) in enumerate(lists):
        parent_off[b] = off
        parent_idx[b, :len(idx)] = idx
    return Drafts(tokens, kept, score, local, parent_off, parent_idx, pos_rank, cand_tok, cand_prob)
