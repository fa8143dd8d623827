"""Toy masked-diffusion decoder for the losslessness invariant -- TEST
INFRASTRUCTURE ONLY (see ``oracle/__init__.py``).

App. A proves that Algorithm 1 is lossless: when the distribution computed for
a draft block equals the one the same block would get as the true block, the
speculative run passes through exactly the states of plain one-step-at-a-time
decoding, and accepting M drafts saves M model calls (Sec. 4.3).  This module
builds the smallest setting in which that can be checked end to end: a random,
deterministic one-layer "model" whose only sequence mixing is the packed
attention of Sec. 4.3, a plain decoding loop, and a speculative loop around
Algorithm 1.  The three numeric back ends (attention, decide, walk) are
arguments, so the same loops run on the oracle or on any other implementation.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

import oracle as _o


# ----------------------------------------------------------------------------
# Draft-graph structure (Sec. 4.4.1, Eqs. draft-graph-1..3)
# ----------------------------------------------------------------------------
def is_structural_parent(a, c, mask_id) -> bool:
    """True when block state ``c`` can follow ``a`` in the denoising process:
    the unmasked positions of ``a`` are a strict subset of those of ``c`` and
    the two agree on them (Eq. draft-graph-3; the count condition of
    Eq. draft-graph-2 is implied when the number of newly unmasked tokens is
    left free, as it is under threshold unmasking)."""
    a = np.asarray(a)
    c = np.asarray(c)
    ua, uc = a != mask_id, c != mask_id
    if not np.all(uc[ua]):
        return False
    if ua.sum() >= uc.sum():
        return False
    return bool(np.all(a[ua] == c[ua]))


def parent_lists(states, mask_id):
    """CSR parent lists (offsets [N+1], indices) holding every structural
    parent with a smaller index.  ``states`` [N,L], node 0 the true block."""
    states = np.asarray(states)
    n = states.shape[0]
    off = [0]
    idx = []
    for c in range(n):
        for a in range(c):
            if is_structural_parent(states[a], states[c], mask_id):
                idx.append(a)
        off.append(len(idx))
    return np.asarray(off, dtype=np.int32), np.asarray(idx, dtype=np.int32)


def pad_parent_lists(off, idx, cap=None):
    """Shape one sequence's CSR as the [1,N+1] / [1,cap] arrays of the ABI."""
    cap = max(1, len(idx)) if cap is None else cap
    out = np.zeros((1, cap), dtype=np.int32)
    out[0, :len(idx)] = idx
    return off.reshape(1, -1).astype(np.int32), out


# ----------------------------------------------------------------------------
# The toy model
# ----------------------------------------------------------------------------
def _default_attention(q, kp, vp, kb, vb):
    return _o.graph_attention(q, kp, vp, kb, vb)


def _default_decide(logits, states, mask_id, rule, top_s, threshold):
    d = _o.unmask_decide(logits, states, mask_id, rule, top_s, threshold)
    return d.top_tok, d.unmask_bits


def _default_walk(states, off, idx, top_tok, unmask_bits, mask_id):
    bits = unmask_bits.astype(np.uint64)
    pos = (bits[..., None] >> np.arange(states.shape[-1], dtype=np.uint64)) & np.uint64(1)
    nxt = np.where(pos.astype(bool), top_tok, states).astype(np.int32)
    w = _o.accept_walk(states, off, idx, nxt, bits)
    return w.accepted_node, w.n_accepted, w.path, w.next_block


@dataclass
class ToyModel:
    """logits = unembed(attention(embed(tokens) + pos)) over a fixed random
    context; float32-representable weights so that every back end sees the
    same inputs."""
    vocab: int = 24
    block_len: int = 8
    prefix_len: int = 16
    n_q_heads: int = 2
    n_kv_heads: int = 1
    head_dim: int = 64
    seed: int = 0
    sharpness: float = 1.0
    attention: callable = field(default=_default_attention, repr=False)

    def __post_init__(self):
        r = np.random.default_rng(self.seed)
        D = 32
        f = lambda *s: r.standard_normal(s).astype(np.float32)
        self.mask_id = self.vocab - 1
        self.emb = f(self.vocab, D)
        self.pos = f(self.block_len, D)
        self.wq = f(D, self.n_q_heads * self.head_dim) / np.float32(np.sqrt(D))
        self.wk = f(D, self.n_kv_heads * self.head_dim) / np.float32(np.sqrt(D))
        self.wv = f(D, self.n_kv_heads * self.head_dim) / np.float32(np.sqrt(D))
        self.wu = f(self.n_q_heads * self.head_dim, self.vocab)
        self.ctx_k = f(1, self.prefix_len, self.n_kv_heads, self.head_dim)
        self.ctx_v = f(1, self.prefix_len, self.n_kv_heads, self.head_dim)
        self.calls = 0

    def __call__(self, states):
        """states [N,L] int -> logits [1,N,L,V] float32 (one packed call)."""
        states = np.asarray(states)
        n, L = states.shape
        x = self.emb[states] + self.pos[None, :L]
        q = (x @ self.wq).astype(np.float32).reshape(1, n, L, self.n_q_heads, self.head_dim)
        k = (x @ self.wk).astype(np.float32).reshape(1, n, L, self.n_kv_heads, self.head_dim)
        v = (x @ self.wv).astype(np.float32).reshape(1, n, L, self.n_kv_heads, self.head_dim)
        o = np.asarray(self.attention(q, self.ctx_k, self.ctx_v, k, v), dtype=np.float64)
        # round the mixing result to float32 so that the unembedding (plain
        # numpy, outside the path under test) is identical for every back end
        h = o.astype(np.float32).reshape(n, L, -1).astype(np.float64)
        logits = (h @ self.wu.astype(np.float64)) * self.sharpness
        logits[..., self.mask_id] = -1e4  # the model never predicts MASK
        self.calls += 1
        return logits.astype(np.float32).reshape(1, n, L, self.vocab)


# ----------------------------------------------------------------------------
# Decoding loops
# ----------------------------------------------------------------------------
def vanilla_decode(model, state0, rule, top_s=1, threshold=0.9, decide=_default_decide):
    """Plain decoding (Sec. 3.1): one model call per denoising step.  Returns
    the list of block states visited, state0 first."""
    mask_id = model.mask_id
    state = np.asarray(state0, dtype=np.int32).copy()
    traj = [state.copy()]
    while np.any(state == mask_id):
        logits = model(state[None])
        top_tok, bits = decide(logits, state[None, None], mask_id, rule, top_s, threshold)
        L = state.shape[0]
        sel = ((int(bits[0, 0]) >> np.arange(L)) & 1).astype(bool)
        state = np.where(sel, top_tok[0, 0], state).astype(np.int32)
        traj.append(state.copy())
    return traj


def speculative_decode(model, state0, drafter, rule, top_s=1, threshold=0.9,
                       decide=_default_decide, walk=_default_walk):
    """Decoding with Algorithm 1.  ``drafter(state, call_index)`` returns an
    array [D,L] of draft blocks (possibly empty).  A drafter with the attribute
    ``uses_last_logits`` is called as ``drafter(state, call_index, logits)``
    with the distribution [L,V] of the last node accepted by the previous call
    (None before the first call): the distribution ``state`` was unmasked from.
    Returns (states visited, per call the number of accepted drafts whose
    distribution was used)."""
    mask_id = model.mask_id
    state = np.asarray(state0, dtype=np.int32).copy()
    L = state.shape[0]
    traj = [state.copy()]
    accepted = []
    call = 0
    last_logits = None
    while np.any(state == mask_id):
        if getattr(drafter, "uses_last_logits", False):
            drafts = drafter(state, call, last_logits)
        else:
            drafts = drafter(state, call)
        drafts = np.asarray(drafts, dtype=np.int32).reshape(-1, L)
        # order drafts by how many tokens they unmask so that parents precede
        # children, and drop exact duplicates
        if len(drafts):
            keep = []
            seen = {tuple(state)}
            for i in np.argsort((drafts != mask_id).sum(1), kind="stable"):
                t = tuple(drafts[i])
                if t not in seen:
                    seen.add(t)
                    keep.append(drafts[i])
            drafts = np.asarray(keep, dtype=np.int32).reshape(-1, L)
        states = np.concatenate([state[None], drafts], 0)
        off, idx = pad_parent_lists(*parent_lists(states, mask_id))
        logits = model(states)
        top_tok, bits = decide(logits, states[None], mask_id, rule, top_s, threshold)
        acc, hops, path, next_block = walk(states[None], off, idx, top_tok, bits, mask_id)
        # every node on the accepted path contributes its next state
        for node in path[0][: int(hops[0]) + 1]:
            if int(bits[0, node]) == 0:  # a fully unmasked draft was accepted
                continue
            sel = ((int(bits[0, node]) >> np.arange(L)) & 1).astype(bool)
            traj.append(np.where(sel, top_tok[0, node], states[node]).astype(np.int32))
        assert np.array_equal(traj[-1], next_block[0])
        state = next_block[0].astype(np.int32).copy()
        last_logits = np.asarray(logits)[0, int(path[0][int(hops[0])])]
        # an accepted draft saves a model call only when its distribution is
        # used, i.e. when it still had something to unmask
        accepted.append(sum(1 for node in path[0][1: int(hops[0]) + 1]
                            if int(bits[0, node]) != 0))
        call += 1
    return traj, accepted


# ----------------------------------------------------------------------------
# Drafters
# ----------------------------------------------------------------------------
def peeking_drafter(vanilla_traj, depth=3, wrong_prob=0.3, seed=0, vocab=None):
    """Drafts taken from a recorded plain trajectory (so that deep accepts do
    happen), each spoiled with probability ``wrong_prob``; plus one sibling per
    level that is always wrong."""
    rng = np.random.default_rng(seed)
    index = {tuple(s): i for i, s in enumerate(vanilla_traj)}

    def drafter(state, call):
        i = index.get(tuple(state))
        if i is None:  # the run has left the recorded trajectory
            return np.zeros((0, len(state)), dtype=np.int32)
        out = []
        for k in range(1, depth + 1):
            if i + k >= len(vanilla_traj):
                break
            d = vanilla_traj[i + k].copy()
            if rng.random() < wrong_prob:
                new = np.flatnonzero(d != state)
                d[rng.choice(new)] = rng.integers(0, vocab - 1)
            out.append(d)
            w = vanilla_traj[i + k].copy()
            new = np.flatnonzero(w != state)
            w[new[0]] = (w[new[0]] + 1) % (vocab - 1)
            out.append(w)
        return np.asarray(out, dtype=np.int32).reshape(-1, len(state))

    return drafter


def random_drafter(mask_id, n_drafts=4, seed=0, vocab=None):
    """Drafts that unmask random positions with random tokens."""
    rng = np.random.default_rng(seed)

    def drafter(state, call):
        out = []
        masked = np.flatnonzero(state == mask_id)
        cur = state.copy()
        for _ in range(min(n_drafts, len(masked))):
            cur = cur.copy()
            free = np.flatnonzero(cur == mask_id)
            cur[rng.choice(free)] = rng.integers(0, vocab - 1)
            out.append(cur)
        return np.asarray(out, dtype=np.int32).reshape(-1, len(state))

    return drafter


def auto_drafter(model, formulas, children, budget, top_k, draft=None):
    """Auto-speculation (Sec. 4.4.2): drafts are built from the target
    distribution of the current block with fixed draft formulas and pruned to
    ``budget`` (Sec. 4.4.4).  ``model`` is a twin of the decoder's model (same
    weights), so that the decoder's own call count is not disturbed; ``draft``
    replaces the oracle's drafting step (the CUDA library in the GPU tests)."""
    from . import drafting

    def default_draft(logits, state, mask_id):
        return drafting.draft_blocks(logits, state, mask_id, formulas, children, budget, top_k).tokens

    build = draft or default_draft

    def drafter(state, call):
        logits = model(state[None])[:, 0]  # [1, L, V]: p_TD of the current block
        tokens = build(np.ascontiguousarray(logits, dtype=np.float32), state[None].astype(np.int32),
                       model.mask_id)
        return np.asarray(tokens)[0, 1:]

    return drafter


def carry_over_drafter(mask_id, formulas, children, budget, top_k, draft=None):
    """Auto-speculation without any extra model call: the drafts of a call are
    built from the distribution of the last node accepted by the previous call
    (Algorithm 1 hands that distribution on; Sec. 4.4.2 drafts from the
    distribution at hand), with the ranks taken over the positions still masked
    in the new current block.  The first call has no distribution yet and
    carries no drafts."""
    from . import drafting

    def default_draft(logits, state, mask):
        return drafting.draft_blocks(logits, state, mask, formulas, children, budget, top_k).tokens

    build = draft or default_draft

    def drafter(state, call, logits):
        if logits is None:
            return np.zeros((0, len(state)), dtype=np.int32)
        tokens = build(np.ascontiguousarray(logits[None], dtype=np.float32), state[None].astype(np.int32), mask_id)
        return np.asarray(tokens)[0, 1:]

    drafter.uses_last_logits = True
    return drafter
