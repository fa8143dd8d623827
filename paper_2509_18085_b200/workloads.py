"""Seeded synthetic workloads for one Spiffy verification step.

This module only *draws inputs*: tensors, block states and draft graphs with
the shapes and value distributions of the five benchmark configurations.  It
computes nothing of the method (no softmax, no argmax, no unmasking rule, no
graph walk): wherever an input has to be consistent with a decision the target
model would take -- a draft block is "the parent's next state, sometimes
spoiled" -- that decision is known *by construction*, because the generator
plants the winning token and its approximate confidence into the logits it
draws.  A caller that wants drafts derived from an actual evaluation of the
logits passes its own ``proposer`` callback.

Both the CUDA library and the CPU checker consume these inputs; neither is
imported here.

Value recipe (all rounded to the configuration's dtype):
  q, k, v        i.i.d. N(0, 1)
  root state     L/4 random positions already unmasked with random tokens
                 (none when L < 8); mask id = V - 1, never planted or drawn
  logits         per still-masked row: N(0, sigma = 2) noise; then
     "sharp"     noise clipped to +-4 sigma and one planted token raised to
                 ln(V-1) + sigma^2/2 + logit(c), i.e. to a top-1 probability of
                 about c (the expected log-sum-exp of the noise is analytic);
                 per node a few rows get c in [0.92, 0.999], the rest
                 c in [0.05, 0.85], so that a 0.9 threshold does fire
     "literal"   one random token per row raised by U[0, 8]; the winner of such
                 a row is not known by construction, so drafts built without a
                 ``proposer`` are mostly wrong (a poor drafter) -- the kernels'
                 run time does not depend on the values
  draft graph    levels 1..depth filled evenly; a node's primary parent sits one
                 level up; its state is the parent's designed next state with
                 each new token replaced by a random one with probability
                 p_wrong; later siblings swap one position for the next-ranked
                 one; finally every structural parent (strict subset of the
                 unmasked positions, equal tokens there: Eqs. draft-graph-2/3
                 of Sec. 4.4.1) goes into the parent lists
"""
from __future__ import annotations

import itertools
import math
from dataclasses import dataclass, field, replace
from typing import Callable, Optional

import numpy as np
import torch

RULE_TOPS = 0
RULE_THRESHOLD = 1


@dataclass(frozen=True)
class Config:
    name: str
    batch: int
    n_nodes: int
    block_len: int
    prefix_len: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str            # "f32" | "bf16"
    vocab: int
    rule: int
    top_s: int = 1
    threshold: float = 0.9
    depth: int = 3
    p_wrong: float = 0.3
    graph: str = "levels"  # "levels" | "diamond" | "formulas"
    logits_mode: str = "sharp"
    sigma: float = 2.0

    @property
    def mask_id(self) -> int:
        return self.vocab - 1


def config(index: int, n_nodes: Optional[int] = None, **over) -> Config:
    """The five benchmark configurations (1-based).  Configuration 5 is a
    sweep over the node count: pass ``n_nodes``."""
    table = {
        1: Config("tiny", 1, 4, 8, 128, 4, 4, 64, "f32", 1024, RULE_TOPS, depth=2,
                  p_wrong=0.3, graph="diamond"),
        2: Config("llada8b", 1, 8, 32, 512, 32, 32, 128, "bf16", 126464,
                  RULE_THRESHOLD, depth=3, p_wrong=0.3),
        3: Config("dream7b-gqa", 1, 16, 32, 1024, 28, 4, 128, "bf16", 152064,
                  RULE_TOPS, depth=4, p_wrong=0.2),
        4: Config("long-batched", 4, 32, 32, 4096, 32, 32, 128, "bf16", 126464,
                  RULE_THRESHOLD, depth=5, p_wrong=0.25),
        5: Config("short-wide", 1, 8, 4, 2048, 32, 8, 128, "bf16", 151936,
                  RULE_THRESHOLD, depth=3, p_wrong=0.25, graph="formulas"),
    }
    cfg = table[index]
    if n_nodes is not None:
        cfg = replace(cfg, n_nodes=n_nodes)
    return replace(cfg, **over) if over else cfg


def seed_for(index: int, case: int = 0) -> int:
    return 1000 * index + case


@dataclass
class Workload:
    cfg: Config
    seed: int
    q: np.ndarray              # [B,N,L,Hq,d] float32 holding dtype-representable values
    k_prefix: np.ndarray       # [B,P,Hkv,d]
    v_prefix: np.ndarray
    k_block: np.ndarray        # [B,N,L,Hkv,d]
    v_block: np.ndarray
    logits: np.ndarray         # [B,N,L,V] float32 holding dtype-representable values
    block_tokens: np.ndarray   # [B,N,L] int32
    parent_off: np.ndarray     # [B,N+1] int32
    parent_idx: np.ndarray     # [B,cap] int32
    planted_tok: np.ndarray    # [B,N,L] int32, -1 at unmasked positions
    planted_conf: np.ndarray   # [B,N,L] float32 design confidence, nan if none
    level: np.ndarray          # [B,N] int32
    info: dict = field(default_factory=dict)


def round_to(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round float32 values to ``dtype`` and return them as float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if dtype == "f32":
        return x
    t = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32)
    return t.numpy()


def _normal(rng, shape, dtype, scale=1.0):
    x = rng.standard_normal(shape, dtype=np.float32)
    if scale != 1.0:
        x *= np.float32(scale)
    return round_to(x, dtype)


def attention_inputs(cfg: Config, seed: int):
    rng = np.random.default_rng([seed, 1])
    B, N, L, P = cfg.batch, cfg.n_nodes, cfg.block_len, cfg.prefix_len
    Hq, Hkv, d = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    return dict(q=_normal(rng, (B, N, L, Hq, d), cfg.dtype),
                k_prefix=_normal(rng, (B, P, Hkv, d), cfg.dtype),
                v_prefix=_normal(rng, (B, P, Hkv, d), cfg.dtype),
                k_block=_normal(rng, (B, N, L, Hkv, d), cfg.dtype),
                v_block=_normal(rng, (B, N, L, Hkv, d), cfg.dtype))


# ----------------------------------------------------------------------------
# Draft-graph structure
# ----------------------------------------------------------------------------
def structural_parent_lists(states: np.ndarray, mask_id: int):
    """Parent lists with every earlier node whose unmasked positions are a
    strict subset of the child's and whose tokens agree there."""
    states = np.asarray(states)
    n = states.shape[0]
    un = states != mask_id
    cnt = un.sum(1)
    off = np.zeros(n + 1, dtype=np.int32)
    idx = []
    for c in range(n):
        for a in range(c):
            if cnt[a] < cnt[c] and not np.any(un[a] & ~un[c]) and \
                    np.array_equal(states[a][un[a]], states[c][un[a]]):
                idx.append(a)
        off[c + 1] = len(idx)
    return off, np.asarray(idx, dtype=np.int32)


def _pack_parents(per_seq, n_nodes):
    cap = max(1, max(len(i) for _, i in per_seq))
    cap = (cap + 3) // 4 * 4
    off = np.zeros((len(per_seq), n_nodes + 1), dtype=np.int32)
    idx = np.zeros((len(per_seq), cap), dtype=np.int32)
    for b, (o, i) in enumerate(per_seq):
        off[b] = o
        idx[b, :len(i)] = i
    return off, idx


# ----------------------------------------------------------------------------
# One node's logits and the decision they are designed to produce
# ----------------------------------------------------------------------------
@dataclass
class _Design:
    tok: np.ndarray      # [L] planted winner per position (-1 where unmasked)
    conf: np.ndarray     # [L] design confidence (nan where unmasked / unknown)
    ranked: list         # masked positions, most confident first (by design)
    unmask: list         # positions the node is designed to unmask


def _design_conf(cfg: Config, rng, n_masked: int) -> np.ndarray:
    """Design confidences of a node's masked rows, with a guard band around the
    decision boundary so that rounding cannot flip the rule."""
    if n_masked == 0:
        return np.zeros(0, dtype=np.float64)
    if cfg.rule == RULE_THRESHOLD:
        k = int(rng.integers(1, 4))
        k = min(k, n_masked)
        c = rng.uniform(0.05, 0.85, size=n_masked)
        hi = rng.choice(n_masked, size=k, replace=False)
        c[hi] = rng.uniform(0.92, 0.999, size=k)
        return c
    c = np.sort(rng.uniform(0.05, 0.80, size=n_masked))[::-1].copy()
    take = min(cfg.top_s, n_masked)
    c[:take] = np.sort(rng.uniform(0.90, 0.999, size=take))[::-1]
    # keep the designed order strict with visible gaps
    for i in range(1, take):
        c[i] = min(c[i], c[i - 1] - 0.01)
    return c[rng.permutation(n_masked)]


def _node_logits(cfg: Config, rng, state: np.ndarray, hint: Optional[dict] = None):
    """Draw the logits rows of one node and return (rows [L,V], _Design)."""
    L, V, mask = cfg.block_len, cfg.vocab, cfg.mask_id
    sig = np.float32(cfg.sigma)
    rows = rng.standard_normal((L, V), dtype=np.float32) * sig
    masked = np.flatnonzero(state == mask)
    tok = np.full(L, -1, dtype=np.int32)
    conf = np.full(L, np.nan, dtype=np.float64)
    if cfg.logits_mode == "sharp":
        np.clip(rows, -4 * sig, 4 * sig, out=rows)
        c = _design_conf(cfg, rng, len(masked))
        t = rng.integers(0, V - 1, size=len(masked))
        if hint is not None:  # stay close to another node's distribution
            for i, l in enumerate(masked):
                t[i] = hint["tok"][l] if rng.random() >= cfg.p_wrong else hint["alt"][l]
            order = [l for l in hint["ranked"] if state[l] == mask]
            cs = np.sort(c)[::-1]
            for r, l in enumerate(order):
                c[list(masked).index(l)] = cs[r]
        lse = math.log(V - 1) + float(sig) ** 2 / 2.0
        for i, l in enumerate(masked):
            rows[l, t[i]] = lse + math.log(c[i] / (1.0 - c[i]))
            tok[l] = t[i]
            conf[l] = c[i]
    elif cfg.logits_mode == "literal":
        t = rng.integers(0, V - 1, size=len(masked))
        boost = rng.uniform(0.0, 8.0, size=len(masked)).astype(np.float32)
        for i, l in enumerate(masked):
            rows[l, t[i]] += boost[i]
            tok[l] = t[i]
            conf[l] = boost[i] / 8.0  # only an ordering hint
    else:
        raise ValueError(cfg.logits_mode)
    rows = round_to(rows, cfg.dtype)
    ranked = sorted(masked.tolist(), key=lambda l: (-conf[l], l))
    if cfg.rule == RULE_THRESHOLD and cfg.logits_mode == "sharp":
        unmask = [l for l in ranked if conf[l] > cfg.threshold] or ranked[:1]
    else:
        unmask = ranked[:cfg.top_s if cfg.rule == RULE_TOPS else 1]
    return rows, _Design(tok, conf, ranked, unmask)


Proposer = Callable[[np.ndarray, np.ndarray], tuple]
"""proposer(rows [L,V], state [L]) -> (top_tok [L], unmask positions (list),
ranked masked positions (list)): lets a caller derive drafts from an actual
evaluation of the logits instead of from the planted design."""


def _apply_proposer(proposer, rows, state, design: _Design) -> _Design:
    if proposer is None:
        return design
    top_tok, unmask, ranked = proposer(rows, state)
    return _Design(np.asarray(top_tok, dtype=np.int32), design.conf, list(ranked), list(unmask))


def _spoil(cfg, rng, tok):
    """A random token different from ``tok`` (never the mask id)."""
    t = int(rng.integers(0, cfg.vocab - 2))
    return t + 1 if t >= tok else t


def _child_state(cfg, rng, parent_state, des: _Design, sibling: int):
    s = parent_state.copy()
    unmask = list(des.unmask)
    if sibling > 0:
        rest = [l for l in des.ranked if l not in unmask]
        if rest:
            unmask[(sibling - 1) % len(unmask)] = rest[(sibling - 1) % len(rest)]
        elif unmask:
            l = unmask[(sibling - 1) % len(unmask)]
            s[l] = _spoil(cfg, rng, int(des.tok[l]))
            unmask = [u for u in unmask if u != l] + [l]
            for u in unmask[:-1]:
                s[u] = des.tok[u]
            return s
    for l in unmask:
        t = int(des.tok[l])
        s[l] = _spoil(cfg, rng, t) if rng.random() < cfg.p_wrong else t
    return s


def _root_state(cfg, rng):
    L = cfg.block_len
    s = np.full(L, cfg.mask_id, dtype=np.int32)
    u0 = L // 4 if L >= 8 else 0
    known = rng.choice(L, size=u0, replace=False)
    s[known] = rng.integers(0, cfg.vocab - 1, size=u0)
    return s


def _level_sizes(n_drafts, depth):
    depth = max(1, min(depth, n_drafts)) if n_drafts else 0
    base, extra = divmod(n_drafts, depth) if depth else (0, 0)
    return [base + (1 if i < extra else 0) for i in range(depth)]


def _sequence_levels(cfg, rng, proposer, logits_out, states_out, ptok, pconf, level):
    """Graph kinds "levels" and "diamond"."""
    N, L = cfg.n_nodes, cfg.block_len
    states = [_root_state(cfg, rng)]
    designs = []
    rows, des = _node_logits(cfg, rng, states[0])
    logits_out[0] = rows
    designs.append(_apply_proposer(proposer, rows, states[0], des))
    lev = [0]
    if cfg.graph == "diamond" and N == 4:
        # root R; A = R + a; B = R + b; C = R + {a, b} with parents A and B
        d0 = designs[0]
        a, b = d0.ranked[0], d0.ranked[1]
        plan = [(1, [a]), (1, [b]), (2, [a, b])]
        for lv, pos in plan:
            s = states[0].copy()
            for l in pos:
                t = int(d0.tok[l])
                s[l] = _spoil(cfg, rng, t) if rng.random() < cfg.p_wrong else t
            if lv == 2:  # C agrees with A on a and with B on b whenever they are right
                s[a] = states[1][a]
                s[b] = states[2][b]
            states.append(s)
            lev.append(lv)
        # the drafts' own distributions stay close to the root's, so that the
        # two-hop paths R -> A -> C and R -> B -> C can be taken
        alt = np.array([_spoil(cfg, rng, int(t)) if t >= 0 else -1 for t in d0.tok],
                       dtype=np.int32)
        hint = dict(tok=d0.tok, alt=alt, ranked=d0.ranked)
        for i in range(1, N):
            rows, des = _node_logits(cfg, rng, states[i], hint=hint)
            logits_out[i] = rows
            designs.append(_apply_proposer(proposer, rows, states[i], des))
    else:
        sizes = _level_sizes(N - 1, cfg.depth)
        prev = [0]
        for lv, size in enumerate(sizes, start=1):
            cur = []
            n_sib = {}
            for j in range(size):
                par = prev[j % len(prev)]
                while len(designs) <= par:
                    i = len(designs)
                    rows, des = _node_logits(cfg, rng, states[i])
                    logits_out[i] = rows
                    designs.append(_apply_proposer(proposer, rows, states[i], des))
                sib = n_sib.get(par, 0)
                n_sib[par] = sib + 1
                pd = designs[par]
                s = states[par].copy()
                if pd.unmask:
                    s = _child_state(cfg, rng, states[par], pd, sib)
                    tries = 0
                    while any(np.array_equal(s, o) for o in states) and tries < 8:
                        new = np.flatnonzero(s != states[par])
                        s[rng.choice(new)] = int(rng.integers(0, cfg.vocab - 1))
                        tries += 1
                cur.append(len(states))
                states.append(s)
                lev.append(lv)
            prev = cur or prev
    for i in range(len(designs), N):
        rows, des = _node_logits(cfg, rng, states[i])
        logits_out[i] = rows
        designs.append(_apply_proposer(proposer, rows, states[i], des))
    for i in range(N):
        states_out[i] = states[i]
        ptok[i] = designs[i].tok if proposer is None else -1
        pconf[i] = designs[i].conf
        level[i] = lev[i]


def _sequence_formulas(cfg, rng, proposer, logits_out, states_out, ptok, pconf, level):
    """Graph kind "formulas": drafts are the root state plus a set of
    (position rank i, vocabulary rank j) choices, j in {0, 1}, enumerated in
    breadth-first order by (size, ranks, variant) and truncated to N - 1 -- the
    draft formulas of Sec. 4.4.3 without a calibration run."""
    N, L, V = cfg.n_nodes, cfg.block_len, cfg.vocab
    root = _root_state(cfg, rng)
    rows, des = _node_logits(cfg, rng, root)
    des = _apply_proposer(proposer, rows, root, des)
    alt = np.array([_spoil(cfg, rng, int(t)) if t >= 0 else -1 for t in des.tok], dtype=np.int32)
    logits_out[0] = rows
    states = [root]
    lev = [0]
    designs = [des]
    ranked = des.ranked
    formulas = []
    for size in range(1, min(3, len(ranked)) + 1):
        for subset in itertools.combinations(range(len(ranked)), size):
            for variant in itertools.product((0, 1), repeat=size):
                formulas.append((subset, variant))
    for subset, variant in formulas[:N - 1]:
        s = root.copy()
        for i, j in zip(subset, variant):
            l = ranked[i]
            s[l] = des.tok[l] if j == 0 else alt[l]
        states.append(s)
        lev.append(len(subset))
    while len(states) < N:  # more nodes asked for than formulas exist
        s = states[-1].copy()
        free = np.flatnonzero(s == cfg.mask_id)
        if len(free):
            s[free[0]] = int(rng.integers(0, V - 1))
        states.append(s)
        lev.append(lev[-1] + 1)
    hint = dict(tok=des.tok, alt=alt, ranked=ranked)
    for i in range(1, N):
        rows, d = _node_logits(cfg, rng, states[i], hint=hint)
        logits_out[i] = rows
        designs.append(d)
    for i in range(N):
        states_out[i] = states[i]
        ptok[i] = designs[i].tok if (proposer is None or i > 0) else -1
        pconf[i] = designs[i].conf
        level[i] = lev[i]


def decision_inputs(cfg: Config, seed: int, proposer: Optional[Proposer] = None):
    """Logits, block states and parent lists of every sequence."""
    B, N, L, V = cfg.batch, cfg.n_nodes, cfg.block_len, cfg.vocab
    logits = np.empty((B, N, L, V), dtype=np.float32)
    states = np.empty((B, N, L), dtype=np.int32)
    ptok = np.empty((B, N, L), dtype=np.int32)
    pconf = np.empty((B, N, L), dtype=np.float64)
    level = np.zeros((B, N), dtype=np.int32)
    per_seq = []
    build = _sequence_formulas if cfg.graph == "formulas" else _sequence_levels
    for b in range(B):
        rng = np.random.default_rng([seed, 2, b])
        build(cfg, rng, proposer, logits[b], states[b], ptok[b], pconf[b], level[b])
        # nodes are created level by level, so parents precede children
        per_seq.append(structural_parent_lists(states[b], cfg.mask_id))
    off, idx = _pack_parents(per_seq, N)
    return dict(logits=logits, block_tokens=states, parent_off=off, parent_idx=idx,
                planted_tok=ptok, planted_conf=pconf.astype(np.float32), level=level)


def make(cfg: Config, seed: int, proposer: Optional[Proposer] = None,
         attention: bool = True, decision: bool = True) -> Workload:
    """Draw one verification step's inputs for ``cfg``."""
    B, N, L = cfg.batch, cfg.n_nodes, cfg.block_len
    z = np.zeros((0,), dtype=np.float32)
    att = attention_inputs(cfg, seed) if attention else dict(
        q=z, k_prefix=z, v_prefix=z, k_block=z, v_block=z)
    dec = decision_inputs(cfg, seed, proposer) if decision else dict(
        logits=z, block_tokens=np.zeros((B, N, L), np.int32),
        parent_off=np.zeros((B, N + 1), np.int32), parent_idx=np.zeros((B, 4), np.int32),
        planted_tok=np.zeros((B, N, L), np.int32), planted_conf=np.zeros((B, N, L), np.float32),
        level=np.zeros((B, N), np.int32))
    return Workload(cfg=cfg, seed=seed, **att, **dec)
