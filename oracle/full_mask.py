"""CPU oracle of the verification attention for full-sequence bidirectional
models without a suffix cache -- TEST INFRASTRUCTURE ONLY.

Fig. 3 (caption): the true sequence keeps attending to itself; each draft block
attends to itself and to all blocks of the true sequence except the block it is
a draft of.  With a cached prefix X', the block being decoded X_2 (node 0 of the
draft graph) and trailing, still fully masked blocks X_3 that are recomputed in
every call (App. A.2), the packed call has

    keys     [ prefix | X_2 (true block) | X_3 (suffix) | draft block 1 | ... ]
    queries  [ X_2 rows | X_3 rows | rows of draft 1 | ... ]

and the mask, written out here as a boolean matrix:
    X_2 and X_3 rows see prefix, X_2 and X_3;
    rows of draft m see prefix, X_3 and draft m.

Plain numpy in float64 with the mask materialised; nothing in the product
package imports this module and it imports nothing from it.

blockwise_causal_attention is the same packed call for block-causal models
(last sentence of the caption of Fig. 3, App. A.2): a block attends to the
blocks before it and to itself, never forward, so for the block being decoded
the mask keeps the earlier blocks and the node's own block and hides every later
block of the sequence.

Pins (tests/test_oracle_full_mask.py): the node rows equal the packed-attention
oracle with the suffix appended to the context; the suffix rows equal a library
scaled-dot-product attention over the true sequence; without a suffix the result
is the packed-attention oracle's; a draft's output does not change when the true
block's keys do.  Block-causal variant: each node's rows equal a library
scaled-dot-product attention with a block-causal mask over the sequence in
which that node stands in place of the block being decoded.
"""
from __future__ import annotations

import numpy as np


def full_sequence_attention(q_nodes, q_suffix, k_prefix, v_prefix, k_suffix, v_suffix, k_block, v_block,
                            scale=None):
    """q_nodes [B,N,L,Hq,d], q_suffix [B,S,Hq,d], k/v_prefix [B,P,Hkv,d],
    k/v_suffix [B,S,Hkv,d], k/v_block [B,N,L,Hkv,d] (node 0 = the true block).
    Returns (out_nodes [B,N,L,Hq,d], out_suffix [B,S,Hq,d])."""
    f = lambda a: np.asarray(a, dtype=np.float64)
    q_nodes, q_suffix, k_prefix, v_prefix = f(q_nodes), f(q_suffix), f(k_prefix), f(v_prefix)
    k_suffix, v_suffix, k_block, v_block = f(k_suffix), f(v_suffix), f(k_block), f(v_block)
    B, N, L, Hq, d = q_nodes.shape
    P, Hkv = k_prefix.shape[1], k_prefix.shape[2]
    S = q_suffix.shape[1]
    rep = Hq // Hkv
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    # key axis: prefix | node 0 | suffix | nodes 1..N-1
    keys = np.concatenate([k_prefix, k_block[:, 0], k_suffix, k_block[:, 1:].reshape(B, (N - 1) * L, Hkv, d)], 1)
    vals = np.concatenate([v_prefix, v_block[:, 0], v_suffix, v_block[:, 1:].reshape(B, (N - 1) * L, Hkv, d)], 1)
    # query axis: node 0 | suffix | nodes 1..N-1
    qs = np.concatenate([q_nodes[:, 0], q_suffix, q_nodes[:, 1:].reshape(B, (N - 1) * L, Hq, d)], 1)
    nq, nk = qs.shape[1], keys.shape[1]
    mask = np.zeros((nq, nk), dtype=bool)
    true_rows = slice(0, L + S)
    mask[true_rows, :P + L + S] = True                       # the true sequence attends to itself
    for m in range(1, N):
        rows = slice(L + S + (m - 1) * L, L + S + m * L)
        mask[rows, :P] = True                                # a draft sees the prefix,
        mask[rows, P + L:P + L + S] = True                   # the suffix (every true block but the one it drafts)
        mask[rows, P + L + S + (m - 1) * L:P + L + S + m * L] = True  # and itself
    out = np.empty((B, nq, Hq, d))
    for b in range(B):
        for h in range(Hq):
            g = h // rep
            s = (qs[b, :, h] @ keys[b, :, g].T) * scale
            s = np.where(mask, s, -np.inf)
            p = np.exp(s - s.max(axis=1, keepdims=True))
            p /= p.sum(axis=1, keepdims=True)
            out[b, :, h] = p @ vals[b, :, g]
    out_nodes = np.empty((B, N, L, Hq, d))
    out_nodes[:, 0] = out[:, :L]
    out_nodes[:, 1:] = out[:, L + S:].reshape(B, N - 1, L, Hq, d)
    return out_nodes, out[:, L:L + S]


def blockwise_causal_attention(q_nodes, k_seq, v_seq, k_block, v_block, block_index, scale=None):
    """Verification attention of a block-causal model for block ``block_index``.
    q_nodes [B,N,L,Hq,d]; k_seq, v_seq [B,n_blocks*L,Hkv,d]: keys and values of
    the whole sequence (what is stored for blocks >= block_index is never
    visible); k/v_block [B,N,L,Hkv,d]: the nodes' own blocks.  Returns
    [B,N,L,Hq,d]."""
    f = lambda a: np.asarray(a, dtype=np.float64)
    q_nodes, k_seq, v_seq, k_block, v_block = f(q_nodes), f(k_seq), f(v_seq), f(k_block), f(v_block)
    B, N, L, Hq, d = q_nodes.shape
    T, Hkv = k_seq.shape[1], k_seq.shape[2]
    rep = Hq // Hkv
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    # key axis: the sequence | block of node 0 | block of node 1 | ...
    keys = np.concatenate([k_seq, k_block.reshape(B, N * L, Hkv, d)], 1)
    vals = np.concatenate([v_seq, v_block.reshape(B, N * L, Hkv, d)], 1)
    mask = np.zeros((N * L, T + N * L), dtype=bool)
    for n in range(N):
        rows = slice(n * L, (n + 1) * L)
        for j in range(T):
            mask[rows, j] = (j // L) < block_index            # earlier blocks only: never forward
        mask[rows, T + n * L:T + (n + 1) * L] = True            # the node's own block, both directions
    qs = q_nodes.reshape(B, N * L, Hq, d)
    out = np.empty((B, N * L, Hq, d))
    for b in range(B):
        for h in range(Hq):
            g = h // rep
            s = (qs[b, :, h] @ keys[b, :, g].T) * scale
            s = np.where(mask, s, -np.inf)
            p = np.exp(s - s.max(axis=1, keepdims=True))
            p /= p.sum(axis=1, keepdims=True)
            out[b, :, h] = p @ vals[b, :, g]
    return out.reshape(B, N, L, Hq, d)
