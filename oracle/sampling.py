"""CPU oracle of the decision step at sampling temperature T > 0 -- TEST
INFRASTRUCTURE ONLY.

The paper evaluates Spiffy at temperatures above zero (Sec. 5.3, SDAR at T = 1)
without spelling the sampler out; the reading taken here (listed with the
others in the design notes):

  - per still-masked position the token is drawn from softmax(x / T) by the
    Gumbel-max construction: token = argmax_v (x_v / T + g_v), g_v = -ln(-ln u_v)
    with u_v uniform on (0, 1); its confidence is its probability under that
    same distribution, softmax(x / T)[token]; the unmasking rule of Sec. 3.1 is
    then applied to the confidences as at T = 0;
  - losslessness (App. A) needs a draft block and the true block that equals it
    to draw the same token, so the noise may depend on the sequence, the
    position, the vocabulary entry and on how far the block has been denoised
    (its number of still-masked positions), never on the node's index;
  - the uniforms come from the counter-based generator Philox4x32-10 (Salmon,
    Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC 2011):
    counter = (v // 4, l, b, masked positions of the node), key = the two halves
    of a 64-bit seed, vocabulary entry v takes output word v % 4, and
    u = (word + 0.5) / 2^32.

Everything is numpy; floating point in float64.  Nothing in the product package
imports this module and it imports nothing from it.

Pins (tests/test_oracle_sampling.py): the generator's published known-answer
vectors; the drawn tokens follow softmax(x / T) (frequencies over many seeds);
T -> 0 gives the arg-max; the noise ignores the node index and follows the
masked count; on the toy model the speculative run equals plain sampled decoding.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

import oracle as _o

M0, M1 = 0xD2511F53, 0xCD9E8D57   # Philox4x32 multipliers
W0, W1 = 0x9E3779B9, 0xBB67AE85   # Weyl key increments (golden ratio, sqrt(3) - 1)
MASK32 = 0xFFFFFFFF


def philox4x32_10(counter, key):
    """counter [..., 4] and key [..., 2] (or [2]) of 32-bit words -> [..., 4] words."""
    c = np.asarray(counter, dtype=np.uint64) & MASK32
    k = np.broadcast_to(np.asarray(key, dtype=np.uint64) & MASK32, c.shape[:-1] + (2,)).copy()
    c0, c1, c2, c3 = (c[..., i].copy() for i in range(4))
    k0, k1 = k[..., 0], k[..., 1]
    for _ in range(10):
        p0 = np.uint64(M0) * c0
        p1 = np.uint64(M1) * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & MASK32
        hi1, lo1 = p1 >> np.uint64(32), p1 & MASK32
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
        k0 = (k0 + np.uint64(W0)) & MASK32
        k1 = (k1 + np.uint64(W1)) & MASK32
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint64)


def uniforms(seed, b, l, masked_count, vocab):
    """u_v in (0, 1) for v = 0..vocab-1 at (sequence b, position l, masked count)."""
    n4 = (vocab + 3) // 4
    ctr = np.zeros((n4, 4), dtype=np.uint64)
    ctr[:, 0] = np.arange(n4)
    ctr[:, 1] = l
    ctr[:, 2] = b
    ctr[:, 3] = masked_count
    key = np.array([seed & MASK32, (seed >> 32) & MASK32], dtype=np.uint64)
    words = philox4x32_10(ctr, key).reshape(-1)[:vocab]
    return (words.astype(np.float64) + 0.5) / 4294967296.0


def gumbel(seed, b, l, masked_count, vocab):
    return -np.log(-np.log(uniforms(seed, b, l, masked_count, vocab)))


def apply_rule(conf, tokens, mask_id, rule, top_s, threshold):
    """Sec. 3.1 on given confidences: the top_s most confident masked positions
    (ties to the lower position), or every masked position above the threshold
    and, if there is none, the most confident one.  Returns (bits, count,
    margin): margin is how far a confidence is from changing the outcome."""
    B, N, L = tokens.shape
    bits = np.zeros((B, N), dtype=np.uint64)
    count = np.zeros((B, N), dtype=np.int32)
    margin = np.full((B, N), np.inf)
    for b in range(B):
        for n in range(N):
            masked = [l for l in range(L) if tokens[b, n, l] == mask_id]
            if not masked:
                continue
            ranked = sorted(masked, key=lambda l: (-conf[b, n, l], l))
            c = [conf[b, n, l] for l in ranked]
            if rule == _o.RULE_TOPS:
                take = ranked[:top_s]
                if len(ranked) > top_s:
                    margin[b, n] = c[top_s - 1] - c[top_s]
            else:
                take = [l for l in masked if conf[b, n, l] > threshold]  # strict
                margin[b, n] = min(abs(x - threshold) for x in c)
                if not take:
                    take = ranked[:1]
                    if len(ranked) > 1:
                        margin[b, n] = min(margin[b, n], c[0] - c[1])
            for l in take:
                bits[b, n] |= np.uint64(1) << np.uint64(l)
            count[b, n] = len(take)
    return bits, count, margin


@dataclass
class SampledDecision:
    conf: np.ndarray         # [B,N,L] probability of the drawn token, -inf at unmasked positions
    top_tok: np.ndarray      # [B,N,L] drawn token; the existing token at unmasked positions
    unmask_bits: np.ndarray  # [B,N] uint64
    n_unmask: np.ndarray     # [B,N]
    next_tokens: np.ndarray  # [B,N,L]
    draw_gap: np.ndarray     # [B,N,L] best minus second best noisy score (inf at unmasked positions)
    margin: np.ndarray       # [B,N] how far the rule's decision is from flipping


def sampled_decide(logits, block_tokens, mask_id, rule, top_s, threshold, temperature, seed):
    logits = np.asarray(logits, dtype=np.float64)
    tokens = np.asarray(block_tokens, dtype=np.int32)
    B, N, L, V = logits.shape
    conf = np.full((B, N, L), -np.inf)
    tok = tokens.copy()
    gap = np.full((B, N, L), np.inf)
    for b in range(B):
        for n in range(N):
            masked = tokens[b, n] == mask_id
            count = int(masked.sum())
            for l in np.flatnonzero(masked):
                z = logits[b, n, l] / temperature
                y = z + gumbel(seed, b, int(l), count, V)
                order = np.lexsort((np.arange(V), -y))  # value descending, index ascending
                t = int(order[0])
                p = np.exp(z - z.max())
                conf[b, n, l] = p[t] / p.sum()
                tok[b, n, l] = t
                gap[b, n, l] = y[order[0]] - y[order[1]] if V > 1 else np.inf
    bits, n_unmask, margin = apply_rule(conf, tokens, mask_id, rule, top_s, threshold)
    pos = (bits[..., None] >> np.arange(L, dtype=np.uint64)) & np.uint64(1)
    nxt = np.where(pos.astype(bool), tok, tokens).astype(np.int32)
    return SampledDecision(conf, tok, bits, n_unmask, nxt, gap, margin)
