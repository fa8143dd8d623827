"""CPU oracle of the decision step at sampling temperature T > 0 -- TEST
INFRASTRUCTURE ONLY.

The paper evaluates Spiffy at temperatures above zero (Sec. 5.3, SDAR at T = 1)
without spelling the sampler out; the reading taken here (listed with the
others in the design notes):

  - per still-masked position the token is drawn from softmax(z), z = x / T, in
    two levels over vocabulary slices of `slice_width` consecutive entries
    (slice s holds the entries s * slice_width ... ; the width is a parameter of
    the sampler):
      1. the slice: s* = argmax_s (ln Z_s + g_s), Z_s = sum of exp(z_v) over the
         slice, g_s = -ln(-ln u_s) -- the Gumbel-max construction on the slices'
         total weights (ties to the lower slice; a slice of weight 0 never wins);
      2. the entry inside it, by inverting the running sum with one more
         uniform: the first entry v of slice s* (ascending) whose running sum
         C_v = sum_{w <= v in s*} exp(z_w) reaches u' * Z_{s*};
    the token's confidence is its probability softmax(z)[token]; the unmasking
    rule of Sec. 3.1 is then applied to the confidences as at T = 0;
  - losslessness (App. A) needs a draft block and the true block that equals it
    to draw the same token, so the noise may depend on the sequence, the
    position, the slice and on how far the block has been denoised (its number
    of still-masked positions), never on the node's index;
  - the uniforms come from the counter-based generator Philox4x32-10 (Salmon,
    Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC 2011):
    counter = (s, l, b, masked positions of the node), key = the two halves of a
    64-bit seed; output word 0 gives u_s, output word 1 gives u' (used for the
    chosen slice only), and u = (word + 0.5) / 2^32.

Everything is numpy; floating point in float64.  Nothing in the product package
imports this module and it imports nothing from it.

Pins (tests/test_oracle_sampling.py): the generator's published known-answer
vectors; the drawn tokens follow softmax(x / T) for one and for several slices
(frequencies over many seeds); with one slice the draw is numpy's searchsorted
on the cumulative distribution; T -> 0 gives the arg-max; the noise ignores the
node index and follows the masked count; on the toy model the speculative run
equals plain sampled decoding.
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


def slice_uniforms(seed, b, l, masked_count, n_slices):
    """(u_s, u'_s) in (0, 1) for slices s = 0..n_slices-1 at (sequence b, position l,
    masked count): output words 0 and 1 of the counter (s, l, b, masked count)."""
    ctr = np.zeros((n_slices, 4), dtype=np.uint64)
    ctr[:, 0] = np.arange(n_slices)
    ctr[:, 1] = l
    ctr[:, 2] = b
    ctr[:, 3] = masked_count
    key = np.array([seed & MASK32, (seed >> 32) & MASK32], dtype=np.uint64)
    words = philox4x32_10(ctr, key)
    to_unit = lambda w: (w.astype(np.float64) + 0.5) / 4294967296.0
    return to_unit(words[:, 0]), to_unit(words[:, 1])


def draw_token(z, u_slice, u_inside, slice_width):
    """One two-level draw from softmax(z).  Returns (token, slice_gap, cdf_gap):
    slice_gap is the best minus the second best slice score (inf with one
    live slice), cdf_gap how far u' * Z is from the nearest edge of the chosen
    token's interval of the running sum, as a fraction of Z."""
    V = z.shape[0]
    n_slices = (V + slice_width - 1) // slice_width
    e = np.exp(z - z.max())                 # a common factor changes neither level
    score = np.full(n_slices, -np.inf)
    for s in range(n_slices):
        Z = e[s * slice_width:(s + 1) * slice_width].sum()
        if Z > 0:
            score[s] = np.log(Z) - np.log(-np.log(u_slice[s]))
    order = np.lexsort((np.arange(n_slices), -score))   # score descending, slice ascending
    s_star = int(order[0])
    slice_gap = score[order[0]] - score[order[1]] if n_slices > 1 else np.inf
    w = e[s_star * slice_width:(s_star + 1) * slice_width]
    C = np.cumsum(w)
    target = u_inside[s_star] * C[-1]
    hit = np.flatnonzero(C >= target)
    i = int(hit[0]) if hit.size else int(np.flatnonzero(w > 0)[-1])
    below = C[i - 1] if i > 0 else 0.0
    cdf_gap = min(target - below, C[i] - target) / C[-1]
    return s_star * slice_width + i, slice_gap, cdf_gap


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
    slice_gap: np.ndarray    # [B,N,L] best minus second best slice score (inf at unmasked positions)
    cdf_gap: np.ndarray      # [B,N,L] distance of u' Z from the token's interval edges, over Z (inf at unmasked)
    margin: np.ndarray       # [B,N] how far the rule's decision is from flipping


def sampled_decide(logits, block_tokens, mask_id, rule, top_s, threshold, temperature, seed, slice_width):
    logits = np.asarray(logits, dtype=np.float64)
    tokens = np.asarray(block_tokens, dtype=np.int32)
    B, N, L, V = logits.shape
    n_slices = (V + slice_width - 1) // slice_width
    conf = np.full((B, N, L), -np.inf)
    tok = tokens.copy()
    slice_gap = np.full((B, N, L), np.inf)
    cdf_gap = np.full((B, N, L), np.inf)
    for b in range(B):
        for n in range(N):
            masked = tokens[b, n] == mask_id
            count = int(masked.sum())
            for l in np.flatnonzero(masked):
                z = logits[b, n, l] / temperature
                u_slice, u_inside = slice_uniforms(seed, b, int(l), count, n_slices)
                t, slice_gap[b, n, l], cdf_gap[b, n, l] = draw_token(z, u_slice, u_inside, slice_width)
                p = np.exp(z - z.max())
                conf[b, n, l] = p[t] / p.sum()
                tok[b, n, l] = t
    bits, n_unmask, margin = apply_rule(conf, tokens, mask_id, rule, top_s, threshold)
    pos = (bits[..., None] >> np.arange(L, dtype=np.uint64)) & np.uint64(1)
    nxt = np.where(pos.astype(bool), tok, tokens).astype(np.int32)
    return SampledDecision(conf, tok, bits, n_unmask, nxt, slice_gap, cdf_gap, margin)
