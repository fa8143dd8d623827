"""Pins of the decision oracle (Algorithm 1 steps 1-4; rules of Sec. 3.1)."""
import itertools

import numpy as np
import pytest
import torch

import oracle

MASK = 15


def decide(logits, tokens, rule=oracle.RULE_TOPS, top_s=1, tau=0.9, mask=MASK):
    logits = np.asarray(logits, dtype=np.float32)
    tokens = np.asarray(tokens, dtype=np.int32)
    while logits.ndim < 4:
        logits = logits[None]
    while tokens.ndim < 3:
        tokens = tokens[None]
    return oracle.unmask_decide(logits, tokens, mask, rule, top_s, tau)


def test_naive_long_double_softmax_and_library_softmax():
    r = np.random.default_rng(0)
    x = (r.standard_normal((1, 3, 6, 16)) * 2).astype(np.float32)
    tok = np.full((1, 3, 6), MASK, dtype=np.int32)
    d = decide(x, tok)
    e = np.exp(x.astype(np.longdouble))  # no max subtraction: |x| is small
    p = e / e.sum(-1, keepdims=True)
    np.testing.assert_allclose(d.conf, p.max(-1).astype(np.float64), rtol=1e-13)
    assert np.array_equal(d.top_tok, p.argmax(-1))
    pt = torch.softmax(torch.from_numpy(x).double(), -1)
    np.testing.assert_allclose(d.conf, pt.max(-1).values.numpy(), rtol=1e-13)
    assert np.array_equal(d.top_tok, pt.argmax(-1).numpy())


def test_uniform_row_and_shift_invariance_and_large_values():
    V = 16
    tok = np.full((1, 1, 2), MASK, dtype=np.int32)
    x = np.zeros((1, 1, 2, V), dtype=np.float32)
    x[0, 0, 1] = 7.5
    d = decide(x, tok)
    np.testing.assert_allclose(d.conf, 1.0 / V, rtol=1e-15)
    assert np.all(d.top_tok == 0)  # every entry ties: lowest index
    r = np.random.default_rng(1)
    y = r.standard_normal((1, 1, 2, V)).astype(np.float32)
    a = decide(y, tok)
    b = decide(y + np.float32(64.0), tok)  # exact in float32 for these magnitudes? compare loosely
    np.testing.assert_allclose(a.conf, b.conf, rtol=1e-5)
    big = y * 0 + 1e4  # exp(1e4) overflows without max subtraction
    big[..., 3] = 1e4 + 2
    c = decide(big, tok)
    np.testing.assert_allclose(c.conf, 1.0 / (1.0 + (V - 1) * np.exp(-2.0)), rtol=1e-14)
    assert np.all(c.top_tok == 3)


def test_planted_confidence_closed_form():
    """x_peak = LSE(rest) + logit(c)  =>  conf = c (after accounting for the
    float32 rounding of x_peak)."""
    r = np.random.default_rng(2)
    V = 64
    rest = (r.standard_normal(V) * 0.3).astype(np.float32)
    for c in (0.2, 0.5, 0.9, 0.97):
        x = rest.copy()
        others = np.delete(x.astype(np.float64), 10)
        lse = np.log(np.exp(others).sum())
        x[10] = np.float32(lse + np.log(c / (1 - c)))
        exact = 1.0 / (1.0 + np.exp(lse - float(x[10])))
        d = decide(x[None], np.array([[MASK]]))
        np.testing.assert_allclose(d.conf[0, 0, 0], exact, rtol=1e-13)
        assert abs(d.conf[0, 0, 0] - c) < 1e-6
        assert d.top_tok[0, 0, 0] == 10


def test_argmax_ties_take_lowest_index_and_negative_zero():
    x = np.full((1, 1, 1, 16), -1.0, dtype=np.float32)
    x[..., 9] = 2.0
    x[..., 4] = 2.0
    assert decide(x, [[MASK]]).top_tok[0, 0, 0] == 4
    z = np.full((1, 1, 1, 16), -3.0, dtype=np.float32)
    z[..., 7] = -0.0
    z[..., 11] = 0.0
    assert decide(z, [[MASK]]).top_tok[0, 0, 0] == 7


def test_unmasked_positions_and_full_node():
    r = np.random.default_rng(3)
    x = r.standard_normal((1, 2, 4, 16)).astype(np.float32)
    tok = np.array([[[MASK, 3, MASK, 5], [1, 2, 3, 4]]], dtype=np.int32)
    x[0, 0, 1] = np.nan  # rows of unmasked positions are never read
    x[0, 1] = np.inf
    d = decide(x, tok)
    assert d.conf[0, 0, 1] == -np.inf and d.conf[0, 0, 3] == -np.inf
    assert d.top_tok[0, 0, 1] == 3 and d.top_tok[0, 0, 3] == 5
    assert d.unmask_bits[0, 1] == 0 and d.n_unmask[0, 1] == 0
    assert np.array_equal(d.next_tokens[0, 1], [1, 2, 3, 4])
    assert d.bad_row.sum() == 0
    assert bin(int(d.unmask_bits[0, 0])).count("1") == 1
    assert int(d.unmask_bits[0, 0]) & 0b1010 == 0


def test_nonfinite_row_is_flagged():
    x = np.zeros((1, 1, 2, 16), dtype=np.float32)
    x[0, 0, 1, 3] = np.nan
    assert decide(x, [[MASK, MASK]]).bad_row[0, 0] == 1
    x[0, 0, 1, 3] = np.inf
    assert decide(x, [[MASK, MASK]]).bad_row[0, 0] == 1
    x[0, 0, 1, :] = -np.inf
    assert decide(x, [[MASK, MASK]]).bad_row[0, 0] == 1


def rows_with_conf(confs, V=16, seed=0):
    """Logit rows whose top-1 probability is the requested value: peak at a
    random index, the rest uniform."""
    r = np.random.default_rng(seed)
    x = np.zeros((len(confs), V), dtype=np.float64)
    peaks = []
    for i, c in enumerate(confs):
        p = int(r.integers(0, V - 1))
        x[i, p] = np.log(c / (1 - c)) + np.log(V - 1)
        peaks.append(p)
    return x.astype(np.float32), peaks


def brute_force_rule(conf, masked, rule, S, tau):
    pos = [l for l in range(len(conf)) if masked[l]]
    order = sorted(pos, key=lambda l: (-conf[l], l))
    if not order:
        return set()
    if rule == oracle.RULE_TOPS:
        return set(order[:S])
    u = {l for l in pos if conf[l] > tau}
    return u if u else {order[0]}


@pytest.mark.parametrize("rule,S", [(oracle.RULE_TOPS, 1), (oracle.RULE_TOPS, 2),
                                    (oracle.RULE_TOPS, 9), (oracle.RULE_THRESHOLD, 1)])
def test_rule_against_enumeration(rule, S):
    L = 6
    grid = [0.30, 0.55, 0.80, 0.95]
    r = np.random.default_rng(4)
    for trial in range(60):
        confs = list(r.choice(grid, size=L) + r.uniform(0, 0.03, size=L))
        masked = r.random(L) < 0.7
        x, peaks = rows_with_conf(confs, seed=trial)
        tok = np.where(masked, MASK, 1).astype(np.int32)
        d = decide(x[None, None], tok[None, None], rule=rule, top_s=S, tau=0.9)
        want = brute_force_rule(d.conf[0, 0], masked, rule, S, 0.9)
        got = {l for l in range(L) if (int(d.unmask_bits[0, 0]) >> l) & 1}
        assert got == want
        assert d.n_unmask[0, 0] == len(want)
        nxt = tok.copy()
        for l in want:
            nxt[l] = peaks[l]
        assert np.array_equal(d.next_tokens[0, 0], nxt)
        np.testing.assert_allclose(d.conf[0, 0][masked], np.asarray(confs)[masked], atol=1e-6)


def test_threshold_hand_built_cases():
    tok = np.full((1, 1, 4), MASK, dtype=np.int32)
    # none pass: fall back to the single best position (ties: lowest position)
    x, _ = rows_with_conf([0.5, 0.7, 0.7, 0.2])
    x[2] = x[1]
    d = decide(x[None, None], tok, rule=oracle.RULE_THRESHOLD, tau=0.9)
    assert int(d.unmask_bits[0, 0]) == 0b0010
    # all pass
    x, _ = rows_with_conf([0.95, 0.92, 0.99, 0.91])
    d = decide(x[None, None], tok, rule=oracle.RULE_THRESHOLD, tau=0.9)
    assert int(d.unmask_bits[0, 0]) == 0b1111 and d.n_unmask[0, 0] == 4
    # exactly tau does not pass (strict >): two equal logits give conf = 0.5
    y = np.full((1, 1, 4, 16), -np.inf, dtype=np.float32)
    y[..., 0] = 0.0
    y[..., 1] = 0.0
    d = decide(y, tok, rule=oracle.RULE_THRESHOLD, tau=0.5)
    assert np.all(d.conf == 0.5)
    assert int(d.unmask_bits[0, 0]) == 0b0001  # fallback, not all four
    d = decide(y, tok, rule=oracle.RULE_THRESHOLD, tau=0.4999999)
    assert int(d.unmask_bits[0, 0]) == 0b1111


def test_margin_reports_distance_to_flip():
    tok = np.full((1, 1, 3), MASK, dtype=np.int32)
    x, _ = rows_with_conf([0.95, 0.86, 0.40])
    d = decide(x[None, None], tok, rule=oracle.RULE_THRESHOLD, tau=0.9)
    np.testing.assert_allclose(d.margin[0, 0], 0.04, atol=1e-5)
    d = decide(x[None, None], tok, rule=oracle.RULE_TOPS, top_s=1)
    np.testing.assert_allclose(d.margin[0, 0], 0.09, atol=1e-5)
    d = decide(x[None, None], tok, rule=oracle.RULE_TOPS, top_s=2)
    np.testing.assert_allclose(d.margin[0, 0], 0.46, atol=1e-5)


def test_row_stride_view():
    r = np.random.default_rng(5)
    buf = r.standard_normal((1, 2, 3, 24)).astype(np.float32)
    view = buf[..., :16]
    tok = np.full((1, 2, 3), MASK, dtype=np.int32)
    a = oracle.unmask_decide(view, tok, MASK, oracle.RULE_TOPS)
    b = oracle.unmask_decide(np.ascontiguousarray(view), tok, MASK, oracle.RULE_TOPS)
    assert np.array_equal(a.conf, b.conf) and np.array_equal(a.top_tok, b.top_tok)
