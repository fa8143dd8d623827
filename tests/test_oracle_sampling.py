"""Pins of the sampled decision oracle (temperature > 0): the generator against
its published known-answer vectors, the sampler against the distribution it
must draw from, the rule against the verification oracle's own, and the
losslessness invariant of App. A under sampling."""
import numpy as np
import pytest

import oracle
from oracle import sampling as S
from oracle import toy


def golden_vectors():
    import os
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "philox4x32_10_kat.txt")
    rows = []
    with open(path) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                w = [int(x, 16) for x in line.split()]
                rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def test_philox_known_answers():
    """The test vectors published with the generator (tests/golden/philox4x32_10_kat.txt)."""
    rows = golden_vectors()
    assert len(rows) == 3
    for ctr, key, want in rows:
        assert S.philox4x32_10(ctr, key).tolist() == want


def test_uniforms_are_open_interval_and_counter_dependent():
    u, w = S.slice_uniforms(seed=5, b=1, l=2, masked_count=3, n_slices=4099)
    for x in (u, w):
        assert x.shape == (4099,) and x.min() > 0.0 and x.max() < 1.0
        assert abs(x.mean() - 0.5) < 0.02
    assert abs(np.corrcoef(u, w)[0, 1]) < 0.05   # the two words of one counter are independent
    for other in (S.slice_uniforms(6, 1, 2, 3, 4099), S.slice_uniforms(5, 0, 2, 3, 4099),
                  S.slice_uniforms(5, 1, 3, 3, 4099), S.slice_uniforms(5, 1, 2, 4, 4099)):
        assert np.mean(other[0] == u) < 0.01 and np.mean(other[1] == w) < 0.01
    # slice s is counter word 0 = s: a prefix of a longer row
    assert np.array_equal(S.slice_uniforms(5, 1, 2, 3, 10)[0], u[:10])
    # the words are those of the generator itself: counter (s, l, b, masked count), key = seed halves
    words = S.philox4x32_10([7, 2, 1, 3], [5, 0])
    assert u[7] == (float(words[0]) + 0.5) / 2.0 ** 32 and w[7] == (float(words[1]) + 0.5) / 2.0 ** 32


@pytest.mark.parametrize("width", [1, 2, 4, 6, 100])
def test_drawn_tokens_follow_the_tempered_softmax(width):
    """Whatever the slice width (one entry per slice = plain Gumbel-max, one
    slice = plain inversion, or in between), the draw is from softmax(x / T)."""
    x = np.array([[[[1.0, 0.2, -0.5, 2.0, 0.0, -30.0]]]])
    state = np.array([[[5]]], dtype=np.int32)  # token 5 is the mask token
    for T in (0.7, 2.5):
        p = np.exp(x[0, 0, 0] / T)
        p /= p.sum()
        n = 3000
        counts = np.zeros(6)
        for seed in range(n):
            d = S.sampled_decide(x, state, 5, oracle.RULE_TOPS, 1, 0.0, T, seed, width)
            counts[d.top_tok[0, 0, 0]] += 1
            assert abs(d.conf[0, 0, 0] - p[d.top_tok[0, 0, 0]]) < 1e-12
        sigma = np.sqrt(p * (1 - p) / n)
        assert np.all(np.abs(counts / n - p) < 4 * sigma + 1e-9), (T, counts / n, p)


def test_pairs_of_positions_draw_independently():
    """Two positions of one block: the joint frequencies are the product of the marginals."""
    x = np.zeros((1, 1, 2, 3))
    x[0, 0, :, 2] = -40.0                      # the mask token is never drawn
    state = np.full((1, 1, 2), 2, dtype=np.int32)
    n = 4000
    joint = np.zeros((2, 2))
    for seed in range(n):
        d = S.sampled_decide(x, state, 2, oracle.RULE_TOPS, 1, 0.0, 1.0, seed, 2)
        joint[d.top_tok[0, 0, 0], d.top_tok[0, 0, 1]] += 1
    assert np.all(np.abs(joint / n - 0.25) < 4 * np.sqrt(0.25 * 0.75 / n))


def test_one_slice_is_inversion_of_the_cumulative_distribution():
    """With the whole vocabulary in one slice, level 1 has nothing to choose and
    the token is numpy's searchsorted of u' on the cumulative distribution."""
    r = np.random.default_rng(4)
    V = 50
    for trial in range(40):
        z = r.standard_normal(V) * 2
        p = np.exp(z - z.max())
        p /= p.sum()
        _, w = S.slice_uniforms(trial, 0, 0, 1, 1)
        x = z.reshape(1, 1, 1, V).copy()
        d = S.sampled_decide(x, np.full((1, 1, 1), V, dtype=np.int32), V, oracle.RULE_TOPS, 1, 0.0, 1.0, trial, 64)
        want = int(np.searchsorted(np.cumsum(p), w[0], side="left"))
        if d.cdf_gap[0, 0, 0] > 1e-12:
            assert d.top_tok[0, 0, 0] == want
        assert np.isinf(d.slice_gap[0, 0, 0])


def test_slice_choice_is_gumbel_max_on_slice_weights():
    """Level 1 by hand on a case with three slices: the scores are the logs of
    the slices' weights plus the Gumbel noise of the slices' own uniforms, and
    the token comes from the winning slice."""
    z = np.log(np.array([0.1, 0.2, 0.05, 0.25, 0.3, 0.1]))
    x = z.reshape(1, 1, 1, 6)
    state = np.full((1, 1, 1), 6, dtype=np.int32)   # no logit column belongs to the mask token here
    seen = set()
    for seed in range(200):
        u, w = S.slice_uniforms(seed, 0, 0, 1, 3)
        score = np.log(np.array([0.3, 0.3, 0.4])) - np.log(-np.log(u))
        s_star = int(np.argmax(score))
        d = S.sampled_decide(x, state, 6, oracle.RULE_TOPS, 1, 0.0, 1.0, seed, 2)
        assert d.top_tok[0, 0, 0] // 2 == s_star
        pair = np.exp(z[2 * s_star:2 * s_star + 2])
        assert d.top_tok[0, 0, 0] % 2 == (0 if w[s_star] * pair.sum() <= pair[0] else 1)
        assert abs(d.slice_gap[0, 0, 0] - (np.sort(score)[-1] - np.sort(score)[-2])) < 1e-12
        seen.add(int(d.top_tok[0, 0, 0]))
    assert seen == set(range(6))


def test_weightless_slices_and_entries_are_never_drawn():
    x = np.full((1, 1, 1, 9), -np.inf)
    x[0, 0, 0, 4] = 0.3
    x[0, 0, 0, 7] = 0.1
    state = np.full((1, 1, 1), 8, dtype=np.int32)
    for seed in range(50):
        d = S.sampled_decide(x, state, 8, oracle.RULE_TOPS, 1, 0.0, 1.0, seed, 3)
        assert d.top_tok[0, 0, 0] in (4, 7)


def test_low_temperature_gives_the_arg_max():
    r = np.random.default_rng(0)
    x = r.standard_normal((2, 3, 5, 40)).astype(np.float32)
    x[..., 39] = -30
    state = np.where(r.random((2, 3, 5)) < 0.3, 1, 39).astype(np.int32)
    d = S.sampled_decide(x, state, 39, oracle.RULE_TOPS, 1, 0.0, 1e-4, seed=9, slice_width=16)
    o = oracle.unmask_decide(x, state, 39, oracle.RULE_TOPS)
    assert np.array_equal(d.top_tok, o.top_tok)
    assert np.all(d.conf[state == 39] > 0.99)


@pytest.mark.parametrize("rule,S_,tau", [(oracle.RULE_TOPS, 1, 0.0), (oracle.RULE_TOPS, 3, 0.0),
                                          (oracle.RULE_THRESHOLD, 1, 0.35)])
def test_rule_agrees_with_the_verification_oracle(rule, S_, tau):
    """apply_rule is written here in numpy; the verification oracle has its own
    in C++.  Fed the same confidences they must pick the same positions."""
    r = np.random.default_rng(1)
    x = (r.standard_normal((3, 4, 9, 30)) * 2).astype(np.float32)
    state = np.where(r.random((3, 4, 9)) < 0.3, 2, 29).astype(np.int32)
    state[0, 0] = 2  # a node with nothing left to unmask
    o = oracle.unmask_decide(x, state, 29, rule, S_, tau)
    bits, count, _ = S.apply_rule(o.conf, state, 29, rule, S_, tau)
    assert np.array_equal(bits, o.unmask_bits) and np.array_equal(count, o.n_unmask)


def test_noise_follows_the_state_not_the_node():
    r = np.random.default_rng(2)
    row = r.standard_normal((1, 1, 6, 50)).astype(np.float32)
    x = np.repeat(row, 3, axis=1)                      # three nodes with the same distributions
    state = np.full((1, 3, 6), 49, dtype=np.int32)
    state[0, 2, 0] = 7                                  # node 2 is one step further
    d = S.sampled_decide(x, state, 49, oracle.RULE_TOPS, 1, 0.0, 1.0, seed=3, slice_width=8)
    assert np.array_equal(d.top_tok[0, 0], d.top_tok[0, 1])          # equal states draw equal tokens
    assert np.array_equal(d.conf[0, 0], d.conf[0, 1])
    assert not np.array_equal(d.top_tok[0, 0, 1:], d.top_tok[0, 2, 1:])  # another masked count, other noise


def sampled_backend(T, seed):
    def decide(logits, states, mask_id, rule, top_s, threshold):
        d = S.sampled_decide(logits, states, mask_id, rule, top_s, threshold, T, seed, 5)
        return d.top_tok, d.unmask_bits
    return decide


@pytest.mark.parametrize("rule,S_,tau", [(oracle.RULE_TOPS, 1, 0.0), (oracle.RULE_THRESHOLD, 1, 0.5)])
@pytest.mark.parametrize("seed", range(3))
def test_sampled_decoding_is_lossless(rule, S_, tau, seed):
    """App. A at temperature 1: the speculative run visits the states of plain
    sampled decoding and saves one model call per accepted draft."""
    model = toy.ToyModel(seed=seed)
    r = np.random.default_rng(seed)
    s0 = np.full(model.block_len, model.mask_id, dtype=np.int32)
    s0[r.integers(0, model.block_len)] = 1
    decide = sampled_backend(1.0, seed + 50)
    vanilla = toy.vanilla_decode(model, s0, rule, S_, tau, decide=decide)
    calls = model.calls
    model.calls = 0
    drafter = toy.peeking_drafter(vanilla, depth=3, wrong_prob=0.2, seed=seed, vocab=model.vocab)
    traj, accepted = toy.speculative_decode(model, s0, drafter, rule, S_, tau, decide=decide)
    assert len(traj) == len(vanilla) and all(np.array_equal(a, b) for a, b in zip(traj, vanilla))
    assert model.calls == calls - sum(accepted) and sum(accepted) > 0


def test_sampling_changes_what_is_decoded():
    differ = 0
    for seed in range(6):
        model = toy.ToyModel(seed=seed)
        s0 = np.full(model.block_len, model.mask_id, dtype=np.int32)
        greedy = toy.vanilla_decode(model, s0, oracle.RULE_TOPS)
        sampled = toy.vanilla_decode(model, s0, oracle.RULE_TOPS, decide=sampled_backend(2.0, seed))
        differ += not np.array_equal(greedy[-1], sampled[-1])
    assert differ >= 4
