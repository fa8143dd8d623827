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
    u = S.uniforms(seed=5, b=1, l=2, masked_count=3, vocab=4099)
    assert u.shape == (4099,) and u.min() > 0.0 and u.max() < 1.0
    assert abs(u.mean() - 0.5) < 0.02
    for other in (S.uniforms(6, 1, 2, 3, 4099), S.uniforms(5, 0, 2, 3, 4099),
                  S.uniforms(5, 1, 3, 3, 4099), S.uniforms(5, 1, 2, 4, 4099)):
        assert np.mean(other == u) < 0.01
    # vocabulary entry v is word v % 4 of block v // 4: a prefix of a longer row
    assert np.array_equal(S.uniforms(5, 1, 2, 3, 10), u[:10])


def test_drawn_tokens_follow_the_tempered_softmax():
    x = np.array([[[[1.0, 0.2, -0.5, 2.0, 0.0, -30.0]]]])
    state = np.array([[[5]]], dtype=np.int32)  # token 5 is the mask token
    for T in (0.7, 1.0, 2.5):
        p = np.exp(x[0, 0, 0] / T)
        p /= p.sum()
        n = 3000
        counts = np.zeros(6)
        for seed in range(n):
            d = S.sampled_decide(x, state, 5, oracle.RULE_TOPS, 1, 0.0, T, seed)
            counts[d.top_tok[0, 0, 0]] += 1
            assert abs(d.conf[0, 0, 0] - p[d.top_tok[0, 0, 0]]) < 1e-12
        sigma = np.sqrt(p * (1 - p) / n)
        assert np.all(np.abs(counts / n - p) < 4 * sigma + 1e-9), (T, counts / n, p)


def test_low_temperature_gives_the_arg_max():
    r = np.random.default_rng(0)
    x = r.standard_normal((2, 3, 5, 40)).astype(np.float32)
    x[..., 39] = -30
    state = np.where(r.random((2, 3, 5)) < 0.3, 1, 39).astype(np.int32)
    d = S.sampled_decide(x, state, 39, oracle.RULE_TOPS, 1, 0.0, 1e-4, seed=9)
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
    d = S.sampled_decide(x, state, 49, oracle.RULE_TOPS, 1, 0.0, 1.0, seed=3)
    assert np.array_equal(d.top_tok[0, 0], d.top_tok[0, 1])          # equal states draw equal tokens
    assert np.array_equal(d.conf[0, 0], d.conf[0, 1])
    assert not np.array_equal(d.top_tok[0, 0, 1:], d.top_tok[0, 2, 1:])  # another masked count, other noise


def sampled_backend(T, seed):
    def decide(logits, states, mask_id, rule, top_s, threshold):
        d = S.sampled_decide(logits, states, mask_id, rule, top_s, threshold, T, seed)
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
