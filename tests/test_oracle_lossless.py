"""The losslessness invariant of App. A on a toy model: the speculative run
visits exactly the states of plain decoding, and accepting M drafts saves M
model calls (Sec. 4.3)."""
import numpy as np
import pytest

import oracle
from oracle import toy


def start_state(model, seed):
    r = np.random.default_rng(seed)
    s = np.full(model.block_len, model.mask_id, dtype=np.int32)
    known = r.choice(model.block_len, size=model.block_len // 4, replace=False)
    s[known] = r.integers(0, model.vocab - 1, size=len(known))
    return s


@pytest.mark.parametrize("rule,S,tau", [(oracle.RULE_TOPS, 1, 0.0), (oracle.RULE_TOPS, 2, 0.0),
                                        (oracle.RULE_THRESHOLD, 1, 0.8)])
@pytest.mark.parametrize("seed", range(4))
def test_speculative_trajectory_equals_vanilla(rule, S, tau, seed):
    model = toy.ToyModel(seed=seed)
    s0 = start_state(model, seed)
    vanilla = toy.vanilla_decode(model, s0, rule, S, tau)
    calls_vanilla = model.calls
    assert not np.any(vanilla[-1] == model.mask_id)
    for drafter in (toy.peeking_drafter(vanilla, depth=3, wrong_prob=0.3, seed=seed, vocab=model.vocab),
                    toy.random_drafter(model.mask_id, n_drafts=4, seed=seed, vocab=model.vocab),
                    lambda state, call: np.zeros((0, len(state)), dtype=np.int32)):
        model.calls = 0
        traj, accepted = toy.speculative_decode(model, s0, drafter, rule, S, tau)
        assert len(traj) == len(vanilla)
        assert all(np.array_equal(a, b) for a, b in zip(traj, vanilla))
        # T vanilla steps cost T - M calls when M drafts are accepted
        assert model.calls == calls_vanilla - sum(accepted)


def test_peeking_drafter_does_reach_deep_accepts():
    total = 0
    for seed in range(6):
        model = toy.ToyModel(seed=seed)
        s0 = start_state(model, seed)
        vanilla = toy.vanilla_decode(model, s0, oracle.RULE_TOPS)
        d = toy.peeking_drafter(vanilla, depth=3, wrong_prob=0.0, seed=seed, vocab=model.vocab)
        _, accepted = toy.speculative_decode(model, s0, d, oracle.RULE_TOPS)
        assert max(accepted) == 3  # all three levels accepted in one call
        total += sum(accepted)
    assert total > 0


def test_a_planted_mistake_breaks_the_invariant():
    """If drafts could see one another's blocks (a wrong mask), a draft's
    distribution would differ from the true block's and the runs diverge: the
    invariant does detect a broken attention rule."""
    def leaky(q, kp, vp, kb, vb):
        # every node additionally sees node 0's block as if it were context
        kp2 = np.concatenate([kp, kb[:, 0]], 1)
        vp2 = np.concatenate([vp, vb[:, 0]], 1)
        return oracle.graph_attention(q, kp2, vp2, kb, vb)

    diverged = 0
    for seed in range(6):
        good = toy.ToyModel(seed=seed)
        s0 = start_state(good, seed)
        vanilla = toy.vanilla_decode(good, s0, oracle.RULE_TOPS)
        bad = toy.ToyModel(seed=seed, attention=leaky)
        vanilla_bad = toy.vanilla_decode(bad, s0, oracle.RULE_TOPS)
        d = toy.peeking_drafter(vanilla_bad, depth=3, wrong_prob=0.0, seed=seed, vocab=bad.vocab)
        traj, _ = toy.speculative_decode(bad, s0, d, oracle.RULE_TOPS)
        same = len(traj) == len(vanilla_bad) and all(
            np.array_equal(a, b) for a, b in zip(traj, vanilla_bad))
        diverged += not same
    assert diverged > 0


def test_auto_speculation_with_the_drafting_oracle_is_lossless_and_saves_calls():
    """Drafts built from the target distribution with fixed formulas (Sec. 4.4.2)
    and pruned (Sec. 4.4.4): the first-rank chain is what plain decoding does
    next, so drafts are accepted, and the trajectory stays the plain one."""
    formulas = [[(0, 0)], [(0, 1)], [(0, 0), (1, 0)], [(0, 0), (1, 1)], [(0, 0), (1, 0), (2, 0)]]
    children = [[2, 3], [], [4], [], []]
    saved = 0
    for seed in range(4):
        model = toy.ToyModel(seed=seed)
        s0 = start_state(model, seed)
        vanilla = toy.vanilla_decode(model, s0, oracle.RULE_TOPS)
        calls_vanilla = model.calls
        model.calls = 0
        drafter = toy.auto_drafter(toy.ToyModel(seed=seed), formulas, children, budget=3, top_k=2)
        traj, accepted = toy.speculative_decode(model, s0, drafter, oracle.RULE_TOPS)
        assert len(traj) == len(vanilla) and all(np.array_equal(a, b) for a, b in zip(traj, vanilla))
        assert model.calls == calls_vanilla - sum(accepted)
        saved += sum(accepted)
    assert saved > 0
