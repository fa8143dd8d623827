"""Offline calibration (Algorithm 2, App. D.1): pins of the oracle against hand
-worked examples and invariants, the package's host implementation against the
oracle, and the closed loop calibrate -> draft -> verify on the toy model."""
import numpy as np
import pytest

import oracle
from oracle import calibration as ocal
from oracle import toy
from paper_2509_18085_b200 import calibration as pcal

M = 3  # mask id of the hand example (V = 4)


def hand_run():
    """Three positions, four tokens; worked by hand in the comments."""
    states = [np.array(s) for s in ([M, M, M], [M, 2, M], [0, 2, M], [0, 2, 1])]
    logits = [
        # t=0: confidences 0.506 / 0.909 / 0.490 -> position ranks: pos1 -> 0, pos0 -> 1, pos2 -> 2
        np.array([[1.0, 0.5, 0.0, -30], [0.0, 0.0, 3.0, -30], [0.0, 2.0, 1.9, -30]]),
        # t=1: pos1 is unmasked; confidences pos0 0.787, pos2 0.844 -> pos2 -> 0, pos0 -> 1
        np.array([[2.0, 0.0, 0.0, -30], [9.0, 0.0, 0.0, -30], [0.0, 1.0, 3.0, -30]]),
        # t=2: only pos2 masked; token 1 ties with token 2 behind token 0 -> vocabulary rank 1
        np.array([[9.0, 0.0, 0.0, -30], [9.0, 0.0, 0.0, -30], [5.0, 0.0, 0.0, -30]]),
    ]
    return states, logits


HAND_SEQUENCES = [
    [(1, frozenset({(0, 0)})), (2, frozenset({(1, 0)})), (3, frozenset({(2, 0)}))],
    [(1, frozenset({(1, 0)})), (2, frozenset({(0, 1)}))],
    [(1, frozenset({(0, 1)}))],
]


@pytest.mark.parametrize("impl", [ocal.rewind, pcal.record])
def test_rewind_hand_example(impl):
    states, logits = hand_run()
    assert impl(states, logits, M, 3, 3) == HAND_SEQUENCES
    # a vocabulary rank that cannot be named ends the look-ahead of that timestep
    assert impl(states, logits, M, 3, 1) == [HAND_SEQUENCES[0], HAND_SEQUENCES[1][:1], []]
    # the look-ahead length cuts every sequence
    assert impl(states, logits, M, 1, 3) == [s[:1] for s in HAND_SEQUENCES]


@pytest.mark.parametrize("impl", [ocal.candidate_graph, pcal.build_graph])
def test_candidate_graph_hand_example(impl):
    f = frozenset
    g = impl(HAND_SEQUENCES, 3)
    assert g == [(1, f({(0, 0)}), 1), (1, f({(0, 1)}), 1), (1, f({(1, 0)}), 1),
                 (2, f({(0, 0), (1, 0)}), 1), (2, f({(0, 1), (1, 0)}), 1),
                 (3, f({(0, 0), (1, 0), (2, 0)}), 1)]
    # counts add up over repeated sequences and only the `top` most frequent stay
    seqs = HAND_SEQUENCES * 2 + [HAND_SEQUENCES[2]] * 3 + [[(1, f({(5, 0)}))]]
    g = impl(seqs, 2, top=2)
    assert g == [(1, f({(0, 1)}), 5), (1, f({(0, 0)}), 2),
                 (2, f({(0, 0), (1, 0)}), 2), (2, f({(0, 1), (1, 0)}), 2)]


def hand_graph():
    f = frozenset
    return [(1, f("a"), 10), (1, f("b"), 9), (1, f("c"), 1),
            (2, f("ab"), 8), (2, f("ac"), 2), (2, f("bd"), 1),
            (3, f("ace"), 20), (3, f("abf"), 3), (3, f("xyz"), 50)]


def test_best_subgraph_hand_example():
    """Node 8 is the most frequent one but has no parent in the graph, node 6
    needs one of {a}, {c}, {a,c} beside it (App. D.1)."""
    g = hand_graph()
    assert ocal.best_subgraph(g, 1) == ([0], 10)
    assert ocal.best_subgraph(g, 2) == ([0, 6], 30)
    assert ocal.best_subgraph(g, 3) == ([0, 1, 6], 39)
    assert ocal.best_subgraph(g, 4) == ([0, 1, 3, 6], 47)
    # all nine nodes: node 8 can never be connected, so no 9-subset qualifies
    assert ocal.best_subgraph(g, 9) == ([], -1)
    assert ocal.best_subgraph(g, 8) == (list(range(8)), 54)
    formulas, children = ocal.formulas_of(g, [0, 1, 3, 6])
    assert formulas == [["a"], ["b"], ["a", "b"], ["a", "c", "e"]]
    assert children == [[2, 3], [2], [], []]


def test_connectivity_definition():
    g = hand_graph()
    assert ocal.is_connected(g, (0, 1, 2, 3, 4, 5))  # levels 1 and 2 are roots
    assert not ocal.is_connected(g, (6,))
    assert ocal.is_connected(g, (2, 6)) and ocal.is_connected(g, (4, 6))
    assert not ocal.is_connected(g, (1, 6)) and not ocal.is_connected(g, (3, 6))  # {a,b} is no subset of {a,c,e}
    assert not ocal.is_connected(g, (0, 8))


def random_graph(r, lookahead=4, top=3, alphabet=6):
    g = []
    for k in range(1, lookahead + 1):
        seen = set()
        for _ in range(int(r.integers(1, top + 1))):
            node = frozenset((int(i), 0) for i in r.choice(alphabet, size=min(k, alphabet), replace=False))
            if node not in seen:
                seen.add(node)
                g.append((k, node, int(r.integers(1, 8))))
    return g


def test_selection_matches_brute_force_on_random_graphs():
    r = np.random.default_rng(0)
    nontrivial = 0
    for _ in range(150):
        g = random_graph(r)
        for D in (1, 3, 5, 7, len(g), len(g) + 2):
            subset, score = ocal.best_subgraph(g, D)
            formulas, children, pscore = pcal.calibrate(g, D)
            assert pscore == score
            of, oc = ocal.formulas_of(g, subset)
            assert formulas == of and children == oc
            if subset:
                greedy = sorted(range(len(g)), key=lambda a: -g[a][2])[:len(subset)]
                nontrivial += sorted(greedy) != subset
    assert nontrivial > 20  # connectivity did change the answer in many cases


def toy_runs(seeds, rule=oracle.RULE_TOPS, S=1, tau=0.0, sharpness=3.0):
    runs = []
    for seed in seeds:
        model = toy.ToyModel(seed=7, sharpness=sharpness)  # one model, many prompts
        r = np.random.default_rng(seed)
        s0 = np.full(model.block_len, model.mask_id, dtype=np.int32)
        known = r.choice(model.block_len, size=2, replace=False)
        s0[known] = r.integers(0, model.vocab - 1, size=2)
        states = toy.vanilla_decode(model, s0, rule, S, tau)
        logits = [model(s[None])[0, 0] for s in states[:-1]]
        runs.append((states, logits, model.mask_id))
    return runs


def test_record_matches_rewind_on_toy_runs():
    for rule, S, tau in ((oracle.RULE_TOPS, 1, 0.0), (oracle.RULE_TOPS, 2, 0.0), (oracle.RULE_THRESHOLD, 1, 0.6)):
        for states, logits, mask in toy_runs(range(6), rule, S, tau):
            assert pcal.record(states, logits, mask, 3, 3) == ocal.rewind(states, logits, mask, 3, 3)


def test_plain_top1_decoding_fixes_the_first_level():
    """Under the top-1 rule the token unmasked from a distribution is, by the
    definition of the two ranks, the candidate (0, 0) of that distribution: the
    level-1 node of every timestep is {(0, 0)} and it is inside every deeper node."""
    seqs = []
    for states, logits, mask in toy_runs(range(8)):
        seqs += ocal.rewind(states, logits, mask, 3, 24)
    assert all(s[0] == (1, frozenset({(0, 0)})) for s in seqs)
    g = ocal.candidate_graph(seqs, 3)
    assert g[0] == (1, frozenset({(0, 0)}), len(seqs)) and [lv for lv, _, _ in g].count(1) == 1
    assert all((0, 0) in node and len(node) == lv for lv, node, _ in g)
    # a node's count never exceeds that of the level above it summed over its subsets
    assert all(c <= len(seqs) for _, _, c in g)


def test_top_s_decoding_gives_s_tokens_per_level():
    seqs = []
    for states, logits, mask in toy_runs(range(4), oracle.RULE_TOPS, 2):
        seqs += ocal.rewind(states, logits, mask, 2, 24)
    full = [s for s in seqs if len(s) == 2]
    assert full and all(s[0][1] == frozenset({(0, 0), (1, 0)}) for s in seqs)
    assert all(len(s[1][1]) in (1, 2) for s in full)  # the last step of a block may unmask one token


def prompts(seeds):
    for seed in seeds:
        model = toy.ToyModel(seed=7, sharpness=3.0)
        r = np.random.default_rng(seed)
        s0 = np.full(model.block_len, model.mask_id, dtype=np.int32)
        known = r.choice(model.block_len, size=2, replace=False)
        s0[known] = r.integers(0, model.vocab - 1, size=2)
        yield model, s0


def closed_loop(make_drafter, rule, S, tau):
    """Decode unseen prompts; returns (drafts accepted, plain steps) after
    checking the trajectory and the call count against plain decoding (App. A)."""
    accepted_total = steps = 0
    per_prompt = []
    for model, s0 in prompts(range(100, 108)):
        vanilla = toy.vanilla_decode(model, s0, rule, S, tau)
        calls_vanilla = model.calls
        model.calls = 0
        traj, accepted = toy.speculative_decode(model, s0, make_drafter(model), rule, S, tau)
        assert len(traj) == len(vanilla) and all(np.array_equal(a, b) for a, b in zip(traj, vanilla))
        assert model.calls == calls_vanilla - sum(accepted)
        accepted_total += sum(accepted)
        steps += len(vanilla) - 1
        per_prompt.append((sum(accepted), len(vanilla) - 1))
    closed_loop.per_prompt = per_prompt
    return accepted_total, steps


RULES = [(oracle.RULE_TOPS, 1, 0.0), (oracle.RULE_TOPS, 2, 0.0), (oracle.RULE_THRESHOLD, 1, 0.97)]


@pytest.mark.parametrize("rule,S,tau", RULES)
def test_calibrated_graph_same_step_distribution(rule, S, tau):
    """Ranks taken under the distribution of the block itself: level 1 is the
    block's own next state, so every call accepts at least one draft as long as
    pruning keeps the graph whole."""
    seqs = []
    for states, logits, mask in toy_runs(range(10), rule, S, tau):
        seqs += pcal.record(states, logits, mask, 3, 3)
    graph = pcal.build_graph(seqs, 3)
    assert graph == ocal.candidate_graph(seqs, 3)
    formulas, children, score = pcal.calibrate(graph, 5)
    subset, oscore = ocal.best_subgraph(graph, 5)
    assert score == oscore and (formulas, children) == ocal.formulas_of(graph, subset)
    D = len(formulas)
    assert 1 <= D <= 5
    twin = toy.ToyModel(seed=7, sharpness=3.0)
    acc, steps = closed_loop(lambda m: toy.auto_drafter(twin, formulas, children, budget=D, top_k=3), rule, S, tau)
    if rule == oracle.RULE_TOPS:
        # level 1 is one fixed node: every call but the one that finishes the block advances two steps or more
        assert all(a >= n // 2 for a, n in closed_loop.per_prompt)
    else:
        # under the threshold rule the number of tokens per step varies and so does the level-1 node
        assert acc > 0
    # pruned to three drafts the run is still the plain one
    closed_loop(lambda m: toy.auto_drafter(twin, formulas, children, budget=3, top_k=3), rule, S, tau)


@pytest.mark.parametrize("rule,S,tau", RULES)
def test_calibrated_graph_carried_over_distribution(rule, S, tau):
    """No extra model call: a call's drafts come from the distribution of the
    last node the previous call accepted.  Calibration pairs every state with
    the distribution of the state before it, decoding does the same."""
    seqs = []
    for states, logits, mask in toy_runs(range(10), rule, S, tau):
        if len(states) > 2:
            seqs += pcal.record(states[1:], logits[:-1], mask, 3, 3)
    graph = pcal.build_graph(seqs, 3)
    assert graph == ocal.candidate_graph(seqs, 3)
    formulas, children, score = pcal.calibrate(graph, 6)
    subset, oscore = ocal.best_subgraph(graph, 6)
    assert score == oscore and (formulas, children) == ocal.formulas_of(graph, subset)
    D = len(formulas)
    acc, steps = closed_loop(
        lambda m: toy.carry_over_drafter(m.mask_id, formulas, children, budget=D, top_k=3), rule, S, tau)
    if rule == oracle.RULE_TOPS and S == 1:  # long runs: enough steps for the graph to pay off
        assert acc >= steps // 4, (acc, steps, formulas)
    # an uncalibrated graph of the same size (deep ranks nobody unmasks next) gets nothing
    far = [[(5, 2)], [(4, 2)], [(5, 1)], [(4, 2), (5, 2)]][:D]
    acc_far, _ = closed_loop(
        lambda m: toy.carry_over_drafter(m.mask_id, far, [[] for _ in far], budget=len(far), top_k=3), rule, S, tau)
    assert acc_far <= acc and (acc_far < acc or acc == 0)
