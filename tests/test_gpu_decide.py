"""GPU parity of spiffy_unmask_decide + spiffy_accept_walk (Algorithm 1) with
the CPU oracle, through the C ABI, on the seeded synthetic workloads."""
import numpy as np
import pytest
import torch

import oracle
from oracle import toy
from paper_2509_18085_b200 import spiffy
from paper_2509_18085_b200 import workloads as W

import gpu_util as G

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("index,n_nodes,cases", [(1, None, 10), (2, None, 2), (3, None, 2),
                                                 (5, 1, 2), (5, 2, 1), (5, 4, 1), (5, 8, 1), (5, 16, 1),
                                                 (5, 32, 1), (5, 64, 1)])
def test_configs_sharp(index, n_nodes, cases):
    hops = []
    for case in range(cases):
        cfg = W.config(index, n_nodes)
        w = W.make(cfg, W.seed_for(index, case), attention=False)
        dec, walk = G.gpu_decide(w)
        odec, owalk = G.oracle_decide(w)
        compared = G.assert_decision_parity(w, dec, walk, odec, owalk, G.TOL[cfg.dtype], G.MARGIN[cfg.dtype])
        # the generator's guard band keeps every decision away from the boundary:
        # the walk of every sequence was compared with the oracle's own
        assert compared == cfg.batch
        hops += owalk.n_accepted.tolist()
    if index in (1, 2, 3):
        assert max(hops) >= 1  # the workloads do exercise accepted drafts


@pytest.mark.parametrize("index,n_nodes", [(1, None), (2, None), (3, None)])
def test_configs_literal_with_evaluated_drafts(index, n_nodes):
    """The benchmark text's literal logit recipe (noise plus a U[0,8] boost):
    the 0.9 threshold never fires, so this covers the fallback branch; drafts
    are the parent's actual top tokens."""
    cfg = W.config(index, n_nodes, logits_mode="literal")
    w = W.make(cfg, W.seed_for(index, 50), proposer=G.oracle_proposer(cfg), attention=False)
    dec, walk = G.gpu_decide(w)
    odec, owalk = G.oracle_decide(w)
    # literal rows are flat: confidences are tiny and close together, so the
    # decision margin is judged at the precision of fp32 confidences
    compared = G.assert_decision_parity(w, dec, walk, odec, owalk, G.TOL[cfg.dtype], 1e-5)
    assert compared >= 1


def small_case(B, N, L, V, dtype, seed, rule=spiffy.RULE_TOPS, top_s=1, tau=0.9, p_unmasked=0.3):
    r = np.random.default_rng(seed)
    cfg = W.Config("small", B, N, L, 0, 1, 1, 64, dtype, V, rule, top_s=top_s, threshold=tau)
    logits = W.round_to((r.standard_normal((B, N, L, V)) * 3).astype(np.float32), dtype)
    tokens = np.where(r.random((B, N, L)) < p_unmasked, r.integers(0, V - 1, (B, N, L)),
                      V - 1).astype(np.int32)
    return cfg, logits, tokens


@pytest.mark.parametrize("V", [7, 8, 1000, 1001, 4096, 4097, 33000])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_ragged_vocab_and_odd_block(V, dtype):
    cfg, logits, tokens = small_case(2, 3, 5, V, dtype, seed=V)
    # rows must start on 16-byte boundaries: pad the row stride
    per16 = 8 if dtype == "bf16" else 4
    stride = (V + per16 - 1) // per16 * per16 + per16
    buf = torch.zeros((2, 3, 5, stride), dtype=G.tdtype(cfg), device="cuda")
    buf[..., :V] = G.to_dev(logits, G.tdtype(cfg))
    buf[..., V:] = 1e4  # never read
    view = buf[..., :V]
    dec = spiffy.spiffy_unmask_decide(view, G.to_dev(tokens), cfg.mask_id, cfg.rule)
    torch.cuda.synchronize()
    o = oracle.unmask_decide(logits, tokens, cfg.mask_id, cfg.rule)
    masked = tokens == cfg.mask_id
    assert np.array_equal(dec.top_tok.cpu().numpy(), o.top_tok)
    np.testing.assert_allclose(dec.conf.cpu().numpy()[masked], o.conf[masked], atol=G.TOL[dtype])
    safe = o.margin >= 1e-4
    assert np.array_equal(G.bits_np(dec.unmask_bits)[safe], o.unmask_bits[safe])


def test_argmax_ties_across_slices_and_lanes():
    V = 126464
    cfg, logits, tokens = small_case(1, 1, 8, V, "bf16", seed=3, p_unmasked=0.0)
    logits[:] = np.minimum(logits, 2.0)
    spots = [(5, 100000), (0, 7), (4095, 4096), (V - 1, 17), (64000, 63999), (12, 13), (8191, 8192),
             (90000, 30000)]
    for l, (a, b) in enumerate(spots):
        logits[0, 0, l, a] = 9.0
        logits[0, 0, l, b] = 9.0
    dec = spiffy.spiffy_unmask_decide(G.to_dev(logits, torch.bfloat16), G.to_dev(tokens),
                                      cfg.mask_id, cfg.rule)
    assert dec.top_tok.cpu().numpy()[0, 0].tolist() == [min(s) for s in spots]
    o = oracle.unmask_decide(logits, tokens, cfg.mask_id, cfg.rule)
    assert np.array_equal(dec.top_tok.cpu().numpy(), o.top_tok)


@pytest.mark.parametrize("rule,top_s,tau", [(spiffy.RULE_TOPS, 1, 0.0), (spiffy.RULE_TOPS, 3, 0.0),
                                            (spiffy.RULE_TOPS, 80, 0.0),
                                            (spiffy.RULE_THRESHOLD, 1, 0.02),
                                            (spiffy.RULE_THRESHOLD, 1, 0.9)])
def test_rules_on_wide_blocks(rule, top_s, tau):
    """L = 64 uses every bit of the unmask word; nodes with no masked position
    and with every position masked are both present."""
    cfg, logits, tokens = small_case(3, 4, 64, 512, "f32", seed=11, rule=rule, top_s=top_s, tau=tau)
    tokens[0, 0] = 5
    tokens[1, 2] = cfg.mask_id
    dec = spiffy.spiffy_unmask_decide(G.to_dev(logits), G.to_dev(tokens), cfg.mask_id, rule, top_s, tau)
    o = oracle.unmask_decide(logits, tokens, cfg.mask_id, rule, top_s, tau)
    safe = o.margin >= 1e-5
    assert safe.mean() > 0.8
    assert np.array_equal(G.bits_np(dec.unmask_bits)[safe], o.unmask_bits[safe])
    assert np.array_equal(dec.n_unmask.cpu().numpy()[safe], o.n_unmask[safe])
    assert dec.n_unmask.cpu().numpy()[0, 0] == 0 and G.bits_np(dec.unmask_bits)[0, 0] == 0
    assert np.array_equal(dec.top_tok.cpu().numpy(), o.top_tok)


def test_exact_ties_in_confidence_go_to_the_lower_position():
    cfg, logits, tokens = small_case(1, 2, 6, 64, "f32", seed=1, p_unmasked=0.0)
    logits[0, 0, :] = logits[0, 0, 0]          # six identical rows
    logits[0, 1, 3] = logits[0, 1, 1]
    logits[0, 1, 1, 5] = logits[0, 1, 3, 5] = 30.0  # two equal, dominant rows
    for rule, S, tau in [(spiffy.RULE_TOPS, 2, 0.0), (spiffy.RULE_THRESHOLD, 1, 0.999999)]:
        dec = spiffy.spiffy_unmask_decide(G.to_dev(logits), G.to_dev(tokens), cfg.mask_id, rule, S, tau)
        o = oracle.unmask_decide(logits, tokens, cfg.mask_id, rule, S, tau)
        assert np.array_equal(G.bits_np(dec.unmask_bits), o.unmask_bits)
    dec = spiffy.spiffy_unmask_decide(G.to_dev(logits), G.to_dev(tokens), cfg.mask_id, spiffy.RULE_TOPS, 2)
    assert G.bits_np(dec.unmask_bits).tolist() == [[0b000011, 0b001010]]


def test_nonfinite_rows_set_the_status_bit_only():
    cfg, logits, tokens = small_case(3, 2, 4, 256, "f32", seed=2, p_unmasked=0.0)
    logits[0, 1, 2, 100] = np.nan
    logits[2, 0, 0, :] = -np.inf
    tokens[1, 0, 1] = 3
    logits[1, 0, 1, :] = np.nan  # an unmasked position's row is never read
    logits[1, 1, 3, 7] = -np.inf  # a single -inf entry is an ordinary value
    dec = spiffy.spiffy_unmask_decide(G.to_dev(logits), G.to_dev(tokens), cfg.mask_id, cfg.rule)
    assert dec.dev_status.cpu().tolist() == [spiffy.DEV_NONFINITE, 0, spiffy.DEV_NONFINITE]
    o = oracle.unmask_decide(logits, tokens, cfg.mask_id, cfg.rule)
    assert o.bad_row.tolist() == [[0, 1], [0, 0], [1, 0]]
    good = np.ones(tokens.shape, dtype=bool)
    good[0, 1, 2] = good[2, 0, 0] = False
    assert np.array_equal(dec.top_tok.cpu().numpy()[good], o.top_tok[good])


def test_repeated_calls_are_bit_identical_and_workspace_is_reusable():
    cfg = W.config(2)
    w = W.make(cfg, W.seed_for(2, 7), attention=False)
    logits = G.to_dev(w.logits, torch.bfloat16)
    tokens = G.to_dev(w.block_tokens)
    desc = spiffy.decide_desc(logits, tokens, cfg.mask_id, cfg.rule, cfg.top_s, cfg.threshold)
    ws = torch.full((spiffy.spiffy_unmask_decide_workspace(desc),), 0xAB, dtype=torch.uint8, device="cuda")
    a = spiffy.spiffy_unmask_decide(logits, tokens, cfg.mask_id, cfg.rule, cfg.top_s, cfg.threshold, workspace=ws)
    b = spiffy.spiffy_unmask_decide(logits, tokens, cfg.mask_id, cfg.rule, cfg.top_s, cfg.threshold, workspace=ws)
    for f in ("conf", "top_tok", "unmask_bits", "n_unmask"):
        assert torch.equal(getattr(a, f), getattr(b, f))


def test_walk_on_random_tiny_graphs_in_one_batch():
    """Hundreds of random graphs, one per sequence of the batch."""
    import test_oracle_walk as T
    rng = np.random.default_rng(7)
    B, N, L = 600, 8, 6
    states = np.empty((B, N, L), dtype=np.int32)
    top = np.empty((B, N, L), dtype=np.int32)
    bits = np.empty((B, N), dtype=np.uint64)
    lists = []
    for b in range(B):
        states[b], top[b], bits[b] = T.random_graph(rng, N, L)
        lists.append(toy.parent_lists(states[b], T.MASK))
    off, idx = W._pack_parents(lists, N)
    nxt = np.stack([T.next_states(states[b], top[b], bits[b]) for b in range(B)])
    o = oracle.accept_walk(states, off, idx, nxt, bits)
    g = spiffy.spiffy_accept_walk(G.to_dev(states), G.to_dev(off), G.to_dev(idx), G.to_dev(top),
                                  G.to_dev(bits.view(np.int64)))
    for name in ("accepted_node", "n_accepted", "path", "next_block"):
        assert np.array_equal(getattr(g, name).cpu().numpy(), getattr(o, name)), name
    assert int(g.dev_status.cpu().sum()) == 0
    assert o.n_accepted.max() >= 3


def test_walk_flags_malformed_parent_lists():
    states = np.full((2, 3, 4), 9, dtype=np.int32)
    top = np.zeros((2, 3, 4), dtype=np.int32)
    bits = np.ones((2, 3), dtype=np.int64)
    off = np.array([[0, 0, 1, 2], [0, 0, 1, 2]], dtype=np.int32)
    idx = np.array([[0, 0, 0, 0], [0, 5, 0, 0]], dtype=np.int32)  # parent 5 >= child 2
    g = spiffy.spiffy_accept_walk(G.to_dev(states), G.to_dev(off), G.to_dev(idx), G.to_dev(top),
                                  G.to_dev(bits))
    assert g.dev_status.cpu().tolist() == [0, spiffy.DEV_BADGRAPH]
    assert g.accepted_node.cpu().tolist() == [0, 0]


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_wide_logit_range(dtype):
    """Logits spread over +-80 with the row maximum anywhere in the row: the sums
    of exponentials must neither overflow nor lose the small terms' order."""
    V = 40000
    cfg, logits, tokens = small_case(1, 2, 8, V, dtype, seed=5, p_unmasked=0.0)
    r = np.random.default_rng(6)
    logits *= 8.0
    for l in range(8):
        logits[0, 0, l, int(r.integers(0, V - 1))] = 80.0 - l   # one dominant token per row
        logits[0, 1, l, int(r.integers(0, V - 1))] = -80.0      # a far-away minimum changes nothing
    logits = W.round_to(logits, dtype)
    dec = spiffy.spiffy_unmask_decide(G.to_dev(logits, G.tdtype(cfg)), G.to_dev(tokens), cfg.mask_id,
                                      spiffy.RULE_THRESHOLD, 1, 0.9)
    o = oracle.unmask_decide(logits, tokens, cfg.mask_id, oracle.RULE_THRESHOLD, 1, 0.9)
    assert np.array_equal(dec.top_tok.cpu().numpy(), o.top_tok)
    np.testing.assert_allclose(dec.conf.cpu().numpy(), o.conf, atol=G.TOL[dtype])
    safe = o.margin >= 1e-3
    assert np.array_equal(G.bits_np(dec.unmask_bits)[safe], o.unmask_bits[safe])
    assert int(dec.dev_status.cpu().sum()) == 0


def test_degenerate_shapes():
    """A graph without drafts, a block of one position, uniform rows and a tiny vocabulary."""
    # N = 1, L = 1: the walk has nowhere to go
    logits = np.zeros((2, 1, 1, 16), dtype=np.float32)
    logits[0, 0, 0, 5] = 3.0
    tokens = np.full((2, 1, 1), 15, dtype=np.int32)
    dec = spiffy.spiffy_unmask_decide(G.to_dev(logits), G.to_dev(tokens), 15, spiffy.RULE_TOPS)
    o = oracle.unmask_decide(logits, tokens, 15, oracle.RULE_TOPS)
    assert dec.top_tok.cpu().numpy().tolist() == [[[5]], [[0]]]       # uniform row: lowest token id
    np.testing.assert_allclose(dec.conf.cpu().numpy(), o.conf, atol=1e-6)
    assert abs(float(dec.conf[1, 0, 0]) - 1.0 / 16) < 1e-6
    off = np.zeros((2, 2), dtype=np.int32)
    idx = np.zeros((2, 4), dtype=np.int32)
    walk = spiffy.spiffy_accept_walk(G.to_dev(tokens), G.to_dev(off), G.to_dev(idx), dec.top_tok, dec.unmask_bits)
    assert walk.accepted_node.cpu().tolist() == [0, 0] and walk.n_accepted.cpu().tolist() == [0, 0]
    assert walk.next_block.cpu().numpy().tolist() == [[5], [0]]
    # V = 4 (half a 128-bit vector of fp32... one vector exactly), every position unmasked in node 1
    logits = np.arange(2 * 3 * 4, dtype=np.float32).reshape(1, 2, 3, 4) % 5
    tokens = np.array([[[3, 3, 1], [0, 1, 2]]], dtype=np.int32)
    dec = spiffy.spiffy_unmask_decide(G.to_dev(logits), G.to_dev(tokens), 3, spiffy.RULE_THRESHOLD, 1, 0.5)
    o = oracle.unmask_decide(logits, tokens, 3, oracle.RULE_THRESHOLD, 1, 0.5)
    assert np.array_equal(dec.top_tok.cpu().numpy(), o.top_tok)
    assert np.array_equal(G.bits_np(dec.unmask_bits), o.unmask_bits)
    assert dec.n_unmask.cpu().numpy().tolist() == o.n_unmask.tolist() and o.n_unmask[0, 1] == 0
