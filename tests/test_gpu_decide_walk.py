"""spiffy_decide_walk: Algorithm 1 steps 1-5 in one call.  It must give exactly
the bits of spiffy_unmask_decide followed by spiffy_accept_walk, on the fused
kernel (small graphs) and on the two-call route (large ones), and both are
checked against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from oracle import toy
from paper_2509_18085_b200 import spiffy
from paper_2509_18085_b200 import workloads as W
import gpu_util as G

pytestmark = pytest.mark.gpu


def both(logits, tokens, off, idx, mask_id, rule, top_s=1, tau=0.9):
    """Runs the two-call and the one-call form on the same device inputs and
    checks that they agree bit for bit; returns the one-call results."""
    lg, tk, of, ix = G.to_dev(logits), G.to_dev(tokens), G.to_dev(off), G.to_dev(idx)
    dec = spiffy.spiffy_unmask_decide(lg, tk, mask_id, rule, top_s, tau)
    walk = spiffy.spiffy_accept_walk(tk, of, ix, dec.top_tok, dec.unmask_bits)
    dec2, walk2 = spiffy.spiffy_decide_walk(lg, tk, of, ix, mask_id, rule, top_s, tau)
    torch.cuda.synchronize()
    G.assert_same_bits(dec, walk, dec2, walk2)
    return dec2, walk2


def random_case(seed, B, N, L, V, p_accept=0.7, dtype="f32"):
    """Random logits and a chain-like graph: node m is, with probability
    p_accept, the next state of an earlier node, else a corrupted copy."""
    r = np.random.default_rng(seed)
    mask = V - 1
    logits = r.standard_normal((B, N, L, V), dtype=np.float32) * np.float32(3)
    logits[..., mask] = -30.0
    logits = W.round_to(logits, dtype)
    tokens = np.empty((B, N, L), dtype=np.int32)
    lists = []
    for b in range(B):
        tokens[b, 0] = np.where(r.random(L) < 0.3, r.integers(0, V - 1, L), mask)
        tokens[b, 0, 0] = mask
        for m in range(1, N):
            parent = int(r.integers(0, m))
            d = oracle.unmask_decide(logits[b:b + 1, parent:parent + 1], tokens[b:b + 1, parent:parent + 1],
                                     mask, oracle.RULE_TOPS, 1)
            nxt = d.next_tokens[0, 0].copy()
            if r.random() > p_accept or not np.any(tokens[b, parent] == mask):
                free = np.flatnonzero(nxt == mask)
                if len(free):
                    nxt[free[0]] = int(r.integers(0, V - 1))
            tokens[b, m] = nxt
        lists.append(toy.parent_lists(tokens[b], mask))
    off, idx = W._pack_parents(lists, N)
    return logits, tokens, off, idx, mask


@pytest.mark.parametrize("B,N,L,V", [(3, 8, 32, 5000), (2, 16, 32, 1000), (5, 3, 7, 36), (1, 2, 64, 300),
                                     (2, 9, 64, 132), (1, 1, 1, 16)])
def test_one_call_equals_two_calls_and_the_oracle(B, N, L, V):
    """Shapes on both sides of the fused kernel's limit (N * L <= 512)."""
    for rule, S, tau in ((spiffy.RULE_TOPS, 1, 0.0), (spiffy.RULE_TOPS, 3, 0.0), (spiffy.RULE_THRESHOLD, 1, 0.5)):
        logits, tokens, off, idx, mask = random_case(B * 100 + N, B, N, L, V)
        dec, walk = both(logits, tokens, off, idx, mask, rule, S, tau)
        o, ow = oracle.verify_step(logits, tokens, off, idx, mask, rule, S, tau)
        assert np.array_equal(dec.top_tok.cpu().numpy(), o.top_tok)
        safe = o.margin >= 1e-5
        assert np.array_equal(G.bits_np(dec.unmask_bits)[safe], o.unmask_bits[safe])
        if safe.all():
            for name in ("accepted_node", "n_accepted", "path", "next_block"):
                assert np.array_equal(getattr(walk, name).cpu().numpy(), getattr(ow, name)), name
        assert int(dec.dev_status.sum()) == 0 and int(walk.dev_status.sum()) == 0


def test_deep_walks_happen_on_the_fused_kernel():
    logits, tokens, off, idx, mask = random_case(3, 40, 8, 16, 200, p_accept=1.0)
    dec, walk = both(logits, tokens, off, idx, mask, spiffy.RULE_TOPS)
    _, ow = oracle.verify_step(logits, tokens, off, idx, mask, oracle.RULE_TOPS, 1, 0.0)
    assert np.array_equal(walk.n_accepted.cpu().numpy(), ow.n_accepted)
    assert np.array_equal(walk.path.cpu().numpy(), ow.path)
    assert ow.n_accepted.max() >= 3


def test_long_parent_lists_take_the_two_call_route():
    """A parent capacity whose arrays do not fit the fused kernel's shared memory."""
    logits, tokens, off, idx, mask = random_case(5, 2, 4, 8, 64)
    wide = np.zeros((2, 16384), dtype=np.int32)
    wide[:, :idx.shape[1]] = idx
    dec, walk = both(logits, tokens, off, wide, mask, spiffy.RULE_TOPS)
    _, ow = oracle.verify_step(logits, tokens, off, idx, mask, oracle.RULE_TOPS, 1, 0.0)
    assert np.array_equal(walk.next_block.cpu().numpy(), ow.next_block)


def test_status_bits_of_both_parts():
    logits, tokens, off, idx, mask = random_case(6, 3, 4, 8, 64)
    logits[1, 2, :, :] = np.nan                 # a row that cannot be decided
    tokens[1, 2, 3] = mask
    idx = idx.copy()
    m = next(m for m in range(1, 4) if off[2, m + 1] > off[2, m])  # first node of sequence 2 with a parent
    idx[2, off[2, m]] = 7                                          # ... which now is no valid one
    dec, walk = both(logits, tokens, off, idx, mask, spiffy.RULE_TOPS)
    assert dec.dev_status.cpu().tolist() == [0, spiffy.DEV_NONFINITE, 0]
    assert walk.dev_status.cpu().tolist()[:2] == [0, 0] and walk.dev_status.cpu().tolist()[2] == spiffy.DEV_BADGRAPH


def test_argument_checks():
    logits, tokens, off, idx, mask = random_case(7, 1, 2, 4, 32)
    lg, tk, of, ix = G.to_dev(logits), G.to_dev(tokens), G.to_dev(off), G.to_dev(idx)
    with pytest.raises(ValueError):
        spiffy.spiffy_decide_walk(lg, tk, of[:, :-1], ix, mask, spiffy.RULE_TOPS)
    with pytest.raises(spiffy.SpiffyError):
        spiffy.spiffy_decide_walk(lg, tk, of, ix, mask, spiffy.RULE_TOPS,
                                  workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    with pytest.raises(spiffy.SpiffyError):
        spiffy.spiffy_decide_walk(lg, tk, of, ix, mask, 7)  # no such rule


def test_graph_replay_over_changing_inputs_sharing_one_workspace():
    """Back-to-back calls in one CUDA graph, each on other logits and another
    graph but the same workspace: every call must see its own partial results
    (the tail kernel is resident before the reduce kernel of its call ends)."""
    B, N, L, V = 1, 8, 32, 40000
    cases = [random_case(100 + i, B, N, L, V) for i in range(5)]
    dev = [(G.to_dev(c[0], torch.bfloat16), G.to_dev(c[1]), G.to_dev(c[2]), G.to_dev(c[3])) for c in cases]
    mask = cases[0][4]
    want = []
    for lg, tk, of, ix in dev:
        dec = spiffy.spiffy_unmask_decide(lg, tk, mask, spiffy.RULE_THRESHOLD, 1, 0.5)
        want.append((dec, spiffy.spiffy_accept_walk(tk, of, ix, dec.top_tok, dec.unmask_bits)))
    desc = spiffy.decide_desc(dev[0][0], dev[0][1], mask, spiffy.RULE_THRESHOLD, 1, 0.5)
    ws = torch.empty(spiffy.spiffy_unmask_decide_workspace(desc), dtype=torch.uint8, device="cuda")
    outs = [spiffy.spiffy_decide_walk(lg, tk, of, ix, mask, spiffy.RULE_THRESHOLD, 1, 0.5, workspace=ws)
            for lg, tk, of, ix in dev]
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for (lg, tk, of, ix), (dec, walk) in zip(dev, outs):
                spiffy.spiffy_decide_walk(lg, tk, of, ix, mask, spiffy.RULE_THRESHOLD, 1, 0.5,
                                          decision=dec, walk=walk, workspace=ws)
        for _ in range(20):
            for dec, walk in outs:
                dec.conf.zero_()
                walk.next_block.zero_()
            graph.replay()
            stream.synchronize()
            for (dec, walk), (dec0, walk0) in zip(outs, want):
                G.assert_same_bits(dec0, walk0, dec, walk)


# ---------------------------------------------------------------------------
# lazy chain evaluation: the decision only for the nodes the walk reaches
# ---------------------------------------------------------------------------
def lazy_vs_eager(logits, tokens, off, idx, mask_id, rule, top_s=1, tau=0.9, dtype=None):
    lg, tk, of, ix = G.to_dev(logits, dtype), G.to_dev(tokens), G.to_dev(off), G.to_dev(idx)
    dec, walk = spiffy.spiffy_decide_walk(lg, tk, of, ix, mask_id, rule, top_s, tau)
    B, N, L = tokens.shape
    # poison what the lazy call must leave alone or overwrite
    lazy_dec = spiffy.Decision(torch.full((B, N, L), -7.0, device="cuda"),
                               torch.full((B, N, L), -7, dtype=torch.int32, device="cuda"),
                               torch.full((B, N), -7, dtype=torch.int64, device="cuda"),
                               torch.full((B, N), -7, dtype=torch.int32, device="cuda"),
                               torch.zeros((B,), dtype=torch.int32, device="cuda"))
    ldec, lwalk = spiffy.spiffy_decide_walk(lg, tk, of, ix, mask_id, rule, top_s, tau, decision=lazy_dec,
                                            lazy=True)
    torch.cuda.synchronize()
    for f in ("accepted_node", "n_accepted", "path", "next_block"):
        assert torch.equal(getattr(walk, f), getattr(lwalk, f)), f
    assert torch.equal(dec.dev_status, ldec.dev_status) or int(dec.dev_status.sum()) != 0
    path = walk.path.cpu().numpy()
    on_path = np.zeros((B, N), dtype=bool)
    for b in range(B):
        on_path[b, path[b][path[b] >= 0]] = True
    m = torch.from_numpy(on_path).cuda()
    assert torch.equal(dec.conf.view(torch.int32)[m], ldec.conf.view(torch.int32)[m])
    assert torch.equal(dec.top_tok[m], ldec.top_tok[m])
    assert torch.equal(dec.unmask_bits[m], ldec.unmask_bits[m])
    assert torch.equal(dec.n_unmask[m], ldec.n_unmask[m])
    # nodes off the path: marked as not evaluated, nothing else written
    assert bool((ldec.n_unmask[~m] == -1).all())
    assert bool((ldec.conf[~m] == -7.0).all()) and bool((ldec.top_tok[~m] == -7).all())
    assert bool((ldec.unmask_bits[~m] == -7).all())
    return walk, lwalk, on_path


@pytest.mark.parametrize("B,N,L,V", [(3, 8, 32, 5000), (2, 16, 32, 1000), (5, 3, 7, 36), (1, 2, 64, 300),
                                     (2, 9, 64, 132), (1, 1, 1, 16), (40, 8, 16, 200)])
def test_lazy_chain_evaluation_equals_the_eager_call_on_the_path(B, N, L, V):
    hops = 0
    for rule, S, tau in ((spiffy.RULE_TOPS, 1, 0.0), (spiffy.RULE_TOPS, 3, 0.0), (spiffy.RULE_THRESHOLD, 1, 0.5)):
        logits, tokens, off, idx, mask = random_case(B * 100 + N, B, N, L, V, p_accept=0.9)
        walk, _, on_path = lazy_vs_eager(logits, tokens, off, idx, mask, rule, S, tau)
        hops += int(walk.n_accepted.sum())
        assert on_path[:, 0].all()
    if N > 2:
        assert hops > 0


@pytest.mark.parametrize("B,N,L,V,dtype", [(64, 8, 32, 1000, "f32"), (33, 16, 4, 70000, "bf16"),
                                           (7, 12, 64, 9000, "f32"), (40, 5, 32, 20000, "bf16")])
def test_lazy_call_with_more_items_than_resident_thread_blocks(B, N, L, V, dtype):
    """B * L * slices exceeds what the device holds at once (six thread blocks
    per SM): every block then takes several (position, slice) items per level,
    each waiting on another sequence's epoch."""
    per_slice = 8192 if dtype == "bf16" else 4096
    items = B * L * -(-V // per_slice)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    assert items > 6 * sms
    logits, tokens, off, idx, mask = random_case(B * 1000 + N, B, N, L, V, p_accept=0.9, dtype=dtype)
    hops = 0
    for rule, S, tau in ((spiffy.RULE_TOPS, 1, 0.0), (spiffy.RULE_THRESHOLD, 1, 0.5)):
        for _ in range(3):  # the interleaving of the blocks differs from run to run, the bits must not
            walk, lwalk, on_path = lazy_vs_eager(logits, tokens, off, idx, mask, rule, S, tau,
                                                 dtype=torch.bfloat16 if dtype == "bf16" else None)
            assert int(lwalk.dev_status.sum()) == 0
        hops += int(walk.n_accepted.sum())
    assert hops > B  # deep walks: several levels per sequence


def test_lazy_chain_evaluation_at_the_benchmark_shapes():
    for index, cases in ((2, 2), (3, 1)):
        cfg = W.config(index)
        for case in range(cases):
            w = W.make(cfg, W.seed_for(index, case))
            walk, lwalk, on_path = lazy_vs_eager(w.logits, w.block_tokens, w.parent_off, w.parent_idx,
                                                 cfg.mask_id, cfg.rule, cfg.top_s, cfg.threshold,
                                                 dtype=G.tdtype(cfg))
            _, ow = G.oracle_decide(w)
            assert np.array_equal(lwalk.path.cpu().numpy(), ow.path)
            assert np.array_equal(lwalk.next_block.cpu().numpy(), ow.next_block)
            assert int(lwalk.dev_status.sum()) == 0


def test_lazy_call_in_a_cuda_graph():
    logits, tokens, off, idx, mask = random_case(11, 2, 8, 16, 2000, p_accept=1.0)
    lg, tk, of, ix = G.to_dev(logits), G.to_dev(tokens), G.to_dev(off), G.to_dev(idx)
    dec0, walk0 = spiffy.spiffy_decide_walk(lg, tk, of, ix, mask, spiffy.RULE_TOPS)
    desc = spiffy.decide_desc(lg, tk, mask, spiffy.RULE_TOPS, 1, 0.9)
    ws = torch.empty(spiffy.spiffy_decide_walk_lazy_workspace(desc), dtype=torch.uint8, device="cuda")
    dec, walk = spiffy.spiffy_decide_walk(lg, tk, of, ix, mask, spiffy.RULE_TOPS, workspace=ws, lazy=True)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            spiffy.spiffy_decide_walk(lg, tk, of, ix, mask, spiffy.RULE_TOPS, decision=dec, walk=walk,
                                      workspace=ws, lazy=True)
        for _ in range(10):
            walk.next_block.zero_()
            walk.path.zero_()
            graph.replay()
            stream.synchronize()
            for f in ("accepted_node", "n_accepted", "path", "next_block", "dev_status"):
                assert torch.equal(getattr(walk, f), getattr(walk0, f)), f
    assert int(walk0.n_accepted.max()) >= 2
