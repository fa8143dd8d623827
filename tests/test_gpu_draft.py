"""GPU parity of spiffy_draft_blocks (Sec. 4.4.2 drafting, Sec. 4.4.4 pruning)
with the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import drafting
from paper_2509_18085_b200 import spiffy
from paper_2509_18085_b200 import workloads as W

import gpu_util as G

pytestmark = pytest.mark.gpu

# a calibrated-graph stand-in: D = 10 formulas over position ranks 0..3 and vocabulary ranks 0..2
FORMULAS = [[(0, 0)], [(0, 1)], [(1, 0)], [(0, 0), (1, 0)], [(0, 0), (1, 1)], [(0, 1), (1, 0)],
            [(0, 0), (2, 0)], [(0, 0), (1, 0), (2, 0)], [(0, 0), (1, 0), (2, 2)], [(0, 0), (1, 0), (2, 0), (3, 0)]]
CHILDREN = [[3, 4, 6], [5], [3, 5], [7, 8], [], [], [7], [9], [], []]


def run_both(logits, state, mask_id, budget, top_k, dtype, formulas=FORMULAS, children=CHILDREN):
    graph = spiffy.draft_graph(formulas, children)
    got = spiffy.spiffy_draft_blocks(G.to_dev(logits, dtype), G.to_dev(state), mask_id, graph, budget, top_k)
    torch.cuda.synchronize()
    want = drafting.draft_blocks(logits, state, mask_id, formulas, children, budget, top_k)
    return got, want


def assert_parity(got, want, tol=1e-4):
    sc, ws = got.score.cpu().numpy().astype(np.float64), want.score
    assert np.array_equal(np.isneginf(sc), np.isneginf(ws))
    fin = ~np.isneginf(ws)
    assert np.max(np.abs(sc[fin] - ws[fin]), initial=0.0) <= tol
    checked = 0
    for b in range(ws.shape[0]):
        # the kept set is compared where the last kept and the first dropped score are
        # further apart than the fp32 noise (the order inside the kept set does not matter)
        s = np.sort(ws[b][fin[b]])[::-1]
        budget = want.kept.shape[1]
        if len(s) > budget and s[budget - 1] - s[budget] < 10 * tol:
            continue
        checked += 1
        assert np.array_equal(got.kept[b].cpu().numpy(), want.kept[b])
        assert np.array_equal(got.tokens[b].cpu().numpy(), want.tokens[b])
        off = got.parent_off[b].cpu().numpy()
        assert np.array_equal(off, want.parent_off[b])
        assert np.array_equal(got.parent_idx[b].cpu().numpy()[:off[-1]], want.parent_idx[b][:off[-1]])
    assert int(got.dev_status.cpu().sum()) == 0
    return checked


@pytest.mark.parametrize("index,n_nodes", [(2, None), (3, None), (5, 8)])
def test_configs(index, n_nodes):
    """Draft from the root node's distribution of each configuration's workload."""
    cfg = W.config(index, n_nodes)
    w = W.make(cfg, W.seed_for(index, 60), attention=False)
    logits = np.ascontiguousarray(w.logits[:, 0])        # [B, L, V]: the true block's distribution
    state = np.ascontiguousarray(w.block_tokens[:, 0])
    got, want = run_both(logits, state, cfg.mask_id, 3, 3, torch.bfloat16)
    assert assert_parity(got, want) == cfg.batch
    assert (want.kept >= 0).all()


@pytest.mark.parametrize("dtype,V", [("f32", 1000), ("bf16", 4097), ("f32", 37), ("bf16", 33000)])
def test_ragged_vocabularies_and_budgets(dtype, V):
    r = np.random.default_rng(V)
    B, L = 3, 7
    logits = W.round_to((r.standard_normal((B, L, V)) * 3).astype(np.float32), dtype)
    per16 = 8 if dtype == "bf16" else 4
    stride = (V + per16 - 1) // per16 * per16 + per16
    state = np.where(r.random((B, L)) < 0.3, 5, V - 1).astype(np.int32)
    state[0, :] = V - 1
    state[1, 1:] = 4   # a single masked position: most formulas cannot be built
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    buf = torch.full((B, L, stride), 1e4, dtype=tdt, device="cuda")
    buf[..., :V] = G.to_dev(logits, tdt)
    graph = spiffy.draft_graph(FORMULAS, CHILDREN)
    for budget in (1, 4, 10):
        got = spiffy.spiffy_draft_blocks(buf[..., :V], G.to_dev(state), V - 1, graph, budget, 3)
        want = drafting.draft_blocks(logits, state, V - 1, FORMULAS, CHILDREN, budget, 3)
        assert assert_parity(got, want) >= 2
        assert want.kept[1].tolist()[:2] == [0, 1][:budget] or budget == 1


def test_drafts_feed_the_walk():
    """The blocks and parent lists come out in the layout the acceptance walk reads."""
    cfg = W.config(2)
    w = W.make(cfg, W.seed_for(2, 61), attention=False)
    logits, state = np.ascontiguousarray(w.logits[:, 0]), np.ascontiguousarray(w.block_tokens[:, 0])
    graph = spiffy.draft_graph(FORMULAS, CHILDREN)
    d = spiffy.spiffy_draft_blocks(G.to_dev(logits, torch.bfloat16), G.to_dev(state), cfg.mask_id, graph, 4, 3)
    # pretend the target unmasks exactly the last kept draft's tokens at the root: the walk must
    # reach that node in one hop (the current block is a parent of every draft)
    tokens = d.tokens.cpu().numpy()
    kept = d.kept.cpu().numpy()[0].tolist()
    assert all(q >= 0 for q in kept)
    node = len(kept)
    top = np.broadcast_to(tokens[:, node:node + 1], tokens.shape).astype(np.int32).copy()
    bits = np.zeros((1, 5), dtype=np.int64)
    changed = np.flatnonzero(tokens[0, node] != tokens[0, 0])
    bits[0, 0] = sum(1 << int(l) for l in changed)
    walk = spiffy.spiffy_accept_walk(d.tokens, d.parent_off, d.parent_idx, G.to_dev(top), G.to_dev(bits))
    assert walk.accepted_node.cpu().tolist() == [node] and walk.n_accepted.cpu().tolist() == [1]
    assert int(walk.dev_status.cpu().sum()) == 0


def test_nothing_left_to_draft_and_single_rank():
    """A fully unmasked block yields no draft; top_k = 1 and budget = D keep every buildable formula."""
    V, L = 64, 4
    r = np.random.default_rng(3)
    logits = (r.standard_normal((2, L, V)) * 2).astype(np.float32)
    state = np.array([[1, 2, 3, 4], [V - 1, V - 1, 7, V - 1]], dtype=np.int32)
    formulas = [[(0, 0)], [(1, 0)], [(0, 0), (1, 0)], [(0, 0), (1, 0), (2, 0)], [(3, 0)]]
    children = [[2], [2], [3], [], []]
    got, want = run_both(logits, state, V - 1, 5, 1, torch.float32, formulas, children)
    assert_parity(got, want)
    assert got.kept[0].cpu().tolist() == [-1] * 5 and got.kept[1].cpu().tolist() == [0, 1, 2, 3, -1]
    assert torch.equal(got.tokens[0], torch.from_numpy(state[0]).cuda().expand(6, L))


def test_more_than_32_vocabulary_slices():
    """A vocabulary long enough (fp32, more than 32 slices of 4096) for the build
    kernel's general slice merge, and all ten drafts kept (a parent list per node)."""
    r = np.random.default_rng(3)
    B, L, V = 2, 5, 140000
    logits = (r.standard_normal((B, L, V)) * 3).astype(np.float32)
    logits[..., V - 1] = -30.0
    state = np.full((B, L), V - 1, dtype=np.int32)
    state[1, 3] = 11
    got, want = run_both(logits, state, V - 1, 10, 3, torch.float32)
    assert assert_parity(got, want) == B
    assert int(want.parent_off[0, -1]) > 10
