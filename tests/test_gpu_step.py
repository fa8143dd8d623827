"""Whole verification steps on the GPU: the full-size decision of the long
batched configuration on sampled rows, and the losslessness invariant of
App. A with the CUDA library as the back end of the toy decoder."""
import numpy as np
import pytest
import torch

import oracle
from oracle import toy
from paper_2509_18085_b200 import spiffy
from paper_2509_18085_b200 import workloads as W

import gpu_util as G

pytestmark = pytest.mark.gpu


_full_size = {}


def long_batched_workload():
    """Configuration 4's decision inputs (2 GB on the host), drawn once."""
    if "w" not in _full_size:
        cfg = W.config(4)
        _full_size["w"] = W.make(cfg, W.seed_for(4, 0), attention=False)
    return _full_size["w"]


def test_full_size_long_batched_decision_sampled():
    """Configuration 4 at full size: 4 x 32 x 32 rows of 126464 logits.  The
    oracle evaluates a sample of nodes; the walk is then checked by running
    the oracle's walk on the GPU's own per-node decisions (integer work)."""
    cfg = W.config(4)
    w = long_batched_workload()
    dec, walk = G.gpu_decide(w)
    conf = dec.conf.cpu().numpy()
    top = dec.top_tok.cpu().numpy()
    bits = G.bits_np(dec.unmask_bits)
    rng = np.random.default_rng(1)
    for _ in range(12):
        b, n = int(rng.integers(0, cfg.batch)), int(rng.integers(0, cfg.n_nodes))
        o = oracle.unmask_decide(w.logits[b:b + 1, n:n + 1], w.block_tokens[b:b + 1, n:n + 1],
                                 cfg.mask_id, cfg.rule, cfg.top_s, cfg.threshold)
        masked = w.block_tokens[b, n] == cfg.mask_id
        assert np.array_equal(top[b, n], o.top_tok[0, 0])
        assert np.max(np.abs(conf[b, n][masked] - o.conf[0, 0][masked]), initial=0) <= G.TOL["bf16"]
        if o.margin[0, 0] >= G.MARGIN["bf16"]:
            assert bits[b, n] == o.unmask_bits[0, 0]
    # planted winners: with a 4-sigma clip the planted token is the argmax by construction
    masked = w.block_tokens == cfg.mask_id
    assert np.array_equal(top[masked], w.planted_tok[masked])
    sel = (bits[..., None] >> np.arange(cfg.block_len, dtype=np.uint64)) & np.uint64(1)
    nxt = np.where(sel.astype(bool), top, w.block_tokens).astype(np.int32)
    ow = oracle.accept_walk(w.block_tokens, w.parent_off, w.parent_idx, nxt, bits)
    for name in ("accepted_node", "n_accepted", "path", "next_block"):
        assert np.array_equal(getattr(walk, name).cpu().numpy(), getattr(ow, name)), name
    assert ow.n_accepted.max() >= 1


def test_full_size_long_batched_lazy_call_equals_the_eager_one():
    """Configuration 4 at full size through spiffy_decide_walk_lazy: 4 x 32 x 16
    (position, slice) items, more than the device holds thread blocks, so every
    block loops over items of several sequences.  Walk outputs and the on-path
    decisions must be the eager call's bits; the walk itself is checked with the
    oracle's walk on the eager call's per-node decisions."""
    import test_gpu_decide_walk as T
    cfg = W.config(4)
    w = long_batched_workload()
    for _ in range(2):
        walk, lwalk, on_path = T.lazy_vs_eager(w.logits, w.block_tokens, w.parent_off, w.parent_idx,
                                               cfg.mask_id, cfg.rule, cfg.top_s, cfg.threshold,
                                               dtype=torch.bfloat16)
        assert int(lwalk.dev_status.sum()) == 0
    lg, tk = G.to_dev(w.logits, torch.bfloat16), G.to_dev(w.block_tokens)
    dec = spiffy.spiffy_unmask_decide(lg, tk, cfg.mask_id, cfg.rule, cfg.top_s, cfg.threshold)
    ow = G.assert_walk_follows_decisions(w, dec, lwalk)
    assert ow.n_accepted.max() >= 1 and on_path.sum() > cfg.batch
    _full_size.clear()  # 2 GB of host memory


def gpu_backends(dtype=torch.float32, kernel=spiffy.ATTN_AUTO):
    def attention(q, kp, vp, kb, vb):
        t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda().to(dtype)
        out = spiffy.spiffy_graph_attention(t(q), t(kp), t(vp), t(kb), t(vb), kernel=kernel)
        return out.float().cpu().numpy()

    def decide(logits, states, mask_id, rule, top_s, threshold):
        d = spiffy.spiffy_unmask_decide(G.to_dev(logits), G.to_dev(states.astype(np.int32)), mask_id,
                                        rule, top_s, threshold)
        return d.top_tok.cpu().numpy(), G.bits_np(d.unmask_bits)

    def walk(states, off, idx, top_tok, unmask_bits, mask_id):
        g = spiffy.spiffy_accept_walk(G.to_dev(states.astype(np.int32)), G.to_dev(off), G.to_dev(idx),
                                      G.to_dev(top_tok.astype(np.int32)),
                                      G.to_dev(unmask_bits.view(np.int64)))
        return (g.accepted_node.cpu().numpy(), g.n_accepted.cpu().numpy(), g.path.cpu().numpy(),
                g.next_block.cpu().numpy())

    return attention, decide, walk


@pytest.mark.parametrize("rule,S,tau", [(oracle.RULE_TOPS, 1, 0.0), (oracle.RULE_THRESHOLD, 1, 0.8)])
@pytest.mark.parametrize("seed", range(3))
def test_losslessness_with_the_cuda_library(rule, S, tau, seed):
    """Speculative decoding through the CUDA kernels visits exactly the states
    of plain decoding through the same kernels and saves one model call per
    accepted draft; both equal the oracle's trajectory."""
    attention, decide, walk = gpu_backends()
    start = np.full(8, 23, dtype=np.int32)
    start[seed] = seed + 1
    ref_model = toy.ToyModel(seed=seed)
    ref_traj = toy.vanilla_decode(ref_model, start, rule, S, tau)
    model = toy.ToyModel(seed=seed, attention=attention)
    vanilla = toy.vanilla_decode(model, start, rule, S, tau, decide=decide)
    calls = model.calls
    assert len(vanilla) == len(ref_traj) and all(np.array_equal(a, b) for a, b in zip(vanilla, ref_traj))
    total = 0
    for wrong_prob in (0.3, 0.0):  # spoiled drafts and perfect ones
        drafter = toy.peeking_drafter(vanilla, depth=3, wrong_prob=wrong_prob, seed=seed, vocab=model.vocab)
        model.calls = 0
        traj, accepted = toy.speculative_decode(model, start, drafter, rule, S, tau, decide=decide, walk=walk)
        assert len(traj) == len(vanilla) and all(np.array_equal(a, b) for a, b in zip(traj, vanilla))
        assert model.calls == calls - sum(accepted)
        total += sum(accepted)
    assert total > 0


def test_graph_replay_at_the_benchmark_configuration_matches_the_oracle():
    """The launch configuration the benchmark times: one verification step of
    the LLaDA-8B-shaped configuration captured in a CUDA graph and replayed.
    Decisions and the walk are compared bit-exactly, confidences and a sample of
    attention rows within tolerance."""
    from paper_2509_18085_b200.step import VerifyStep, inputs_from_workload
    cfg = W.config(2)
    w = W.make(cfg, W.seed_for(2, 100))
    x = inputs_from_workload(w)
    step = VerifyStep(cfg)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        step.run(x)
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            step.run(x)
        step.attn_out.zero_()
        step.decision.top_tok.zero_()
        step.walk.next_block.zero_()
        for _ in range(3):
            graph.replay()
        stream.synchronize()
    odec, owalk = G.oracle_decide(w)
    n = G.assert_decision_parity(w, step.decision, step.walk, odec, owalk, G.TOL["bf16"], G.MARGIN["bf16"])
    assert n == cfg.batch
    got = step.attn_out.float().cpu().numpy()
    for node in (0, 3, 7):
        want = oracle.graph_attention(w.q[:, node:node + 1], w.k_prefix, w.v_prefix,
                                      w.k_block[:, node:node + 1], w.v_block[:, node:node + 1])
        assert np.max(np.abs(got[:, node] - want[:, 0])) <= G.TOL["bf16"]
    assert int(step.attn_status.item()) == 0


def test_auto_speculation_through_the_cuda_drafting_call():
    """The closed loop of the method on the toy model: draft with
    spiffy_draft_blocks, verify with the CUDA decision and walk; the trajectory
    is plain decoding's and accepted drafts save model calls."""
    formulas = [[(0, 0)], [(0, 1)], [(0, 0), (1, 0)], [(0, 0), (1, 1)], [(0, 0), (1, 0), (2, 0)]]
    children = [[2, 3], [], [4], [], []]
    graph = spiffy.draft_graph(formulas, children)
    _, decide, walk = gpu_backends()

    def draft(logits, state, mask_id):
        d = spiffy.spiffy_draft_blocks(G.to_dev(logits), G.to_dev(state), mask_id, graph, 3, 2)
        return d.tokens.cpu().numpy()

    saved = 0
    for seed in range(3):
        start = np.full(8, 23, dtype=np.int32)
        start[seed] = seed + 1
        model = toy.ToyModel(seed=seed)
        vanilla = toy.vanilla_decode(model, start, oracle.RULE_TOPS, decide=decide)
        calls = model.calls
        model.calls = 0
        drafter = toy.auto_drafter(toy.ToyModel(seed=seed), formulas, children, 3, 2, draft=draft)
        traj, accepted = toy.speculative_decode(model, start, drafter, oracle.RULE_TOPS, decide=decide, walk=walk)
        assert len(traj) == len(vanilla) and all(np.array_equal(a, b) for a, b in zip(traj, vanilla))
        assert model.calls == calls - sum(accepted)
        saved += sum(accepted)
    assert saved > 0


def test_calibrated_graph_with_carried_over_distribution_on_the_cuda_path():
    """Offline calibration (Algorithm 2) on plain runs, then decoding where every
    call's drafts are built by spiffy_draft_blocks from the distribution of the
    last node the previous call accepted: no extra model call, the trajectory is
    plain decoding's (App. A) and the calibrated graph saves calls."""
    from paper_2509_18085_b200 import calibration

    def prompt(seed):
        model = toy.ToyModel(seed=7, sharpness=3.0)
        r = np.random.default_rng(seed)
        start = np.full(model.block_len, model.mask_id, dtype=np.int32)
        known = r.choice(model.block_len, size=2, replace=False)
        start[known] = r.integers(0, model.vocab - 1, size=2)
        return model, start

    _, decide, walk = gpu_backends()
    sequences = []
    for seed in range(10):
        model, start = prompt(seed)
        states = toy.vanilla_decode(model, start, oracle.RULE_TOPS, decide=decide)
        logits = [model(s[None])[0, 0] for s in states[:-1]]
        sequences += calibration.record(states[1:], logits[:-1], model.mask_id, 3, 3)
    formulas, children, _ = calibration.calibrate(calibration.build_graph(sequences, 3), 6)
    assert len(formulas) == 6
    graph = spiffy.draft_graph(formulas, children)

    def draft(logits, state, mask_id):
        d = spiffy.spiffy_draft_blocks(G.to_dev(logits), G.to_dev(state), mask_id, graph, len(formulas), 3)
        assert int(d.dev_status.max().item()) == 0
        return d.tokens.cpu().numpy()

    saved = steps = 0
    for seed in range(100, 106):
        model, start = prompt(seed)
        vanilla = toy.vanilla_decode(model, start, oracle.RULE_TOPS, decide=decide)
        calls = model.calls
        model.calls = 0
        drafter = toy.carry_over_drafter(model.mask_id, formulas, children, len(formulas), 3, draft=draft)
        traj, accepted = toy.speculative_decode(model, start, drafter, oracle.RULE_TOPS, decide=decide, walk=walk)
        assert len(traj) == len(vanilla) and all(np.array_equal(a, b) for a, b in zip(traj, vanilla))
        assert model.calls == calls - sum(accepted)
        saved += sum(accepted)
        steps += len(vanilla) - 1
    assert saved >= steps // 5


@pytest.mark.parametrize("config,pinned", [(1, True), (2, True), (1, False)])
def test_end_to_end_call_from_host_memory(config, pinned):
    """spiffy_verify_step_host: inputs in host memory, verdict back in host
    memory.  From pinned memory only the logits rows of still-masked positions
    cross the bus: with the whole device workspace poisoned beforehand (NaN in
    every row that is not copied) the verdict still equals the oracle's walk and
    the device path's, and the byte count reported is what crossed the bus.
    Pageable memory takes the plain-copy route."""
    from paper_2509_18085_b200.step import VerifyStep, inputs_from_workload
    cfg = W.config(config)
    w = W.make(cfg, W.seed_for(config, 7))
    host = inputs_from_workload(w, device="cpu", pin=pinned)
    step = VerifyStep(cfg)
    step.run_host(host)            # allocates the device workspace
    step.host_ws.fill_(0xFF)       # bf16 / fp32 NaN patterns everywhere
    acc, hops, path, nxt, status = [t.clone() for t in step.run_host(host)]
    assert status.tolist() == [0] * (1 + 2 * cfg.batch)
    odec, owalk = G.oracle_decide(w)
    assert (odec.margin >= G.MARGIN[cfg.dtype]).all()  # the generator's guard band
    assert np.array_equal(acc.numpy(), owalk.accepted_node)
    assert np.array_equal(hops.numpy(), owalk.n_accepted)
    assert np.array_equal(path.numpy(), owalk.path)
    assert np.array_equal(nxt.numpy(), owalk.next_block)
    dev_walk = step.run(inputs_from_workload(w))
    torch.cuda.synchronize()
    assert np.array_equal(acc.numpy(), dev_walk.accepted_node.cpu().numpy())
    assert np.array_equal(nxt.numpy(), dev_walk.next_block.cpu().numpy())
    masked = int((w.block_tokens == cfg.mask_id).sum())
    esz = host.logits.element_size()
    assert step.h2d_bytes(host) == host.nbytes() - (host.logits.shape[:-1].numel() - masked) * cfg.vocab * esz
    assert step.d2h_bytes() == sum(t.numel() * 4 for t in (acc, hops, path, nxt, status))


@pytest.mark.parametrize("dtype,V", [(torch.bfloat16, 126464), (torch.float32, 1000), (torch.bfloat16, 8),
                                     (torch.float32, 2052)])
@pytest.mark.parametrize("pinned", [True, False])
def test_stage_masked_rows_copies_exactly_the_masked_rows(dtype, V, pinned):
    """From pinned host memory or device memory: masked rows arrive bit for
    bit, every other row of the destination keeps what it held."""
    rows = 37
    g = torch.Generator().manual_seed(V)
    src = torch.randn((rows, V), generator=g).to(dtype)
    tokens = torch.where(torch.rand(rows, generator=g) < 0.6, 9, 3).to(torch.int32)
    tokens[0], tokens[-1] = 9, 3
    if pinned:
        src_in, tok_in = src.pin_memory(), tokens.pin_memory()
    else:
        src_in, tok_in = src.cuda(), tokens.cuda()
    dst = torch.full((rows, V), 5.0, dtype=dtype, device="cuda")
    spiffy.spiffy_stage_masked_rows(src_in, dst, tok_in, 9)
    torch.cuda.synchronize()
    got = dst.cpu()
    masked = tokens == 9
    assert torch.equal(got[masked].view(torch.uint8), src[masked].view(torch.uint8))
    assert bool((got[~masked] == 5.0).all())
    with pytest.raises(ValueError):
        spiffy.spiffy_stage_masked_rows(src, dst, tok_in, 9)  # pageable host memory
