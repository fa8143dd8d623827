"""Helpers of the GPU parity tests: move a synthetic workload to the device,
run the CUDA library through its C ABI, run the CPU oracle on the same inputs."""
import numpy as np
import torch

import oracle
from paper_2509_18085_b200 import spiffy
from paper_2509_18085_b200 import workloads as W

TOL = {"bf16": 2e-2, "f32": 1e-4}     # max abs error of attention outputs and confidences
MARGIN = {"bf16": 1e-3, "f32": 1e-5}  # decisions are compared when the oracle's margin exceeds this


def tdtype(cfg):
    return torch.bfloat16 if cfg.dtype == "bf16" else torch.float32


def to_dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(dtype) if dtype is not None else t


def oracle_proposer(cfg):
    """Drafts derived from an evaluation of the parent's logits (used for the
    'literal' logit recipe, whose winners are not known by construction)."""
    def proposer(rows, state):
        d = oracle.unmask_decide(rows[None, None], state[None, None], cfg.mask_id, cfg.rule,
                                 cfg.top_s, cfg.threshold)
        masked = np.flatnonzero(state == cfg.mask_id)
        ranked = sorted(masked.tolist(), key=lambda l: (-d.conf[0, 0, l], l))
        unmask = [l for l in range(len(state)) if (int(d.unmask_bits[0, 0]) >> l) & 1]
        return d.top_tok[0, 0], unmask, ranked
    return proposer


def gpu_attention(w, kernel=spiffy.ATTN_AUTO, scale=0.0):
    dt = tdtype(w.cfg)
    out = spiffy.spiffy_graph_attention(
        to_dev(w.q, dt), to_dev(w.k_prefix, dt) if w.cfg.prefix_len else None,
        to_dev(w.v_prefix, dt) if w.cfg.prefix_len else None,
        to_dev(w.k_block, dt), to_dev(w.v_block, dt), scale=scale, kernel=kernel)
    torch.cuda.synchronize()
    return out.float().cpu().numpy().astype(np.float64)


def gpu_decide(w, logits_dev=None):
    cfg = w.cfg
    logits = to_dev(w.logits, tdtype(cfg)) if logits_dev is None else logits_dev
    tokens = to_dev(w.block_tokens)
    dec = spiffy.spiffy_unmask_decide(logits, tokens, cfg.mask_id, cfg.rule, cfg.top_s, cfg.threshold)
    walk = spiffy.spiffy_accept_walk(tokens, to_dev(w.parent_off), to_dev(w.parent_idx),
                                     dec.top_tok, dec.unmask_bits)
    # the one-call form gives the same bits, whichever kernels it takes
    dec2, walk2 = spiffy.spiffy_decide_walk(logits, tokens, to_dev(w.parent_off), to_dev(w.parent_idx),
                                            cfg.mask_id, cfg.rule, cfg.top_s, cfg.threshold)
    torch.cuda.synchronize()
    assert_same_bits(dec, walk, dec2, walk2)
    return dec, walk


def assert_same_bits(dec, walk, dec2, walk2):
    """Two runs of the decision and the walk agree bit for bit (confidences are
    compared as integers so that a NaN equals itself)."""
    assert torch.equal(dec.conf.view(torch.int32), dec2.conf.view(torch.int32))
    for f in ("top_tok", "unmask_bits", "n_unmask", "dev_status"):
        assert torch.equal(getattr(dec, f), getattr(dec2, f)), f
    for f in ("accepted_node", "n_accepted", "path", "next_block", "dev_status"):
        assert torch.equal(getattr(walk, f), getattr(walk2, f)), f


def oracle_decide(w):
    cfg = w.cfg
    return oracle.verify_step(w.logits, w.block_tokens, w.parent_off, w.parent_idx, cfg.mask_id,
                              cfg.rule, cfg.top_s, cfg.threshold)


def bits_np(t):
    return t.cpu().numpy().view(np.uint64)


def assert_decision_parity(w, dec, walk, odec, owalk, tol, margin):
    """conf within tol; argmax tokens bit-exact; unmask sets, accepted node,
    hop count, path and next block bit-exact wherever the oracle certifies that
    no confidence sits within ``margin`` of the decision boundary."""
    cfg = w.cfg
    masked = w.block_tokens == cfg.mask_id
    conf = dec.conf.cpu().numpy().astype(np.float64)
    assert np.all(np.isneginf(conf[~masked]))
    assert np.max(np.abs(conf[masked] - odec.conf[masked]), initial=0.0) <= tol
    assert np.array_equal(dec.top_tok.cpu().numpy(), odec.top_tok)
    assert int(dec.dev_status.cpu().abs().sum()) == 0 and int(walk.dev_status.cpu().abs().sum()) == 0
    safe = odec.margin >= margin
    assert safe.mean() > 0.9, "the generator's guard band should keep decisions away from the boundary"
    assert np.array_equal(bits_np(dec.unmask_bits)[safe], odec.unmask_bits[safe])
    assert np.array_equal(dec.n_unmask.cpu().numpy()[safe], odec.n_unmask[safe])
    seq_safe = safe.all(axis=1)
    for name in ("accepted_node", "n_accepted", "path", "next_block"):
        got = getattr(walk, name).cpu().numpy()
        assert np.array_equal(got[seq_safe], getattr(owalk, name)[seq_safe]), name
    # The walk is integer work: whatever the margins, it must equal the oracle's
    # walk run on the GPU's own per-node decisions, for every sequence.
    assert_walk_follows_decisions(w, dec, walk)
    return int(seq_safe.sum())


def assert_walk_follows_decisions(w, dec, walk):
    """The GPU's walk against the oracle's walk on the GPU's own (top_tok,
    unmask_bits): bit-exact for every sequence."""
    cfg = w.cfg
    top = dec.top_tok.cpu().numpy()
    bits = bits_np(dec.unmask_bits)
    sel = (bits[..., None] >> np.arange(cfg.block_len, dtype=np.uint64)) & np.uint64(1)
    nxt = np.where(sel.astype(bool), top, w.block_tokens).astype(np.int32)
    ow = oracle.accept_walk(w.block_tokens, w.parent_off, w.parent_idx, nxt, bits)
    for name in ("accepted_node", "n_accepted", "path", "next_block"):
        assert np.array_equal(getattr(walk, name).cpu().numpy(), getattr(ow, name)), name
    return ow
