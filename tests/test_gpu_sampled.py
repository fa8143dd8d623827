"""spiffy_unmask_decide_sampled against the sampling oracle: drawn tokens bit
for bit wherever the oracle's two decisions are not within rounding of a tie
(best and second best slice score; u' Z and the edges of the token's interval
of the running sum), confidences within tolerance, the rule's decision where
its margin allows, and the losslessness invariant through the CUDA call."""
import numpy as np
import pytest
import torch

import oracle
from oracle import sampling as S
from oracle import toy
from paper_2509_18085_b200 import spiffy
from paper_2509_18085_b200 import workloads as W
import gpu_util as G

pytestmark = pytest.mark.gpu

SLICE_GAP = 1e-4  # fp32 slice scores (logarithm of an fp32 sum plus fp32 noise) against the oracle's float64
CDF_GAP = 3e-7    # running sums of fp32 exponentials (relative error 2^-22 each) as a fraction of the slice's weight


def case(seed, B, N, L, V, dtype, p_unmasked=0.3):
    r = np.random.default_rng(seed)
    logits = W.round_to((r.standard_normal((B, N, L, V)) * 2).astype(np.float32), dtype)
    mask = V - 1
    logits[..., mask] = W.round_to(np.float32(-30.0), dtype)
    tokens = np.where(r.random((B, N, L)) < p_unmasked, r.integers(0, V - 1, (B, N, L)), mask).astype(np.int32)
    tokens[:, :, 0] = mask
    return logits, tokens, mask


def check(logits, tokens, mask, dtype, rule, top_s, tau, T, seed):
    dec = spiffy.spiffy_unmask_decide_sampled(G.to_dev(logits, torch.bfloat16 if dtype == "bf16" else None),
                                              G.to_dev(tokens), mask, rule, T, seed, top_s, tau)
    torch.cuda.synchronize()
    dl = G.to_dev(logits, torch.bfloat16 if dtype == "bf16" else None)
    width = spiffy.spiffy_sampled_slice_width(spiffy.decide_desc(dl, G.to_dev(tokens), mask, rule, top_s, tau))
    assert 0 < width <= (8192 if dtype == "bf16" else 4096)
    o = S.sampled_decide(logits, tokens, mask, rule, top_s, tau, T, seed, width)
    sure = (o.slice_gap > SLICE_GAP) & (o.cdf_gap > CDF_GAP)
    got_tok = dec.top_tok.cpu().numpy()
    assert np.array_equal(got_tok[sure], o.top_tok[sure])
    assert sure.mean() > 0.97
    masked = tokens == mask
    ok = sure & masked
    np.testing.assert_allclose(dec.conf.cpu().numpy()[ok], o.conf[ok], atol=G.TOL[dtype] if dtype == "bf16" else 1e-4)
    assert np.all(np.isneginf(dec.conf.cpu().numpy()[~masked]))
    assert np.array_equal(got_tok[~masked], tokens[~masked])
    node_ok = sure.all(axis=2) & (o.margin > (1e-3 if dtype == "bf16" else 1e-4))
    assert np.array_equal(G.bits_np(dec.unmask_bits)[node_ok], o.unmask_bits[node_ok])
    assert np.array_equal(dec.n_unmask.cpu().numpy()[node_ok], o.n_unmask[node_ok])
    if logits.shape[-1] <= 10000:  # with longer vocabularies the confidences are too close to compare the rule
        assert node_ok.any()
    assert int(dec.dev_status.sum()) == 0
    return dec, o


@pytest.mark.parametrize("dtype,V", [("bf16", 8192), ("bf16", 33000), ("f32", 4100), ("f32", 1001 * 4),
                                     ("bf16", 126464), ("f32", 36), ("bf16", 8)])
@pytest.mark.parametrize("T", [0.7, 1.0])
def test_draws_match_the_oracle(dtype, V, T):
    B, N, L = (1, 2, 5) if V > 100000 else (2, 3, 9)
    logits, tokens, mask = case(V, B, N, L, V, dtype)
    for rule, S_, tau in ((spiffy.RULE_TOPS, 2, 0.0), (spiffy.RULE_THRESHOLD, 1, 0.05)):
        check(logits, tokens, mask, dtype, rule, S_, tau, T, seed=1234 + V)


def test_more_slices_than_lanes_and_long_blocks():
    """34 vocabulary slices (the slice choice loops over the lanes twice) and a
    block of 40 positions (the masked count spans two ballots)."""
    logits, tokens, mask = case(5, 1, 2, 3, 270000, "bf16", p_unmasked=0.0)
    check(logits, tokens, mask, "bf16", spiffy.RULE_TOPS, 1, 0.0, 0.9, seed=31)
    logits, tokens, mask = case(6, 1, 2, 40, 9000, "f32")
    check(logits, tokens, mask, "f32", spiffy.RULE_THRESHOLD, 1, 0.05, 1.0, seed=32)


def test_noise_ignores_the_node_and_follows_the_seed_and_the_state():
    logits, tokens, mask = case(3, 1, 1, 6, 5000, "f32", p_unmasked=0.0)
    x = np.repeat(logits, 4, axis=1)
    st = np.repeat(tokens, 4, axis=1)
    st[0, 3, 2] = 17  # node 3 is one step further
    run = lambda seed: spiffy.spiffy_unmask_decide_sampled(G.to_dev(x), G.to_dev(st), mask, spiffy.RULE_TOPS,
                                                           1.0, seed).top_tok.cpu().numpy()
    a, b, c = run(5), run(5), run(6)
    assert np.array_equal(a, b)                       # deterministic
    assert np.array_equal(a[0, 0], a[0, 1]) and np.array_equal(a[0, 0], a[0, 2])
    assert not np.array_equal(a[0, 0], c[0, 0])       # another seed, other draws
    keep = np.arange(6) != 2
    assert not np.array_equal(a[0, 0][keep], a[0, 3][keep])  # another masked count, other noise


def test_draw_frequencies_follow_the_tempered_softmax():
    """One call with many sequences: each sequence index is part of the counter,
    so the B draws of position 0 are independent samples of one distribution."""
    B, V, T = 4000, 8, 1.3
    x = np.array([1.0, 0.2, -0.5, 2.0, 0.0, 0.7, -1.0, -30.0], dtype=np.float32)
    logits = np.broadcast_to(x, (B, 1, 1, V)).copy()
    tokens = np.full((B, 1, 1), V - 1, dtype=np.int32)
    dec = spiffy.spiffy_unmask_decide_sampled(G.to_dev(logits), G.to_dev(tokens), V - 1, spiffy.RULE_TOPS, T, 77)
    tok = dec.top_tok.cpu().numpy().reshape(-1)
    p = np.exp(x.astype(np.float64) / T)
    p /= p.sum()
    freq = np.bincount(tok, minlength=V) / B
    assert np.all(np.abs(freq - p) < 4 * np.sqrt(p * (1 - p) / B) + 1e-9), (freq, p)
    np.testing.assert_allclose(dec.conf.cpu().numpy().reshape(-1), p[tok], atol=1e-5)


def test_draw_frequencies_across_slices():
    """The live entries sit in three different slices of a long vocabulary:
    level 1 (Gumbel-max over slice weights) and level 2 (inversion inside the
    slice) together must still draw from softmax(x / T)."""
    B, V, T = 3000, 20000, 0.8
    live = {5: 1.0, 4000: 0.3, 7000: -0.4, 9000: 1.5, 15000: 0.0, 19998: 0.6}
    row = np.full(V, -np.inf, dtype=np.float32)
    for v, x in live.items():
        row[v] = x
    logits = np.broadcast_to(row, (B, 1, 1, V)).copy()
    tokens = np.full((B, 1, 1), V - 1, dtype=np.int32)
    dl, dt = G.to_dev(logits, torch.bfloat16), G.to_dev(tokens)
    width = spiffy.spiffy_sampled_slice_width(spiffy.decide_desc(dl, dt, V - 1, spiffy.RULE_TOPS))
    assert len({v // width for v in live}) == 3
    dec = spiffy.spiffy_unmask_decide_sampled(dl, dt, V - 1, spiffy.RULE_TOPS, T, 4242)
    tok = dec.top_tok.cpu().numpy().reshape(-1)
    xs = np.array([float(torch.tensor(x).to(torch.bfloat16)) for x in live.values()], dtype=np.float64)
    p = np.exp(xs / T)
    p /= p.sum()
    ids = np.array(list(live))
    assert set(tok.tolist()) <= set(ids.tolist())
    freq = np.array([(tok == v).mean() for v in ids])
    assert np.all(np.abs(freq - p) < 4 * np.sqrt(p * (1 - p) / B) + 1e-9), (freq, p)
    got = dec.conf.cpu().numpy().reshape(-1)
    np.testing.assert_allclose(got, p[np.searchsorted(ids, tok)], atol=1e-5)
    assert int(dec.dev_status.sum()) == 0


def test_unusable_rows_set_the_status_bit_and_spare_the_rest():
    logits, tokens, mask = case(11, 3, 2, 4, 9000, "f32", p_unmasked=0.0)
    logits[0, 1, 2, 17] = np.nan
    logits[1, 0, 3, :] = -np.inf
    logits[1, 1, 0, 5] = np.inf
    dec = spiffy.spiffy_unmask_decide_sampled(G.to_dev(logits), G.to_dev(tokens), mask, spiffy.RULE_TOPS, 1.0, 3)
    torch.cuda.synchronize()
    status = dec.dev_status.cpu().numpy()
    assert status[0] & spiffy.DEV_NONFINITE and status[1] & spiffy.DEV_NONFINITE and status[2] == 0
    width = spiffy.spiffy_sampled_slice_width(spiffy.decide_desc(G.to_dev(logits), G.to_dev(tokens), mask,
                                                                 spiffy.RULE_TOPS))
    o = S.sampled_decide(logits[2:], tokens[2:], mask, spiffy.RULE_TOPS, 1, 0.0, 1.0, 3, width)
    # sequence 2 alone in the oracle is sequence 0 there: compare with a run that has it first
    dec2 = spiffy.spiffy_unmask_decide_sampled(G.to_dev(logits[2:]), G.to_dev(tokens[2:]), mask,
                                               spiffy.RULE_TOPS, 1.0, 3)
    sure = (o.slice_gap > SLICE_GAP) & (o.cdf_gap > CDF_GAP)
    assert np.array_equal(dec2.top_tok.cpu().numpy()[sure], o.top_tok[sure])


def test_argument_checks():
    logits, tokens, mask = case(1, 1, 2, 4, 64, "f32")
    lg, tk = G.to_dev(logits), G.to_dev(tokens)
    for bad_t in (0.0, -1.0, float("nan"), float("inf")):
        with pytest.raises(spiffy.SpiffyError):
            spiffy.spiffy_unmask_decide_sampled(lg, tk, mask, spiffy.RULE_TOPS, bad_t, 1)
    with pytest.raises(spiffy.SpiffyError):
        spiffy.spiffy_unmask_decide_sampled(lg, tk, mask, spiffy.RULE_TOPS, 1.0, 1,
                                            workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))


@pytest.mark.parametrize("seed", range(2))
def test_sampled_decoding_through_the_cuda_call_is_lossless(seed):
    """App. A at T = 1 with the CUDA sampled decision and the CUDA walk."""
    def decide(logits, states, mask_id, rule, top_s, threshold):
        d = spiffy.spiffy_unmask_decide_sampled(G.to_dev(logits), G.to_dev(states.astype(np.int32)), mask_id,
                                                rule, 1.0, 900 + seed, top_s, threshold)
        return d.top_tok.cpu().numpy(), G.bits_np(d.unmask_bits)

    def walk(states, off, idx, top_tok, unmask_bits, mask_id):
        g = spiffy.spiffy_accept_walk(G.to_dev(states.astype(np.int32)), G.to_dev(off), G.to_dev(idx),
                                      G.to_dev(top_tok.astype(np.int32)), G.to_dev(unmask_bits.view(np.int64)))
        return (g.accepted_node.cpu().numpy(), g.n_accepted.cpu().numpy(), g.path.cpu().numpy(),
                g.next_block.cpu().numpy())

    model = toy.ToyModel(seed=seed)
    s0 = np.full(model.block_len, model.mask_id, dtype=np.int32)
    s0[seed] = 2
    vanilla = toy.vanilla_decode(model, s0, oracle.RULE_TOPS, decide=decide)
    calls = model.calls
    model.calls = 0
    drafter = toy.peeking_drafter(vanilla, depth=3, wrong_prob=0.2, seed=seed, vocab=model.vocab)
    traj, accepted = toy.speculative_decode(model, s0, drafter, oracle.RULE_TOPS, decide=decide, walk=walk)
    assert len(traj) == len(vanilla) and all(np.array_equal(a, b) for a, b in zip(traj, vanilla))
    assert model.calls == calls - sum(accepted) and sum(accepted) > 0
