"""Out-of-bounds and determinism checks for every call of the library, in place
of a memory checker: each output tensor and each workspace is a window of a
larger buffer whose margins hold a sentinel pattern, the call runs on ragged
shapes (L = 5, P = 127, V = 1000 and the like), and afterwards the margins must
be untouched.  Each call then runs a second time and must write the same bits
(fixed reduction orders)."""
import numpy as np
import pytest
import torch

from paper_2509_18085_b200 import spiffy
from paper_2509_18085_b200 import workloads as W
import gpu_util as G

pytestmark = pytest.mark.gpu

PAD = 256          # sentinel bytes on either side of a window (keeps 256-byte alignment)
SENTINEL = 0xA5


class Fenced:
    """Tensors carved out of sentinel-filled byte buffers."""

    def __init__(self):
        self.buffers = []

    def tensor(self, shape, dtype):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        room = (n + 255) // 256 * 256
        raw = torch.full((PAD + room + PAD,), SENTINEL, dtype=torch.uint8, device="cuda")
        assert raw.data_ptr() % 256 == 0
        self.buffers.append((raw, n))
        return raw[PAD:PAD + n].view(dtype).view(*shape)

    def bytes(self, n):
        return self.tensor((max(int(n), 16),), torch.uint8)

    def check(self):
        torch.cuda.synchronize()
        for raw, n in self.buffers:
            assert bool((raw[:PAD] == SENTINEL).all()), "a write landed in front of a buffer"
            assert bool((raw[PAD + n:] == SENTINEL).all()), "a write landed behind a buffer"

    def decision(self, B, N, L):
        d = spiffy.Decision(self.tensor((B, N, L), torch.float32), self.tensor((B, N, L), torch.int32),
                            self.tensor((B, N), torch.int64), self.tensor((B, N), torch.int32),
                            self.tensor((B,), torch.int32))
        d.dev_status.zero_()
        return d

    def walk(self, B, N, L):
        w = spiffy.Walk(self.tensor((B,), torch.int32), self.tensor((B,), torch.int32),
                        self.tensor((B, N), torch.int32), self.tensor((B, L), torch.int32),
                        self.tensor((B,), torch.int32))
        w.dev_status.zero_()
        return w


def snapshot(*objs):
    out = []
    for o in objs:
        ts = [o] if isinstance(o, torch.Tensor) else [getattr(o, f) for f in o.__dataclass_fields__]
        out += [t.clone().view(torch.uint8) for t in ts]
    return out


def same(a, b):
    return all(torch.equal(x, y) for x, y in zip(a, b))


ATTENTION_SHAPES = [
    # fp32 / d = 64: CUDA-core kernel
    (dict(batch=2, n_nodes=3, block_len=5, prefix_len=127, n_q_heads=6, n_kv_heads=2, head_dim=64), "f32"),
    # tensor-core kernel: one CTA per M-tile, a cluster pair, the workspace route, two M-tiles per CTA
    (dict(batch=1, n_nodes=3, block_len=7, prefix_len=257, n_q_heads=16, n_kv_heads=16, head_dim=128), "bf16"),
    (dict(batch=1, n_nodes=8, block_len=32, prefix_len=512, n_q_heads=16, n_kv_heads=16, head_dim=128), "bf16"),
    (dict(batch=1, n_nodes=9, block_len=8, prefix_len=1000, n_q_heads=3, n_kv_heads=3, head_dim=128), "bf16"),
    (dict(batch=3, n_nodes=9, block_len=32, prefix_len=300, n_q_heads=32, n_kv_heads=32, head_dim=128), "bf16"),
    (dict(batch=2, n_nodes=4, block_len=12, prefix_len=129, n_q_heads=6, n_kv_heads=2, head_dim=128), "bf16"),
]


@pytest.mark.parametrize("shape,dtype", ATTENTION_SHAPES)
def test_attention_stays_inside_its_buffers(shape, dtype):
    cfg = W.Config("fenced", dtype=dtype, vocab=16, rule=0, **shape)
    w = W.make(cfg, 3, decision=False)
    dt = G.tdtype(cfg)
    q, kp, vp, kb, vb = (G.to_dev(a, dt) for a in (w.q, w.k_prefix, w.v_prefix, w.k_block, w.v_block))
    f = Fenced()
    out = f.tensor(tuple(q.shape), dt)
    status = f.tensor((1,), torch.int32)
    status.zero_()
    ws = f.bytes(spiffy.spiffy_graph_attention_workspace(spiffy.attn_desc(q, kp, kb)))
    runs = []
    for _ in range(2):
        out.view(torch.uint8).fill_(0x5A)
        spiffy.spiffy_graph_attention(q, kp, vp, kb, vb, out=out, dev_status=status, workspace=ws)
        f.check()
        runs.append(snapshot(out))
    assert same(*runs)
    assert int(status[0]) == 0
    assert torch.isfinite(out.float()).all()   # every output element was written


DECISION_SHAPES = [(2, 3, 5, 1000, "f32"), (1, 2, 9, 8200, "bf16"), (3, 4, 33, 36, "f32"), (1, 8, 32, 33000, "bf16")]


def decision_case(B, N, L, V, dtype, seed=1):
    cfg = W.Config("fenced", dtype=dtype, vocab=V, rule=spiffy.RULE_THRESHOLD, threshold=0.3, batch=B,
                   n_nodes=N, block_len=L, prefix_len=0, n_q_heads=1, n_kv_heads=1, head_dim=64)
    w = W.make(cfg, seed, attention=False)
    return cfg, G.to_dev(w.logits, G.tdtype(cfg)), G.to_dev(w.block_tokens), G.to_dev(w.parent_off), \
        G.to_dev(w.parent_idx)


@pytest.mark.parametrize("B,N,L,V,dtype", DECISION_SHAPES)
def test_decision_calls_stay_inside_their_buffers(B, N, L, V, dtype):
    cfg, logits, tokens, off, idx = decision_case(B, N, L, V, dtype)
    desc = spiffy.decide_desc(logits, tokens, cfg.mask_id, cfg.rule, cfg.top_s, cfg.threshold)
    args = (cfg.mask_id, cfg.rule, cfg.top_s, cfg.threshold)

    def twice(run, *objs):
        runs = []
        for _ in range(2):
            run()
            f.check()
            runs.append(snapshot(*objs))
        assert same(*runs)

    # decision, walk
    f = Fenced()
    dec, walk = f.decision(B, N, L), f.walk(B, N, L)
    ws = f.bytes(spiffy.spiffy_unmask_decide_workspace(desc))
    twice(lambda: spiffy.spiffy_unmask_decide(logits, tokens, *args, out=dec, workspace=ws), dec)
    twice(lambda: spiffy.spiffy_accept_walk(tokens, off, idx, dec.top_tok, dec.unmask_bits, out=walk), walk)
    # both in one call, eager and lazy
    for lazy in (False, True):
        f = Fenced()
        dec2, walk2 = f.decision(B, N, L), f.walk(B, N, L)
        need = spiffy.spiffy_decide_walk_lazy_workspace(desc) if lazy else spiffy.spiffy_unmask_decide_workspace(desc)
        ws = f.bytes(need)
        twice(lambda: spiffy.spiffy_decide_walk(logits, tokens, off, idx, *args, decision=dec2, walk=walk2,
                                                workspace=ws, lazy=lazy), walk2)
        G.assert_same_bits(dec, walk, dec, walk2) if lazy else G.assert_same_bits(dec, walk, dec2, walk2)
    # sampled
    f = Fenced()
    dec3 = f.decision(B, N, L)
    ws = f.bytes(int(spiffy.lib().spiffy_unmask_decide_sampled_workspace(desc)))
    twice(lambda: spiffy.spiffy_unmask_decide_sampled(logits, tokens, cfg.mask_id, cfg.rule, 0.9, 17, cfg.top_s,
                                                      cfg.threshold, out=dec3, workspace=ws), dec3)
    assert int(dec3.dev_status.sum()) == 0
    # static scratch
    f = Fenced()
    dec4 = f.decision(B, N, L)
    twice(lambda: spiffy.spiffy_unmask_decide_static(logits, tokens, cfg.mask_id, cfg.rule, dec4, cfg.top_s,
                                                     cfg.threshold), dec4)
    G.assert_same_bits(dec, walk, dec4, walk)


def test_full_sequence_attention_stays_inside_its_buffers():
    B, N, L, P, S, H, d = 1, 3, 16, 200, 40, 4, 128
    g = torch.Generator(device="cuda")
    g.manual_seed(5)
    mk = lambda *s: torch.randn(*s, device="cuda", generator=g).to(torch.bfloat16)
    qn, qs = mk(B, N, L, H, d), mk(B, S, H, d)
    kp, vp, ks, vs, kb, vb = mk(B, P, H, d), mk(B, P, H, d), mk(B, S, H, d), mk(B, S, H, d), mk(B, N, L, H, d), \
        mk(B, N, L, H, d)
    f = Fenced()
    on, os_ = f.tensor((B, N, L, H, d), torch.bfloat16), f.tensor((B, S, H, d), torch.bfloat16)
    status = f.tensor((1,), torch.int32)
    status.zero_()
    import ctypes
    desc = spiffy.attn_desc(qn, kp, kb, 0.0, spiffy.ATTN_TCGEN05)
    ws = f.bytes(int(spiffy.lib().spiffy_full_sequence_attention_workspace(ctypes.byref(desc), S)))
    runs = []
    for _ in range(2):
        spiffy.spiffy_full_sequence_attention(qn, qs, kp, vp, ks, vs, kb, vb, out_nodes=on, out_suffix=os_,
                                              dev_status=status, workspace=ws)
        f.check()
        runs.append(snapshot(on, os_))
    assert same(*runs)
    assert int(status[0]) == 0 and torch.isfinite(on.float()).all() and torch.isfinite(os_.float()).all()
