"""One whole verification step as a user drives it: device buffers, one stream,
the three library calls in order.  Plumbing only (torch for memory, streams and
copies); all arithmetic happens inside ``libspiffy.so``.

``VerifyStep`` owns preallocated outputs and workspaces so that a step issues
no allocation and can be captured into a CUDA graph.  ``run`` takes device
tensors; ``run_host`` takes host tensors (pinned for speed) and makes the whole
step one C-ABI call that copies them in, runs the step and brings the verdict
back -- the end-to-end call.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass

import torch

from . import spiffy
from .workloads import Config


@dataclass
class StepInputs:
    q: torch.Tensor
    k_prefix: torch.Tensor
    v_prefix: torch.Tensor
    k_block: torch.Tensor
    v_block: torch.Tensor
    logits: torch.Tensor
    block_tokens: torch.Tensor
    parent_off: torch.Tensor
    parent_idx: torch.Tensor

    def tensors(self):
        return [self.q, self.k_prefix, self.v_prefix, self.k_block, self.v_block, self.logits,
                self.block_tokens, self.parent_off, self.parent_idx]

    def nbytes(self) -> int:
        return sum(t.numel() * t.element_size() for t in self.tensors())


def inputs_from_workload(w, device="cuda", pin=False) -> StepInputs:
    """Move a synthetic workload to ``device`` in the configuration's dtype."""
    dt = torch.bfloat16 if w.cfg.dtype == "bf16" else torch.float32

    def mv(a, dtype=None):
        t = torch.from_numpy(a)
        if dtype is not None:
            t = t.to(dtype)
        if device == "cpu":
            return t.pin_memory() if pin else t
        return t.to(device)

    return StepInputs(mv(w.q, dt), mv(w.k_prefix, dt), mv(w.v_prefix, dt), mv(w.k_block, dt),
                      mv(w.v_block, dt), mv(w.logits, dt), mv(w.block_tokens), mv(w.parent_off),
                      mv(w.parent_idx))


class VerifyStep:
    def __init__(self, cfg: Config, device="cuda", attn_kernel=spiffy.ATTN_AUTO):
        self.cfg = cfg
        self.device = torch.device(device)
        B, N, L = cfg.batch, cfg.n_nodes, cfg.block_len
        dt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
        dev = self.device
        self.attn_kernel = attn_kernel
        self.attn_out = torch.empty((B, N, L, cfg.n_q_heads, cfg.head_dim), dtype=dt, device=dev)
        self.attn_status = torch.zeros((1,), dtype=torch.int32, device=dev)
        adesc = spiffy.AttnDesc(B, N, L, cfg.prefix_len, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim,
                                spiffy.BF16 if cfg.dtype == "bf16" else spiffy.F32, 0.0, attn_kernel)
        self.attn_ws = torch.empty((max(16, spiffy.spiffy_graph_attention_workspace(adesc)),),
                                   dtype=torch.uint8, device=dev)
        ddesc = spiffy.DecideDesc(B, N, L, cfg.vocab, adesc.dtype, cfg.vocab, cfg.mask_id, cfg.rule,
                                  cfg.top_s, cfg.threshold)
        self.decide_ws = torch.empty((max(16, spiffy.spiffy_unmask_decide_workspace(ddesc)),),
                                     dtype=torch.uint8, device=dev)
        self.decision = spiffy.Decision(
            torch.empty((B, N, L), dtype=torch.float32, device=dev),
            torch.empty((B, N, L), dtype=torch.int32, device=dev),
            torch.empty((B, N), dtype=torch.int64, device=dev),
            torch.empty((B, N), dtype=torch.int32, device=dev),
            torch.zeros((B,), dtype=torch.int32, device=dev))
        self.walk = spiffy.Walk(
            torch.empty((B,), dtype=torch.int32, device=dev),
            torch.empty((B,), dtype=torch.int32, device=dev),
            torch.empty((B, N), dtype=torch.int32, device=dev),
            torch.empty((B, L), dtype=torch.int32, device=dev),
            torch.zeros((B,), dtype=torch.int32, device=dev))
        self.host_ws = None
        self.host_desc = None
        self.host_verdict = None
        self.lazy_ws = None
        self.sampled_ws = None

    # the three calls of one step, asynchronous on the current stream
    def attention(self, x: StepInputs):
        return spiffy.spiffy_graph_attention(x.q, x.k_prefix, x.v_prefix, x.k_block, x.v_block,
                                             out=self.attn_out, kernel=self.attn_kernel,
                                             dev_status=self.attn_status, workspace=self.attn_ws)

    def decide(self, x: StepInputs):
        c = self.cfg
        return spiffy.spiffy_unmask_decide(x.logits, x.block_tokens, c.mask_id, c.rule, c.top_s,
                                           c.threshold, out=self.decision, workspace=self.decide_ws)

    def accept(self, x: StepInputs):
        return spiffy.spiffy_accept_walk(x.block_tokens, x.parent_off, x.parent_idx,
                                         self.decision.top_tok, self.decision.unmask_bits,
                                         out=self.walk)

    def decide_accept(self, x: StepInputs):
        c = self.cfg
        spiffy.spiffy_decide_walk(x.logits, x.block_tokens, x.parent_off, x.parent_idx, c.mask_id,
                                  c.rule, c.top_s, c.threshold, decision=self.decision,
                                  walk=self.walk, workspace=self.decide_ws)
        return self.walk

    def decide_sampled(self, x: StepInputs, temperature: float = 1.0, seed: int = 1):
        """The decision at sampling temperature T > 0 (spiffy_unmask_decide_sampled)."""
        c = self.cfg
        if self.sampled_ws is None:
            desc = spiffy.decide_desc(x.logits, x.block_tokens, c.mask_id, c.rule, c.top_s, c.threshold)
            need = int(spiffy.lib().spiffy_unmask_decide_sampled_workspace(ctypes.byref(desc)))
            self.sampled_ws = torch.empty((max(16, need),), dtype=torch.uint8, device=self.device)
        return spiffy.spiffy_unmask_decide_sampled(x.logits, x.block_tokens, c.mask_id, c.rule, temperature,
                                                   seed, c.top_s, c.threshold, out=self.decision,
                                                   workspace=self.sampled_ws)

    def decide_accept_lazy(self, x: StepInputs):
        """The decision only for the nodes the walk reaches (spiffy_decide_walk_lazy)."""
        c = self.cfg
        if self.lazy_ws is None:
            desc = spiffy.decide_desc(x.logits, x.block_tokens, c.mask_id, c.rule, c.top_s, c.threshold)
            self.lazy_ws = torch.empty((max(16, spiffy.spiffy_decide_walk_lazy_workspace(desc)),),
                                       dtype=torch.uint8, device=self.device)
        spiffy.spiffy_decide_walk(x.logits, x.block_tokens, x.parent_off, x.parent_idx, c.mask_id,
                                  c.rule, c.top_s, c.threshold, decision=self.decision,
                                  walk=self.walk, workspace=self.lazy_ws, lazy=True)
        return self.walk

    def run(self, x: StepInputs):
        self.attention(x)
        return self.decide_accept(x)

    def run_host(self, host: StepInputs):
        """End to end from pinned host memory through the C ABI's host-buffer
        entry (spiffy_verify_step_host): the step's inputs are copied in -- of
        the logits only the rows of still-masked positions cross the bus --, the
        step runs, and the verdict (accepted node, hop count, path, next block)
        is in host memory when the call returns."""
        c = self.cfg
        B, N, L = c.batch, c.n_nodes, c.block_len
        if self.host_ws is None:
            self.host_desc = spiffy.step_desc(host.q, host.k_prefix, host.k_block, host.logits, host.block_tokens,
                                              host.parent_idx, c.mask_id, c.rule, c.top_s, c.threshold,
                                              kernel=self.attn_kernel)
            need = spiffy.spiffy_verify_step_host_workspace(self.host_desc)
            self.host_ws = torch.empty((need + 256,), dtype=torch.uint8, device=self.device)
            off = (-self.host_ws.data_ptr()) % 256
            self.host_ws = self.host_ws[off:off + need]
            pin = lambda *shape: torch.empty(shape, dtype=torch.int32).pin_memory()
            self.host_verdict = (pin(B), pin(B), pin(B, N), pin(B, L), pin(1 + 2 * B))
        kp = host.k_prefix if c.prefix_len else None
        vp = host.v_prefix if c.prefix_len else None
        return spiffy.spiffy_verify_step_host(self.host_desc, host.q, kp, vp, host.k_block, host.v_block,
                                              host.logits, host.block_tokens, host.parent_off, host.parent_idx,
                                              *self.host_verdict, self.host_ws)

    def h2d_bytes(self, host: StepInputs) -> int:
        """Bytes ``run_host`` copies to the device for this input."""
        rows = int((host.block_tokens == self.cfg.mask_id).sum())
        V = host.logits.shape[-1]
        return host.nbytes() - host.logits.numel() * host.logits.element_size() \
            + rows * V * host.logits.element_size()

    def d2h_bytes(self) -> int:
        c = self.cfg
        B, N, L = c.batch, c.n_nodes, c.block_len
        return 4 * (B + B + B * N + B * L + 1 + 2 * B)
