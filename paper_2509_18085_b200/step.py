"""One whole verification step as a user drives it: device buffers, one stream,
the three library calls in order.  Plumbing only (torch for memory, streams and
copies); all arithmetic happens inside ``libspiffy.so``.

``VerifyStep`` owns preallocated outputs and workspaces so that a step issues
no allocation and can be captured into a CUDA graph.  ``run`` takes device
tensors; ``run_host`` takes pinned host tensors, copies them in, runs the step
and copies the verdict back -- the end-to-end call.
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
        # the verdict a caller reads back: accepted node, hop count, next block
        pin = dev.type == "cuda"
        host = lambda t: torch.empty_like(t, device="cpu").pin_memory() if pin else None
        self.verdict_host = (host(self.walk.accepted_node), host(self.walk.n_accepted),
                             host(self.walk.next_block))
        self.staging = None
        self.lazy_ws = None
        self.sampled_ws = None
        self.copy_stream = None
        self.copy_events = None

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

    @staticmethod
    def _masked_row_runs(host: StepInputs, mask_id: int):
        """[start, stop) runs of logit rows whose position is still masked: the
        only rows the decision step reads (Algorithm 1 ranks masked positions)."""
        m = (host.block_tokens.reshape(-1) == mask_id).to(torch.int8)
        edges = torch.diff(m, prepend=m.new_zeros(1), append=m.new_zeros(1)).nonzero().reshape(-1).tolist()
        return list(zip(edges[0::2], edges[1::2]))

    def run_host(self, host: StepInputs):
        """End to end from pinned host memory: copy the step's inputs in, run
        it, read the verdict (accepted node, hop count, next block) back.  Of
        the logits only the rows of still-masked positions cross the bus
        (spiffy_stage_masked_rows reads them from the pinned buffer); the
        staging rows of unmasked positions keep whatever they held and no
        kernel reads them."""
        if self.staging is None:
            self.staging = StepInputs(*[torch.empty_like(t, device=self.device) for t in host.tensors()])
        main = torch.cuda.current_stream()
        if self.copy_stream is None:
            self.copy_stream = torch.cuda.Stream(self.device)
            self.copy_events = (torch.cuda.Event(), torch.cuda.Event())
        # the small tensors go through the copy engine on a side stream while one kernel pulls
        # the masked logits rows over the bus; both start once the staging buffers are free
        self.copy_events[0].record(main)
        self.copy_stream.wait_event(self.copy_events[0])
        with torch.cuda.stream(self.copy_stream):
            for dst, src in zip(self.staging.tensors(), host.tensors()):
                if src is not host.logits:
                    dst.copy_(src, non_blocking=True)
            self.copy_events[1].record(self.copy_stream)
        spiffy.spiffy_stage_masked_rows(host.logits, self.staging.logits, host.block_tokens, self.cfg.mask_id)
        main.wait_event(self.copy_events[1])
        w = self.run(self.staging)
        for dst, src in zip(self.verdict_host, (w.accepted_node, w.n_accepted, w.next_block)):
            dst.copy_(src, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        return self.verdict_host

    def h2d_bytes(self, host: StepInputs) -> int:
        """Bytes ``run_host`` copies to the device for this input."""
        rows = sum(b - a for a, b in self._masked_row_runs(host, self.cfg.mask_id))
        V = host.logits.shape[-1]
        return host.nbytes() - host.logits.numel() * host.logits.element_size() \
            + rows * V * host.logits.element_size()

    def d2h_bytes(self) -> int:
        return sum(t.numel() * t.element_size() for t in self.verdict_host)
