"""ctypes binding of ``libspiffy.so`` -- argument marshalling only.

The three entry points carry the names of the C ABI (``include/spiffy.h``) and
take torch CUDA tensors; every step of the path runs in the library's kernels.
There is no CPU fallback: when the library has not been built, or a tensor is
not on a CUDA device, the call raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libspiffy.so")

OK, EINVAL, EUNSUPPORTED, EWORKSPACE, EGRAPH, ECUDA = range(6)
F32, BF16 = 0, 1
RULE_TOPS, RULE_THRESHOLD = 0, 1
DEV_NONFINITE, DEV_BADGRAPH, DEV_TIMEOUT = 1, 2, 4
ATTN_AUTO, ATTN_SIMT, ATTN_TCGEN05 = 0, 1, 2
ATTN_EARLY_DEPENDENTS = 0x100  # flag OR-ed into the kernel selection

DECIDE_STATIC_BYTES = 2 << 20


class SpiffyError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().spiffy_status_string(status).decode()
        super().__init__(f"{where}: {msg} (status {status})")


class AttnDesc(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("n_nodes", ctypes.c_int32),
                ("block_len", ctypes.c_int32), ("prefix_len", ctypes.c_int32),
                ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("scale", ctypes.c_float), ("kernel", ctypes.c_int32)]


class DecideDesc(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("n_nodes", ctypes.c_int32),
                ("block_len", ctypes.c_int32), ("vocab", ctypes.c_int32),
                ("logits_dtype", ctypes.c_int32), ("row_stride", ctypes.c_int64),
                ("mask_token_id", ctypes.c_int32), ("rule", ctypes.c_int32),
                ("top_s", ctypes.c_int32), ("threshold", ctypes.c_float)]


class StepDesc(ctypes.Structure):
    _fields_ = [("attn", AttnDesc), ("decide", DecideDesc), ("parent_cap", ctypes.c_int32)]


class SampleDesc(ctypes.Structure):
    _fields_ = [("temperature", ctypes.c_float), ("reserved", ctypes.c_uint32), ("seed", ctypes.c_uint64)]


class DraftDesc(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("block_len", ctypes.c_int32), ("vocab", ctypes.c_int32),
                ("logits_dtype", ctypes.c_int32), ("row_stride", ctypes.c_int64),
                ("mask_token_id", ctypes.c_int32), ("n_formulas", ctypes.c_int32),
                ("top_k", ctypes.c_int32), ("budget", ctypes.c_int32), ("parent_cap", ctypes.c_int32)]


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library; raises when it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with "
                "`python -m paper_2509_18085_b200.build` (there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, sz, i32 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int32
        L.spiffy_graph_attention_workspace.restype = sz
        L.spiffy_graph_attention_workspace.argtypes = [ctypes.POINTER(AttnDesc)]
        L.spiffy_graph_attention.restype = ctypes.c_int
        L.spiffy_graph_attention.argtypes = [ctypes.POINTER(AttnDesc)] + [vp] * 8 + [sz, vp]
        L.spiffy_full_sequence_attention_workspace.restype = sz
        L.spiffy_full_sequence_attention_workspace.argtypes = [ctypes.POINTER(AttnDesc), i32]
        L.spiffy_full_sequence_attention.restype = ctypes.c_int
        L.spiffy_full_sequence_attention.argtypes = [ctypes.POINTER(AttnDesc), i32] + [vp] * 12 + [sz, vp]
        L.spiffy_unmask_decide_workspace.restype = sz
        L.spiffy_unmask_decide_workspace.argtypes = [ctypes.POINTER(DecideDesc)]
        L.spiffy_unmask_decide.restype = ctypes.c_int
        L.spiffy_unmask_decide.argtypes = [ctypes.POINTER(DecideDesc)] + [vp] * 8 + [sz, vp]
        L.spiffy_unmask_decide_static.restype = ctypes.c_int
        L.spiffy_unmask_decide_static.argtypes = [ctypes.POINTER(DecideDesc)] + [vp] * 8
        L.spiffy_draft_blocks_workspace.restype = sz
        L.spiffy_draft_blocks_workspace.argtypes = [ctypes.POINTER(DraftDesc)]
        L.spiffy_draft_blocks.restype = ctypes.c_int
        L.spiffy_draft_blocks.argtypes = [ctypes.POINTER(DraftDesc)] + [vp] * 14 + [sz, vp]
        L.spiffy_accept_walk.restype = ctypes.c_int
        L.spiffy_accept_walk.argtypes = [ctypes.POINTER(DecideDesc), vp, vp, vp, i32] + [vp] * 8
        L.spiffy_decide_walk.restype = ctypes.c_int
        L.spiffy_decide_walk.argtypes = [ctypes.POINTER(DecideDesc), vp, vp, vp, vp, i32] + [vp] * 11 + [sz, vp]
        L.spiffy_decide_walk_lazy_workspace.restype = sz
        L.spiffy_decide_walk_lazy_workspace.argtypes = [ctypes.POINTER(DecideDesc)]
        L.spiffy_decide_walk_lazy.restype = ctypes.c_int
        L.spiffy_decide_walk_lazy.argtypes = L.spiffy_decide_walk.argtypes
        L.spiffy_stage_masked_rows.restype = ctypes.c_int
        L.spiffy_stage_masked_rows.argtypes = [vp, vp, ctypes.c_int64, vp, i32, ctypes.c_int64, vp]
        L.spiffy_unmask_decide_sampled_workspace.restype = sz
        L.spiffy_unmask_decide_sampled_workspace.argtypes = [ctypes.POINTER(DecideDesc)]
        L.spiffy_sampled_slice_width.restype = ctypes.c_int64
        L.spiffy_sampled_slice_width.argtypes = [ctypes.POINTER(DecideDesc)]
        L.spiffy_unmask_decide_sampled.restype = ctypes.c_int
        L.spiffy_unmask_decide_sampled.argtypes = [ctypes.POINTER(DecideDesc), ctypes.POINTER(SampleDesc)] + \
            [vp] * 8 + [sz, vp]
        L.spiffy_lmhead_decide_workspace.restype = sz
        L.spiffy_lmhead_decide_workspace.argtypes = [ctypes.POINTER(DecideDesc), i32]
        L.spiffy_lmhead_decide.restype = ctypes.c_int
        L.spiffy_lmhead_decide.argtypes = [ctypes.POINTER(DecideDesc), i32] + [vp] * 9 + [sz, vp]
        L.spiffy_verify_step_host_workspace.restype = sz
        L.spiffy_verify_step_host_workspace.argtypes = [ctypes.POINTER(StepDesc)]
        L.spiffy_verify_step_host.restype = ctypes.c_int
        L.spiffy_verify_step_host.argtypes = [ctypes.POINTER(StepDesc)] + [vp] * 15 + [sz, vp]
        L.spiffy_status_string.restype = ctypes.c_char_p
        L.spiffy_status_string.argtypes = [ctypes.c_int]
        L.spiffy_launch_count.restype = ctypes.c_uint64
        L.spiffy_launch_count.argtypes = []
        L.spiffy_set_wait_limits.restype = None
        L.spiffy_set_wait_limits.argtypes = [ctypes.c_int64, ctypes.c_int64, i32]
        _lib = L
    return _lib


def launch_count() -> int:
    return int(lib().spiffy_launch_count())


def set_wait_limits(mbarrier_polls: int = -1, flag_polls: int = -1, lazy_extra_arrivals: int = 0):
    """Failure-detection hook (spiffy_set_wait_limits): lowers the poll limits of
    the library's bounded device-side waits so that a test can see one run out;
    called without arguments it restores the defaults."""
    lib().spiffy_set_wait_limits(int(mbarrier_polls), int(flag_polls), int(lazy_extra_arrivals))


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _dev(t: Optional[torch.Tensor], name: str, dtype=None) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must live on a CUDA device (no CPU path exists)")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    return t.data_ptr()


def _stream(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def _check(status: int, where: str):
    if status != OK:
        raise SpiffyError(status, where)


def attn_desc(q, k_prefix, k_block, scale=0.0, kernel=ATTN_AUTO) -> AttnDesc:
    B, N, L, Hq, d = q.shape
    P = 0 if k_prefix is None else k_prefix.shape[1]
    Hkv = k_block.shape[3]
    return AttnDesc(B, N, L, P, Hq, Hkv, d, _dtype_code(q), float(scale), int(kernel))


def spiffy_graph_attention_workspace(desc: AttnDesc) -> int:
    return int(lib().spiffy_graph_attention_workspace(ctypes.byref(desc)))


def spiffy_graph_attention(q, k_prefix, v_prefix, k_block, v_block, out=None,
                           scale: float = 0.0, kernel: int = ATTN_AUTO,
                           dev_status=None, workspace=None, stream=None):
    """Packed draft-graph attention.  q [B,N,L,Hq,d]; k/v_prefix [B,P,Hkv,d];
    k/v_block [B,N,L,Hkv,d]; returns out [B,N,L,Hq,d] (allocated when None)."""
    desc = attn_desc(q, k_prefix, k_block, scale, kernel)
    if out is None:
        out = torch.empty_like(q)
    need = spiffy_graph_attention_workspace(desc)
    if need and workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    st = lib().spiffy_graph_attention(
        ctypes.byref(desc), _dev(q, "q"), _dev(k_prefix, "k_prefix", q.dtype),
        _dev(v_prefix, "v_prefix", q.dtype), _dev(k_block, "k_block", q.dtype),
        _dev(v_block, "v_block", q.dtype), _dev(out, "out", q.dtype),
        _dev(dev_status, "dev_status", torch.int32), _dev(workspace, "workspace"),
        ws_bytes, _stream(stream))
    _check(st, "spiffy_graph_attention")
    return out


def decide_desc(logits, block_tokens, mask_token_id, rule, top_s=1, threshold=0.9) -> DecideDesc:
    B, N, L = block_tokens.shape
    V = logits.shape[-1]
    row_stride = logits.stride(-2) if logits.dim() >= 2 else V
    return DecideDesc(B, N, L, V, _dtype_code(logits), int(row_stride), int(mask_token_id),
                      int(rule), int(top_s), float(threshold))


def spiffy_unmask_decide_workspace(desc: DecideDesc) -> int:
    return int(lib().spiffy_unmask_decide_workspace(ctypes.byref(desc)))


def spiffy_full_sequence_attention(q_nodes, q_suffix, k_prefix, v_prefix, k_suffix, v_suffix, k_block,
                                   v_block, scale: float = 0.0, out_nodes=None, out_suffix=None,
                                   dev_status=None, workspace=None, stream=None):
    """The verification attention of a full-sequence bidirectional model that
    caches only its prefix (Fig. 3 caption, App. A.2): the block being decoded
    (node 0) and the trailing masked blocks attend to the whole true sequence,
    every draft block to the prefix, the trailing blocks and itself.
    q_nodes [B,N,L,Hq,d], q_suffix [B,S,Hq,d], k/v_prefix [B,P,Hkv,d], k/v_suffix
    [B,S,Hkv,d], k/v_block [B,N,L,Hkv,d], all bf16, d = 128, S <= 1024.
    Returns (out_nodes [B,N,L,Hq,d], out_suffix [B,S,Hq,d])."""
    desc = attn_desc(q_nodes, k_prefix, k_block, scale, ATTN_TCGEN05)
    S = int(q_suffix.shape[1])
    if out_nodes is None:
        out_nodes = torch.empty_like(q_nodes)
    if out_suffix is None:
        out_suffix = torch.empty_like(q_suffix)
    need = int(lib().spiffy_full_sequence_attention_workspace(ctypes.byref(desc), S))
    if need and workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=q_nodes.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    dt = q_nodes.dtype
    st = lib().spiffy_full_sequence_attention(
        ctypes.byref(desc), S, _dev(q_nodes, "q_nodes"), _dev(q_suffix, "q_suffix", dt),
        _dev(k_prefix, "k_prefix", dt), _dev(v_prefix, "v_prefix", dt), _dev(k_suffix, "k_suffix", dt),
        _dev(v_suffix, "v_suffix", dt), _dev(k_block, "k_block", dt), _dev(v_block, "v_block", dt),
        _dev(out_nodes, "out_nodes", dt), _dev(out_suffix, "out_suffix", dt),
        _dev(dev_status, "dev_status", torch.int32), _dev(workspace, "workspace"), ws_bytes, _stream(stream))
    _check(st, "spiffy_full_sequence_attention")
    return out_nodes, out_suffix


@dataclass
class Decision:
    conf: torch.Tensor         # [B,N,L] float32
    top_tok: torch.Tensor      # [B,N,L] int32
    unmask_bits: torch.Tensor  # [B,N] int64 holding the uint64 bit sets
    n_unmask: torch.Tensor     # [B,N] int32
    dev_status: torch.Tensor   # [B] int32


def _logits_ptr(logits: torch.Tensor) -> int:
    if not logits.is_cuda:
        raise ValueError("logits must live on a CUDA device (no CPU path exists)")
    if logits.stride(-1) != 1:
        raise ValueError("logits rows must be dense")
    if logits.dim() == 4:
        B, N, L, _ = logits.shape
        rs = logits.stride(2)
        if (N > 1 and logits.stride(1) != L * rs) or (B > 1 and logits.stride(0) != N * L * rs):
            raise ValueError("logits rows must be equally spaced")
    return logits.data_ptr()


def spiffy_unmask_decide(logits, block_tokens, mask_token_id: int, rule: int,
                         top_s: int = 1, threshold: float = 0.9, out: Optional[Decision] = None,
                         workspace=None, stream=None) -> Decision:
    """Steps 1-4 of Algorithm 1 for every node.  logits [B,N,L,V] (rows may be
    a strided view of a wider buffer), block_tokens [B,N,L] int32."""
    desc = decide_desc(logits, block_tokens, mask_token_id, rule, top_s, threshold)
    B, N, L = block_tokens.shape
    dev = logits.device
    if out is None:
        out = _new_decision(B, N, L, dev)
    need = spiffy_unmask_decide_workspace(desc)
    if workspace is None:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
    st = lib().spiffy_unmask_decide(
        ctypes.byref(desc), _logits_ptr(logits), _dev(block_tokens, "block_tokens", torch.int32),
        _dev(out.conf, "conf", torch.float32), _dev(out.top_tok, "top_tok", torch.int32),
        _dev(out.unmask_bits, "unmask_bits", torch.int64),
        _dev(out.n_unmask, "n_unmask", torch.int32),
        _dev(out.dev_status, "dev_status", torch.int32), _dev(workspace, "workspace"),
        workspace.numel() * workspace.element_size(), _stream(stream))
    _check(st, "spiffy_unmask_decide")
    return out


def spiffy_unmask_decide_sampled(logits, block_tokens, mask_token_id: int, rule: int, temperature: float,
                                 seed: int, top_s: int = 1, threshold: float = 0.9,
                                 out: Optional[Decision] = None, workspace=None, stream=None) -> Decision:
    """Steps 1-4 of Algorithm 1 at sampling temperature T > 0: tokens drawn from
    softmax(x / T) in two levels (Gumbel-max over vocabulary slices, inversion
    of the running sum inside the chosen slice) with Philox4x32-10 noise that
    follows the block's state (sequence, position, slice, masked count), never
    the node's index; conf is the drawn token's probability."""
    desc = decide_desc(logits, block_tokens, mask_token_id, rule, top_s, threshold)
    sample = SampleDesc(float(temperature), 0, int(seed) & 0xFFFFFFFFFFFFFFFF)
    B, N, L = block_tokens.shape
    dev = logits.device
    if out is None:
        out = _new_decision(B, N, L, dev)
    if workspace is None:
        need = int(lib().spiffy_unmask_decide_sampled_workspace(ctypes.byref(desc)))
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
    st = lib().spiffy_unmask_decide_sampled(
        ctypes.byref(desc), ctypes.byref(sample), _logits_ptr(logits),
        _dev(block_tokens, "block_tokens", torch.int32),
        _dev(out.conf, "conf", torch.float32), _dev(out.top_tok, "top_tok", torch.int32),
        _dev(out.unmask_bits, "unmask_bits", torch.int64),
        _dev(out.n_unmask, "n_unmask", torch.int32),
        _dev(out.dev_status, "dev_status", torch.int32), _dev(workspace, "workspace"),
        workspace.numel() * workspace.element_size(), _stream(stream))
    _check(st, "spiffy_unmask_decide_sampled")
    return out


def spiffy_sampled_slice_width(desc: DecideDesc) -> int:
    """Width of the vocabulary slices of the sampled decision's two-level draw."""
    return int(lib().spiffy_sampled_slice_width(ctypes.byref(desc)))


def spiffy_lmhead_decide(hidden_states, weight, block_tokens, mask_token_id: int, rule: int,
                         top_s: int = 1, threshold: float = 0.9, out: Optional[Decision] = None,
                         workspace=None, stream=None) -> Decision:
    """Steps 1-4 of Algorithm 1 straight from the hidden states: logits =
    hidden_states @ weight.T are formed and reduced on the tensor cores without
    ever being written.  hidden_states [B,N,L,H] bf16 (H a multiple of 128),
    weight [V,H] bf16, block_tokens [B,N,L] int32."""
    B, N, L = block_tokens.shape
    H = hidden_states.shape[-1]
    V = weight.shape[0]
    if hidden_states.dtype != torch.bfloat16 or weight.dtype != torch.bfloat16:
        raise ValueError("hidden_states and weight must be bf16")
    if tuple(hidden_states.shape) != (B, N, L, H) or weight.shape[1] != H:
        raise ValueError("hidden_states must be [B,N,L,H] and weight [V,H]")
    if not hidden_states.is_contiguous() or not weight.is_contiguous():
        raise ValueError("hidden_states and weight must be contiguous")
    desc = DecideDesc(B, N, L, V, BF16, V, int(mask_token_id), int(rule), int(top_s), float(threshold))
    dev = hidden_states.device
    if out is None:
        out = _new_decision(B, N, L, dev)
    if workspace is None:
        need = int(lib().spiffy_lmhead_decide_workspace(ctypes.byref(desc), int(H)))
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
    st = lib().spiffy_lmhead_decide(
        ctypes.byref(desc), int(H), _dev(hidden_states, "hidden_states"), _dev(weight, "weight"),
        _dev(block_tokens, "block_tokens", torch.int32),
        _dev(out.conf, "conf", torch.float32), _dev(out.top_tok, "top_tok", torch.int32),
        _dev(out.unmask_bits, "unmask_bits", torch.int64),
        _dev(out.n_unmask, "n_unmask", torch.int32),
        _dev(out.dev_status, "dev_status", torch.int32), _dev(workspace, "workspace"),
        workspace.numel() * workspace.element_size(), _stream(stream))
    _check(st, "spiffy_lmhead_decide")
    return out


def spiffy_unmask_decide_static(logits, block_tokens, mask_token_id: int, rule: int, out: Decision,
                                top_s: int = 1, threshold: float = 0.9, stream=None) -> Decision:
    """The decision step without any workspace: scratch lives in a fixed array
    inside the library (``DECIDE_STATIC_BYTES``), for callers that cannot
    allocate device memory at call time.  ``out`` must be preallocated by the
    caller -- this wrapper allocates nothing either.  Calls that overlap on the
    GPU share that array and race; shapes that need more scratch raise
    ``SpiffyError`` with status ``EUNSUPPORTED``."""
    desc = decide_desc(logits, block_tokens, mask_token_id, rule, top_s, threshold)
    st = lib().spiffy_unmask_decide_static(
        ctypes.byref(desc), _logits_ptr(logits), _dev(block_tokens, "block_tokens", torch.int32),
        _dev(out.conf, "conf", torch.float32), _dev(out.top_tok, "top_tok", torch.int32),
        _dev(out.unmask_bits, "unmask_bits", torch.int64),
        _dev(out.n_unmask, "n_unmask", torch.int32),
        _dev(out.dev_status, "dev_status", torch.int32), _stream(stream))
    _check(st, "spiffy_unmask_decide_static")
    return out


@dataclass
class Walk:
    accepted_node: torch.Tensor  # [B] int32
    n_accepted: torch.Tensor     # [B] int32
    path: torch.Tensor           # [B,N] int32
    next_block: torch.Tensor     # [B,L] int32
    dev_status: torch.Tensor     # [B] int32


def spiffy_accept_walk(block_tokens, parent_off, parent_idx, top_tok, unmask_bits,
                       out: Optional[Walk] = None, stream=None) -> Walk:
    """Step 5 of Algorithm 1.  parent_off [B,N+1], parent_idx [B,cap] int32."""
    B, N, L = block_tokens.shape
    dev = block_tokens.device
    desc = DecideDesc(B, N, L, 0, F32, 0, 0, 0, 1, 0.0)
    if out is None:
        out = _new_walk(B, N, L, dev)
    if tuple(parent_off.shape) != (B, N + 1) or parent_idx.dim() != 2 or parent_idx.shape[0] != B:
        raise ValueError("parent_off must be [B,N+1] and parent_idx [B,cap]")
    st = lib().spiffy_accept_walk(
        ctypes.byref(desc), _dev(block_tokens, "block_tokens", torch.int32),
        _dev(parent_off, "parent_off", torch.int32), _dev(parent_idx, "parent_idx", torch.int32),
        int(parent_idx.shape[1]), _dev(top_tok, "top_tok", torch.int32),
        _dev(unmask_bits, "unmask_bits", torch.int64),
        _dev(out.accepted_node, "accepted_node", torch.int32),
        _dev(out.n_accepted, "n_accepted", torch.int32), _dev(out.path, "path", torch.int32),
        _dev(out.next_block, "next_block", torch.int32),
        _dev(out.dev_status, "dev_status", torch.int32), _stream(stream))
    _check(st, "spiffy_accept_walk")
    return out


def _new_decision(B, N, L, dev) -> Decision:
    return Decision(torch.empty((B, N, L), dtype=torch.float32, device=dev),
                    torch.empty((B, N, L), dtype=torch.int32, device=dev),
                    torch.empty((B, N), dtype=torch.int64, device=dev),
                    torch.empty((B, N), dtype=torch.int32, device=dev),
                    torch.zeros((B,), dtype=torch.int32, device=dev))


def _new_walk(B, N, L, dev) -> Walk:
    return Walk(torch.empty((B,), dtype=torch.int32, device=dev),
                torch.empty((B,), dtype=torch.int32, device=dev),
                torch.empty((B, N), dtype=torch.int32, device=dev),
                torch.empty((B, L), dtype=torch.int32, device=dev),
                torch.zeros((B,), dtype=torch.int32, device=dev))


def spiffy_decide_walk_lazy_workspace(desc: DecideDesc) -> int:
    return int(lib().spiffy_decide_walk_lazy_workspace(ctypes.byref(desc)))


def spiffy_decide_walk(logits, block_tokens, parent_off, parent_idx, mask_token_id: int, rule: int,
                       top_s: int = 1, threshold: float = 0.9, decision: Optional[Decision] = None,
                       walk: Optional[Walk] = None, workspace=None, stream=None, lazy: bool = False):
    """Steps 1-5 of Algorithm 1 in one call: spiffy_unmask_decide followed by
    spiffy_accept_walk, fused on the device for small graphs.  With ``lazy`` the
    decision is evaluated only for the nodes the walk reaches
    (spiffy_decide_walk_lazy): the Decision then holds those nodes' entries and
    n_unmask = -1 everywhere else.  Returns (Decision, Walk)."""
    desc = decide_desc(logits, block_tokens, mask_token_id, rule, top_s, threshold)
    B, N, L = block_tokens.shape
    dev = logits.device
    decision = decision or _new_decision(B, N, L, dev)
    walk = walk or _new_walk(B, N, L, dev)
    if tuple(parent_off.shape) != (B, N + 1) or parent_idx.dim() != 2 or parent_idx.shape[0] != B:
        raise ValueError("parent_off must be [B,N+1] and parent_idx [B,cap]")
    need = spiffy_decide_walk_lazy_workspace(desc) if lazy else spiffy_unmask_decide_workspace(desc)
    if workspace is None:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
    entry = lib().spiffy_decide_walk_lazy if lazy else lib().spiffy_decide_walk
    st = entry(
        ctypes.byref(desc), _logits_ptr(logits), _dev(block_tokens, "block_tokens", torch.int32),
        _dev(parent_off, "parent_off", torch.int32), _dev(parent_idx, "parent_idx", torch.int32),
        int(parent_idx.shape[1]),
        _dev(decision.conf, "conf", torch.float32), _dev(decision.top_tok, "top_tok", torch.int32),
        _dev(decision.unmask_bits, "unmask_bits", torch.int64),
        _dev(decision.n_unmask, "n_unmask", torch.int32),
        _dev(decision.dev_status, "decide_status", torch.int32),
        _dev(walk.accepted_node, "accepted_node", torch.int32),
        _dev(walk.n_accepted, "n_accepted", torch.int32), _dev(walk.path, "path", torch.int32),
        _dev(walk.next_block, "next_block", torch.int32),
        _dev(walk.dev_status, "walk_status", torch.int32), _dev(workspace, "workspace"),
        workspace.numel() * workspace.element_size(), _stream(stream))
    _check(st, "spiffy_decide_walk_lazy" if lazy else "spiffy_decide_walk")
    return decision, walk


def spiffy_stage_masked_rows(src_logits, dst_logits, tokens, mask_token_id: int, stream=None):
    """Copies the logits rows of still-masked positions from ``src_logits`` (a
    pinned host tensor, or a device tensor) into the device tensor
    ``dst_logits`` of the same shape; ``tokens`` (pinned host or device int32)
    has one entry per row."""
    if not dst_logits.is_cuda or not dst_logits.is_contiguous():
        raise ValueError("dst_logits must be a contiguous CUDA tensor")
    for name, t in (("src_logits", src_logits), ("tokens", tokens)):
        if not (t.is_cuda or t.is_pinned()) or not t.is_contiguous():
            raise ValueError(f"{name} must be a contiguous CUDA or pinned host tensor")
    if src_logits.shape != dst_logits.shape or src_logits.dtype != dst_logits.dtype:
        raise ValueError("src_logits and dst_logits differ in shape or dtype")
    if tokens.dtype != torch.int32 or tokens.numel() != src_logits.numel() // src_logits.shape[-1]:
        raise ValueError("tokens must be int32 with one entry per logits row")
    row_bytes = src_logits.shape[-1] * src_logits.element_size()
    st = lib().spiffy_stage_masked_rows(ctypes.c_void_p(src_logits.data_ptr()),
                                        ctypes.c_void_p(dst_logits.data_ptr()), row_bytes,
                                        ctypes.c_void_p(tokens.data_ptr()), int(mask_token_id),
                                        tokens.numel(), _stream(stream))
    _check(st, "spiffy_stage_masked_rows")
    return dst_logits


def _host(t: Optional[torch.Tensor], name: str, dtype=None) -> Optional[int]:
    if t is None:
        return None
    if t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous host tensor")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    return t.data_ptr()


def step_desc(q, k_prefix, k_block, logits, block_tokens, parent_idx, mask_token_id, rule, top_s=1,
              threshold=0.9, scale=0.0, kernel=ATTN_AUTO) -> StepDesc:
    return StepDesc(attn_desc(q, k_prefix, k_block, scale, kernel),
                    decide_desc(logits, block_tokens, mask_token_id, rule, top_s, threshold),
                    int(parent_idx.shape[1]))


def spiffy_verify_step_host_workspace(desc: StepDesc) -> int:
    return int(lib().spiffy_verify_step_host_workspace(ctypes.byref(desc)))


def spiffy_verify_step_host(desc: StepDesc, q, k_prefix, v_prefix, k_block, v_block, logits, block_tokens,
                            parent_off, parent_idx, accepted_node, n_accepted, path, next_block, status,
                            device_workspace, stream=None):
    """One whole verification step from HOST tensors (pinned for speed): the
    inputs are copied in, attention + decision + walk run on the device, and the
    verdict (accepted_node [B], n_accepted [B], path [B,N], next_block [B,L], all
    int32 host tensors, plus status [1+2B]) is back when the call returns."""
    i32 = torch.int32
    dt = q.dtype
    st = lib().spiffy_verify_step_host(
        ctypes.byref(desc), _host(q, "q"), _host(k_prefix, "k_prefix", dt), _host(v_prefix, "v_prefix", dt),
        _host(k_block, "k_block", dt), _host(v_block, "v_block", dt), _host(logits, "logits"),
        _host(block_tokens, "block_tokens", i32), _host(parent_off, "parent_off", i32),
        _host(parent_idx, "parent_idx", i32), _host(accepted_node, "accepted_node", i32),
        _host(n_accepted, "n_accepted", i32), _host(path, "path", i32), _host(next_block, "next_block", i32),
        _host(status, "status", i32), _dev(device_workspace, "device_workspace"),
        device_workspace.numel() * device_workspace.element_size(), _stream(stream))
    _check(st, "spiffy_verify_step_host")
    return accepted_node, n_accepted, path, next_block, status


@dataclass
class DraftGraph:
    """The calibrated draft graph on the device: D formulas of (position rank,
    vocabulary rank) pairs and each formula's children, both in CSR form."""
    formula_off: torch.Tensor  # [D+1] int32
    formula_i: torch.Tensor
    formula_j: torch.Tensor
    child_off: torch.Tensor    # [D+1] int32
    child_idx: torch.Tensor

    @property
    def n_formulas(self) -> int:
        return self.formula_off.numel() - 1


def draft_graph(formulas, children, device="cuda") -> DraftGraph:
    """formulas: list of lists of (i, j); children: list of lists of formula indices."""
    def csr(lists, width):
        off, flat = [0], []
        for x in lists:
            flat += list(x)
            off.append(len(flat))
        flat = flat or [(0,) * width if width > 1 else 0]
        return off, flat
    foff, pairs = csr(formulas, 2)
    coff, kids = csr(children, 1)
    t = lambda a: torch.tensor(a, dtype=torch.int32, device=device)
    return DraftGraph(t(foff), t([p[0] for p in pairs]), t([p[1] for p in pairs]), t(coff), t(kids))


@dataclass
class Drafts:
    tokens: torch.Tensor      # [B, D*+1, L] int32
    kept: torch.Tensor        # [B, D*] int32
    score: torch.Tensor       # [B, D] float32
    parent_off: torch.Tensor  # [B, D*+2] int32
    parent_idx: torch.Tensor  # [B, cap] int32
    dev_status: torch.Tensor  # [B] int32


def spiffy_draft_blocks(logits, state, mask_token_id: int, graph: DraftGraph, budget: int, top_k: int,
                        parent_cap: int = 0, out: Optional[Drafts] = None, workspace=None,
                        stream=None) -> Drafts:
    """Drafting and pruning.  logits [B,L,V] (rows may be a strided view), state [B,L] int32."""
    B, L = state.shape
    V = logits.shape[-1]
    D = graph.n_formulas
    cap = parent_cap or max(4, (budget + 1) * budget // 2)
    row_stride = logits.stride(-2)
    if B > 1 and logits.stride(0) != L * row_stride:
        raise ValueError("logits rows must be equally spaced")
    desc = DraftDesc(B, L, V, _dtype_code(logits), int(row_stride), int(mask_token_id), D, int(top_k),
                     int(budget), int(cap))
    dev = logits.device
    if out is None:
        out = Drafts(torch.empty((B, budget + 1, L), dtype=torch.int32, device=dev),
                     torch.empty((B, budget), dtype=torch.int32, device=dev),
                     torch.empty((B, D), dtype=torch.float32, device=dev),
                     torch.empty((B, budget + 2), dtype=torch.int32, device=dev),
                     torch.zeros((B, cap), dtype=torch.int32, device=dev),
                     torch.zeros((B,), dtype=torch.int32, device=dev))
    need = int(lib().spiffy_draft_blocks_workspace(ctypes.byref(desc)))
    if workspace is None:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
    i32 = torch.int32
    st = lib().spiffy_draft_blocks(
        ctypes.byref(desc), _logits_ptr(logits) if logits.dim() == 4 else logits.data_ptr(),
        _dev(state, "state", i32), _dev(graph.formula_off, "formula_off", i32),
        _dev(graph.formula_i, "formula_i", i32), _dev(graph.formula_j, "formula_j", i32),
        _dev(graph.child_off, "child_off", i32), _dev(graph.child_idx, "child_idx", i32),
        _dev(out.tokens, "tokens", i32), _dev(out.kept, "kept", i32),
        _dev(out.score, "score", torch.float32), _dev(out.parent_off, "parent_off", i32),
        _dev(out.parent_idx, "parent_idx", i32), _dev(out.dev_status, "dev_status", i32),
        _dev(workspace, "workspace"), workspace.numel() * workspace.element_size(), _stream(stream))
    _check(st, "spiffy_draft_blocks")
    return out
