"""CPU oracle of the Spiffy verification step -- TEST INFRASTRUCTURE ONLY.

Thin numpy/ctypes front end of ``spiffy_oracle.cpp`` (plain C++, double
precision).  Nothing in the product package may import this module: it is used
by the tests, by the smoke check and by the benchmark's CPU-baseline leg.  It
imports nothing from the CUDA package.

Functions mirror the paper: :func:`graph_attention` is the packed attention of
Sec. 4.3 with the mask of Fig. 3, :func:`unmask_decide` is steps 1-4 of
Algorithm 1, :func:`accept_walk` is step 5.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "spiffy_oracle.cpp")
_LIB = os.path.join(_HERE, "libspiffy_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (OpenMP on) when missing or stale."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    subprocess.run(["g++", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c++17",
                    "-o", tmp, _SRC], check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_max_threads.restype = ctypes.c_int
    return _lib


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def set_threads(n: int) -> None:
    _load().oracle_set_threads(ctypes.c_int(int(n)))


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def graph_attention(q, k_prefix, v_prefix, k_block, v_block, scale=None,
                    return_probs=False):
    """Sec. 4.3 attention.  q: [B,N,L,Hq,d]; k/v_prefix: [B,P,Hkv,d];
    k/v_block: [B,N,L,Hkv,d]; all float32-representable.  Returns float64
    ``out`` [B,N,L,Hq,d] (and the softmax rows [B,N,L,Hq,P+L] on request)."""
    q = _f32(q)
    kb, vb = _f32(k_block), _f32(v_block)
    B, N, L, Hq, d = q.shape
    Hkv = kb.shape[3]
    kp, vp = _f32(k_prefix), _f32(v_prefix)
    P = kp.shape[1]
    assert kp.shape == (B, P, Hkv, d) and vp.shape == kp.shape
    assert kb.shape == (B, N, L, Hkv, d) and vb.shape == kb.shape
    assert Hq % Hkv == 0
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    out = np.empty((B, N, L, Hq, d), dtype=np.float64)
    probs = np.empty((B, N, L, Hq, P + L), dtype=np.float64) if return_probs else None
    _load().oracle_graph_attention(
        B, N, L, P, Hq, Hkv, d, ctypes.c_double(scale), _ptr(q), _ptr(kp),
        _ptr(vp), _ptr(kb), _ptr(vb), _ptr(out),
        _ptr(probs) if return_probs else None)
    return (out, probs) if return_probs else out


RULE_TOPS = 0
RULE_THRESHOLD = 1


@dataclass
class Decision:
    conf: np.ndarray         # [B,N,L] float64, -inf at unmasked positions
    top_tok: np.ndarray      # [B,N,L] int32
    unmask_bits: np.ndarray  # [B,N] uint64
    n_unmask: np.ndarray     # [B,N] int32
    next_tokens: np.ndarray  # [B,N,L] int32, the state after step 4
    margin: np.ndarray       # [B,N] float64, distance of the decision from flipping
    bad_row: np.ndarray      # [B,N] int32


def unmask_decide(logits, block_tokens, mask_id, rule, top_s=1, threshold=0.9):
    """Algorithm 1 steps 1-4 for every node.  logits: [B,N,L,V] (float32-
    representable; the last axis may be a strided view), block_tokens [B,N,L]."""
    logits = np.asarray(logits)
    if logits.dtype != np.float32 or logits.strides[-1] != 4:
        logits = _f32(logits)
    B, N, L, V = logits.shape
    if logits.flags["C_CONTIGUOUS"]:
        row_stride = V
    else:  # rows of a wider buffer: [B,N,L,stride] sliced to V columns
        row_stride = logits.strides[2] // 4
        assert L == 1 or logits.strides[2] % 4 == 0 and row_stride >= V
        assert N == 1 or logits.strides[1] == L * row_stride * 4
        assert B == 1 or logits.strides[0] == N * L * row_stride * 4
        assert L > 1, "strided rows need L > 1 to define the stride"
    bt = _i32(block_tokens)
    assert bt.shape == (B, N, L) and L <= 64
    conf = np.empty((B, N, L), dtype=np.float64)
    top_tok = np.empty((B, N, L), dtype=np.int32)
    bits = np.empty((B, N), dtype=np.uint64)
    n_unmask = np.empty((B, N), dtype=np.int32)
    nxt = np.empty((B, N, L), dtype=np.int32)
    margin = np.empty((B, N), dtype=np.float64)
    bad = np.empty((B, N), dtype=np.int32)
    _load().oracle_unmask_decide(
        B, N, L, V, ctypes.c_longlong(row_stride), int(mask_id), int(rule),
        int(top_s), ctypes.c_double(threshold), _ptr(logits), _ptr(bt),
        _ptr(conf), _ptr(top_tok), _ptr(bits), _ptr(n_unmask), _ptr(nxt),
        _ptr(margin), _ptr(bad))
    return Decision(conf, top_tok, bits, n_unmask, nxt, margin, bad)


@dataclass
class Walk:
    accepted_node: np.ndarray  # [B]
    n_accepted: np.ndarray     # [B] hops
    path: np.ndarray           # [B,N], -1 padded
    next_block: np.ndarray     # [B,L]


def accept_walk(block_tokens, parent_off, parent_idx, next_tokens, unmask_bits):
    """Algorithm 1 step 5.  parent_off [B,N+1] and parent_idx [B,cap] are the
    per-sequence CSR parent lists; next_tokens/unmask_bits come from
    :func:`unmask_decide`."""
    bt = _i32(block_tokens)
    B, N, L = bt.shape
    off = _i32(parent_off)
    idx = _i32(parent_idx)
    assert off.shape == (B, N + 1) and idx.ndim == 2 and idx.shape[0] == B
    cap = idx.shape[1]
    nxt = _i32(next_tokens)
    bits = np.ascontiguousarray(unmask_bits, dtype=np.uint64)
    acc = np.empty((B,), dtype=np.int32)
    hops = np.empty((B,), dtype=np.int32)
    path = np.empty((B, N), dtype=np.int32)
    nb = np.empty((B, L), dtype=np.int32)
    _load().oracle_accept_walk(B, N, L, _ptr(bt), _ptr(off), _ptr(idx), cap,
                               _ptr(nxt), _ptr(bits), _ptr(acc), _ptr(hops),
                               _ptr(path), _ptr(nb))
    return Walk(acc, hops, path, nb)


def verify_step(logits, block_tokens, parent_off, parent_idx, mask_id, rule,
                top_s=1, threshold=0.9):
    """Steps 1-5 of Algorithm 1 in one call: (Decision, Walk)."""
    dec = unmask_decide(logits, block_tokens, mask_id, rule, top_s, threshold)
    walk = accept_walk(block_tokens, parent_off, parent_idx, dec.next_tokens,
                       dec.unmask_bits)
    return dec, walk
