#!/usr/bin/env python
"""Benchmark of the Spiffy verification step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One *step* is one pass of the whole hot path over one batch of synthetic input
at the LLaDA-8B-shaped configuration: one packed draft-graph attention call
(one layer), one decision call (Algorithm 1 steps 1-4 for all nodes) and one
acceptance walk (step 5).  The metric is verify steps per second.

`value`   : inputs resident in HBM, K steps replayed from a CUDA graph that
            rotates over several distinct input sets (together larger than
            L2), timed with CUDA events on the launching stream.
`e2e`     : the same step from pinned host memory through ONE C-ABI call,
            spiffy_verify_step_host (host-to-device copies of everything the
            step reads -- of the logits, the rows of still-masked positions --
            and the device-to-host read of the verdict inside the timed region).
`roofline`: the kernel with the largest share of a step (the attention kernel)
            against the roof that binds it at this shape, timed alone by
            replaying its call over the same rotation of input sets; the
            decision kernel likewise under `roofline_decision`.
`composite_model_step`: a step as a whole model runs it, one attention call
            per layer on distinct q/K/V, then one decision + walk.
`other_shapes`: the attention and decision calls at the configurations where
            the tensor and HBM rooflines bind.
`cpu_baseline` / `--impl reference`: the CPU oracle as it stands, timed on the
            host cores (a reported baseline, not a target).

With N > 1 (launched by torchrun) every rank runs an independent replica: the
path has no sharded dimension at this configuration and no collective.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "draft-graph verify steps/sec at LLaDA-8B shape"
UNIT = "steps/s"
WORKLOAD = "config2-llada8b: B=1 N=8 L=32 P=512 Hq=Hkv=32 d=128 bf16, V=126464, threshold 0.9"
N_SETS = 6  # rotating input sets; 6 x 79.4 MB = 477 MB > 126 MB of L2


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=6000)
    ap.add_argument("--warmup", type=int, default=60)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, help="workload configuration (2 = headline)")
    ap.add_argument("--nodes", type=int, default=None, help="node count for configuration 5")
    ap.add_argument("--attn-kernel", default="auto", choices=["auto", "simt", "tcgen05"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-composite", action="store_true", help="skip the whole-model (one attention call per layer) step")
    ap.add_argument("--no-other-shapes", action="store_true", help="skip the timing of the other configurations")
    ap.add_argument("--profile", action="store_true",
                    help="bounded run for a profiler: one timed region of exactly the asked steps (rounded up to "
                         "whole rotations), no per-call timing repeats, no whole-model step, other shapes, "
                         "end-to-end or CPU-baseline legs")
    ap.add_argument("--no-early-dependents", action="store_true",
                    help="whole-model step without SPIFFY_ATTN_EARLY_DEPENDENTS on the layers' attention calls")
    ap.add_argument("--part", default="step", choices=["step", "attention", "full_sequence", "decide", "decide_walk", "decide_walk_lazy", "decide_sampled", "lmhead", "draft"],
                    help="time one library call alone on any configuration (for profiling); "
                         "the benchmark line itself is --part step")
    ap.add_argument("--sets", type=int, default=0, help="rotating input sets for --part (0 = enough to exceed L2)")
    return ap.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """nvidia-smi clock and throttle-reason samples while the GPU is busy."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.path = f"/tmp/spiffy_clocks_{os.getpid()}.csv"

    def start(self):
        try:
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "50"], stdout=self.out,
                stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    sm.append(float(parts[1]))
                    mx.append(float(parts[2]))
                    power.append(float(parts[3]))
                except ValueError:
                    continue
                for name, val in zip(names, parts[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        try:
            os.remove(self.path)
        except OSError:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        # samples under load: the upper half by power draw
        order = sorted(range(len(sm)), key=lambda i: power[i])
        loaded = [sm[i] for i in order[len(order) // 2:]]
        return {"sm_mhz": statistics.median(loaded), "sm_max_mhz": max(mx), "samples": len(sm),
                "power_w_max": max(power), "reasons": sorted(reasons)}


def algorithmic_bytes(cfg, n_masked_rows):
    e = 2 if cfg.dtype == "bf16" else 4
    B, N, L, P = cfg.batch, cfg.n_nodes, cfg.block_len, cfg.prefix_len
    attn = e * B * (2 * N * L * cfg.n_q_heads * cfg.head_dim + 2 * P * cfg.n_kv_heads * cfg.head_dim
                    + 2 * N * L * cfg.n_kv_heads * cfg.head_dim)
    decide = n_masked_rows * cfg.vocab * e + n_masked_rows * 12
    flops = 4 * B * cfg.n_q_heads * N * L * (P + L) * cfg.head_dim
    return attn, decide, flops


def oracle_step_time(cfg, w, repeats, fraction=1.0):
    """Seconds per verification step of the CPU oracle as it stands.  With
    fraction < 1 each part runs on a bounded sample of the step's work (a
    prefix of the nodes; below one node, a prefix of that node's kv-head groups
    for the attention and of its positions for the decision) and its time is
    scaled by the inverse of the sampled share.  Returns (seconds, description)."""
    import oracle
    N, L = cfg.n_nodes, cfg.block_len
    group = cfg.n_q_heads // cfg.n_kv_heads
    n = min(N, max(1, int(round(N * fraction))))
    hk, rows = cfg.n_kv_heads, L
    if N * fraction < 1.0:
        hk = min(cfg.n_kv_heads, max(1, int(round(cfg.n_kv_heads * N * fraction))))
        rows = min(L, max(1, int(round(L * N * fraction))))
    sl = slice(0, n)
    q = w.q[:, sl, :, :hk * group]
    kp, vp = w.k_prefix[:, :, :hk], w.v_prefix[:, :, :hk]
    kb, vb = w.k_block[:, sl, :, :hk], w.v_block[:, sl, :, :hk]
    share_attn = (n * hk) / (N * cfg.n_kv_heads)
    if n == N and rows == L:
        logits, tokens = w.logits, w.block_tokens
        share_dec = 1.0
    else:
        tokens = w.block_tokens[:, sl].copy()
        tokens[:, :, rows:] = 0  # positions outside the sample count as unmasked
        logits = w.logits[:, sl]
        share_dec = max(1, int((tokens == cfg.mask_id).sum())) / max(1, int((w.block_tokens == cfg.mask_id).sum()))
    off = w.parent_off[:, :n + 1].copy()
    times = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        oracle.graph_attention(q, kp, vp, kb, vb)
        t1 = time.perf_counter()
        dec = oracle.unmask_decide(logits, tokens, cfg.mask_id, cfg.rule, cfg.top_s, cfg.threshold)
        t2 = time.perf_counter()
        oracle.accept_walk(tokens, off, w.parent_idx, dec.next_tokens, dec.unmask_bits)
        t3 = time.perf_counter()
        times.append((t1 - t0) / share_attn + (t2 - t1) / share_dec + (t3 - t2))
    what = (f"{n} of {N} nodes, {hk} of {cfg.n_kv_heads} kv-head groups (attention share "
            f"{share_attn:.4f}), decision share {share_dec:.4f}; each part's time divided by its share")
    return statistics.median(times), what


def run_reference(args):
    """The reference arm: the CPU oracle, unmodified, on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2509_18085_b200 import workloads as W
    cfg = W.config(args.config, args.nodes)
    w = W.make(cfg, W.seed_for(args.config, 0))
    cores = oracle.max_threads()
    t1, _ = oracle_step_time(cfg, w, 1)
    budget = 120.0
    frac = min(1.0, budget / max(1e-9, t1 * (args.steps + args.warmup)))
    for _ in range(args.warmup):
        oracle_step_time(cfg, w, 1, frac)
    t0 = time.perf_counter()
    per_step = []
    for _ in range(args.steps):
        t, what = oracle_step_time(cfg, w, 1, frac)
        per_step.append(t)
    wall = time.perf_counter() - t0
    sec = statistics.mean(per_step)
    sample = f"{args.steps} steps, each over {what}; {wall:.1f} s of CPU work"
    value = 1.0 / sec
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": WORKLOAD if args.config == 2 else cfg.name},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def run_part(args):
    """One library call alone: graph replay over rotating input sets, CUDA events.
    Prints its own small JSON line; used for profiling the other configurations."""
    import numpy as np
    import torch
    from paper_2509_18085_b200 import spiffy
    from paper_2509_18085_b200 import workloads as W
    from paper_2509_18085_b200.step import VerifyStep, inputs_from_workload

    torch.cuda.set_device(0)
    cfg = W.config(args.config, args.nodes)
    if args.part == "draft":
        return run_draft_part(args, cfg)
    if args.part == "lmhead":
        return run_lmhead_part(args, cfg)
    if args.part == "full_sequence":
        return run_full_sequence_part(args, cfg)
    attn = args.part == "attention"
    probe = W.make(cfg, W.seed_for(args.config, 100), attention=attn, decision=not attn)
    masked = int((probe.block_tokens == cfg.mask_id).sum())
    attn_bytes, decide_bytes, attn_flops = algorithmic_bytes(cfg, masked)
    per_set = attn_bytes if attn else decide_bytes
    n_sets = args.sets or max(2, min(16, int(300e6 // per_set) + 1))
    work = [probe] + [W.make(cfg, W.seed_for(args.config, 100 + i), attention=attn, decision=not attn)
                      for i in range(1, n_sets)]
    sets = [inputs_from_workload(w) for w in work]
    kernel = {"auto": spiffy.ATTN_AUTO, "simt": spiffy.ATTN_SIMT, "tcgen05": spiffy.ATTN_TCGEN05}[args.attn_kernel]
    step = VerifyStep(cfg, attn_kernel=kernel)
    call = {"attention": step.attention, "decide": step.decide, "decide_walk": step.decide_accept,
            "decide_walk_lazy": step.decide_accept_lazy, "decide_sampled": step.decide_sampled}[args.part]
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for x in sets:
            call(x)
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for x in sets:
                call(x)
        for _ in range(max(3, args.warmup // n_sets)):
            g.replay()
        stream.synchronize()
        reps = max(1, args.steps // n_sets)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            g.replay()
        e1.record(stream)
        stream.synchronize()
        sec = e0.elapsed_time(e1) * 1e-3 / (reps * n_sets)
    peaks = measured_peaks()
    masked_all = float(np.mean([(w.block_tokens == cfg.mask_id).sum() for w in work]))
    out = {"part": args.part, "config": f"config{args.config}-{cfg.name}", "n_nodes": cfg.n_nodes,
           "us_per_call": sec * 1e6, "input_sets": n_sets, "calls_timed": reps * n_sets}
    if attn:
        out.update(tflops=attn_flops / sec / 1e12, frac_of_bf16_peak=attn_flops / sec / 1e12 / peaks["bf16_tflops"],
                   gbs=attn_bytes / sec / 1e9, frac_of_hbm=attn_bytes / sec / 1e9 / peaks["hbm_gbs"],
                   algorithmic_flops=attn_flops, algorithmic_bytes=attn_bytes)
    else:
        by = algorithmic_bytes(cfg, masked_all)[1]
        out.update(gbs=by / sec / 1e9, frac_of_hbm=by / sec / 1e9 / peaks["hbm_gbs"], algorithmic_bytes=by,
                   masked_rows=masked_all)
        if args.part == "decide_walk_lazy":
            # what the lazy call has to read: the still-masked rows of the nodes on the accepted path
            rows, hops = [], []
            for x, w in zip(sets, work):
                walk = call(x)
                torch.cuda.synchronize()
                path = walk.path.cpu().numpy()
                hops.append(float(walk.n_accepted.float().mean()))
                rows.append(sum(int((w.block_tokens[b, n] == cfg.mask_id).sum())
                                for b in range(cfg.batch) for n in path[b] if n >= 0))
            lazy_by = algorithmic_bytes(cfg, float(np.mean(rows)))[1]
            out.update(rows_on_path=float(np.mean(rows)), mean_accepted=float(np.mean(hops)),
                       lazy_algorithmic_bytes=lazy_by, lazy_gbs=lazy_by / sec / 1e9,
                       note="gbs counts the eager call's bytes (every node); lazy_gbs the bytes this call reads")
    out["peaks"] = peaks["source"]
    print(json.dumps(out))


def run_full_sequence_part(args, cfg):
    """spiffy_full_sequence_attention alone: the configuration's nodes plus three
    trailing masked blocks as extra queries (Fig. 3 caption, App. A.2)."""
    import torch
    from paper_2509_18085_b200 import spiffy
    B, N, L, P = cfg.batch, cfg.n_nodes, cfg.block_len, cfg.prefix_len
    S = 3 * L
    g = torch.Generator(device="cuda").manual_seed(17)
    r = lambda *shape: torch.randn(shape, generator=g, device="cuda").to(torch.bfloat16)
    per_set = 2 * B * (2 * (N * L + S) * cfg.n_q_heads + 2 * (P + N * L + S) * cfg.n_kv_heads) * cfg.head_dim
    n_sets = args.sets or max(2, min(16, int(300e6 // per_set) + 1))
    sets = [(r(B, N, L, cfg.n_q_heads, cfg.head_dim), r(B, S, cfg.n_q_heads, cfg.head_dim),
             r(B, P, cfg.n_kv_heads, cfg.head_dim), r(B, P, cfg.n_kv_heads, cfg.head_dim),
             r(B, S, cfg.n_kv_heads, cfg.head_dim), r(B, S, cfg.n_kv_heads, cfg.head_dim),
             r(B, N, L, cfg.n_kv_heads, cfg.head_dim), r(B, N, L, cfg.n_kv_heads, cfg.head_dim)) for _ in range(n_sets)]
    out_n, out_s = spiffy.spiffy_full_sequence_attention(*sets[0])
    desc = spiffy.attn_desc(sets[0][0], sets[0][2], sets[0][6], 0.0, spiffy.ATTN_TCGEN05)
    ws = torch.empty(max(16, int(spiffy.lib().spiffy_full_sequence_attention_workspace(
        __import__("ctypes").byref(desc), S))), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        timer = GraphTimer(stream)
        fns = [lambda x=x: spiffy.spiffy_full_sequence_attention(*x, out_nodes=out_n, out_suffix=out_s, workspace=ws)
               for x in sets]
        for fn in fns:
            fn()
        stream.synchronize()
        sec, replays, _ = timer.measure(timer.capture(fns))
    sec /= n_sets
    peaks = measured_peaks()
    print(json.dumps({"part": "full_sequence", "config": f"config{args.config}-{cfg.name}", "suffix_rows": S,
                      "us_per_call": sec * 1e6, "launches_per_call": 2, "input_sets": n_sets,
                      "algorithmic_bytes": per_set, "gbs": per_set / sec / 1e9,
                      "frac_of_hbm": per_set / sec / 1e9 / peaks["hbm_gbs"], "peaks": peaks["source"]}))


def run_lmhead_part(args, cfg):
    """spiffy_lmhead_decide alone: the decision fused into the output projection
    at the configuration's rows and vocabulary, hidden size 4096 (LLaDA-8B),
    random bf16 operands.  The 1 GB weight matrix is larger than L2 by itself."""
    import ctypes
    import torch
    from paper_2509_18085_b200 import spiffy
    hidden = 4096
    B, N, L, V = cfg.batch, cfg.n_nodes, cfg.block_len, cfg.vocab
    g = torch.Generator().manual_seed(11)
    hs = torch.randn((B, N, L, hidden), generator=g).to(torch.bfloat16).cuda()
    w = (torch.randn((V, hidden), generator=g) * (2.0 / hidden ** 0.5)).to(torch.bfloat16).cuda()
    tokens = torch.where(torch.rand((B, N, L), generator=g) < 0.36, 3, cfg.mask_id).to(torch.int32).cuda()
    desc = spiffy.DecideDesc(B, N, L, V, spiffy.BF16, V, cfg.mask_id, cfg.rule, cfg.top_s, cfg.threshold)
    ws = torch.empty(int(spiffy.lib().spiffy_lmhead_decide_workspace(ctypes.byref(desc), hidden)),
                     dtype=torch.uint8, device="cuda")
    call = lambda out=None: spiffy.spiffy_lmhead_decide(hs, w, tokens, cfg.mask_id, cfg.rule, cfg.top_s,
                                                        cfg.threshold, out=out, workspace=ws)
    out = call()
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for _ in range(max(3, args.warmup // 10)):
            call(out)
        stream.synchronize()
        reps = max(5, args.steps // 100)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            call(out)
        e1.record(stream)
        stream.synchronize()
        sec = e0.elapsed_time(e1) * 1e-3 / reps
    peaks = measured_peaks()
    flops = 2.0 * B * N * L * V * hidden
    by = (V + B * N * L) * hidden * 2.0
    print(json.dumps({"part": "lmhead", "config": f"config{args.config}-{cfg.name}", "us_per_call": sec * 1e6,
                      "rows": B * N * L, "hidden": hidden, "vocab": V, "calls_timed": reps,
                      "tflops": flops / sec / 1e12, "frac_of_bf16_peak": flops / sec / 1e12 / peaks["bf16_tflops"],
                      "gbs": by / sec / 1e9, "frac_of_hbm": by / sec / 1e9 / peaks["hbm_gbs"],
                      "algorithmic_flops": flops, "algorithmic_bytes": by, "peaks": peaks["source"],
                      "dev_status": int(out.dev_status.max().item())}))


def run_draft_part(args, cfg):
    """spiffy_draft_blocks alone (drafting + pruning from the true block's
    distribution): ten formulas over position ranks 0..3 and vocabulary ranks
    0..2, pruned to three drafts -- the paper's operating point (D = 10, D* = 3)."""
    import torch
    from paper_2509_18085_b200 import spiffy
    from paper_2509_18085_b200 import workloads as W
    formulas = [[(0, 0)], [(0, 1)], [(1, 0)], [(0, 0), (1, 0)], [(0, 0), (1, 1)], [(0, 1), (1, 0)],
                [(0, 0), (2, 0)], [(0, 0), (1, 0), (2, 0)], [(0, 0), (1, 0), (2, 2)],
                [(0, 0), (1, 0), (2, 0), (3, 0)]]
    children = [[3, 4, 6], [5], [3, 5], [7, 8], [], [], [7], [9], [], []]
    graph = spiffy.draft_graph(formulas, children)
    n_sets = args.sets or 24
    dt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    sets, masked = [], 0
    for i in range(n_sets):
        w = W.make(W.config(args.config, 1), W.seed_for(args.config, 300 + i), attention=False)
        sets.append((torch.from_numpy(w.logits[:, 0]).to(dt).cuda(), torch.from_numpy(w.block_tokens[:, 0]).cuda()))
        masked += int((w.block_tokens[:, 0] == cfg.mask_id).sum())
    out = spiffy.spiffy_draft_blocks(sets[0][0], sets[0][1], cfg.mask_id, graph, 3, 3)
    ws = torch.empty(1 << 22, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        call = lambda x: spiffy.spiffy_draft_blocks(x[0], x[1], cfg.mask_id, graph, 3, 3, out=out, workspace=ws)
        for x in sets:
            call(x)
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for x in sets:
                call(x)
        g.replay()
        stream.synchronize()
        reps = max(1, args.steps // n_sets)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            g.replay()
        e1.record(stream)
        stream.synchronize()
        sec = e0.elapsed_time(e1) * 1e-3 / (reps * n_sets)
    by = masked / n_sets * cfg.vocab * (2 if cfg.dtype == "bf16" else 4)
    peaks = measured_peaks()
    print(json.dumps({"part": "draft", "config": f"config{args.config}-{cfg.name}", "us_per_call": sec * 1e6,
                      "formulas": len(formulas), "budget": 3, "top_k": 3, "masked_rows": masked / n_sets,
                      "algorithmic_bytes": by, "gbs": by / sec / 1e9, "frac_of_hbm": by / sec / 1e9 / peaks["hbm_gbs"],
                      "input_sets": n_sets, "peaks": peaks["source"], "dev_status": int(out.dev_status.max())}))


def kernel_sources_digest(files):
    """sha256 over the named kernel sources: ties a stored ncu figure to the code it was taken from."""
    import hashlib
    h = hashlib.sha256()
    for name in files:
        with open(os.path.join(ROOT, "paper_2509_18085_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def ncu_traffic(key):
    """DRAM bytes per launch of a kernel as ncu counted them (profiles/ncu_traffic.json, written
    next to the summary the figure comes from).  None when there is no record or the kernel's
    sources have changed since the capture."""
    path = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    try:
        with open(path) as f:
            rec = json.load(f)[key]
        if rec["sources_sha256_16"] != kernel_sources_digest(rec["sources"]):
            return None, f"stale: {rec['sources']} changed since the capture in {rec['summary']}"
        return float(rec["dram_bytes_per_launch"]), f"ncu dram read+write bytes per launch, {rec['summary']}"
    except (OSError, KeyError, ValueError):
        return None, "no ncu record"


class GraphTimer:
    """Times CUDA graphs on one stream with CUDA events: every measurement is the
    median of `repeats` regions, each region replaying the graph until at least
    `min_region_s` of device time has passed."""

    def __init__(self, stream, repeats=5, min_region_s=0.04):
        import torch
        self.torch = torch
        self.stream = stream
        self.repeats = repeats
        self.min_region_s = min_region_s

    def capture(self, fns):
        torch = self.torch
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=self.stream):
            for fn in fns:
                fn()
        return g

    def region(self, graph, replays):
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(self.stream)
        for _ in range(replays):
            graph.replay()
        e1.record(self.stream)
        self.stream.synchronize()
        return e0.elapsed_time(e1) * 1e-3

    def measure(self, graph, min_replays=1, warm_replays=3):
        """(seconds per replay: median over the regions, replays per region, all regions' values)."""
        for _ in range(max(1, warm_replays)):
            graph.replay()
        self.stream.synchronize()
        replays = max(1, min_replays)
        t = self.region(graph, replays)
        while t < self.min_region_s and replays < (1 << 20):  # grow the region to the minimum length
            replays = max(replays + 1, int(replays * min(8.0, 1.3 * self.min_region_s / max(t, 1e-7))))
            t = self.region(graph, replays)
        per = [self.region(graph, replays) / replays for _ in range(self.repeats)]
        return statistics.median(per), replays, per


def device_attention_inputs(cfg, n_sets, seed):
    """Random q/k/v of the configuration's shapes drawn on the device (N(0,1), bf16): input
    data for timing the shapes whose parity the tests cover."""
    import torch
    g = torch.Generator(device="cuda").manual_seed(seed)
    B, N, L, P = cfg.batch, cfg.n_nodes, cfg.block_len, cfg.prefix_len
    r = lambda *shape: torch.randn(shape, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    return [(r(B, N, L, cfg.n_q_heads, cfg.head_dim), r(B, P, cfg.n_kv_heads, cfg.head_dim),
             r(B, P, cfg.n_kv_heads, cfg.head_dim), r(B, N, L, cfg.n_kv_heads, cfg.head_dim),
             r(B, N, L, cfg.n_kv_heads, cfg.head_dim)) for _ in range(n_sets)]


def other_shapes(timer, peaks):
    """The attention call where the tensor roofline binds (configurations 3, 4, 5 with 64
    nodes) and the decision call where HBM binds (3, 4), each alone on L2-cold inputs."""
    import torch
    from paper_2509_18085_b200 import spiffy
    from paper_2509_18085_b200 import workloads as W
    out = {"attention": {}, "decision": {}}
    for index, nodes in ((3, None), (4, None), (5, 64)):
        cfg = W.config(index, nodes)
        attn_bytes, _, flops = algorithmic_bytes(cfg, 0)
        n_sets = max(1, min(16, int(300e6 // attn_bytes) + 1))
        sets = device_attention_inputs(cfg, n_sets, 40 + index)
        outs = torch.empty_like(sets[0][0])
        desc = spiffy.attn_desc(sets[0][0], sets[0][1], sets[0][3], 0.0, spiffy.ATTN_TCGEN05)
        ws = torch.empty(max(16, spiffy.spiffy_graph_attention_workspace(desc)), dtype=torch.uint8, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        fns = [lambda x=x: spiffy.spiffy_graph_attention(*x, out=outs, kernel=spiffy.ATTN_TCGEN05,
                                                         dev_status=status, workspace=ws) for x in sets]
        for fn in fns:
            fn()
        timer.stream.synchronize()
        sec, replays, _ = timer.measure(timer.capture(fns))
        sec /= n_sets
        tf = flops / sec / 1e12
        name = f"config{index}" + (f"-N{nodes}" if nodes else "")
        out["attention"][name] = {
            "us_per_call": sec * 1e6, "tflops": tf, "frac_of_bf16_burst_peak": tf / peaks["bf16_tflops"],
            "frac_of_bf16_sustained_peak": tf / peaks["bf16_tflops_sustained"],
            "gbs": attn_bytes / sec / 1e9, "frac_of_hbm": attn_bytes / sec / 1e9 / peaks["hbm_gbs"],
            "input_sets": n_sets, "calls_timed": replays * n_sets * timer.repeats, "dev_status": int(status)}
        del sets, outs, ws, fns
        torch.cuda.empty_cache()
    for index in (3, 4):
        cfg = W.config(index)
        B, N, L, V = cfg.batch, cfg.n_nodes, cfg.block_len, cfg.vocab
        g = torch.Generator(device="cuda").manual_seed(60 + index)
        # every sequence's nodes keep about 0.55-0.7 of their positions masked, as the generated graphs do
        tokens = torch.where(torch.rand((B, N, L), generator=g, device="cuda") < 0.62, cfg.mask_id, 3).to(torch.int32)
        masked = int((tokens == cfg.mask_id).sum())
        by = masked * V * 2 + masked * 12
        n_sets = max(1, min(4, int(300e6 // by) + 1))
        sets = []
        for _ in range(n_sets):
            lg = torch.empty((B, N, L, V), dtype=torch.bfloat16, device="cuda")
            for b in range(B):  # N(0, 2) drawn sequence by sequence: bounded scratch
                lg[b] = (torch.randn((N, L, V), generator=g, device="cuda") * 2.0).to(torch.bfloat16)
            sets.append(lg)
        dec = None
        desc = spiffy.decide_desc(sets[0], tokens, cfg.mask_id, cfg.rule, cfg.top_s, cfg.threshold)
        ws = torch.empty(max(16, spiffy.spiffy_unmask_decide_workspace(desc)), dtype=torch.uint8, device="cuda")
        dec = spiffy.spiffy_unmask_decide(sets[0], tokens, cfg.mask_id, cfg.rule, cfg.top_s, cfg.threshold, workspace=ws)
        fns = [lambda lg=lg: spiffy.spiffy_unmask_decide(lg, tokens, cfg.mask_id, cfg.rule, cfg.top_s, cfg.threshold,
                                                         out=dec, workspace=ws) for lg in sets]
        timer.stream.synchronize()
        sec, replays, _ = timer.measure(timer.capture(fns))
        sec /= n_sets
        out["decision"][f"config{index}"] = {
            "us_per_call": sec * 1e6, "gbs": by / sec / 1e9, "frac_of_hbm": by / sec / 1e9 / peaks["hbm_gbs"],
            "algorithmic_bytes": by, "masked_rows": masked, "input_sets": n_sets,
            "calls_timed": replays * n_sets * timer.repeats, "dev_status": int(dec.dev_status.max())}
        del sets, ws, fns, dec
        torch.cuda.empty_cache()
    out["inputs"] = ("random tensors of the configurations' shapes and dtypes drawn on the device "
                     "(timing is value-independent; parity of these shapes is the tests' job)")
    return out


def main():
    args = parse()
    if args.impl == "reference":
        return run_reference(args)
    if args.part != "step":
        return run_part(args)

    import numpy as np
    import torch
    from paper_2509_18085_b200 import replicas
    from paper_2509_18085_b200 import spiffy
    from paper_2509_18085_b200 import workloads as W
    from paper_2509_18085_b200.step import VerifyStep, inputs_from_workload

    ranks = replicas.from_env()
    world, rank, local = ranks.world, ranks.rank, ranks.local
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    replicas.init(ranks, "nccl", torch.device("cuda", local))
    spiffy.lib()  # fail loudly now if the library is missing

    cfg = W.config(args.config, args.nodes)
    kernel = {"auto": spiffy.ATTN_AUTO, "simt": spiffy.ATTN_SIMT, "tcgen05": spiffy.ATTN_TCGEN05}[args.attn_kernel]
    first_case = 100 + replicas.case_offset(ranks, N_SETS)
    work = [W.make(cfg, W.seed_for(args.config, first_case + i)) for i in range(N_SETS)]
    sets = [inputs_from_workload(w) for w in work]
    host0 = inputs_from_workload(work[0], device="cpu", pin=True)
    step = VerifyStep(cfg, attn_kernel=kernel)
    masked_rows = float(np.mean([(w.block_tokens == cfg.mask_id).sum() for w in work]))
    attn_bytes, decide_bytes, attn_flops = algorithmic_bytes(cfg, masked_rows)
    set_bytes = sets[0].nbytes()
    peaks = measured_peaks()

    stream = torch.cuda.Stream()
    sampler = ClockSampler(local)
    with torch.cuda.stream(stream):
        timer = GraphTimer(stream, repeats=1, min_region_s=0.0) if args.profile else GraphTimer(stream)
        # eager warm-up (also loads the kernels), then capture one rotation over the input sets
        for i in range(max(3, min(args.warmup, 2 * N_SETS))):
            step.run(sets[i % N_SETS])
        stream.synchronize()
        # what the walk accepts on each input set: hops from the true block to the accepted node
        accepted_depth = []
        for x in sets:
            step.run(x)
            stream.synchronize()
            accepted_depth += step.walk.n_accepted.tolist()
        before = spiffy.launch_count()
        graph = timer.capture([lambda x=x: step.run(x) for x in sets])
        launches_per_step = (spiffy.launch_count() - before) / N_SETS
        # whole rotations only: the asked-for counts are rounded up, never down
        min_replays = max(1, -(-args.steps // N_SETS))
        warm_replays = max(1, -(-max(3, args.warmup) // N_SETS))

        sampler.start()
        replicas.barrier(ranks)
        torch.cuda.synchronize()
        sec_replay, replays, regions = timer.measure(graph, min_replays, warm_replays)
        replicas.barrier(ranks)
        torch.cuda.synchronize()
        steps = replays * N_SETS
        ms_total = sec_replay * replays * 1e3  # the median region

        # each library call alone, over the same rotation of input sets
        def call_seconds(fn):
            before = spiffy.launch_count()
            g = timer.capture([lambda x=x: fn(x) for x in sets])
            kernels = (spiffy.launch_count() - before) / N_SETS
            sec, _, _ = timer.measure(g)
            return sec / N_SETS, kernels

        t_attn, k_attn = call_seconds(step.attention)
        t_dec, k_dec = call_seconds(step.decide)
        t_walk, _ = call_seconds(step.accept)
        t_dw, k_dw = call_seconds(step.decide_accept)

        # one verification step of a whole model: the attention runs once per layer, each layer
        # on its own q/K/V (32 layers x 16.8 MB: L2-cold by construction), then one decision + walk
        composite = None
        if args.config in (2, 3, 4, 5) and not args.no_composite and not args.profile:
            layers = 28 if args.config == 3 else 32
            layer_sets = device_attention_inputs(cfg, layers, 7)
            # in a layer loop the next kernel may begin its set-up while this one drains
            layer_kernel = kernel if args.no_early_dependents else kernel | spiffy.ATTN_EARLY_DEPENDENTS
            layer_fns = [lambda x=x: spiffy.spiffy_graph_attention(*x, out=step.attn_out, kernel=layer_kernel,
                                                                   dev_status=step.attn_status,
                                                                   workspace=step.attn_ws) for x in layer_sets]
            for fn in layer_fns[:2]:
                fn()
            stream.synchronize()
            before = spiffy.launch_count()
            cg = timer.capture([fn for fn in layer_fns] + [lambda: step.decide_accept(sets[0]),
                                                           ] + [fn for fn in layer_fns] +
                               [lambda: step.decide_accept(sets[1])])
            launches_c = (spiffy.launch_count() - before) / 2
            sec_c, replays_c, _ = timer.measure(cg)
            sec_c /= 2
            ag = timer.capture(layer_fns)
            sec_layers, _, _ = timer.measure(ag)
            composite = {
                "layers_per_step": layers, "layer_count_source": "public model card, not the paper",
                "value": 1.0 / sec_c, "unit": UNIT, "ms_per_step": sec_c * 1e3,
                "attention_us_per_layer": sec_layers / layers * 1e6,
                "attention_share": sec_layers / sec_c, "gpu_launches_per_step": launches_c,
                "steps_timed": replays_c * 2 * timer.repeats,
                "attention_frac_of_binding_roofline":
                    max(attn_flops / (peaks["bf16_tflops"] * 1e12), attn_bytes / (peaks["hbm_gbs"] * 1e9))
                    / (sec_layers / layers),
                "early_dependents": not args.no_early_dependents,
                "inputs": "per-layer q/K/V drawn on the device, N(0,1) bf16; logits of the step's own sets"}
            del layer_sets, layer_fns, cg, ag

        shapes = None
        if rank == 0 and world == 1 and args.config == 2 and not args.no_other_shapes and not args.profile:
            shapes = other_shapes(timer, peaks)

        # end to end from pinned host memory
        n_e2e = 1 if args.profile else max(5, min(50, steps))
        for _ in range(3):
            step.run_host(host0)
        torch.cuda.synchronize()
        e2e_regions = []
        for _ in range(3):
            h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            h0.record(stream)
            for _ in range(n_e2e):
                step.run_host(host0)
            h1.record(stream)
            stream.synchronize()
            e2e_regions.append(h0.elapsed_time(h1) / n_e2e)
        ms_e2e = statistics.median(e2e_regions)
        clocks = sampler.stop()
        status = int(step.attn_status.item()) | int(step.decision.dev_status.max().item()) | \
            int(step.walk.dev_status.max().item())

    # max over ranks
    ms_total, ms_e2e = replicas.max_over_ranks(ranks, [ms_total, ms_e2e], device="cuda")
    ms_per_step = ms_total / steps
    value = replicas.whole_job_rate(ranks, steps, ms_total)
    e2e_value = replicas.whole_job_rate(ranks, 1, ms_e2e)

    # rooflines: every kernel against the roof that binds it at this shape
    t_tensor = attn_flops / (peaks["bf16_tflops"] * 1e12)
    t_hbm = attn_bytes / (peaks["hbm_gbs"] * 1e9)
    attn_bound = "tensor" if t_tensor > t_hbm else "hbm"
    attn_tc = attn_flops / t_attn / 1e12
    tr_attn, tr_attn_note = ncu_traffic("graph_attention_tc_kernel@config%d" % args.config)
    attention_roof = {
        "kernel": "graph_attention_tc_kernel" + (" (+ graph_attention_combine_kernel)" if k_attn > 1 else ""),
        "timed_as": f"the spiffy_graph_attention call alone ({k_attn:g} kernel(s) per call), graph replay over "
                    f"{N_SETS} L2-cold input sets, CUDA events on the launching stream",
        "bound": attn_bound,
        "achieved": attn_bytes / t_attn / 1e9 if attn_bound == "hbm" else attn_tc,
        "peak": peaks["hbm_gbs"] if attn_bound == "hbm" else peaks["bf16_tflops"],
        "unit": "GB/s" if attn_bound == "hbm" else "TFLOP/s",
        "frac": max(t_tensor, t_hbm) / t_attn,
        "peak_source": peaks["source"] + (" (burst copy)" if attn_bound == "hbm" else " (burst GEMM)"),
        "traffic": tr_attn, "traffic_note": tr_attn_note,
        "seconds": t_attn, "algorithmic_bytes": attn_bytes, "algorithmic_flops": attn_flops,
        "tflops": attn_tc, "frac_of_bf16_peak": attn_tc / peaks["bf16_tflops"],
        "gbs": attn_bytes / t_attn / 1e9, "frac_of_hbm": attn_bytes / t_attn / 1e9 / peaks["hbm_gbs"],
        "share_of_step": t_attn / (t_attn + t_dw),
    }
    tr_dec, tr_dec_note = ncu_traffic("decide_reduce_kernel@config%d" % args.config)
    decision_roof = {
        "kernel": "decide_reduce_kernel" + (" + decide_finalize_kernel" if k_dec > 1 else ""),
        "timed_as": f"the spiffy_unmask_decide call alone ({k_dec:g} kernel(s) per call), same protocol",
        "bound": "hbm", "achieved": decide_bytes / t_dec / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
        "frac": decide_bytes / t_dec / 1e9 / peaks["hbm_gbs"], "peak_source": peaks["source"] + " (burst copy)",
        "traffic": tr_dec, "traffic_note": tr_dec_note, "seconds": t_dec, "algorithmic_bytes": decide_bytes,
        "share_of_step": t_dw / (t_attn + t_dw),
    }
    dominant_is_attention = (composite is not None) or t_attn >= t_dw
    roofline = dict(attention_roof if dominant_is_attention else decision_roof)
    roofline["why_this_kernel"] = (
        "largest share of a whole-model step (one attention call per layer)" if composite is not None
        else "largest share of the single-layer step")

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
        "warmup": warm_replays * N_SETS, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "config": {"workload": WORKLOAD if args.config == 2 else f"config{args.config}-{cfg.name}",
                   "layers_per_step": 1, "multi_gpu": "independent replicas, no collective",
                   "l2": f"rotating {N_SETS} input sets ({N_SETS * set_bytes / 1e6:.0f} MB) > 126 MB L2",
                   "launch": "CUDA graph of one rotation, replayed",
                   "protocol": f"median of {timer.repeats} regions of {steps} steps each "
                               f"(asked: --steps {args.steps} --warmup {args.warmup}, rounded up to whole rotations "
                               f"and to regions of at least {timer.min_region_s * 1e3:.0f} ms)",
                   "attention_kernel": args.attn_kernel, "masked_rows": masked_rows},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": step.h2d_bytes(host0),
                "d2h_bytes_per_step": step.d2h_bytes(), "ms_per_step": ms_e2e},
        "gpu_launches": int(round(launches_per_step * steps)),
        "roofline": roofline, "roofline_attention": attention_roof, "roofline_decision": decision_roof,
        "per_call_us": {"graph_attention": t_attn * 1e6, "unmask_decide": t_dec * 1e6,
                        "accept_walk": t_walk * 1e6, "decide_walk": t_dw * 1e6},
        "regions_ms_per_step": [r / N_SETS * 1e3 for r in regions],
        "dev_status": status,
        "accepted_depth": {"per_input_set_and_sequence": accepted_depth,
                           "histogram": {str(d): accepted_depth.count(d) for d in sorted(set(accepted_depth))}},
    }
    if composite is not None:
        line["composite_model_step"] = composite
    if shapes is not None:
        line["other_shapes"] = shapes
    if rank == 0 and world == 1 and not args.no_cpu_baseline and not args.profile:
        import oracle
        sec, what = oracle_step_time(cfg, work[0], 80)  # about ten seconds of CPU work
        line["cpu_baseline"] = {"value": 1.0 / sec, "unit": UNIT, "cores": oracle.max_threads(),
                                "kind": "oracle",
                                "sample": f"median of 80 full steps of the same workload ({what})"}
    if rank == 0:
        print(json.dumps(line))
    replicas.finish(ranks)


if __name__ == "__main__":
    main()
