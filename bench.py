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
`e2e`     : the same step driven from pinned host memory through
            VerifyStep.run_host (host-to-device copies of everything the step
            reads -- of the logits, the rows of still-masked positions -- and
            the device-to-host read of the verdict inside the timed region).
`roofline`: the dominant kernel (the decision reduce) against the measured HBM
            copy bandwidth; its duration comes from a second pass that replays
            the decision call alone over the same rotation of input sets.
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
# dram__bytes_read.sum + dram__bytes_write.sum of one decide_reduce_kernel launch at this workload
# (ncu capture summarised under profiles/); set to None whenever that kernel changes
NCU_REDUCE_TRAFFIC_BYTES = 41.77e6


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
    ap.add_argument("--part", default="step", choices=["step", "attention", "decide", "decide_walk", "decide_walk_lazy", "decide_sampled", "lmhead", "draft"],
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

    stream = torch.cuda.Stream()
    sampler = ClockSampler(local)
    with torch.cuda.stream(stream):
        # eager warm-up (also loads the kernels), then capture one rotation
        for i in range(max(3, min(args.warmup, 2 * N_SETS))):
            step.run(sets[i % N_SETS])
        stream.synchronize()
        before = spiffy.launch_count()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for x in sets:
                step.run(x)
        launches_per_step = (spiffy.launch_count() - before) / N_SETS
        replays = max(1, args.steps // N_SETS)
        steps = replays * N_SETS
        warm_replays = max(1, -(-args.warmup // N_SETS))

        sampler.start()
        for _ in range(warm_replays):
            graph.replay()
        stream.synchronize()
        replicas.barrier(ranks)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(replays):
            graph.replay()
        e1.record(stream)
        stream.synchronize()
        replicas.barrier(ranks)
        torch.cuda.synchronize()
        ms_total = e0.elapsed_time(e1)

        # per-call durations: the same rotation, one library call per graph node
        def call_seconds(fn):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for x in sets:
                    fn(x)
            reps = max(2, min(replays, 200))
            g.replay()
            stream.synchronize()
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record(stream)
            for _ in range(reps):
                g.replay()
            a1.record(stream)
            stream.synchronize()
            return a0.elapsed_time(a1) * 1e-3 / (reps * N_SETS)

        t_attn = call_seconds(step.attention)
        t_dec = call_seconds(step.decide)
        t_walk = call_seconds(step.accept)
        t_dw = call_seconds(step.decide_accept)

        # end to end from pinned host memory
        n_e2e = max(3, min(50, steps))
        for _ in range(3):
            step.run_host(host0)
        torch.cuda.synchronize()
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record(stream)
        for _ in range(n_e2e):
            step.run_host(host0)
        h1.record(stream)
        stream.synchronize()
        ms_e2e = h0.elapsed_time(h1) / n_e2e
        clocks = sampler.stop()
        status = int(step.attn_status.item()) | int(step.decision.dev_status.max().item()) | \
            int(step.walk.dev_status.max().item())

    # max over ranks
    ms_total, ms_e2e = replicas.max_over_ranks(ranks, [ms_total, ms_e2e], device="cuda")
    ms_per_step = ms_total / steps
    value = replicas.whole_job_rate(ranks, steps, ms_total)
    e2e_value = replicas.whole_job_rate(ranks, 1, ms_e2e)

    peaks = measured_peaks()
    roofline = {
        "kernel": "decide_reduce_kernel (timed as the spiffy_unmask_decide call: reduce + finalize)",
        "bound": "hbm", "achieved": decide_bytes / t_dec / 1e9, "peak": peaks["hbm_gbs"],
        "unit": "GB/s", "frac": decide_bytes / t_dec / 1e9 / peaks["hbm_gbs"],
        "peak_source": peaks["source"] + " (burst copy)", "traffic": NCU_REDUCE_TRAFFIC_BYTES,
        "traffic_note": "dram read+write bytes of one decide_reduce_kernel launch, ncu capture in "
                        "profiles/decide_reduce_kernel_config2.md",
        "algorithmic_bytes": decide_bytes, "seconds": t_dec,
    }
    attn_tc = attn_flops / t_attn / 1e12
    attention = {
        "seconds": t_attn, "tflops": attn_tc, "frac_of_bf16_peak": attn_tc / peaks["bf16_tflops"],
        "gbs": attn_bytes / t_attn / 1e9, "frac_of_hbm": attn_bytes / t_attn / 1e9 / peaks["hbm_gbs"],
        "algorithmic_bytes": attn_bytes, "algorithmic_flops": attn_flops,
        "binding_roofline_seconds": max(attn_flops / (peaks["bf16_tflops"] * 1e12),
                                        attn_bytes / (peaks["hbm_gbs"] * 1e9)),
    }
    attention["frac_of_binding_roofline"] = attention["binding_roofline_seconds"] / t_attn

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
        "warmup": warm_replays * N_SETS, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "config": {"workload": WORKLOAD if args.config == 2 else f"config{args.config}-{cfg.name}",
                   "layers_per_step": 1, "multi_gpu": "independent replicas, no collective",
                   "l2": f"rotating {N_SETS} input sets ({N_SETS * set_bytes / 1e6:.0f} MB) > 126 MB L2",
                   "launch": "CUDA graph of one rotation, replayed",
                   "attention_kernel": args.attn_kernel, "masked_rows": masked_rows},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": step.h2d_bytes(host0),
                "d2h_bytes_per_step": step.d2h_bytes(), "ms_per_step": ms_e2e},
        "gpu_launches": int(round(launches_per_step * steps)),
        "roofline": roofline, "attention": attention,
        "per_call_us": {"graph_attention": t_attn * 1e6, "unmask_decide": t_dec * 1e6,
                        "accept_walk": t_walk * 1e6, "decide_walk": t_dw * 1e6},
        "dev_status": status,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
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
