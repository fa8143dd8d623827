"""The multi-GPU path on CPU: two gloo ranks run the replica plumbing of
bench.py (rendezvous, barrier, max-over-ranks timing, whole-job rate)."""
import os
import socket

import torch.multiprocessing as mp

from paper_2509_18085_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(WORLD_SIZE=str(world), RANK=str(rank), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    r = replicas.from_env()
    replicas.init(r, "gloo")
    replicas.barrier(r)
    local_ms = [10.0 + 5.0 * rank, 3.0 - rank]  # rank 1 is slower on the first, faster on the second
    slow = replicas.max_over_ranks(r, local_ms)
    rate = replicas.whole_job_rate(r, 100, slow[0])
    out.put((rank, slow, rate, replicas.case_offset(r, 6)))
    replicas.barrier(r)
    replicas.finish(r)


def test_two_replicas_agree_on_the_slowest_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(i, 2, port, out)) for i in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[0] for g in got] == [0, 1]
    for _, slow, rate, _ in got:
        assert slow == [15.0, 3.0]                 # element-wise maximum over the ranks
        assert abs(rate - 2 * 100 / 15e-3) < 1e-6  # both replicas' steps over the slowest time
    assert [g[3] for g in got] == [0, 6]           # replicas draw distinct cases


def test_single_process_needs_no_group():
    r = replicas.Ranks(1, 0, 0)
    assert replicas.max_over_ranks(r, [1.5, 2.5]) == [1.5, 2.5]
    assert replicas.whole_job_rate(r, 10, 2.0) == 5000.0
    replicas.barrier(r)
    replicas.finish(r)
