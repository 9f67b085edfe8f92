"""The N > 1 path of bench.py on CPU: two gloo ranks.  The data path has no
collective (every rank normalises its own token range); what the ranks share is
the timing protocol: a barrier and the MAX of the per-rank times."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from paper_2608_09160_b200 import workloads as W


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = W.scaled(W.WORKLOADS["C4"], 32)
        mine = W.make_inputs(bench.rank_workload(w, rank))
        dist.barrier()
        slow = 10.0 + 5.0 * rank                       # rank 1 is the slow one
        job_ms = bench.max_over_ranks(slow, dist, "cpu")
        # every rank holds different tokens: exchange a fingerprint to prove it
        fp = torch.tensor([float(mine["q"].float().sum())], dtype=torch.float64)
        got = [torch.zeros_like(fp) for _ in range(world)]
        dist.all_gather(got, fp)
        out.put((rank, job_ms, [float(g) for g in got], bench.job_value(w.algorithmic_bytes, world, job_ms)))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_follow_the_timing_protocol():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    w = W.scaled(W.WORKLOADS["C4"], 32)
    for rank, job_ms, fps, value in res:
        assert job_ms == 15.0                           # MAX over ranks, on every rank
        assert fps[0] != fps[1]                         # the ranks drew different tokens
        assert value == 2 * w.algorithmic_bytes / 15e-3 / 1e9   # units of ALL ranks / slowest time


def test_single_rank_needs_no_process_group():
    assert bench.max_over_ranks(3.5, None, "cpu") == 3.5
    w = W.WORKLOADS["C1"]
    assert bench.rank_workload(w, 0) == w
    assert bench.rank_workload(w, 3).seed == w.seed + 3000
