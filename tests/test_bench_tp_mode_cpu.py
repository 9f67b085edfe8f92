"""`bench.py --parallelism tp` on CPU: two gloo ranks run the whole timed region of the
column-sharded mode with the communicator's stand-ins (an inbox file both processes map, a host
routine in place of the kernel launch).  Under test: every rank keeps ITS column slice of the
same seeded tensors, all ranks make the same numbered sequence of calls, the job time is the
MAX over ranks, the job value counts all ranks' bytes, and rank 0's JSON line carries the contract
keys with the tensor-parallel labels."""
import argparse
import os
import socket
import tempfile

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from paper_2608_09160_b200 import workloads as W
from tests.test_tp_communicator_cpu import FileIpc, host_exchange

STEPS, WARMUP = 3, 2


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, folder, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = W.scaled(W.WORKLOADS["C4"], 16)
        ipc = FileIpc(folder)
        seen = []

        def launch(bufs, N, cap, eps, epoch, wait_limit_us):
            # stands in for the kernel: exchange a word with the peer (bounded poll), remember the call
            ex = host_exchange(ipc, None, payload=1000 * (bufs.rank + 1) + epoch)
            ex(bufs, N, cap, eps, epoch, wait_limit_us)
            seen.append((epoch, tuple(bufs.q.shape), tuple(bufs.k.shape), float(bufs.q.float().sum()), dict(ex.got)))

        rec = bench.run_tp_parallel(w, world, rank, dist, STEPS, WARMUP, device="cpu", ipc=ipc, launch=launch)
        args = argparse.Namespace(steps=STEPS, warmup=WARMUP, dtype="bf16")
        line = bench.tp_line(w, world, args, rec, 6521.1, "measured", "tp", rec["launches"], {"sm_mhz": None})
        full = W.make_inputs(w)
        out.put((rank, rec, seen, line, float(W.shard_columns(full["q"], world)[rank].float().sum())))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_run_the_tensor_parallel_bench_mode():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    with tempfile.TemporaryDirectory() as folder:
        procs = [ctx.Process(target=_worker, args=(r, world, port, folder, out)) for r in range(world)]
        for p in procs:
            p.start()
        res = sorted(out.get(timeout=180) for _ in range(world))
        for p in procs:
            p.join(timeout=60)
            assert p.exitcode == 0
        assert os.listdir(folder) == []                      # the communicator was closed, inboxes destroyed
    w = W.scaled(W.WORKLOADS["C4"], 16)
    assert res[0][1]["ms_per_step"] == res[1][1]["ms_per_step"]       # MAX over ranks, on every rank
    for rank, rec, seen, line, slice_sum in res:
        peer = 1 - rank
        assert [e for e, *_ in seen] == list(range(1, WARMUP + STEPS + 1))          # same numbering everywhere
        assert rec["epochs"] == (WARMUP, WARMUP + STEPS)
        for epoch, q_shape, k_shape, q_sum, got in seen:
            assert q_shape == (16, w.dq // world) and k_shape == (16, w.dk // world)  # a column slice ...
            assert got == {peer: 1000 * (peer + 1) + epoch}                           # ... and the peer's word arrived
        assert seen[0][3] == slice_sum                                                # ... this rank's own slice
        assert rec["job_bytes"] == w.algorithmic_bytes
        assert rec["rank_bytes"] == 2 * 16 * (w.dq + w.dk) // world * 2 + (w.dq + w.dk) // world * 2
        assert line["n_gpus"] == world and line["scaling"] == "strong" and line["metric"] == "qknorm_prefill_GBps"
        assert line["config"]["parallelism"] == "tensor-parallel x2, scalar exchange"
        assert line["value"] == round(w.algorithmic_bytes / (rec["ms_per_step"] * 1e-3) / 1e9, 2)
        assert line["roofline"]["exchange_bytes_per_step_per_gpu"] == 16 * 16 * (world - 1)
        assert line["roofline"]["all_waits_completed"] is True
    assert res[0][4] != res[1][4]                                                      # different slices
