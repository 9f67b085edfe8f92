"""The one-process-per-rank plumbing on ONE GPU, without any kernel waiting on another process.

Process A (rank 0) only owns an inbox and exports its handle.  Process B (rank 1) maps A's inbox
through the handle, fills its OWN inbox from the host with the scalars rank 0 would have pushed
(so its polls find them at once), and runs the tensor-parallel kernel for rank 1 alone: its
pushes go through the inter-process mapping into A's memory.  When B has finished and exited, A
reads its inbox: it must hold rank 1's scalars, tagged with the call's number.  This covers handle
export / open / close across processes, stores into a peer's mapping, and the slot layout as two
different processes see it."""
import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

import oracle
from paper_2608_09160_b200 import tp
from paper_2608_09160_b200 import workloads as W
from tests import gpu_harness as H

pytestmark = pytest.mark.gpu

N, T, DQ, DK, EPOCH = 2, 700, 2048, 512, 5
WORKLOAD = W.Workload("tp_ipc", tokens=T, dq=DQ, dk=DK, shards=(N,), seed=123, sigma=1.5)


def _sharded_oracle(inp):
    res = {}
    for name in ("q", "k"):
        xs = [W.bf16_bits(t) for t in W.shard_columns(inp[name], N)]
        gs = [W.bf16_bits(t) for t in W.shard_columns(inp["gamma_" + name], N)]
        res[name] = oracle.rmsnorm_sharded(xs, gs, WORKLOAD.eps)
    return res


def _words(values, epoch):
    bits = np.asarray(values, dtype=np.float32).view(np.uint32).astype(np.uint64)
    return (np.uint64(epoch) << np.uint64(32)) | bits


def _rank1(handle, out):
    try:
        torch.cuda.set_device(0)
        ipc = tp._LibraryIpc()
        inp = W.make_inputs(WORKLOAD)
        ref = _sharded_oracle(inp)
        mine = ipc.create(N, T)
        peer = ipc.open(handle)
        # what rank 0 would have pushed into this inbox, written from the host
        for tensor, name in ((0, "q"), (1, "k")):
            tp.poke(mine, tp.slot_index(N, T, EPOCH, tensor, 0), _words(ref[name]["partials"][0], EPOCH))
        q = W.shard_columns(inp["q"], N)[1].cuda()
        k = W.shard_columns(inp["k"], N)[1].cuda()
        gq = W.shard_columns(inp["gamma_q"], N)[1].cuda()
        gk = W.shard_columns(inp["gamma_k"], N)[1].cuda()
        bufs = tp.RankBuffers(rank=1, q=q, k=k, gamma_q=gq, gamma_k=gk, out_q=torch.empty_like(q),
                              out_k=torch.empty_like(k), inbox=mine, peer_inbox=[peer, mine],
                              rstd_q=torch.empty(T, device="cuda"), rstd_k=torch.empty(T, device="cuda"))
        tp.qknorm_fwd_tp([bufs], N, T, WORKLOAD.eps, EPOCH, wait_limit_us=100000)
        torch.cuda.synchronize()
        status = tp.status(mine)
        H.compare_output(H.bits(bufs.out_q), ref["q"]["y"][1], "rank 1 q")
        H.compare_output(H.bits(bufs.out_k), ref["k"]["y"][1], "rank 1 k")
        H.compare_stat(bufs.rstd_q, ref["q"]["rstd"], "rank 1 rstd_q")
        ipc.close(peer)
        ipc.destroy(mine)
        out.put(("ok", status))
    except BaseException as e:   # reported to the parent
        out.put(("error", repr(e)))


def test_rank_1_in_another_process_pushes_through_the_ipc_mapping(libqknorm):
    ipc = tp._LibraryIpc()
    inbox = ipc.create(N, T)
    try:
        handle = ipc.export(inbox)
        assert len(handle) == tp.IPC_HANDLE_BYTES
        ctx = mp.get_context("spawn")
        out = ctx.Queue()
        child = ctx.Process(target=_rank1, args=(handle, out))
        child.start()
        kind, detail = out.get(timeout=300)
        child.join(timeout=60)
        assert kind == "ok", detail
        assert detail["status"] == tp.STATUS_OK
        assert child.exitcode == 0
        ref = _sharded_oracle(W.make_inputs(WORKLOAD))
        for tensor, name in ((0, "q"), (1, "k")):
            got = tp.peek(inbox, tp.slot_index(N, T, EPOCH, tensor, 1), T)
            assert np.array_equal(got >> np.uint64(32), np.full(T, EPOCH, dtype=np.uint64))     # every slot tagged
            vals = (got & np.uint64(0xFFFFFFFF)).astype(np.uint32).view(np.float32).astype(np.float64)
            want = ref[name]["partials"][1]
            assert np.max(np.abs(vals - want) / want) < 1e-5
            # rank 0's own row of slots and the other half of the inbox were not touched
            assert not tp.peek(inbox, tp.slot_index(N, T, EPOCH, tensor, 0), T).any()
            assert not tp.peek(inbox, tp.slot_index(N, T, EPOCH + 1, tensor, 1), T).any()
        assert tp.status(inbox)["status"] == tp.STATUS_OK
    finally:
        ipc.destroy(inbox)
