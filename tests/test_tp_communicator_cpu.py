"""Host side of the tensor-parallel path on CPU: two gloo ranks build a Communicator each.

The inbox routines and the kernel launch are replaced by stand-ins that keep the inbox in a
file both processes map: what is under test is the host plumbing -- that peer_inbox[p] really
is rank p's inbox, that all ranks number their calls alike, that empty calls take no number,
that the restart before the number wraps is collective, and that a peer that never calls shows
up as a bounded wait running out, not as a hang."""
import os
import socket
import tempfile
import time

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_09160_b200 import tp

HEADER_WORDS = 32


class FileIpc:
    """Inbox = a file of 64-bit words mapped by every rank; handle = its path."""

    def __init__(self, folder):
        self.folder, self.maps, self.zeroed = folder, {}, 0

    def create(self, num_ranks, cap):
        path = os.path.join(self.folder, f"inbox_{os.getpid()}.bin")
        n = HEADER_WORDS + 4 * num_ranks * cap
        np.zeros(n, dtype=np.uint64).tofile(path)
        return self._map(path)

    def _map(self, path):
        m = np.memmap(path, dtype=np.uint64, mode="r+")
        key = 1 + len(self.maps)
        self.maps[key] = (path, m)
        return key

    def export(self, inbox):
        return self.maps[inbox][0].encode().ljust(tp.IPC_HANDLE_BYTES, b"\0")

    def open(self, handle):
        return self._map(handle.rstrip(b"\0").decode())

    def close(self, mapped):
        del self.maps[mapped]

    def destroy(self, inbox):
        path, _ = self.maps.pop(inbox)
        os.unlink(path)

    def quiesce(self):
        pass

    def zero(self, inbox, num_ranks, cap):
        self.maps[inbox][1][:] = 0
        self.zeroed += 1

    def status(self, inbox):
        m = self.maps[inbox][1]
        return {"status": int(m[0]), "token": 0, "missing_rank": int(m[1])}


def host_exchange(ipc, comm, payload, wait_s=20.0):
    """Stand-in for the kernel: push {epoch, payload} for token 0 of tensor 0 to every peer, then
    poll the own inbox with a bound.  Returns what arrived, per source rank."""
    def launch(bufs, N, cap, eps, epoch, wait_limit_us):
        half = epoch & 1
        word = np.uint64((epoch << 32) | payload)
        for p in range(N):
            if p != bufs.rank:
                m = ipc.maps[bufs.peer_inbox[p]][1]
                m[HEADER_WORDS + ((half * 2 + 0) * N + bufs.rank) * cap] = word
                m.flush()
        own = ipc.maps[bufs.inbox][1]
        got = {}
        limit = time.time() + (wait_limit_us / 1e6 if wait_limit_us else wait_s)
        for p in range(N):
            if p == bufs.rank:
                continue
            while True:
                v = int(own[HEADER_WORDS + ((half * 2 + 0) * N + p) * cap])
                if v >> 32 == epoch:
                    got[p] = v & 0xFFFFFFFF
                    break
                if time.time() > limit:
                    own[0], own[1] = tp.STATUS_PEER_TIMEOUT, p
                    got[p] = None
                    break
                time.sleep(0.001)
        launch.got = got
    return launch


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, folder, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ipc = FileIpc(folder)
        comm = tp.Communicator(16, ipc=ipc)
        x = torch.zeros((4, 8))
        empty = torch.zeros((0, 8))
        log = []
        for call in range(3):
            comm.launch = host_exchange(ipc, comm, payload=100 * (rank + 1) + call)
            e = comm.forward(comm.buffers(x, None, None, None, out_q=x), 1e-6)
            log.append((e, dict(comm.launch.got)))
            assert comm.forward(comm.buffers(empty, None, None, None, out_q=empty), 1e-6) == e   # takes no number
        # just before the 32-bit number wraps every rank restarts together: inbox zeroed, next number is 1
        comm.epochs.last = tp.MAX_EPOCH
        comm.launch = host_exchange(ipc, comm, payload=7 + rank)
        e = comm.forward(comm.buffers(x, None, None, None, out_q=x), 1e-6)
        log.append((e, dict(comm.launch.got)))
        zeroed = ipc.zeroed
        # rank 1 skips a call: rank 0's bounded wait runs out and names the missing rank
        status = None
        if rank == 0:
            comm.launch = host_exchange(ipc, comm, payload=1)
            comm.forward(comm.buffers(x, None, None, None, out_q=x), 1e-6, wait_limit_us=200000)
            status = comm.status()
        dist.barrier()
        comm.close()
        out.put((rank, log, zeroed, status, len(ipc.maps)))
    finally:
        dist.destroy_process_group()


def test_two_ranks_wire_their_inboxes_and_number_calls_alike():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    with tempfile.TemporaryDirectory() as folder:
        procs = [ctx.Process(target=_worker, args=(r, world, port, folder, out)) for r in range(world)]
        for p in procs:
            p.start()
        res = sorted(out.get(timeout=120) for _ in range(world))
        for p in procs:
            p.join(timeout=60)
            assert p.exitcode == 0
        assert os.listdir(folder) == []                       # every inbox destroyed by its owner
    for rank, log, zeroed, status, maps_left in res:
        peer = 1 - rank
        assert [e for e, _ in log] == [1, 2, 3, 1]            # same numbers on both ranks, restart at 1
        for call in range(3):
            assert log[call][1] == {peer: 100 * (peer + 1) + call}   # the peer's word, from the peer
        assert log[3][1] == {peer: 7 + peer}
        assert zeroed == 1 and maps_left == 0
    assert res[0][3] == {"status": tp.STATUS_PEER_TIMEOUT, "token": 0, "missing_rank": 1}


def test_epoch_counter_skips_zero_and_announces_the_wrap():
    c = tp.EpochCounter()
    assert [c.next(), c.next()] == [1, 2] and not c.next_wraps
    c.last = tp.MAX_EPOCH - 1
    assert c.next() == tp.MAX_EPOCH and c.next_wraps
    assert c.next() == 1
