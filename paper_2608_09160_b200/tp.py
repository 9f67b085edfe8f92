"""Python side of the tensor-parallel entry points (include/qknorm_tp.h).

Argument marshalling and the host-side bookkeeping of Algorithm 1's exchange only: who
owns which inbox, which number the next call carries.  Every step of the method runs in
the library's kernel.

Two ways to use it:

* ``EmulatedGroup`` -- all N ranks' buffers on ONE GPU, one cooperative launch serves
  them all.  The protocol (push, tagged slots, bounded polls, one fixed sum order) is the real
  one; only the "link" is the GPU's own memory.  Tests and the benchmark use this.
* ``Communicator`` -- one process per GPU over ``torch.distributed``: each rank creates
  its inbox, the inter-process handles are all-gathered on the host, and every call
  pushes scalars straight into the peers' memory over NVLink.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import torch

from . import binding
from .binding import QKNormError, _check, _ptr, _stream

EXPORTS = (
    "qknorm_tp_inbox_bytes",
    "qknorm_fwd_tp",
    "qknorm_fwd_tp_e4m3",
    "qknorm_tp_status",
    "qknorm_tp_clear_status",
    "qknorm_tp_slot_index",
    "qknorm_tp_inbox_peek",
    "qknorm_tp_inbox_poke",
    "qknorm_tp_inbox_create",
    "qknorm_tp_inbox_zero",
    "qknorm_tp_inbox_destroy",
    "qknorm_tp_ipc_export",
    "qknorm_tp_ipc_open",
    "qknorm_tp_ipc_close",
)

STATUS_OK, STATUS_PEER_TIMEOUT, STATUS_STAGE_TIMEOUT = 0, 1, 2
IPC_HANDLE_BYTES = 64
MAX_EPOCH = 0xFFFFFFFF

_vp = ctypes.c_void_p


class CTpRank(ctypes.Structure):
    """struct qknorm_tp_rank"""
    _fields_ = [
        ("rank", ctypes.c_int32), ("reserved", ctypes.c_int32),
        ("q", _vp), ("k", _vp), ("gamma_q", _vp), ("gamma_k", _vp), ("out_q", _vp), ("out_k", _vp),
        ("rstd_q", _vp), ("rstd_k", _vp), ("partial_q", _vp), ("partial_k", _vp),
        ("inbox", _vp), ("peer_inbox", ctypes.POINTER(_vp)),
    ]


_ready = False


def lib() -> ctypes.CDLL:
    """The loaded library with the prototypes of qknorm_tp.h declared."""
    global _ready
    L = binding.load()
    if _ready:
        return L
    i32, i64, u32, f32 = ctypes.c_int32, ctypes.c_int64, ctypes.c_uint32, ctypes.c_float
    L.qknorm_tp_inbox_bytes.argtypes = [i32, i64, ctypes.POINTER(i64)]
    for fn in (L.qknorm_fwd_tp, L.qknorm_fwd_tp_e4m3):
        fn.argtypes = [ctypes.POINTER(CTpRank), i32, i32, i64, i64, i32, i32, ctypes.POINTER(i64), f32, u32, u32, _vp]
    L.qknorm_tp_status.argtypes = [_vp, ctypes.POINTER(i32)]
    L.qknorm_tp_clear_status.argtypes = [_vp, _vp]
    L.qknorm_tp_slot_index.argtypes = [i32, i64, u32, i32, i32]
    L.qknorm_tp_inbox_peek.argtypes = [_vp, i64, i64, ctypes.POINTER(ctypes.c_uint64)]
    L.qknorm_tp_inbox_poke.argtypes = [_vp, i64, i64, ctypes.POINTER(ctypes.c_uint64)]
    L.qknorm_tp_inbox_create.argtypes = [i32, i64, ctypes.POINTER(_vp)]
    L.qknorm_tp_inbox_zero.argtypes = [_vp, i32, i64, _vp]
    L.qknorm_tp_inbox_destroy.argtypes = [_vp]
    L.qknorm_tp_ipc_export.argtypes = [_vp, ctypes.c_char_p]
    L.qknorm_tp_ipc_open.argtypes = [ctypes.c_char_p, ctypes.POINTER(_vp)]
    L.qknorm_tp_ipc_close.argtypes = [_vp]
    for name in EXPORTS:
        getattr(L, name).restype = ctypes.c_int
    L.qknorm_tp_slot_index.restype = ctypes.c_int64
    _ready = True
    return L


def inbox_bytes(num_ranks: int, token_capacity: int) -> int:
    out = ctypes.c_int64(0)
    _check(lib().qknorm_tp_inbox_bytes(num_ranks, token_capacity, ctypes.byref(out)))
    return out.value


def _addr(x) -> Optional[int]:
    if x is None:
        return None
    if isinstance(x, int):
        return x or None
    return _ptr(x)


@dataclass
class RankBuffers:
    """One rank's view of a call: X_local, W_local, Y_local for Q and K (2-D CUDA tensors,
    possibly row-strided views), the rank's inbox and its peers' inboxes (tensors, or raw device
    addresses for peer mappings)."""
    rank: int
    q: Optional[torch.Tensor]
    k: Optional[torch.Tensor]
    gamma_q: Optional[torch.Tensor]
    gamma_k: Optional[torch.Tensor]
    out_q: Optional[torch.Tensor]
    out_k: Optional[torch.Tensor]
    inbox: object = None
    peer_inbox: Sequence[object] = field(default_factory=list)
    rstd_q: Optional[torch.Tensor] = None
    rstd_k: Optional[torch.Tensor] = None
    partial_q: Optional[torch.Tensor] = None
    partial_k: Optional[torch.Tensor] = None


def _row_view(t: torch.Tensor, what: str):
    if t.dim() != 2 or (t.shape[1] > 0 and t.stride(1) != 1) or (t.shape[0] > 1 and t.stride(0) < t.shape[1]):
        raise QKNormError(binding.QKNORM_ERR_SHAPE, f"{what}: expected a 2-D tensor with unit column stride")
    return t.stride(0) if t.shape[0] > 1 else t.shape[1]


class PreparedTp:
    """A tensor-parallel call with everything marshalled but its number: ``call(epoch)``."""

    def __init__(self, ranks: Sequence[RankBuffers], num_ranks: int, token_capacity: int, eps: float):
        L = lib()
        if not ranks:
            raise QKNormError(binding.QKNORM_ERR_SHARDS, "no ranks")
        r0 = ranks[0]
        ref = r0.q if r0.q is not None else r0.k
        if ref is None:
            raise QKNormError(binding.QKNORM_ERR_NULL, "q and k are both None")
        act = ref.dtype
        if act not in (torch.bfloat16, torch.float8_e4m3fn):
            raise QKNormError(binding.QKNORM_ERR_SHAPE, f"unsupported activation dtype {act}")
        self.cfunc = L.qknorm_fwd_tp if act is torch.bfloat16 else L.qknorm_fwd_tp_e4m3
        self.T = ref.shape[0]
        self.wq = r0.q.shape[1] if r0.q is not None else 0
        self.wk = r0.k.shape[1] if r0.k is not None else 0
        lds = [0, 0, 0, 0]
        self.keep = []
        arr = (CTpRank * len(ranks))()
        for i, r in enumerate(ranks):
            for j, (x, y, g, w, nm) in enumerate(((r.q, r.out_q, r.gamma_q, self.wq, "q"), (r.k, r.out_k, r.gamma_k, self.wk, "k"))):
                if w == 0:
                    if x is not None:
                        raise QKNormError(binding.QKNORM_ERR_SHAPE, f"rank {r.rank}: {nm} given but absent on rank {r0.rank}")
                    continue
                for t, what in ((x, nm), (y, "out_" + nm)):
                    if t is None or not t.is_cuda or t.dtype != act or tuple(t.shape) != (self.T, w):
                        raise QKNormError(binding.QKNORM_ERR_SHAPE, f"rank {r.rank}: {what} must be a CUDA {act} tensor [{self.T}, {w}]")
                if g is None or not g.is_cuda or g.dtype != torch.bfloat16 or tuple(g.shape) != (w,) or not g.is_contiguous():
                    raise QKNormError(binding.QKNORM_ERR_SHAPE, f"rank {r.rank}: gamma_{nm} must be a contiguous CUDA bf16 tensor [{w}]")
                for slot, t in ((j, x), (2 + j, y)):
                    ldv = _row_view(t, nm)
                    if lds[slot] not in (0, ldv):
                        raise QKNormError(binding.QKNORM_ERR_SHAPE, "all ranks must use the same row pitches")
                    lds[slot] = ldv
            for t, what in ((r.rstd_q, "rstd_q"), (r.rstd_k, "rstd_k"), (r.partial_q, "partial_q"), (r.partial_k, "partial_k")):
                if t is not None and (t.dtype != torch.float32 or tuple(t.shape) != (self.T,) or not t.is_contiguous()):
                    raise QKNormError(binding.QKNORM_ERR_SHAPE, f"rank {r.rank}: {what} must be contiguous fp32 [{self.T}]")
            peers = (_vp * num_ranks)(*[_addr(p) for p in r.peer_inbox]) if len(r.peer_inbox) == num_ranks else None
            if peers is None and num_ranks > 1:
                raise QKNormError(binding.QKNORM_ERR_SHARDS, f"rank {r.rank}: peer_inbox needs {num_ranks} entries")
            c = arr[i]
            c.rank, c.reserved = r.rank, 0
            c.q, c.k, c.gamma_q, c.gamma_k = _addr(r.q), _addr(r.k), _addr(r.gamma_q), _addr(r.gamma_k)
            c.out_q, c.out_k = _addr(r.out_q), _addr(r.out_k)
            c.rstd_q, c.rstd_k, c.partial_q, c.partial_k = _addr(r.rstd_q), _addr(r.rstd_k), _addr(r.partial_q), _addr(r.partial_k)
            c.inbox = _addr(r.inbox)
            c.peer_inbox = ctypes.cast(peers, ctypes.POINTER(_vp)) if peers is not None else None
            self.keep.append((r, peers))
        self.arr, self.n_local, self.num_ranks = arr, len(ranks), num_ranks
        self.cap, self.eps = token_capacity, float(eps)
        self.ld = (ctypes.c_int64 * 4)(*lds)

    def __call__(self, epoch: int, stream=None, wait_limit_us: int = 0) -> None:
        status = self.cfunc(self.arr, self.n_local, self.num_ranks, self.T, self.cap, self.wq, self.wk, self.ld,
                            self.eps, epoch, wait_limit_us, _stream(stream))
        if status != binding.QKNORM_OK:
            _check(status)


def qknorm_fwd_tp(ranks: Sequence[RankBuffers], num_ranks: int, token_capacity: int, eps: float, epoch: int, *,
                  wait_limit_us: int = 0, stream=None) -> None:
    """qknorm_fwd_tp / qknorm_fwd_tp_e4m3 (chosen by the activations' dtype): one launch for the
    listed ranks.  Outputs are the tensors in ``ranks``."""
    PreparedTp(ranks, num_ranks, token_capacity, eps)(epoch, stream, wait_limit_us)


def status(inbox) -> dict:
    """The header of an inbox: {'status', 'token', 'missing_rank'}; synchronise the call's stream first."""
    out = (ctypes.c_int32 * 4)()
    _check(lib().qknorm_tp_status(_addr(inbox), out))
    return {"status": out[0], "token": out[1], "missing_rank": out[2]}


def slot_index(num_ranks: int, token_capacity: int, epoch: int, tensor: int, src_rank: int) -> int:
    """Word offset of source rank `src_rank`'s slot for token 0 (tensor 0 = Q, 1 = K) in an inbox."""
    i = lib().qknorm_tp_slot_index(num_ranks, token_capacity, epoch, tensor, src_rank)
    if i < 0:
        raise QKNormError(binding.QKNORM_ERR_SHAPE, "slot index arguments out of range")
    return i


def peek(inbox, first_word: int, n_words: int):
    """n_words 64-bit words of an inbox as a numpy uint64 array (synchronous)."""
    import numpy as np
    out = np.empty(n_words, dtype=np.uint64)
    _check(lib().qknorm_tp_inbox_peek(_addr(inbox), first_word, n_words, out.ctypes.data_as(ctypes.POINTER(ctypes.c_uint64))))
    return out


def poke(inbox, first_word: int, words) -> None:
    """Writes a numpy uint64 array into an inbox from word first_word on (synchronous)."""
    import numpy as np
    w = np.ascontiguousarray(words, dtype=np.uint64)
    _check(lib().qknorm_tp_inbox_poke(_addr(inbox), first_word, w.size, w.ctypes.data_as(ctypes.POINTER(ctypes.c_uint64))))


def clear_status(inbox, stream=None) -> None:
    _check(lib().qknorm_tp_clear_status(_addr(inbox), _stream(stream)))


class EpochCounter:
    """Numbers the calls of a group: 1, 2, ...; ``next_wraps`` tells the owner that the 32-bit number
    is about to start again at 1, before which every rank must quiesce and zero its inbox."""

    def __init__(self, start: int = 0):
        self.last = start

    def next(self) -> int:
        self.last = 1 if self.last >= MAX_EPOCH else self.last + 1
        return self.last

    @property
    def next_wraps(self) -> bool:
        return self.last >= MAX_EPOCH


class EmulatedGroup:
    """N ranks on one GPU: inboxes are zeroed tensors of the current device, every forward is ONE
    cooperative launch that serves all ranks."""

    def __init__(self, num_ranks: int, token_capacity: int, device="cuda"):
        self.N, self.cap = num_ranks, token_capacity
        nbytes = inbox_bytes(num_ranks, token_capacity)
        self.inboxes = [torch.zeros(nbytes // 8, dtype=torch.int64, device=device) for _ in range(num_ranks)]
        self.epochs = EpochCounter()

    def buffers(self, q_slices, k_slices, gq_slices, gk_slices, out_q=None, out_k=None, *, stats: bool = False,
                ranks: Optional[Sequence[int]] = None) -> List[RankBuffers]:
        """RankBuffers for the listed ranks (default: all).  Slices are per-rank lists (or None)."""
        todo = list(range(self.N)) if ranks is None else list(ranks)
        res = []
        for r in todo:
            q = q_slices[r] if q_slices is not None else None
            k = k_slices[r] if k_slices is not None else None
            T = (q if q is not None else k).shape[0]
            mk = (lambda: torch.empty(T, dtype=torch.float32, device=self.inboxes[0].device)) if stats else (lambda: None)
            res.append(RankBuffers(
                rank=r, q=q, k=k,
                gamma_q=gq_slices[r] if q is not None else None, gamma_k=gk_slices[r] if k is not None else None,
                out_q=(out_q[r] if out_q is not None else torch.empty_like(q)) if q is not None else None,
                out_k=(out_k[r] if out_k is not None else torch.empty_like(k)) if k is not None else None,
                inbox=self.inboxes[r], peer_inbox=list(self.inboxes),
                rstd_q=mk() if q is not None else None, rstd_k=mk() if k is not None else None,
                partial_q=mk() if q is not None else None, partial_k=mk() if k is not None else None))
        return res

    def prepare(self, bufs: Sequence[RankBuffers], eps: float) -> PreparedTp:
        return PreparedTp(bufs, self.N, self.cap, eps)

    def forward(self, bufs: Sequence[RankBuffers], eps: float, *, stream=None, wait_limit_us: int = 0) -> int:
        """One numbered call; returns the epoch it used."""
        call = self.prepare(bufs, eps)
        if call.T == 0:
            return self.epochs.last
        if self.epochs.next_wraps:
            torch.cuda.synchronize()
            for b in self.inboxes:
                b.zero_()
        e = self.epochs.next()
        call(e, stream, wait_limit_us)
        return e


class Communicator:
    """One rank of a tensor-parallel group, one process per GPU.

    Construction is collective: every rank creates its inbox on its own GPU, the 64-byte
    inter-process handles are all-gathered over ``group`` (host side, any backend) and each rank
    maps its peers' inboxes.  ``forward`` then makes one numbered call; all ranks must make the same
    sequence of forward calls with the same token counts.

    ``ipc`` is the provider of the four inbox routines (default: the library); tests on CPU pass a
    stand-in, and ``launch`` likewise stands in for the kernel launch there."""

    def __init__(self, token_capacity: int, group=None, *, ipc=None, launch=None):
        import torch.distributed as dist
        self.dist, self.group = dist, group
        self.rank, self.N = dist.get_rank(group), dist.get_world_size(group)
        self.cap = token_capacity
        self.ipc = ipc if ipc is not None else _LibraryIpc()
        self.launch = launch
        self.inbox = self.ipc.create(self.N, token_capacity)
        handle = self.ipc.export(self.inbox)
        handles: List[Optional[bytes]] = [None] * self.N
        dist.all_gather_object(handles, bytes(handle), group=group)
        self.peer_inbox: List[int] = []
        for p, h in enumerate(handles):
            self.peer_inbox.append(self.inbox if p == self.rank else self.ipc.open(h))
        dist.barrier(group=group)  # every inbox is mapped everywhere before anybody pushes
        self.epochs = EpochCounter()
        self.closed = False

    def buffers(self, q, k, gamma_q, gamma_k, out_q=None, out_k=None, **kw) -> RankBuffers:
        return RankBuffers(rank=self.rank, q=q, k=k, gamma_q=gamma_q, gamma_k=gamma_k,
                           out_q=(torch.empty_like(q) if out_q is None else out_q) if q is not None else None,
                           out_k=(torch.empty_like(k) if out_k is None else out_k) if k is not None else None,
                           inbox=self.inbox, peer_inbox=list(self.peer_inbox), **kw)

    def prepare(self, bufs: RankBuffers, eps: float) -> PreparedTp:
        """The call on these buffers with its arguments marshalled once, for a hot loop:
        ``comm.forward(bufs, eps, prepared=call)`` then only numbers and launches it."""
        return PreparedTp([bufs], self.N, self.cap, eps)

    def forward(self, bufs: RankBuffers, eps: float, *, stream=None, wait_limit_us: int = 0,
                prepared: Optional[PreparedTp] = None) -> int:
        ref = bufs.q if bufs.q is not None else bufs.k
        if ref is None or ref.shape[0] == 0:
            return self.epochs.last          # an empty call takes no number
        if ref.shape[0] > self.cap:
            raise QKNormError(binding.QKNORM_ERR_SHAPE, f"{ref.shape[0]} tokens exceed the inbox capacity {self.cap}")
        if self.epochs.next_wraps:
            self._restart()
        e = self.epochs.next()
        if self.launch is not None:
            self.launch(bufs, self.N, self.cap, eps, e, wait_limit_us)
        elif prepared is not None:
            prepared(e, stream, wait_limit_us)
        else:
            qknorm_fwd_tp([bufs], self.N, self.cap, eps, e, wait_limit_us=wait_limit_us, stream=stream)
        return e

    def _restart(self) -> None:
        """Before the 32-bit call number wraps: all ranks finish, zero their inboxes, meet again."""
        self.ipc.quiesce()
        self.dist.barrier(group=self.group)
        self.ipc.zero(self.inbox, self.N, self.cap)
        self.dist.barrier(group=self.group)

    def status(self) -> dict:
        return self.ipc.status(self.inbox)

    def close(self) -> None:
        if self.closed:
            return
        self.closed = True
        self.ipc.quiesce()
        self.dist.barrier(group=self.group)   # nobody pushes any more
        for p, addr in enumerate(self.peer_inbox):
            if p != self.rank:
                self.ipc.close(addr)
        self.dist.barrier(group=self.group)   # nobody has this inbox mapped any more
        self.ipc.destroy(self.inbox)


class _LibraryIpc:
    """The library's inbox routines on the current CUDA device."""

    def create(self, num_ranks: int, token_capacity: int) -> int:
        out = _vp()
        _check(lib().qknorm_tp_inbox_create(num_ranks, token_capacity, ctypes.byref(out)))
        return out.value

    def destroy(self, inbox: int) -> None:
        _check(lib().qknorm_tp_inbox_destroy(inbox))

    def export(self, inbox: int) -> bytes:
        buf = ctypes.create_string_buffer(IPC_HANDLE_BYTES)
        _check(lib().qknorm_tp_ipc_export(inbox, buf))
        return buf.raw

    def open(self, handle: bytes) -> int:
        out = _vp()
        _check(lib().qknorm_tp_ipc_open(handle, ctypes.byref(out)))
        return out.value

    def close(self, mapped: int) -> None:
        _check(lib().qknorm_tp_ipc_close(mapped))

    def quiesce(self) -> None:
        torch.cuda.synchronize()

    def zero(self, inbox: int, num_ranks: int, token_capacity: int) -> None:
        _check(lib().qknorm_tp_inbox_zero(inbox, num_ranks, token_capacity, _stream(None)))
        torch.cuda.synchronize()

    def status(self, inbox: int) -> dict:
        return status(inbox)
