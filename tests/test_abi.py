"""The C-ABI library loads, exports what include/qknorm.h declares, and rejects
bad arguments on the host before anything is launched (no GPU needed)."""
import ctypes
import os
import re

import pytest

from paper_2608_09160_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "qknorm.h")
HEADER_TP = os.path.join(ROOT, "include", "qknorm_tp.h")


def declared_functions(header=HEADER):
    src = open(header).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(qknorm_[a-z0-9_]+)\s*\(", src)))


def test_header_and_binding_agree_on_exports():
    assert declared_functions() == sorted(binding.EXPORTS)


def test_tensor_parallel_header_and_binding_agree_on_exports(libqknorm):
    from paper_2608_09160_b200 import tp
    names = [n for n in declared_functions(HEADER_TP) if n != "qknorm_tp_rank"]
    assert names == sorted(tp.EXPORTS)
    for name in names:
        assert hasattr(libqknorm, name), name


def test_library_exports_every_declared_symbol(libqknorm):
    for name in declared_functions():
        assert hasattr(libqknorm, name), name
    assert libqknorm.qknorm_version() >= 100
    assert libqknorm.qknorm_status_string(0) == b"QKNORM_OK"
    for code in range(1, 8):
        assert libqknorm.qknorm_status_string(code).startswith(b"QKNORM_ERR_")
    assert libqknorm.qknorm_status_string(99) == b"unknown qknorm status"


def test_no_symbol_of_the_oracle_is_linked_in(libqknorm):
    for name in ("qko_rmsnorm", "qko_rmsnorm_sharded", "qko_f64_to_bf16"):
        assert not hasattr(libqknorm, name)


# Fake device addresses: validation never dereferences them and fails before any launch.
A, B, C, D, E, F = (0x10000000 + i * 0x1000000 for i in range(6))


def fwd(lib, q=A, k=B, gq=C, gk=D, T=4, dq=64, dk=64, eps=1e-6, oq=E, ok=F):
    return lib.qknorm_fwd(q, k, gq, gk, T, dq, dk, eps, oq, ok, None)


def test_unsharded_argument_errors(libqknorm):
    lib = libqknorm
    assert fwd(lib, T=0) == binding.QKNORM_OK                   # nothing to do, nothing launched
    assert fwd(lib, T=-1) == binding.QKNORM_ERR_SHAPE
    assert fwd(lib, dq=-8) == binding.QKNORM_ERR_SHAPE
    assert fwd(lib, dq=65536 + 8) == binding.QKNORM_ERR_SHAPE
    assert fwd(lib, dq=0, dk=0) == binding.QKNORM_ERR_SHAPE
    assert fwd(lib, eps=-1.0) == binding.QKNORM_ERR_EPS
    assert fwd(lib, eps=float("nan")) == binding.QKNORM_ERR_EPS
    assert fwd(lib, q=None) == binding.QKNORM_ERR_NULL
    assert fwd(lib, gk=None) == binding.QKNORM_ERR_NULL
    assert fwd(lib, ok=None) == binding.QKNORM_ERR_NULL
    assert fwd(lib, q=A + 1) == binding.QKNORM_ERR_ALIGN
    # partial overlap of an output with its input, with the other tensor, with a gamma
    assert fwd(lib, oq=A + 64) == binding.QKNORM_ERR_ALIAS
    assert fwd(lib, oq=B) == binding.QKNORM_ERR_ALIAS
    assert fwd(lib, oq=C) == binding.QKNORM_ERR_ALIAS
    assert fwd(lib, oq=E, ok=E + 2) == binding.QKNORM_ERR_ALIAS


def test_exact_in_place_passes_validation_and_then_needs_a_gpu(libqknorm):
    import torch
    if torch.cuda.is_available():
        pytest.skip("on a GPU box this call would launch on fake pointers")
    # out == in is legal; the call gets as far as asking CUDA for the device and fails loudly there
    assert fwd(libqknorm, oq=A, ok=B) == binding.QKNORM_ERR_CUDA
    assert libqknorm.qknorm_last_cuda_error() != 0
    assert fwd(libqknorm, dq=0, q=None, gq=None, oq=None) == binding.QKNORM_ERR_CUDA   # K-only is legal too


def sharded(lib, S=4, T=4, dq=64, dk=64, eps=1e-6, q=None, oq=None, k_none=False):
    arr = ctypes.c_void_p * max(S, 1)
    n = max(S, 1)
    mk = lambda base: arr(*[base + i * 0x10000 for i in range(n)])
    qa = mk(A) if q is None else q
    oqa = mk(E) if oq is None else oq
    return lib.qknorm_fwd_sharded(qa, None if k_none else mk(B), mk(C), mk(D), S, T, dq, dk, eps,
                                  oqa, mk(F), None)


def test_sharded_argument_errors(libqknorm):
    lib = libqknorm
    assert sharded(lib, S=0) == binding.QKNORM_ERR_SHARDS
    assert sharded(lib, S=17) == binding.QKNORM_ERR_SHARDS
    assert sharded(lib, S=3, dq=64) == binding.QKNORM_ERR_SHAPE          # 64 % 3 != 0
    assert sharded(lib, T=0) == binding.QKNORM_OK
    assert sharded(lib, k_none=True) == binding.QKNORM_ERR_NULL
    arr = ctypes.c_void_p * 4
    assert sharded(lib, q=arr(A, None, A + 0x20000, A + 0x30000)) == binding.QKNORM_ERR_NULL
    # shard 1's output lands on shard 2's input
    assert sharded(lib, oq=arr(E, A + 0x20000, E + 0x20000, E + 0x30000)) == binding.QKNORM_ERR_ALIAS
    # two output shards overlap each other
    assert sharded(lib, oq=arr(E, E + 16, E + 0x20000, E + 0x30000)) == binding.QKNORM_ERR_ALIAS


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "libqknorm.so"))
    with pytest.raises(binding.QKNormError, match="no fallback"):
        binding.load()


def test_strided_and_headwise_argument_errors(libqknorm):
    lib = libqknorm
    strided = lambda ld_q=192, ld_k=192, oq=A, ok=A + 128, ld_oq=192, ld_ok=192, T=4: lib.qknorm_fwd_strided(
        A, A + 128, C, D, T, 64, 32, ld_q, ld_k, 1e-6, oq, ok, ld_oq, ld_ok, None)
    assert strided(T=0) == binding.QKNORM_OK
    assert strided(ld_q=32) == binding.QKNORM_ERR_SHAPE                 # stride smaller than the width
    assert strided(ld_k=-1) == binding.QKNORM_ERR_SHAPE
    assert strided(oq=A + 64) == binding.QKNORM_ERR_ALIAS               # output columns run into the K columns
    assert strided(oq=A, ld_oq=256) == binding.QKNORM_ERR_ALIAS         # same base, another pitch: not "in place"
    head = lambda hd, dq=256, dk=128: lib.qknorm_fwd_headwise(A, B, C, D, 4, dq, dk, hd, 0, 0, 1e-6, E, F, 0, 0,
                                                               None, None, None)
    assert head(0) == binding.QKNORM_ERR_HEADS
    assert head(96) == binding.QKNORM_ERR_HEADS                         # 256 % 96 != 0
    assert head(64, dk=96) == binding.QKNORM_ERR_HEADS
    assert lib.qknorm_fwd_headwise(A, B, C, D, 0, 256, 128, 64, 0, 0, 1e-6, E, F, 0, 0, None, None, None) == binding.QKNORM_OK


def test_baseline_scratch_errors(libqknorm):
    lib = libqknorm
    arr = ctypes.c_void_p * 2
    mk = lambda base: arr(base, base + 0x10000)
    SC = 0x70000000
    def two_pass(scratch, nbytes, T=4):
        return lib.qknorm_baseline_two_pass(mk(A), mk(B), mk(C), mk(D), 2, T, 64, 64, 1e-6, mk(E), mk(F), scratch, nbytes, None)
    def gather(scratch, nbytes, T=4):
        return lib.qknorm_baseline_gather_then_norm(mk(A), mk(B), mk(C), mk(D), 2, T, 64, 64, 1e-6, mk(E), mk(F),
                                                    scratch, nbytes, None)
    assert two_pass(None, 0, T=0) == binding.QKNORM_OK
    assert two_pass(None, 1 << 20) == binding.QKNORM_ERR_SCRATCH
    assert two_pass(SC, 2 * 2 * 4 * 4 - 1) == binding.QKNORM_ERR_SCRATCH       # one byte short
    assert two_pass(SC + 2, 1 << 20) == binding.QKNORM_ERR_SCRATCH             # not float aligned
    assert two_pass(A, 1 << 20) == binding.QKNORM_ERR_SCRATCH                  # on top of an input
    assert gather(SC, 4 * 128 * 2 - 1) == binding.QKNORM_ERR_SCRATCH
    assert gather(SC + 8, 1 << 20) == binding.QKNORM_ERR_SCRATCH               # not 16-byte aligned
    assert gather(E, 1 << 20) == binding.QKNORM_ERR_SCRATCH                    # on top of an output


# ---- tensor-parallel entry point: everything below is rejected on the host, before any launch ----
def _tp_call(lib, N=2, n_local=2, T=4, cap=8, wq=64, wk=64, eps=1e-6, epoch=1, ranks=(0, 1), patch=None, fn="qknorm_fwd_tp"):
    from paper_2608_09160_b200 import tp
    tp.lib()
    arr = (tp.CTpRank * max(n_local, 1))()
    keep = []
    for i in range(n_local):
        base = 0x20000000 + i * 0x8000000
        peers = (ctypes.c_void_p * N)(*[0x70000000 + p * 0x1000000 for p in range(N)])
        keep.append(peers)
        c = arr[i]
        c.rank = ranks[i]
        c.q, c.k, c.gamma_q, c.gamma_k = base, base + 0x100000, base + 0x200000, base + 0x300000
        c.out_q, c.out_k = base + 0x400000, base + 0x500000
        c.inbox = 0x70000000 + ranks[i] * 0x1000000
        c.peer_inbox = ctypes.cast(peers, ctypes.POINTER(ctypes.c_void_p))
        if patch:
            patch(i, c)
    return getattr(lib, fn)(arr, n_local, N, T, cap, wq, wk, None, eps, epoch, 0, None)


def test_tensor_parallel_argument_errors(libqknorm):
    lib = libqknorm
    B = binding
    assert _tp_call(lib, T=0) == B.QKNORM_OK                        # nothing to do, nothing launched
    assert _tp_call(lib, N=0) == B.QKNORM_ERR_SHARDS
    assert _tp_call(lib, N=17, n_local=1) == B.QKNORM_ERR_SHARDS
    assert _tp_call(lib, N=1, n_local=2) == B.QKNORM_ERR_SHARDS      # more local ranks than ranks
    assert _tp_call(lib, ranks=(0, 0)) == B.QKNORM_ERR_SHARDS        # a rank listed twice
    assert _tp_call(lib, ranks=(0, 2)) == B.QKNORM_ERR_SHARDS        # rank number out of range
    assert _tp_call(lib, T=9, cap=8) == B.QKNORM_ERR_SHAPE           # more tokens than the inboxes hold
    assert _tp_call(lib, wq=0, wk=0) == B.QKNORM_ERR_SHAPE
    assert _tp_call(lib, N=16, n_local=1, wq=8192) == B.QKNORM_ERR_SHAPE   # H_total beyond the maximum
    assert _tp_call(lib, epoch=0) == B.QKNORM_ERR_SHAPE              # 0 is what an empty slot holds
    assert _tp_call(lib, eps=float("nan")) == B.QKNORM_ERR_EPS
    assert _tp_call(lib, wq=60) == B.QKNORM_ERR_ALIGN                # slice row not a multiple of 16 bytes
    assert _tp_call(lib, wq=24, fn="qknorm_fwd_tp_e4m3") == B.QKNORM_ERR_ALIGN

    def no_inbox(i, c):
        c.inbox = None
    assert _tp_call(lib, patch=no_inbox) == B.QKNORM_ERR_NULL

    def skewed(i, c):
        c.q = c.q + 2
    assert _tp_call(lib, patch=skewed) == B.QKNORM_ERR_ALIGN

    def shared_output(i, c):
        c.out_q = 0x60000000
    assert _tp_call(lib, patch=shared_output) == B.QKNORM_ERR_ALIAS   # two ranks write one buffer

    def output_in_inbox(i, c):
        c.out_k = c.inbox + 256
    assert _tp_call(lib, patch=output_in_inbox) == B.QKNORM_ERR_ALIAS
    # a slice row pair too long for a warp's three shared-memory stages
    assert _tp_call(lib, N=2, wq=32768, wk=32768) == B.QKNORM_ERR_SHAPE


def test_tensor_parallel_inbox_size(libqknorm):
    from paper_2608_09160_b200 import tp
    assert tp.inbox_bytes(8, 65536) == 256 + 2 * 2 * 8 * 65536 * 8
    assert tp.inbox_bytes(1, 1) == 256 + 32
    with pytest.raises(binding.QKNormError):
        tp.inbox_bytes(17, 16)
    with pytest.raises(binding.QKNormError):
        tp.inbox_bytes(2, 0)
