"""Thin Python binding of libqknorm's C ABI (argument marshalling only).

Every function here has the name and the arguments of the C entry point it
calls (see include/qknorm.h).  Tensors are used for their device pointers and
shapes; all arithmetic happens in the CUDA kernels.  There is no fallback: if
the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
import threading
from typing import Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libqknorm.so")

EXPORTS = (
    "qknorm_fwd",
    "qknorm_fwd_sharded",
    "qknorm_fwd_ex",
    "qknorm_fwd_sharded_ex",
    "qknorm_fwd_e4m3",
    "qknorm_fwd_strided",
    "qknorm_fwd_strided_e4m3",
    "qknorm_fwd_headwise",
    "qknorm_fwd_headwise_e4m3",
    "qknorm_fwd_headwise_sharded",
    "qknorm_fwd_headwise_sharded_e4m3",
    "qknorm_baseline_gather_then_norm",
    "qknorm_baseline_two_pass",
    "qknorm_baseline_two_pass_static",
    "qknorm_static_scratch_capacity",
    "qknorm_fwd_sharded_e4m3",
    "qknorm_status_string",
    "qknorm_device_error_word",
    "qknorm_last_cuda_error",
    "qknorm_last_variant",
    "qknorm_launch_count",
    "qknorm_version",
)

QKNORM_OK = 0
QKNORM_ERR_NULL = 1
QKNORM_ERR_SHAPE = 2
QKNORM_ERR_ALIGN = 3
QKNORM_ERR_ALIAS = 4
QKNORM_ERR_SHARDS = 5
QKNORM_ERR_EPS = 6
QKNORM_ERR_CUDA = 7
QKNORM_ERR_HEADS = 8
QKNORM_ERR_SCRATCH = 9
QKNORM_ERR_STATIC_LIMIT = 10


class QKNormError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(message)
        self.status = status


_lib = None
_vp = ctypes.c_void_p
_vpp = ctypes.POINTER(ctypes.c_void_p)


def load() -> ctypes.CDLL:
    """Loads libqknorm.so (built by ``python -m paper_2608_09160_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise QKNormError(-1, f"{LIB_PATH} is missing: build it with "
                              f"`python -m paper_2608_09160_b200.build` (there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    i32, i64, f32 = ctypes.c_int32, ctypes.c_int64, ctypes.c_float
    lib.qknorm_fwd.argtypes = [_vp, _vp, _vp, _vp, i64, i32, i32, f32, _vp, _vp, _vp]
    lib.qknorm_fwd.restype = ctypes.c_int
    lib.qknorm_fwd_ex.argtypes = [_vp, _vp, _vp, _vp, i64, i32, i32, f32, _vp, _vp, _vp, _vp, _vp]
    lib.qknorm_fwd_ex.restype = ctypes.c_int
    lib.qknorm_fwd_sharded.argtypes = [_vpp, _vpp, _vpp, _vpp, i32, i64, i32, i32, f32, _vpp, _vpp, _vp]
    lib.qknorm_fwd_sharded.restype = ctypes.c_int
    lib.qknorm_fwd_sharded_ex.argtypes = [_vpp, _vpp, _vpp, _vpp, i32, i64, i32, i32, f32, _vpp, _vpp,
                                          _vp, _vp, _vp, _vp, _vp]
    lib.qknorm_fwd_sharded_ex.restype = ctypes.c_int
    lib.qknorm_fwd_e4m3.argtypes = lib.qknorm_fwd_ex.argtypes
    lib.qknorm_fwd_e4m3.restype = ctypes.c_int
    lib.qknorm_fwd_sharded_e4m3.argtypes = lib.qknorm_fwd_sharded_ex.argtypes
    lib.qknorm_fwd_sharded_e4m3.restype = ctypes.c_int
    lib.qknorm_fwd_strided.argtypes = [_vp, _vp, _vp, _vp, i64, i32, i32, i64, i64, f32, _vp, _vp, i64, i64, _vp]
    lib.qknorm_fwd_strided.restype = ctypes.c_int
    lib.qknorm_fwd_strided_e4m3.argtypes = lib.qknorm_fwd_strided.argtypes
    lib.qknorm_fwd_strided_e4m3.restype = ctypes.c_int
    lib.qknorm_fwd_headwise.argtypes = [_vp, _vp, _vp, _vp, i64, i32, i32, i32, i64, i64, f32, _vp, _vp, i64, i64,
                                        _vp, _vp, _vp]
    lib.qknorm_fwd_headwise.restype = ctypes.c_int
    lib.qknorm_fwd_headwise_e4m3.argtypes = lib.qknorm_fwd_headwise.argtypes
    lib.qknorm_fwd_headwise_e4m3.restype = ctypes.c_int
    for fn in (lib.qknorm_fwd_headwise_sharded, lib.qknorm_fwd_headwise_sharded_e4m3):
        fn.argtypes = [_vpp, _vpp, _vpp, _vpp, i32, i64, i32, i32, i32, f32, _vpp, _vpp, _vp, _vp, _vp]
        fn.restype = ctypes.c_int
    for fn in (lib.qknorm_baseline_gather_then_norm, lib.qknorm_baseline_two_pass):
        fn.argtypes = [_vpp, _vpp, _vpp, _vpp, i32, i64, i32, i32, f32, _vpp, _vpp, _vp, ctypes.c_size_t, _vp]
        fn.restype = ctypes.c_int
    lib.qknorm_baseline_two_pass_static.argtypes = [_vpp, _vpp, _vpp, _vpp, i32, i64, i32, i32, f32, _vpp, _vpp, _vp]
    lib.qknorm_baseline_two_pass_static.restype = ctypes.c_int
    lib.qknorm_static_scratch_capacity.argtypes = []
    lib.qknorm_static_scratch_capacity.restype = ctypes.c_int64
    lib.qknorm_status_string.argtypes = [ctypes.c_int]
    lib.qknorm_status_string.restype = ctypes.c_char_p
    lib.qknorm_device_error_word.argtypes = [ctypes.POINTER(ctypes.c_int)]
    lib.qknorm_device_error_word.restype = ctypes.c_int
    lib.qknorm_last_cuda_error.argtypes = []
    lib.qknorm_last_cuda_error.restype = ctypes.c_int
    lib.qknorm_last_variant.argtypes = []
    lib.qknorm_last_variant.restype = ctypes.c_char_p
    lib.qknorm_launch_count.argtypes = []
    lib.qknorm_launch_count.restype = ctypes.c_int64
    lib.qknorm_version.argtypes = []
    lib.qknorm_version.restype = ctypes.c_int
    _lib = lib
    return lib


def _check(status: int) -> None:
    if status != QKNORM_OK:
        lib = load()
        msg = lib.qknorm_status_string(status).decode()
        if status == QKNORM_ERR_CUDA:
            msg += f" (cudaError {lib.qknorm_last_cuda_error()})"
        raise QKNormError(status, msg)


class PreparedCall:
    """One C-ABI call whose arguments are already marshalled (pointers, sizes, host pointer
    arrays).  Calling the object makes the C call again on the current (or the given) stream:
    nothing but the call itself is left on the host side of a hot loop.  The tensors are kept
    alive by the object; `outputs` is what the wrapper would have returned."""
    __slots__ = ("cfunc", "args", "keep", "outputs")

    def __init__(self, cfunc, args, keep):
        self.cfunc, self.args, self.keep, self.outputs = cfunc, tuple(args), keep, None

    def __call__(self, stream=None):
        status = self.cfunc(*self.args, _stream(stream))
        if status != QKNORM_OK:
            _check(status)


_capture = threading.local()


def _invoke(cfunc, args, stream, keep):
    """Makes the call, or records it when `prepared` is collecting."""
    sink = getattr(_capture, "sink", None)
    if sink is not None:
        sink.append(PreparedCall(cfunc, args, keep))
        return
    _check(cfunc(*args, _stream(stream)))


def prepared(wrapper, *args, **kwargs) -> PreparedCall:
    """prepared(qknorm_fwd_sharded, q_shards, ...) validates and marshals the arguments exactly
    as the wrapper would, makes NO call, and returns a PreparedCall for the one C-ABI call the
    wrapper would have made."""
    _capture.sink = []
    try:
        outs = wrapper(*args, **kwargs)
        sink = _capture.sink
    finally:
        _capture.sink = None
    if len(sink) != 1:
        raise QKNormError(-1, "the wrapper did not make exactly one C-ABI call")
    sink[0].outputs = outs
    return sink[0]


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    return t.data_ptr() or None


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


def _expect(t: Optional[torch.Tensor], shape, dtype, what: str) -> None:
    if t is None:
        raise QKNormError(QKNORM_ERR_NULL, f"{what} is None")
    if not t.is_cuda:
        raise QKNormError(-1, f"{what} must be a CUDA tensor")
    if t.dtype != dtype or tuple(t.shape) != tuple(shape) or not t.is_contiguous():
        raise QKNormError(QKNORM_ERR_SHAPE, f"{what}: expected contiguous {dtype} {tuple(shape)}, "
                                            f"got {t.dtype} {tuple(t.shape)}")


def _array(ts: Optional[Sequence[torch.Tensor]], n: int):
    if ts is None:
        return None
    if len(ts) != n:
        raise QKNormError(QKNORM_ERR_SHARDS, f"expected {n} shards, got {len(ts)}")
    return (ctypes.c_void_p * n)(*[_ptr(t) for t in ts])


def qknorm_fwd_e4m3(q, k, gamma_q, gamma_k, eps: float, out_q=None, out_k=None, *,
                    rstd_q=None, rstd_k=None, stream=None):
    """qknorm_fwd_e4m3: as qknorm_fwd with q, k and the outputs torch.float8_e4m3fn (gamma bf16)."""
    return qknorm_fwd(q, k, gamma_q, gamma_k, eps, out_q, out_k, rstd_q=rstd_q, rstd_k=rstd_k,
                      stream=stream, _act=torch.float8_e4m3fn)


def qknorm_fwd_sharded_e4m3(q_shards, k_shards, gamma_q_shards, gamma_k_shards, eps: float,
                            out_q_shards=None, out_k_shards=None, *, partials_q=None, partials_k=None,
                            rstd_q=None, rstd_k=None, stream=None):
    """qknorm_fwd_sharded_e4m3: as qknorm_fwd_sharded with float8_e4m3fn activations."""
    return qknorm_fwd_sharded(q_shards, k_shards, gamma_q_shards, gamma_k_shards, eps, out_q_shards,
                              out_k_shards, partials_q=partials_q, partials_k=partials_k, rstd_q=rstd_q,
                              rstd_k=rstd_k, stream=stream, _act=torch.float8_e4m3fn)


def qknorm_fwd(q, k, gamma_q, gamma_k, eps: float, out_q=None, out_k=None, *,
               rstd_q=None, rstd_k=None, stream=None, _act=torch.bfloat16):
    """qknorm_fwd / qknorm_fwd_ex.  q [T,dq], k [T,dk] bf16 CUDA tensors (either may
    be None to skip that tensor); out_* default to new tensors, and may be the
    inputs themselves (in place).  Passing rstd_* (fp32 [T]) selects the _ex form.
    Returns (out_q, out_k)."""
    lib = load()
    bf = torch.bfloat16
    act = _act
    ref = q if q is not None else k
    if ref is None:
        raise QKNormError(QKNORM_ERR_NULL, "q and k are both None")
    T = ref.shape[0]
    dq = q.shape[1] if q is not None else 0
    dk = k.shape[1] if k is not None else 0
    if q is not None:
        _expect(q, (T, dq), act, "q")
        _expect(gamma_q, (dq,), bf, "gamma_q")
        out_q = torch.empty_like(q) if out_q is None else out_q
        _expect(out_q, (T, dq), act, "out_q")
    if k is not None:
        _expect(k, (T, dk), act, "k")
        _expect(gamma_k, (dk,), bf, "gamma_k")
        out_k = torch.empty_like(k) if out_k is None else out_k
        _expect(out_k, (T, dk), act, "out_k")
    if rstd_q is not None:
        _expect(rstd_q, (T,), torch.float32, "rstd_q")
    if rstd_k is not None:
        _expect(rstd_k, (T,), torch.float32, "rstd_k")
    args = [_ptr(q), _ptr(k), _ptr(gamma_q) if q is not None else None,
            _ptr(gamma_k) if k is not None else None, T, dq, dk, float(eps),
            _ptr(out_q) if q is not None else None, _ptr(out_k) if k is not None else None]
    keep = (q, k, gamma_q, gamma_k, out_q, out_k, rstd_q, rstd_k)
    if act is not bf:
        _invoke(lib.qknorm_fwd_e4m3, [*args, _ptr(rstd_q), _ptr(rstd_k)], stream, keep)
    elif rstd_q is None and rstd_k is None:
        _invoke(lib.qknorm_fwd, args, stream, keep)
    else:
        _invoke(lib.qknorm_fwd_ex, [*args, _ptr(rstd_q), _ptr(rstd_k)], stream, keep)
    return out_q, out_k


def qknorm_fwd_sharded(q_shards, k_shards, gamma_q_shards, gamma_k_shards, eps: float,
                       out_q_shards=None, out_k_shards=None, *, partials_q=None, partials_k=None,
                       rstd_q=None, rstd_k=None, stream=None, _act=torch.bfloat16):
    """qknorm_fwd_sharded / qknorm_fwd_sharded_ex.  *_shards are lists of S CUDA
    tensors ([T, dq/S], [T, dk/S], [dq/S], [dk/S]); q_shards or k_shards may be
    None to skip that tensor.  Passing partials_* (fp32 [S,T]) or rstd_* (fp32
    [T]) selects the _ex form.  Returns (out_q_shards, out_k_shards)."""
    lib = load()
    bf = torch.bfloat16
    act = _act
    ref = q_shards if q_shards is not None else k_shards
    if ref is None:
        raise QKNormError(QKNORM_ERR_NULL, "q_shards and k_shards are both None")
    S = len(ref)
    if S < 1:
        raise QKNormError(QKNORM_ERR_SHARDS, "need at least one shard")
    T = ref[0].shape[0]
    wq = q_shards[0].shape[1] if q_shards is not None else 0
    wk = k_shards[0].shape[1] if k_shards is not None else 0

    def side(xs, gs, outs, w, name):
        if xs is None:
            return None, None, None
        if outs is None:
            outs = [torch.empty_like(x) for x in xs]
        if len(xs) != S or len(gs) != S or len(outs) != S:
            raise QKNormError(QKNORM_ERR_SHARDS, f"{name}: every list must hold {S} shards")
        for s in range(S):
            _expect(xs[s], (T, w), act, f"{name}_shards[{s}]")
            _expect(gs[s], (w,), bf, f"gamma_{name}_shards[{s}]")
            _expect(outs[s], (T, w), act, f"out_{name}_shards[{s}]")
        return xs, gs, outs

    q_shards, gamma_q_shards, out_q_shards = side(q_shards, gamma_q_shards, out_q_shards, wq, "q")
    k_shards, gamma_k_shards, out_k_shards = side(k_shards, gamma_k_shards, out_k_shards, wk, "k")
    for nm, t, shp in (("partials_q", partials_q, (S, T)), ("partials_k", partials_k, (S, T)),
                       ("rstd_q", rstd_q, (T,)), ("rstd_k", rstd_k, (T,))):
        if t is not None:
            _expect(t, shp, torch.float32, nm)
    args = [_array(q_shards, S), _array(k_shards, S), _array(gamma_q_shards, S), _array(gamma_k_shards, S),
            S, T, wq * S, wk * S, float(eps), _array(out_q_shards, S), _array(out_k_shards, S)]
    keep = (q_shards, k_shards, gamma_q_shards, gamma_k_shards, out_q_shards, out_k_shards,
            partials_q, partials_k, rstd_q, rstd_k)
    extra = [_ptr(partials_q), _ptr(partials_k), _ptr(rstd_q), _ptr(rstd_k)]
    if act is not bf:
        _invoke(lib.qknorm_fwd_sharded_e4m3, [*args, *extra], stream, keep)
    elif all(t is None for t in (partials_q, partials_k, rstd_q, rstd_k)):
        _invoke(lib.qknorm_fwd_sharded, args, stream, keep)
    else:
        _invoke(lib.qknorm_fwd_sharded_ex, [*args, *extra], stream, keep)
    return out_q_shards, out_k_shards


def _expect_rows(t: Optional[torch.Tensor], T: int, d: int, what: str, dtype=torch.bfloat16) -> int:
    """A [T, d] CUDA view of `dtype` whose rows are contiguous; returns its row stride in elements."""
    if t is None:
        raise QKNormError(QKNORM_ERR_NULL, f"{what} is None")
    if (not t.is_cuda or t.dtype != dtype or tuple(t.shape) != (T, d)
            or (d > 1 and t.stride(1) != 1)):
        raise QKNormError(QKNORM_ERR_SHAPE, f"{what}: expected a {dtype} CUDA [{T}, {d}] view with unit column stride")
    return int(t.stride(0)) if T > 1 else d


def qknorm_fwd_strided(q, k, gamma_q, gamma_k, eps: float, out_q=None, out_k=None, *, stream=None):
    """qknorm_fwd_strided: q [T,dq] and k [T,dk] may be column blocks of a wider buffer
    (row stride taken from the tensors); out_* default to the inputs (in place).  bf16, or
    float8_e4m3fn activations (qknorm_fwd_strided_e4m3)."""
    lib = load()
    T, dq, dk = q.shape[0], q.shape[1], k.shape[1]
    cfunc = lib.qknorm_fwd_strided_e4m3 if q.dtype is torch.float8_e4m3fn else lib.qknorm_fwd_strided
    out_q = q if out_q is None else out_q
    out_k = k if out_k is None else out_k
    act = q.dtype if q.dtype is torch.float8_e4m3fn else torch.bfloat16
    ld = [_expect_rows(q, T, dq, "q", act), _expect_rows(k, T, dk, "k", act),
          _expect_rows(out_q, T, dq, "out_q", act), _expect_rows(out_k, T, dk, "out_k", act)]
    _expect(gamma_q, (dq,), torch.bfloat16, "gamma_q")
    _expect(gamma_k, (dk,), torch.bfloat16, "gamma_k")
    _invoke(cfunc, [_ptr(q), _ptr(k), _ptr(gamma_q), _ptr(gamma_k), T, dq, dk, ld[0], ld[1],
                                     float(eps), _ptr(out_q), _ptr(out_k), ld[2], ld[3]], stream,
            (q, k, gamma_q, gamma_k, out_q, out_k))
    return out_q, out_k


def qknorm_fwd_headwise(q, k, gamma_q, gamma_k, head_dim: int, eps: float, out_q=None, out_k=None, *,
                        rstd_q=None, rstd_k=None, stream=None):
    """qknorm_fwd_headwise / qknorm_fwd_headwise_e4m3 (chosen by the activations' dtype): every head of
    head_dim columns normalised on its own.  q, k are [T, d] bf16 or float8_e4m3fn CUDA views with unit
    column stride (either may be None); out_* default to new contiguous tensors; rstd_* are optional
    fp32 [T, d/head_dim]."""
    lib = load()
    ref = q if q is not None else k
    if ref is None:
        raise QKNormError(QKNORM_ERR_NULL, "q and k are both None")
    act = torch.float8_e4m3fn if ref.dtype is torch.float8_e4m3fn else torch.bfloat16
    cfunc = lib.qknorm_fwd_headwise_e4m3 if act is torch.float8_e4m3fn else lib.qknorm_fwd_headwise
    T = ref.shape[0]
    dq = q.shape[1] if q is not None else 0
    dk = k.shape[1] if k is not None else 0
    ld = [0, 0, 0, 0]
    if q is not None:
        out_q = torch.empty((T, dq), dtype=q.dtype, device=q.device) if out_q is None else out_q
        ld[0], ld[2] = _expect_rows(q, T, dq, "q", act), _expect_rows(out_q, T, dq, "out_q", act)
        _expect(gamma_q, (dq,), torch.bfloat16, "gamma_q")
    if k is not None:
        out_k = torch.empty((T, dk), dtype=k.dtype, device=k.device) if out_k is None else out_k
        ld[1], ld[3] = _expect_rows(k, T, dk, "k", act), _expect_rows(out_k, T, dk, "out_k", act)
        _expect(gamma_k, (dk,), torch.bfloat16, "gamma_k")
    hd = int(head_dim)
    if rstd_q is not None:
        _expect(rstd_q, (T, dq // max(hd, 1)), torch.float32, "rstd_q")
    if rstd_k is not None:
        _expect(rstd_k, (T, dk // max(hd, 1)), torch.float32, "rstd_k")
    _invoke(cfunc, [_ptr(q), _ptr(k), _ptr(gamma_q) if q is not None else None,
                    _ptr(gamma_k) if k is not None else None, T, dq, dk, hd, ld[0], ld[1],
                    float(eps), _ptr(out_q) if q is not None else None,
                    _ptr(out_k) if k is not None else None, ld[2], ld[3], _ptr(rstd_q),
                    _ptr(rstd_k)], stream, (q, k, gamma_q, gamma_k, out_q, out_k, rstd_q, rstd_k))
    return out_q, out_k


def qknorm_fwd_headwise_e4m3(q, k, gamma_q, gamma_k, head_dim: int, eps: float, out_q=None, out_k=None, **kw):
    """qknorm_fwd_headwise_e4m3: as qknorm_fwd_headwise with float8_e4m3fn activations."""
    for t, what in ((q, "q"), (k, "k")):
        if t is not None and t.dtype is not torch.float8_e4m3fn:
            raise QKNormError(QKNORM_ERR_SHAPE, f"{what}: expected torch.float8_e4m3fn")
    return qknorm_fwd_headwise(q, k, gamma_q, gamma_k, head_dim, eps, out_q, out_k, **kw)


def qknorm_fwd_headwise_sharded(q_shards, k_shards, gamma_q_shards, gamma_k_shards, head_dim: int, eps: float,
                                out_q_shards=None, out_k_shards=None, *, rstd_q=None, rstd_k=None, stream=None):
    """qknorm_fwd_headwise_sharded / _e4m3 (chosen by the activations' dtype): headwise granularity on
    S column slices in one launch.  *_shards as in qknorm_fwd_sharded; rstd_* are optional fp32
    [T, d/head_dim] with the heads in slice order.  Returns (out_q_shards, out_k_shards)."""
    lib = load()
    ref = q_shards if q_shards is not None else k_shards
    if ref is None:
        raise QKNormError(QKNORM_ERR_NULL, "q_shards and k_shards are both None")
    S = len(ref)
    if S < 1:
        raise QKNormError(QKNORM_ERR_SHARDS, "need at least one shard")
    act = torch.float8_e4m3fn if ref[0].dtype is torch.float8_e4m3fn else torch.bfloat16
    cfunc = lib.qknorm_fwd_headwise_sharded_e4m3 if act is torch.float8_e4m3fn else lib.qknorm_fwd_headwise_sharded
    T = ref[0].shape[0]
    wq = q_shards[0].shape[1] if q_shards is not None else 0
    wk = k_shards[0].shape[1] if k_shards is not None else 0

    def side(xs, gs, outs, w, name):
        if xs is None:
            return None, None, None
        if outs is None:
            outs = [torch.empty_like(x) for x in xs]
        if len(xs) != S or len(gs) != S or len(outs) != S:
            raise QKNormError(QKNORM_ERR_SHARDS, f"{name}: every list must hold {S} shards")
        for s in range(S):
            _expect(xs[s], (T, w), act, f"{name}_shards[{s}]")
            _expect(gs[s], (w,), torch.bfloat16, f"gamma_{name}_shards[{s}]")
            _expect(outs[s], (T, w), act, f"out_{name}_shards[{s}]")
        return xs, gs, outs

    q_shards, gamma_q_shards, out_q_shards = side(q_shards, gamma_q_shards, out_q_shards, wq, "q")
    k_shards, gamma_k_shards, out_k_shards = side(k_shards, gamma_k_shards, out_k_shards, wk, "k")
    hd = int(head_dim)
    if rstd_q is not None:
        _expect(rstd_q, (T, wq * S // max(hd, 1)), torch.float32, "rstd_q")
    if rstd_k is not None:
        _expect(rstd_k, (T, wk * S // max(hd, 1)), torch.float32, "rstd_k")
    _invoke(cfunc, [_array(q_shards, S), _array(k_shards, S), _array(gamma_q_shards, S), _array(gamma_k_shards, S),
                    S, T, wq * S, wk * S, hd, float(eps), _array(out_q_shards, S), _array(out_k_shards, S),
                    _ptr(rstd_q), _ptr(rstd_k)], stream,
            (q_shards, k_shards, gamma_q_shards, gamma_k_shards, out_q_shards, out_k_shards, rstd_q, rstd_k))
    return out_q_shards, out_k_shards


def _baseline(entry, q_shards, k_shards, gamma_q_shards, gamma_k_shards, eps, out_q_shards, out_k_shards,
              scratch, stream):
    S = len(q_shards)
    T = q_shards[0].shape[0]
    wq, wk = q_shards[0].shape[1], k_shards[0].shape[1]
    bf = torch.bfloat16
    out_q_shards = [torch.empty_like(t) for t in q_shards] if out_q_shards is None else out_q_shards
    out_k_shards = [torch.empty_like(t) for t in k_shards] if out_k_shards is None else out_k_shards
    for s in range(S):
        _expect(q_shards[s], (T, wq), bf, f"q_shards[{s}]")
        _expect(k_shards[s], (T, wk), bf, f"k_shards[{s}]")
        _expect(gamma_q_shards[s], (wq,), bf, f"gamma_q_shards[{s}]")
        _expect(gamma_k_shards[s], (wk,), bf, f"gamma_k_shards[{s}]")
        _expect(out_q_shards[s], (T, wq), bf, f"out_q_shards[{s}]")
        _expect(out_k_shards[s], (T, wk), bf, f"out_k_shards[{s}]")
    if scratch is not None and (not scratch.is_cuda or not scratch.is_contiguous()):
        raise QKNormError(QKNORM_ERR_SCRATCH, "scratch must be a contiguous CUDA tensor")
    nbytes = scratch.numel() * scratch.element_size() if scratch is not None else 0
    _invoke(entry, [_array(q_shards, S), _array(k_shards, S), _array(gamma_q_shards, S), _array(gamma_k_shards, S),
                    S, T, wq * S, wk * S, float(eps), _array(out_q_shards, S), _array(out_k_shards, S),
                    _ptr(scratch), nbytes], stream,
            (q_shards, k_shards, gamma_q_shards, gamma_k_shards, out_q_shards, out_k_shards, scratch))
    return out_q_shards, out_k_shards


def qknorm_baseline_gather_then_norm(q_shards, k_shards, gamma_q_shards, gamma_k_shards, eps: float,
                                     out_q_shards=None, out_k_shards=None, *, scratch, stream=None):
    """qknorm_baseline_gather_then_norm; scratch: CUDA tensor of >= T*(dq+dk)*2 bytes."""
    return _baseline(load().qknorm_baseline_gather_then_norm, q_shards, k_shards, gamma_q_shards, gamma_k_shards,
                     eps, out_q_shards, out_k_shards, scratch, stream)


def qknorm_baseline_two_pass(q_shards, k_shards, gamma_q_shards, gamma_k_shards, eps: float,
                             out_q_shards=None, out_k_shards=None, *, scratch, stream=None):
    """qknorm_baseline_two_pass; scratch: CUDA fp32 tensor of >= 2*S*T elements."""
    return _baseline(load().qknorm_baseline_two_pass, q_shards, k_shards, gamma_q_shards, gamma_k_shards,
                     eps, out_q_shards, out_k_shards, scratch, stream)


def qknorm_baseline_two_pass_static(q_shards, k_shards, gamma_q_shards, gamma_k_shards, eps: float,
                                    out_q_shards, out_k_shards, *, stream=None):
    """qknorm_baseline_two_pass_static: the two-pass stand-in with the library's built-in
    1 MiB scratch array, for callers that must not allocate device memory.  Unlike the
    other wrappers this one creates no tensors: the outputs must be passed (they may be the
    inputs).  Calls that can overlap on the GPU race on the shared array; the first call on
    a device should come before any stream capture (see include/qknorm.h)."""
    lib = load()
    S = len(q_shards)
    T = q_shards[0].shape[0]
    wq, wk = q_shards[0].shape[1], k_shards[0].shape[1]
    bf = torch.bfloat16
    for s in range(S):
        _expect(q_shards[s], (T, wq), bf, f"q_shards[{s}]")
        _expect(k_shards[s], (T, wk), bf, f"k_shards[{s}]")
        _expect(gamma_q_shards[s], (wq,), bf, f"gamma_q_shards[{s}]")
        _expect(gamma_k_shards[s], (wk,), bf, f"gamma_k_shards[{s}]")
        _expect(out_q_shards[s], (T, wq), bf, f"out_q_shards[{s}]")
        _expect(out_k_shards[s], (T, wk), bf, f"out_k_shards[{s}]")
    _invoke(lib.qknorm_baseline_two_pass_static,
            [_array(q_shards, S), _array(k_shards, S), _array(gamma_q_shards, S), _array(gamma_k_shards, S), S, T,
             wq * S, wk * S, float(eps), _array(out_q_shards, S), _array(out_k_shards, S)], stream,
            (q_shards, k_shards, gamma_q_shards, gamma_k_shards, out_q_shards, out_k_shards))
    return out_q_shards, out_k_shards


def static_scratch_capacity() -> int:
    return int(load().qknorm_static_scratch_capacity())


def device_error_word() -> int:
    """Synchronises; 0 unless a bounded in-kernel wait ever ran out on the current device."""
    out = ctypes.c_int(-1)
    _check(load().qknorm_device_error_word(ctypes.byref(out)))
    return int(out.value)


def last_variant() -> str:
    return load().qknorm_last_variant().decode()


def launch_count() -> int:
    return int(load().qknorm_launch_count())


def version() -> int:
    return int(load().qknorm_version())
