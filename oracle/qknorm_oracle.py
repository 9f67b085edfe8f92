"""ctypes front end of the C oracle (qknorm_oracle.c).  TEST INFRASTRUCTURE ONLY.

Argument marshalling only: numpy uint16 arrays of bf16 bit patterns go in,
numpy arrays come out.  All arithmetic is in the C file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qknorm_oracle.c")
_LIB = os.path.join(_HERE, "libqknorm_oracle.so")
_lib = None

_u16p = ctypes.POINTER(ctypes.c_uint16)
_f64p = ctypes.POINTER(ctypes.c_double)
_u8p = ctypes.POINTER(ctypes.c_uint8)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (fp64, no fast-math, OpenMP for the timed
    baseline only).  Returns the path of the shared object."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
           "-fno-fast-math", "-ffp-contract=off", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.qko_bf16_to_f64.argtypes = [ctypes.c_uint16]
        lib.qko_bf16_to_f64.restype = ctypes.c_double
        lib.qko_f64_to_bf16.argtypes = [ctypes.c_double]
        lib.qko_f64_to_bf16.restype = ctypes.c_uint16
        lib.qko_rmsnorm.argtypes = [_u16p, _u16p, ctypes.c_int64, ctypes.c_int64, ctypes.c_float,
                                    _u16p, _f64p, _f64p, _f64p, ctypes.c_int]
        lib.qko_rmsnorm.restype = ctypes.c_int
        pp = ctypes.POINTER(_u16p)
        lib.qko_rmsnorm_sharded.argtypes = [pp, pp, ctypes.c_int, ctypes.c_int64, ctypes.c_int64,
                                            ctypes.c_float, pp, _f64p, _f64p, _f64p, ctypes.c_int]
        lib.qko_rmsnorm_sharded.restype = ctypes.c_int
        lib.qko_e4m3_to_f64.argtypes = [ctypes.c_uint8]
        lib.qko_e4m3_to_f64.restype = ctypes.c_double
        lib.qko_f64_to_e4m3.argtypes = [ctypes.c_double]
        lib.qko_f64_to_e4m3.restype = ctypes.c_uint8
        p8 = ctypes.POINTER(_u8p)
        lib.qko_rmsnorm_sharded_e4m3.argtypes = [p8, pp, ctypes.c_int, ctypes.c_int64, ctypes.c_int64,
                                                 ctypes.c_float, p8, _f64p, _f64p, _f64p, _f64p, ctypes.c_int]
        lib.qko_rmsnorm_sharded_e4m3.restype = ctypes.c_int
        lib.qko_rmsnorm_headwise.argtypes = [ctypes.c_void_p, _u16p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
                                             ctypes.c_float, ctypes.c_int, ctypes.c_void_p, _f64p, _f64p, ctypes.c_int]
        lib.qko_rmsnorm_headwise.restype = ctypes.c_int
        lib.qko_max_threads.argtypes = []
        lib.qko_max_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _u16(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16:
        raise TypeError("bf16 data must be passed as uint16 bit patterns")
    return a


def _ptr(a: Optional[np.ndarray], ty):
    return a.ctypes.data_as(ty) if a is not None else ty()


def bf16_to_f64(bits) -> np.ndarray:
    lib = _load()
    b = np.asarray(bits, dtype=np.uint16)
    out = np.empty(b.shape, dtype=np.float64)
    fo, fb = out.reshape(-1), b.reshape(-1)
    for i in range(fb.size):
        fo[i] = lib.qko_bf16_to_f64(int(fb[i]))
    return out


def f64_to_bf16(vals) -> np.ndarray:
    lib = _load()
    v = np.asarray(vals, dtype=np.float64)
    out = np.empty(v.shape, dtype=np.uint16)
    fo, fv = out.reshape(-1), v.reshape(-1)
    for i in range(fv.size):
        fo[i] = lib.qko_f64_to_bf16(float(fv[i]))
    return out


def max_threads() -> int:
    return int(_load().qko_max_threads())


def rmsnorm(x_bits: np.ndarray, gamma_bits: np.ndarray, eps: float, *,
            want_y64: bool = False, nthreads: int = 1, out: Optional[np.ndarray] = None):
    """Eq. 1 on every row of x_bits[T, H].  Returns a dict with
    y (uint16 [T,H]), acc (fp64 [T], sum of squares), rstd (fp64 [T]) and, if
    asked, y64 (fp64 [T,H], the result before rounding to bf16)."""
    lib = _load()
    x = _u16(x_bits)
    g = _u16(gamma_bits)
    if x.ndim != 2 or g.ndim != 1 or g.shape[0] != x.shape[1]:
        raise ValueError("expected x[T,H] and gamma[H]")
    T, H = x.shape
    y = np.empty((T, H), dtype=np.uint16) if out is None else out
    y64 = np.empty((T, H), dtype=np.float64) if want_y64 else None
    acc = np.empty((T,), dtype=np.float64)
    rstd = np.empty((T,), dtype=np.float64)
    rc = lib.qko_rmsnorm(_ptr(x, _u16p), _ptr(g, _u16p), T, H, float(eps), _ptr(y, _u16p),
                         _ptr(y64, _f64p), _ptr(acc, _f64p), _ptr(rstd, _f64p), int(nthreads))
    if rc != 0:
        raise RuntimeError(f"qko_rmsnorm failed ({rc})")
    res = {"y": y, "acc": acc, "rstd": rstd}
    if want_y64:
        res["y64"] = y64
    return res


def rmsnorm_sharded(x_shards: Sequence[np.ndarray], gamma_shards: Sequence[np.ndarray],
                    eps: float, *, nthreads: int = 1):
    """The sharded form: S column slices x_s[T, w] with their gamma slices.
    Returns y (list of uint16 [T,w]), partials (fp64 [S,T]), acc, rstd (fp64 [T])."""
    lib = _load()
    S = len(x_shards)
    if S < 1 or len(gamma_shards) != S:
        raise ValueError("need S >= 1 shards and as many gamma slices")
    xs: List[np.ndarray] = [_u16(a) for a in x_shards]
    gs: List[np.ndarray] = [_u16(a) for a in gamma_shards]
    T, w = xs[0].shape
    for a, g in zip(xs, gs):
        if a.shape != (T, w) or g.shape != (w,):
            raise ValueError("all shards must be [T,w] with gamma [w]")
    ys = [np.empty((T, w), dtype=np.uint16) for _ in range(S)]
    partials = np.empty((S, T), dtype=np.float64)
    acc = np.empty((T,), dtype=np.float64)
    rstd = np.empty((T,), dtype=np.float64)
    arr = _u16p * S
    xa = arr(*[_ptr(a, _u16p) for a in xs])
    ga = arr(*[_ptr(a, _u16p) for a in gs])
    ya = arr(*[_ptr(a, _u16p) for a in ys])
    rc = lib.qko_rmsnorm_sharded(xa, ga, S, T, w * S, float(eps), ya, _ptr(partials, _f64p),
                                 _ptr(acc, _f64p), _ptr(rstd, _f64p), int(nthreads))
    if rc != 0:
        raise RuntimeError(f"qko_rmsnorm_sharded failed ({rc})")
    return {"y": ys, "partials": partials, "acc": acc, "rstd": rstd}


def e4m3_to_f64(bits) -> np.ndarray:
    lib = _load()
    b = np.asarray(bits, dtype=np.uint8)
    out = np.empty(b.shape, dtype=np.float64)
    fo, fb = out.reshape(-1), b.reshape(-1)
    for i in range(fb.size):
        fo[i] = lib.qko_e4m3_to_f64(int(fb[i]))
    return out


def f64_to_e4m3(vals) -> np.ndarray:
    lib = _load()
    v = np.asarray(vals, dtype=np.float64)
    out = np.empty(v.shape, dtype=np.uint8)
    fo, fv = out.reshape(-1), v.reshape(-1)
    for i in range(fv.size):
        fo[i] = lib.qko_f64_to_e4m3(float(fv[i]))
    return out


def rmsnorm_e4m3(x_shards: Sequence[np.ndarray], gamma_shards: Sequence[np.ndarray], eps: float, *,
                 want_y64: bool = False, nthreads: int = 1):
    """Eq. 1 with FP8-E4M3 activations (uint8 bit patterns) and bf16 gamma (uint16 bit
    patterns), given as S column slices (S = 1: unsharded).  Returns y (list of uint8
    [T,w]), partials (fp64 [S,T]), acc, rstd (fp64 [T]) and, if asked, y64 ([T,H])."""
    lib = _load()
    S = len(x_shards)
    if S < 1 or len(gamma_shards) != S:
        raise ValueError("need S >= 1 shards and as many gamma slices")
    xs = [np.ascontiguousarray(a) for a in x_shards]
    gs = [_u16(a) for a in gamma_shards]
    T, w = xs[0].shape
    for a, g in zip(xs, gs):
        if a.dtype != np.uint8 or a.shape != (T, w) or g.shape != (w,):
            raise ValueError("all shards must be uint8 [T,w] with gamma uint16 [w]")
    ys = [np.empty((T, w), dtype=np.uint8) for _ in range(S)]
    y64 = np.empty((T, w * S), dtype=np.float64) if want_y64 else None
    partials = np.empty((S, T), dtype=np.float64)
    acc = np.empty((T,), dtype=np.float64)
    rstd = np.empty((T,), dtype=np.float64)
    xa = (_u8p * S)(*[_ptr(a, _u8p) for a in xs])
    ga = (_u16p * S)(*[_ptr(a, _u16p) for a in gs])
    ya = (_u8p * S)(*[_ptr(a, _u8p) for a in ys])
    rc = lib.qko_rmsnorm_sharded_e4m3(xa, ga, S, T, w * S, float(eps), ya, _ptr(y64, _f64p),
                                      _ptr(partials, _f64p), _ptr(acc, _f64p), _ptr(rstd, _f64p), int(nthreads))
    if rc != 0:
        raise RuntimeError(f"qko_rmsnorm_sharded_e4m3 failed ({rc})")
    res = {"y": ys, "partials": partials, "acc": acc, "rstd": rstd}
    if want_y64:
        res["y64"] = y64
    return res


def rmsnorm_headwise(x_bits: np.ndarray, gamma_bits: np.ndarray, head_dim: int, eps: float, *,
                     want_y64: bool = False, nthreads: int = 1):
    """Headwise granularity: Eq. 1 on every head (head_dim consecutive columns) of every row of
    x_bits[T, H]; uint16 input = bf16, uint8 input = FP8-E4M3; gamma is bf16 [H].
    Returns y (same dtype and shape as x_bits), rstd (fp64 [T, H/head_dim]) and, if asked, y64."""
    lib = _load()
    x = np.ascontiguousarray(x_bits)
    if x.dtype not in (np.uint16, np.uint8):
        raise TypeError("activations must be uint16 (bf16) or uint8 (E4M3) bit patterns")
    g = _u16(gamma_bits)
    T, H = x.shape
    if g.shape != (H,) or head_dim < 1 or H % head_dim:
        raise ValueError("expected gamma[H] and head_dim dividing H")
    y = np.empty_like(x)
    y64 = np.empty((T, H), dtype=np.float64) if want_y64 else None
    rstd = np.empty((T, H // head_dim), dtype=np.float64)
    rc = lib.qko_rmsnorm_headwise(x.ctypes.data, _ptr(g, _u16p), T, H, int(head_dim), float(eps),
                                  1 if x.dtype == np.uint8 else 0, y.ctypes.data, _ptr(y64, _f64p),
                                  _ptr(rstd, _f64p), int(nthreads))
    if rc != 0:
        raise RuntimeError(f"qko_rmsnorm_headwise failed ({rc})")
    res = {"y": y, "rstd": rstd}
    if want_y64:
        res["y64"] = y64
    return res
