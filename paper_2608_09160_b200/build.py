"""Builds libqknorm.so (sm_100a only) with nvcc, in-tree.

    python -m paper_2608_09160_b200.build [--force] [--verbose]

The row kernels are instantiated once per value of N (chunks per thread) in their own translation
unit, so the objects are compiled in parallel and linked into one shared
library next to this file.
"""
from __future__ import annotations

import argparse
import concurrent.futures as cf
import hashlib
import os
import shutil
import subprocess
import sys
from typing import List, Tuple

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG_DIR, "csrc")
INCLUDE = os.path.join(os.path.dirname(PKG_DIR), "include")
BUILD_DIR = os.path.join(PKG_DIR, "build")
LIB_PATH = os.path.join(PKG_DIR, "libqknorm.so")

CHUNKS_PER_THREAD = (1, 2, 3, 4, 6, 8)          # row / ring kernels
CHUNK_SLOTS_PER_LANE = tuple(range(4, 44, 4))    # warp-per-row kernel

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-std=c++17", "-lineinfo",
    "-Xcompiler", "-fPIC",
    "-I", INCLUDE, "-I", CSRC,
]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found; libqknorm cannot be built")
    return exe


def _units() -> List[Tuple[str, str, List[str]]]:
    """(object name, source, extra flags)"""
    units = [("qknorm_api.o", os.path.join(CSRC, "qknorm_api.cu"), [])]
    for n in CHUNKS_PER_THREAD:
        units.append((f"qknorm_rows_n{n}.o", os.path.join(CSRC, "qknorm_rows_inst.cu"), [f"-DQKNORM_N={n}"]))
    for l in CHUNK_SLOTS_PER_LANE:
        for io, tag in (("IoBf16", "bf16"), ("IoE4m3", "e4m3")):
            units.append((f"qknorm_warp_{tag}_l{l}.o", os.path.join(CSRC, "qknorm_warp_inst.cu"),
                          [f"-DQKNORM_L={l}", f"-DQKNORM_IO={io}", f"-DQKNORM_IO_TAG={tag}"]))
    units.append(("qknorm_tp.o", os.path.join(CSRC, "qknorm_tp_inst.cu"), []))
    return units


def _source_digest() -> str:
    h = hashlib.sha256()
    paths = [os.path.join(CSRC, f) for f in sorted(os.listdir(CSRC))]
    paths += [os.path.join(INCLUDE, f) for f in sorted(os.listdir(INCLUDE))]
    paths.append(os.path.abspath(__file__))
    for p in paths:
        if os.path.isfile(p):
            h.update(p.encode())
            with open(p, "rb") as fh:
                h.update(fh.read())
    return h.hexdigest()


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile and link; returns the path of libqknorm.so.  Skips the work when
    the sources have not changed since the library was built."""
    os.makedirs(BUILD_DIR, exist_ok=True)
    stamp = os.path.join(BUILD_DIR, "sources.sha256")
    digest = _source_digest()
    if not force and os.path.exists(LIB_PATH) and os.path.exists(stamp):
        with open(stamp) as fh:
            if fh.read().strip() == digest:
                return LIB_PATH
    nvcc = _nvcc()
    extra = ["-Xptxas", "-v"] if verbose else []

    def compile_one(unit):
        obj, src, flags = unit
        out = os.path.join(BUILD_DIR, obj)
        cmd = [nvcc, *NVCC_FLAGS, *extra, *flags, "-c", src, "-o", out]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed for {obj}:\n{' '.join(cmd)}\n{r.stdout}\n{r.stderr}")
        return out, r.stderr

    units = _units()
    with cf.ThreadPoolExecutor(max_workers=min(len(units), os.cpu_count() or 4)) as pool:
        results = list(pool.map(compile_one, units))
    if verbose:
        for out, log in results:
            sys.stderr.write(f"==== {os.path.basename(out)}\n{log}\n")
    tmp = LIB_PATH + f".tmp{os.getpid()}"
    cmd = [nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp,
           *[o for o, _ in results]]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed:\n{' '.join(cmd)}\n{r.stdout}\n{r.stderr}")
    os.replace(tmp, LIB_PATH)
    with open(stamp, "w") as fh:
        fh.write(digest)
    return LIB_PATH


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--force", action="store_true")
    ap.add_argument("--verbose", action="store_true", help="print ptxas register/shared-memory usage")
    a = ap.parse_args()
    print(build(force=a.force, verbose=a.verbose))
