"""GPU parity at the five full-size workloads, in the launch configuration the
benchmark times (same entry points, same shard counts, in place where the
workload says so)."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2608_09160_b200 import binding
from paper_2608_09160_b200 import workloads as W
from tests import gpu_harness as H

pytestmark = pytest.mark.gpu
NTHREADS = max(1, min(32, os.cpu_count() or 1))
BLOCK_ROWS = 8192         # the oracle walks EVERY row of every workload, this many at a time


@pytest.mark.parametrize("name,S", [(n, S) for n, w in W.WORKLOADS.items() for S in w.shards])
def test_full_size_workload(libqknorm, name, S):
    w = W.WORKLOADS[name]
    inp = W.make_inputs(w)
    T = w.tokens
    dev = {k: v.cuda() for k, v in inp.items()}
    rq = torch.empty((T,), dtype=torch.float32, device="cuda")
    rk = torch.empty((T,), dtype=torch.float32, device="cuda")
    if S == 1:
        oq = dev["q"] if w.in_place else torch.empty_like(dev["q"])
        ok = dev["k"] if w.in_place else torch.empty_like(dev["k"])
        binding.qknorm_fwd(dev["q"], dev["k"], dev["gamma_q"], dev["gamma_k"], w.eps, oq, ok, rstd_q=rq, rstd_k=rk)
        torch.cuda.synchronize()
        out = {"q": oq.cpu(), "k": ok.cpu()}
    else:
        qs, ks = W.shard_columns(dev["q"], S), W.shard_columns(dev["k"], S)
        gqs, gks = W.shard_columns(dev["gamma_q"], S), W.shard_columns(dev["gamma_k"], S)
        del dev["q"], dev["k"]
        oqs = qs if w.in_place else [torch.empty_like(t) for t in qs]
        oks = ks if w.in_place else [torch.empty_like(t) for t in ks]
        binding.qknorm_fwd_sharded(qs, ks, gqs, gks, w.eps, oqs, oks, rstd_q=rq, rstd_k=rk)
        torch.cuda.synchronize()
        out = {"q": W.unshard_columns([t.cpu() for t in oqs]), "k": W.unshard_columns([t.cpu() for t in oks])}
    assert binding.last_variant() != "general"
    # every row of the workload, element by element, in blocks (bounded host memory)
    for nm, r in (("q", rq), ("k", rk)):
        gam = W.bf16_bits(inp["gamma_" + nm])
        r_host = r.cpu()
        worst, ones, count = 0, 0, 0
        for lo in range(0, T, BLOCK_ROWS):
            hi = min(T, lo + BLOCK_ROWS)
            ref = oracle.rmsnorm(W.bf16_bits(inp[nm][lo:hi]), gam, w.eps, nthreads=NTHREADS)
            got = W.bf16_bits(out[nm][lo:hi])
            rep = H.compare_output(got, ref["y"], f"{name}/S={S}/{nm} rows {lo}..{hi}")
            H.compare_stat(r_host[lo:hi], ref["rstd"], f"{name}/S={S}/rstd_{nm} rows {lo}..{hi}")
            worst = max(worst, rep["max_ordinal"])
            ones += rep["rate_dist1"] * got.size
            count += got.size
        print(f"{name} S={S} {nm}: rows checked {T} of {T}, max ordinal {worst}, "
              f"rate at distance 1 {ones / max(count, 1):.2e}")
    # properties that hold for every row at any size: the output is finite and |y| <= |gamma| sqrt(H)
    for nm, d in (("q", w.dq), ("k", w.dk)):
        y = out[nm].float()
        assert bool(torch.isfinite(y).all())
        bound = inp["gamma_" + nm].float().abs() * (d ** 0.5) * (1 + 2 ** -7)
        assert bool((y.abs() <= bound[None, :]).all())


def test_rows_beyond_2_to_the_31_elements(libqknorm):
    """Index arithmetic: a Q tensor of 2.3e9 elements (4.6 GB), so byte and element offsets of
    the last rows do not fit in 32 bits.  The tensor is a 2048-token seeded block repeated along
    the token axis, so every row has a known oracle row; rows near the end are compared."""
    base = W.Workload("big_base", tokens=2048, dq=8192, dk=1024, shards=(8,), seed=21)
    inp = W.make_inputs(base)
    reps = 140                                   # 286720 tokens x 8192 = 2.35e9 elements
    T = base.tokens * reps
    S = 8
    qs = [t.cuda().repeat(reps, 1) for t in W.shard_columns(inp["q"], S)]
    ks = [t.cuda().repeat(reps, 1) for t in W.shard_columns(inp["k"], S)]
    gqs = [t.cuda() for t in W.shard_columns(inp["gamma_q"], S)]
    gks = [t.cuda() for t in W.shard_columns(inp["gamma_k"], S)]
    assert sum(t.numel() for t in qs) > 2 ** 31
    binding.qknorm_fwd_sharded(qs, ks, gqs, gks, base.eps, qs, ks)      # in place
    torch.cuda.synchronize()
    ref = H.oracle_unsharded(inp, base.eps, nthreads=NTHREADS)
    for lo in (0, T // 2 - 1024, T - 2048):                              # first, middle, last block of rows
        got_q = W.unshard_columns([t[lo:lo + 2048].cpu() for t in qs])
        got_k = W.unshard_columns([t[lo:lo + 2048].cpu() for t in ks])
        shift = lo % base.tokens
        want_q = np.roll(ref["q"]["y"], -shift, axis=0)
        want_k = np.roll(ref["k"]["y"], -shift, axis=0)
        H.compare_output(W.bf16_bits(got_q), want_q, f"rows {lo}.. q")
        H.compare_output(W.bf16_bits(got_k), want_k, f"rows {lo}.. k")
