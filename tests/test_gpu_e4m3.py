"""GPU parity of the FP8-E4M3 entry points against the fp64 oracle (same bars as bf16:
at most one ordinal step of the storage format from the fp64 result rounded to it,
statistic within 1e-5)."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2608_09160_b200 import binding
from paper_2608_09160_b200 import workloads as W
from tests import gpu_harness as H
from tests.util import e4m3_ordinal_distance

pytestmark = pytest.mark.gpu
NTHREADS = max(1, min(32, os.cpu_count() or 1))

SHAPES = [
    # name, T, dq, dk, shard counts, expected variant per shard count
    ("e_decode", 8, 4096, 4096, (1, 4), ("rows", "rows")),
    ("e_gqa", 2300, 5120, 1024, (8, 1), ("warp", "warp")),
    ("e_mha", 2100, 5120, 5120, (4,), ("warp",)),
    ("e_odd_width", 650, 1000, 136, (1,), ("general",)),          # not a multiple of 16 elements
    ("e_ragged", 2177, 1008, 144, (1, 3), ("warp", "warp")),       # multiples of 16, ragged over the lanes
    ("e_tiny", 3, 16, 16, (1,), ("rows",)),
    ("e_konly", 2100, 0, 2048, (2,), ("warp",)),
]


def compare_e4m3(got: np.ndarray, ref: np.ndarray, what: str):
    d = e4m3_ordinal_distance(got, ref)
    assert int(d.max()) <= 1, f"{what}: max ordinal distance {int(d.max())}"
    rate = float((d == 1).mean())
    if d.size >= 4096:
        assert rate <= 2e-3, f"{what}: {rate:.2e} of the elements are one step off"
    return rate


def run(w: W.Workload, S: int, in_place: bool):
    inp = W.make_inputs_e4m3(w)
    T = w.tokens
    out = {}
    stats = {}
    names = [n for n, d in (("q", w.dq), ("k", w.dk)) if d > 0]
    xs = {n: [t.cuda() for t in W.shard_columns(inp[n], S)] for n in names}
    gs = {n: [t.cuda() for t in W.shard_columns(inp["gamma_" + n], S)] for n in names}
    outs = {n: (xs[n] if in_place else [torch.full_like(t.view(torch.uint8), 0x7F).view(torch.float8_e4m3fn) for t in xs[n]])
            for n in names}
    rstd = {n: torch.full((T,), float("nan"), device="cuda") for n in names}
    part = {n: torch.full((S, T), float("nan"), device="cuda") for n in names}
    g = lambda d, n: d.get(n)
    if S == 1:
        binding.qknorm_fwd_e4m3(g(xs, "q")[0] if "q" in xs else None, g(xs, "k")[0] if "k" in xs else None,
                                g(gs, "q")[0] if "q" in gs else None, g(gs, "k")[0] if "k" in gs else None, w.eps,
                                g(outs, "q")[0] if "q" in outs else None, g(outs, "k")[0] if "k" in outs else None,
                                rstd_q=g(rstd, "q"), rstd_k=g(rstd, "k"))
    else:
        binding.qknorm_fwd_sharded_e4m3(g(xs, "q"), g(xs, "k"), g(gs, "q"), g(gs, "k"), w.eps, g(outs, "q"), g(outs, "k"),
                                        partials_q=g(part, "q"), partials_k=g(part, "k"),
                                        rstd_q=g(rstd, "q"), rstd_k=g(rstd, "k"))
    torch.cuda.synchronize()
    variant = binding.last_variant()
    for n in names:
        xb = [W.e4m3_bits(t) for t in W.shard_columns(inp[n], S)]
        gb = [W.bf16_bits(t) for t in W.shard_columns(inp["gamma_" + n], S)]
        ref = oracle.rmsnorm_e4m3(xb, gb, w.eps, nthreads=NTHREADS)
        got = np.concatenate([W.e4m3_bits(t.cpu()) for t in outs[n]], axis=1)
        compare_e4m3(got, np.concatenate(ref["y"], axis=1), f"{w.name}/S={S}/{n}")
        H.compare_stat(rstd[n], ref["rstd"], f"{w.name}/S={S}/rstd_{n}")
        if S > 1:
            H.compare_stat(part[n], ref["partials"], f"{w.name}/S={S}/partials_{n}")
    return variant


CASES = [(name, T, dq, dk, S, v) for name, T, dq, dk, shards, vs in SHAPES for S, v in zip(shards, vs)]


@pytest.mark.parametrize("name,T,dq,dk,S,variant", CASES, ids=[f"{c[0]}-S{c[4]}" for c in CASES])
@pytest.mark.parametrize("in_place", [False, True])
def test_e4m3_matches_oracle(libqknorm, name, T, dq, dk, S, variant, in_place):
    w = W.Workload(name, tokens=T, dq=dq, dk=dk, shards=(S,), seed=300 + len(name) + S, sigma=1.5,
                   outlier_frac=0.01 if dq >= 4096 else 0.0)
    assert run(w, S, in_place) == variant


@pytest.mark.parametrize("name,T,dq,dk", [("e_ragged", 2177, 1008, 144), ("e_short", 3001, 2048, 256), ("e_tiny_rows", 2600, 128, 32)])
@pytest.mark.parametrize("forced", ["tile", None])
def test_e4m3_short_unsharded_rows(libqknorm, monkeypatch, name, T, dq, dk, forced):
    """Short FP8 rows: several tokens side by side per warp (variant "warp"), and the three-stage tiled
    kernel when it is asked for."""
    if forced:
        monkeypatch.setenv("QKNORM_FORCE_VARIANT", forced)
    w = W.Workload(name, tokens=T, dq=dq, dk=dk, shards=(1,), seed=340 + len(name), sigma=1.5)
    for in_place in (False, True):
        assert run(w, 1, in_place) == (forced or "warp")


def test_e4m3_saturates_and_propagates_nan(libqknorm):
    T, d = 4, 256
    x = torch.zeros((T, d), dtype=torch.float32)
    x[0, 3] = 1.0                      # one-hot: y_3 = gamma * sqrt(256) = 16 * 200 -> saturates at 448
    x[1] = 2.0
    x[3] = 1.0
    x8 = x.to(torch.float8_e4m3fn)
    bits = x8.view(torch.uint8)
    bits[2, 7] = 0x7F                  # NaN poisons its row
    g = torch.full((d,), 200.0, dtype=torch.bfloat16)
    out, _ = binding.qknorm_fwd_e4m3(x8.cuda(), None, g.cuda(), None, 0.0)
    with np.errstate(all="ignore"):
        ref = oracle.rmsnorm_e4m3([W.e4m3_bits(x8)], [W.bf16_bits(g)], 0.0)["y"][0]
    got = W.e4m3_bits(out.cpu())
    assert e4m3_ordinal_distance(got, ref).max() == 0
    assert got[0, 3] == 0x7E and (got[2] & 0x7F == 0x7F).all()


@pytest.mark.parametrize("name", ["C3", "C4", "C5"])
def test_full_size_e4m3(libqknorm, name):
    w = W.WORKLOADS[name]
    S = w.shards[-1]
    inp = W.make_inputs_e4m3(w)
    qs = [t.cuda() for t in W.shard_columns(inp["q"], S)]
    ks = [t.cuda() for t in W.shard_columns(inp["k"], S)]
    gqs = [t.cuda() for t in W.shard_columns(inp["gamma_q"], S)]
    gks = [t.cuda() for t in W.shard_columns(inp["gamma_k"], S)]
    oqs = qs if w.in_place else [torch.empty_like(t) for t in qs]
    oks = ks if w.in_place else [torch.empty_like(t) for t in ks]
    binding.qknorm_fwd_sharded_e4m3(qs, ks, gqs, gks, w.eps, oqs, oks)
    torch.cuda.synchronize()
    assert binding.last_variant() == "warp"
    # every row, element by element, in blocks of 8192 rows (bounded host memory)
    for nm, outs in (("q", oqs), ("k", oks)):
        gb = [W.bf16_bits(t) for t in W.shard_columns(inp["gamma_" + nm], S)]
        x_sh = W.shard_columns(inp[nm], S)
        host = [t.cpu() for t in outs]
        ones, count = 0.0, 0
        for lo in range(0, w.tokens, 8192):
            hi = min(w.tokens, lo + 8192)
            xb = [W.e4m3_bits(t[lo:hi].contiguous()) for t in x_sh]
            ref = oracle.rmsnorm_e4m3(xb, gb, w.eps, nthreads=NTHREADS)
            got = np.concatenate([W.e4m3_bits(t[lo:hi].contiguous()) for t in host], axis=1)
            rate = compare_e4m3(got, np.concatenate(ref["y"], axis=1), f"{name}/e4m3/{nm} rows {lo}..{hi}")
            ones += rate * got.size
            count += got.size
        print(f"{name} e4m3 {nm}: all {w.tokens} rows, rate at distance 1 {ones / count:.2e}")


@pytest.mark.parametrize("dq,dk,variant", [(2048, 512, "warp"), (8192, 1024, "warp")])
def test_e4m3_gamma_outside_fp16_takes_the_bf16_gamma_path(libqknorm, dq, dk, variant):
    """The prefill kernels keep an fp16 copy of gamma when every value fits fp16; one value that
    does not (2^-20, 1e5) must switch the whole call to the bf16-gamma arithmetic with the same result."""
    w = W.Workload("e_wide_gamma", tokens=2200, dq=dq, dk=dk, shards=(1,), seed=31, sigma=1.5)
    inp = W.make_inputs_e4m3(w)
    gq = inp["gamma_q"].clone()
    gq[5] = 2.0 ** -20
    gq[77] = 1.0e5
    gq[300] = -(2.0 ** -18)
    ref_q = oracle.rmsnorm_e4m3([W.e4m3_bits(inp["q"])], [W.bf16_bits(gq)], w.eps)["y"][0]
    ref_k = oracle.rmsnorm_e4m3([W.e4m3_bits(inp["k"])], [W.bf16_bits(inp["gamma_k"])], w.eps)["y"][0]
    oq, ok = binding.qknorm_fwd_e4m3(inp["q"].cuda(), inp["k"].cuda(), gq.cuda(), inp["gamma_k"].cuda(), w.eps)
    torch.cuda.synchronize()
    assert binding.last_variant() == variant
    compare_e4m3(W.e4m3_bits(oq.cpu()), ref_q, "wide gamma q")
    compare_e4m3(W.e4m3_bits(ok.cpu()), ref_k, "wide gamma k")
    assert (W.e4m3_bits(oq.cpu())[:, 77] & 0x7F == 0x7E).mean() > 0.5     # 1e5 * x saturates


@pytest.mark.parametrize("T,dq,dk,pad,variant", [(2200, 4096, 1024, 0, "warp"), (2300, 1024, 256, 16, "warp"),
                                                  (40, 2048, 512, 32, "rows")])
def test_e4m3_rows_strided_inside_a_fused_qkv_buffer(libqknorm, T, dq, dk, pad, variant):
    """FP8 rows that are column blocks of one fused [T, dq + 2*dk (+ pad)] buffer, normalised in place;
    the V block and the padding keep their bytes."""
    w = W.Workload("e_qkv", tokens=T, dq=dq, dk=dk, shards=(1,), seed=600 + T, sigma=1.5)
    inp = W.make_inputs_e4m3(w)
    ld = dq + 2 * dk + pad
    buf = torch.full((T, ld), 0x55, dtype=torch.uint8, device="cuda").view(torch.float8_e4m3fn)
    buf[:, :dq] = inp["q"].cuda()
    buf[:, dq:dq + dk] = inp["k"].cuda()
    q, k = buf[:, :dq], buf[:, dq:dq + dk]
    binding.qknorm_fwd_strided(q, k, inp["gamma_q"].cuda(), inp["gamma_k"].cuda(), w.eps)
    torch.cuda.synchronize()
    assert binding.last_variant() == variant
    host = buf.cpu()
    for nm, sl in (("q", slice(0, dq)), ("k", slice(dq, dq + dk))):
        ref = oracle.rmsnorm_e4m3([W.e4m3_bits(inp[nm])], [W.bf16_bits(inp["gamma_" + nm])], w.eps)
        compare_e4m3(W.e4m3_bits(host[:, sl].contiguous()), ref["y"][0], f"strided e4m3 {nm}")
    assert bool((host[:, dq + dk:].contiguous().view(torch.uint8) == 0x55).all())
