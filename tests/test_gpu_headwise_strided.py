"""GPU parity of the strided-row and the headwise entry points against the fp64 oracle."""
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
POISON = 0x7FC1


def fused_qkv(w: W.Workload, pad: int = 0):
    """[T, dq + 2*dk + pad] bf16 device buffer holding q | k | v(poison) | pad(poison)."""
    inp = W.make_inputs(w)
    T = w.tokens
    ld = w.dq + 2 * w.dk + pad
    buf = torch.full((T, ld), POISON, dtype=torch.int16, device="cuda").view(torch.bfloat16)
    buf[:, :w.dq] = inp["q"].cuda()
    buf[:, w.dq:w.dq + w.dk] = inp["k"].cuda()
    return inp, buf, ld


@pytest.mark.parametrize("T,dq,dk,pad,variant", [
    (2100, 5120, 1024, 0, "warp"),      # the fused-projection layout at a prefill size
    (16, 4096, 1024, 0, "rows"),       # decode size
    (2150, 2048, 512, 8, "warp"),       # padded rows
    (2300, 512, 128, 8, "warp"),        # short rows inside a padded fused buffer: several tokens per warp
    (33, 1024, 256, 3, "general"),     # row stride not a multiple of 8 elements
])
def test_strided_in_place_in_a_fused_qkv_buffer(libqknorm, T, dq, dk, pad, variant):
    w = W.Workload("qkv", tokens=T, dq=dq, dk=dk, shards=(1,), seed=500 + T)
    inp, buf, ld = fused_qkv(w, pad)
    q, k = buf[:, :dq], buf[:, dq:dq + dk]
    gq, gk = inp["gamma_q"].cuda(), inp["gamma_k"].cuda()
    binding.qknorm_fwd_strided(q, k, gq, gk, w.eps)
    torch.cuda.synchronize()
    assert binding.last_variant() == variant
    ref = H.oracle_unsharded(inp, w.eps, nthreads=NTHREADS)
    host = buf.cpu()
    H.compare_output(W.bf16_bits(host[:, :dq].contiguous()), ref["q"]["y"], "strided q")
    H.compare_output(W.bf16_bits(host[:, dq:dq + dk].contiguous()), ref["k"]["y"], "strided k")
    rest = host[:, dq + dk:].contiguous().view(torch.int16)
    assert bool((rest == POISON).all()), "the V columns or the row padding were written"


def test_strided_out_of_place_and_alias_rules(libqknorm):
    w = W.Workload("qkv", tokens=600, dq=2048, dk=512, shards=(1,), seed=77)
    inp, buf, ld = fused_qkv(w)
    q, k = buf[:, :w.dq], buf[:, w.dq:w.dq + w.dk]
    gq, gk = inp["gamma_q"].cuda(), inp["gamma_k"].cuda()
    oq = torch.empty((w.tokens, w.dq), dtype=torch.bfloat16, device="cuda")
    ok = torch.empty((w.tokens, w.dk), dtype=torch.bfloat16, device="cuda")
    before = buf.clone()
    binding.qknorm_fwd_strided(q, k, gq, gk, w.eps, oq, ok)
    torch.cuda.synchronize()
    assert torch.equal(buf.view(torch.int16), before.view(torch.int16))          # inputs untouched
    ref = H.oracle_unsharded(inp, w.eps, nthreads=NTHREADS)
    H.compare_output(H.bits(oq), ref["q"]["y"], "out-of-place q")
    H.compare_output(H.bits(ok), ref["k"]["y"], "out-of-place k")
    # an output that lands on the K columns of the same buffer is rejected
    with pytest.raises(binding.QKNormError) as ei:
        binding.qknorm_fwd_strided(q, k, gq, gk, w.eps, buf[:, 256:256 + w.dq], ok)
    assert ei.value.status == binding.QKNORM_ERR_ALIAS


HEAD_CASES = [
    # T, dq, dk, head_dim, variant
    (700, 5120, 1024, 128, "head"),
    (5, 4096, 4096, 128, "head"),
    (300, 2048, 512, 64, "head"),
    (300, 2048, 1024, 256, "head"),
    (257, 1920, 480, 96, "head"),       # 12 chunks per head: 16-lane groups with idle lanes
    (100, 960, 240, 24, "head"),
    (50, 1000, 200, 100, "head_general"),   # head_dim not a multiple of 8
    (40, 2048, 1024, 512, "head_general"),  # head wider than one warp step
    (64, 4096, 0, 128, "head"),
]


@pytest.mark.parametrize("T,dq,dk,hd,variant", HEAD_CASES)
def test_headwise_matches_oracle(libqknorm, T, dq, dk, hd, variant):
    w = W.Workload("heads", tokens=T, dq=dq, dk=dk, shards=(1,), seed=700 + T + hd, sigma=2.0)
    inp = W.make_inputs(w)
    q = inp["q"].cuda()
    k = inp["k"].cuda() if dk else None
    rq = torch.full((T, dq // hd), float("nan"), device="cuda")
    rk = torch.full((T, dk // hd), float("nan"), device="cuda") if dk else None
    oq, ok = binding.qknorm_fwd_headwise(q, k, inp["gamma_q"].cuda(), inp["gamma_k"].cuda() if dk else None, hd,
                                         w.eps, rstd_q=rq, rstd_k=rk)
    torch.cuda.synchronize()
    assert binding.last_variant() == variant
    for nm, out, r in (("q", oq, rq), ("k", ok, rk)):
        if out is None:
            continue
        ref = oracle.rmsnorm_headwise(W.bf16_bits(inp[nm]), W.bf16_bits(inp["gamma_" + nm]), hd, w.eps,
                                      nthreads=NTHREADS)
        H.compare_output(H.bits(out), ref["y"], f"headwise {nm} hd={hd}")
        H.compare_stat(r, ref["rstd"], f"headwise rstd {nm} hd={hd}")


def test_headwise_in_place_in_a_fused_qkv_buffer(libqknorm):
    w = W.Workload("qkvh", tokens=900, dq=4096, dk=1024, shards=(1,), seed=91)
    inp, buf, ld = fused_qkv(w)
    q, k = buf[:, :w.dq], buf[:, w.dq:w.dq + w.dk]
    binding.qknorm_fwd_headwise(q, k, inp["gamma_q"].cuda(), inp["gamma_k"].cuda(), 128, w.eps, q, k)
    torch.cuda.synchronize()
    host = buf.cpu()
    for nm, sl in (("q", slice(0, w.dq)), ("k", slice(w.dq, w.dq + w.dk))):
        ref = oracle.rmsnorm_headwise(W.bf16_bits(inp[nm]), W.bf16_bits(inp["gamma_" + nm]), 128, w.eps)
        H.compare_output(W.bf16_bits(host[:, sl].contiguous()), ref["y"], f"fused headwise {nm}")
    assert bool((host[:, w.dq + w.dk:].contiguous().view(torch.int16) == POISON).all())


def test_headwise_general_kernel_on_vector_shapes(libqknorm, monkeypatch):
    monkeypatch.setenv("QKNORM_FORCE_VARIANT", "general")
    w = W.Workload("hg", tokens=70, dq=1024, dk=256, shards=(1,), seed=13)
    inp = W.make_inputs(w)
    oq, ok = binding.qknorm_fwd_headwise(inp["q"].cuda(), inp["k"].cuda(), inp["gamma_q"].cuda(),
                                         inp["gamma_k"].cuda(), 128, w.eps)
    assert binding.last_variant() == "head_general"
    for nm, out in (("q", oq), ("k", ok)):
        ref = oracle.rmsnorm_headwise(W.bf16_bits(inp[nm]), W.bf16_bits(inp["gamma_" + nm]), 128, w.eps)
        H.compare_output(H.bits(out), ref["y"], f"head_general {nm}")


def test_headwise_rejects_bad_head_dim(libqknorm):
    q = torch.zeros((4, 256), dtype=torch.bfloat16, device="cuda")
    g = torch.ones((256,), dtype=torch.bfloat16, device="cuda")
    for hd in (0, 96, -1):
        with pytest.raises(binding.QKNormError) as ei:
            binding.qknorm_fwd_headwise(q, None, g, None, hd, 1e-6)
        assert ei.value.status == binding.QKNORM_ERR_HEADS


# ---- headwise: FP8-E4M3 activations, and column slices in one launch ---------------------------------

def _e4m3_ordinal(bits: np.ndarray) -> np.ndarray:
    b = bits.astype(np.int32)
    mag = b & 0x7F
    return np.where(b & 0x80, -mag, mag)


def _compare_e4m3(got: np.ndarray, ref: np.ndarray, what: str):
    """At most one E4M3 ordinal step from the oracle's rounded value, NaN patterns equal."""
    nan_g, nan_r = (got & 0x7F) == 0x7F, (ref & 0x7F) == 0x7F
    assert np.array_equal(nan_g, nan_r), f"{what}: NaN positions differ"
    d = np.abs(_e4m3_ordinal(got) - _e4m3_ordinal(ref))
    d[nan_r] = 0
    assert int(d.max()) <= 1, f"{what}: max ordinal distance {int(d.max())}"
    if d.size >= 4096:
        assert float((d == 1).mean()) <= 2e-3, f"{what}: too many elements one step off"


E4M3_HEAD_CASES = [
    # T, dq, dk, head_dim, variant
    (700, 5120, 1024, 128, "head"),
    (5, 4096, 4096, 128, "head"),
    (300, 2048, 512, 64, "head"),
    (260, 2048, 1024, 512, "head"),        # a 512-byte head: all 32 lanes on one head
    (257, 1920, 480, 96, "head"),
    (50, 1000, 200, 100, "head_general"),  # head_dim not a multiple of 16
    (64, 0, 1024, 128, "head"),
]


@pytest.mark.parametrize("T,dq,dk,hd,variant", E4M3_HEAD_CASES)
def test_headwise_e4m3_matches_oracle(libqknorm, T, dq, dk, hd, variant):
    w = W.Workload("heads8", tokens=T, dq=dq, dk=dk, shards=(1,), seed=900 + T + hd, sigma=2.0)
    inp = W.make_inputs_e4m3(w)
    q = inp["q"].cuda() if dq else None
    k = inp["k"].cuda() if dk else None
    rq = torch.full((T, dq // hd), float("nan"), device="cuda") if dq else None
    rk = torch.full((T, dk // hd), float("nan"), device="cuda") if dk else None
    oq, ok = binding.qknorm_fwd_headwise_e4m3(q, k, inp["gamma_q"].cuda() if dq else None,
                                              inp["gamma_k"].cuda() if dk else None, hd, w.eps, rstd_q=rq, rstd_k=rk)
    torch.cuda.synchronize()
    assert binding.last_variant() == variant
    for nm, out, r in (("q", oq, rq), ("k", ok, rk)):
        if out is None:
            continue
        ref = oracle.rmsnorm_headwise(W.e4m3_bits(inp[nm]), W.bf16_bits(inp["gamma_" + nm]), hd, w.eps,
                                      nthreads=NTHREADS)
        _compare_e4m3(W.e4m3_bits(out.cpu()), ref["y"], f"headwise e4m3 {nm} hd={hd}")
        H.compare_stat(r, ref["rstd"], f"headwise e4m3 rstd {nm} hd={hd}")


SHARDED_HEAD_CASES = [
    # T, dq, dk, head_dim, S, fp8, variant
    (900, 8192, 1024, 128, 8, False, "head"),      # the C5 shape: a K slice is ONE head
    (900, 8192, 1024, 128, 8, True, "head"),
    (333, 5120, 5120, 128, 4, False, "head"),
    (64, 4096, 1024, 64, 16, False, "head"),
    (120, 3072, 768, 96, 2, True, "head"),
    (77, 1200, 600, 100, 3, False, "head_general"),
    (40, 2048, 0, 128, 4, False, "head"),
]


@pytest.mark.parametrize("T,dq,dk,hd,S,fp8,variant", SHARDED_HEAD_CASES)
@pytest.mark.parametrize("in_place", [False, True])
def test_headwise_sharded_in_one_launch(libqknorm, T, dq, dk, hd, S, fp8, variant, in_place):
    """Heads never straddle a slice, so the oracle is the headwise definition on the gathered row."""
    w = W.Workload("headsS", tokens=T, dq=dq, dk=dk, shards=(S,), seed=1100 + T + S, sigma=1.5)
    inp = (W.make_inputs_e4m3 if fp8 else W.make_inputs)(w)
    to_bits = W.e4m3_bits if fp8 else W.bf16_bits
    dev = {n: ([t.cuda() for t in W.shard_columns(inp[n], S)] if inp[n].shape[-1] else None)
           for n in ("q", "k", "gamma_q", "gamma_k")}
    rq = torch.full((T, dq // hd), float("nan"), device="cuda") if dq else None
    rk = torch.full((T, dk // hd), float("nan"), device="cuda") if dk else None
    n0 = binding.launch_count()
    oq, ok = binding.qknorm_fwd_headwise_sharded(dev["q"], dev["k"], dev["gamma_q"], dev["gamma_k"], hd, w.eps,
                                                 dev["q"] if in_place else None, dev["k"] if in_place else None,
                                                 rstd_q=rq, rstd_k=rk)
    torch.cuda.synchronize()
    assert binding.launch_count() - n0 == 1 and binding.last_variant() == variant
    for nm, outs, r in (("q", oq, rq), ("k", ok, rk)):
        if outs is None:
            continue
        ref = oracle.rmsnorm_headwise(to_bits(inp[nm]), W.bf16_bits(inp["gamma_" + nm]), hd, w.eps, nthreads=NTHREADS)
        got = to_bits(W.unshard_columns([t.cpu() for t in outs]))
        if fp8:
            _compare_e4m3(got, ref["y"], f"sharded headwise e4m3 {nm}")
        else:
            H.compare_output(got, ref["y"], f"sharded headwise {nm}")
        H.compare_stat(r, ref["rstd"], f"sharded headwise rstd {nm}")


def test_headwise_sharded_rejects_a_head_that_straddles_slices(libqknorm):
    S, T = 4, 8
    qs = [torch.zeros((T, 192), dtype=torch.bfloat16, device="cuda") for _ in range(S)]   # 768 wide, slices of 192
    gs = [torch.ones((192,), dtype=torch.bfloat16, device="cuda") for _ in range(S)]
    with pytest.raises(binding.QKNormError) as ei:
        binding.qknorm_fwd_headwise_sharded(qs, None, gs, None, 128, 1e-6)                # 128 divides 768, not 192
    assert ei.value.status == binding.QKNORM_ERR_HEADS
    binding.qknorm_fwd_headwise_sharded(qs, None, gs, None, 96, 1e-6)
    torch.cuda.synchronize()
