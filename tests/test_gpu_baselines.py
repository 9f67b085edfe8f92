"""The one-GPU stand-ins for the paper's comparison paths compute the same result as the
fused sharded kernel: parity with the same oracle, same tolerance."""
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

SHAPES = [(900, 5120, 1024, 8), (64, 4096, 4096, 4), (700, 2048, 512, 1), (37, 1000, 136, 2), (5, 8, 8, 1)]


def setup(T, dq, dk, S, seed):
    w = W.Workload("base", tokens=T, dq=dq, dk=dk, shards=(S,), seed=seed, sigma=1.5)
    inp = W.make_inputs(w)
    dev = {n: [t.cuda() for t in W.shard_columns(inp[n], S)] for n in ("q", "k", "gamma_q", "gamma_k")}
    ref = H.oracle_unsharded(inp, w.eps, nthreads=NTHREADS)
    for n in ("q", "k"):      # every slice's own sum of squares, from the oracle's sharded form
        sh = oracle.rmsnorm_sharded([W.bf16_bits(t) for t in W.shard_columns(inp[n], S)],
                                    [W.bf16_bits(t) for t in W.shard_columns(inp["gamma_" + n], S)], w.eps)
        ref[n]["partials"] = sh["partials"]
    return w, dev, ref


def check(outs_q, outs_k, ref, what):
    H.compare_output(H.bits(W.unshard_columns([t.cpu() for t in outs_q])), ref["q"]["y"], what + " q")
    H.compare_output(H.bits(W.unshard_columns([t.cpu() for t in outs_k])), ref["k"]["y"], what + " k")


@pytest.mark.parametrize("T,dq,dk,S", SHAPES)
@pytest.mark.parametrize("in_place", [False, True])
def test_gather_then_norm(libqknorm, T, dq, dk, S, in_place):
    w, dev, ref = setup(T, dq, dk, S, 800 + T)
    scratch = torch.full((T * (dq + dk) + 64,), 0x7FC1, dtype=torch.int16, device="cuda")
    oq = dev["q"] if in_place else None
    ok = dev["k"] if in_place else None
    n0 = binding.launch_count()
    oq, ok = binding.qknorm_baseline_gather_then_norm(dev["q"], dev["k"], dev["gamma_q"], dev["gamma_k"], w.eps,
                                                      oq, ok, scratch=scratch)
    torch.cuda.synchronize()
    assert binding.launch_count() - n0 == 2
    check(oq, ok, ref, f"gather-then-norm T={T} S={S}")
    assert bool((scratch[T * (dq + dk):] == 0x7FC1).all()), "wrote past the stated scratch size"


@pytest.mark.parametrize("T,dq,dk,S", SHAPES)
@pytest.mark.parametrize("in_place", [False, True])
def test_two_pass(libqknorm, T, dq, dk, S, in_place):
    w, dev, ref = setup(T, dq, dk, S, 900 + T)
    scratch = torch.full((2 * S * T + 16,), float("nan"), dtype=torch.float32, device="cuda")
    oq = dev["q"] if in_place else None
    ok = dev["k"] if in_place else None
    n0 = binding.launch_count()
    oq, ok = binding.qknorm_baseline_two_pass(dev["q"], dev["k"], dev["gamma_q"], dev["gamma_k"], w.eps, oq, ok,
                                              scratch=scratch)
    torch.cuda.synchronize()
    assert binding.launch_count() - n0 == 2 and binding.last_variant() == "two_pass"
    check(oq, ok, ref, f"two-pass T={T} S={S}")
    # the scratch holds every slice's sum of squares: [tensor][slice][token]
    got = scratch[:2 * S * T].view(2, S, T)
    H.compare_stat(got[0], ref["q"]["partials"], "two-pass scratch q")
    H.compare_stat(got[1], ref["k"]["partials"], "two-pass scratch k")
    assert bool(torch.isnan(scratch[2 * S * T:]).all()), "wrote past the stated scratch size"


def test_scratch_is_validated(libqknorm):
    w, dev, ref = setup(40, 1024, 256, 4, 5)
    small = torch.empty((16,), dtype=torch.float32, device="cuda")
    for fn in (binding.qknorm_baseline_gather_then_norm, binding.qknorm_baseline_two_pass):
        with pytest.raises(binding.QKNormError) as ei:
            fn(dev["q"], dev["k"], dev["gamma_q"], dev["gamma_k"], w.eps, scratch=small)
        assert ei.value.status == binding.QKNORM_ERR_SCRATCH
    # scratch that overlaps an input
    with pytest.raises(binding.QKNormError) as ei:
        binding.qknorm_baseline_two_pass(dev["q"], dev["k"], dev["gamma_q"], dev["gamma_k"], w.eps,
                                         scratch=dev["q"][0].view(torch.float32).view(-1))
    assert ei.value.status == binding.QKNORM_ERR_SCRATCH
