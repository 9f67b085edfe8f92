"""qknorm_baseline_two_pass_static: the entry point for callers that may not allocate
device memory (its scratch is an array inside the library image).

It must give what qknorm_baseline_two_pass gives with a caller-owned scratch buffer, on
every call, and both must agree with the CPU oracle: the built-in array is shared by all
calls and keeps the previous call's contents, so the test makes two calls in a row on
different data (the second problem is smaller, so values of the first stay in the array).  The file name makes
pytest collect it last; the test needs nothing from the tests before it and also passes
when it is the only one run in a fresh process.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_09160_b200 import binding
from paper_2608_09160_b200 import workloads as W
from tests import gpu_harness as H
from tests.util import ordinal_distance

pytestmark = pytest.mark.gpu


def device_shards(w: W.Workload, S: int):
    inp = W.make_inputs(w)
    return {n: [t.cuda() for t in W.shard_columns(inp[n], S)] for n in ("q", "k", "gamma_q", "gamma_k")}


def oracle_bits(w: W.Workload):
    """The fp64 definition on the same seeded inputs, rounded once to bf16."""
    inp = W.make_inputs(w)
    return {n: oracle.rmsnorm(W.bf16_bits(inp[n]), W.bf16_bits(inp["gamma_" + n]), w.eps, nthreads=8)["y"]
            for n in ("q", "k")}


def bits(parts):
    return W.bf16_bits(W.unshard_columns([t.cpu() for t in parts]))


def test_static_scratch_matches_caller_scratch_on_two_calls_in_a_row(libqknorm):
    S = 8
    cap = binding.static_scratch_capacity()
    assert cap == 262144
    # two different problems, the second one smaller, so stale values of the first call stay in the array
    problems = [W.Workload("noalloc_a", tokens=3000, dq=5120, dk=1024, shards=(S,), seed=41, sigma=2.0),
                W.Workload("noalloc_b", tokens=777, dq=5120, dk=1024, shards=(S,), seed=42, sigma=0.5)]
    for w in problems:
        assert 2 * S * w.tokens <= cap
        d = device_shards(w, S)
        # existing entry point, caller-owned scratch
        scratch = torch.empty((2 * S * w.tokens,), dtype=torch.float32, device="cuda")
        want_q, want_k = binding.qknorm_baseline_two_pass(d["q"], d["k"], d["gamma_q"], d["gamma_k"], w.eps,
                                                          scratch=scratch)
        # new entry point: outputs are passed in, nothing is allocated by the call
        got_q = [torch.empty_like(t) for t in d["q"]]
        got_k = [torch.empty_like(t) for t in d["k"]]
        torch.cuda.synchronize()
        n0 = binding.launch_count()
        binding.qknorm_baseline_two_pass_static(d["q"], d["k"], d["gamma_q"], d["gamma_k"], w.eps, got_q, got_k)
        torch.cuda.synchronize()
        assert binding.launch_count() - n0 == 2
        ref = oracle_bits(w)
        for name, got in (("q", got_q), ("k", got_k)):
            H.compare_output(bits(got), ref[name], f"{w.name} {name}: built-in scratch against the oracle")
        for name, got, want in (("q", got_q, want_q), ("k", got_k, want_k)):
            dist = ordinal_distance(bits(got), bits(want))
            assert int(dist.max()) <= 1, f"{w.name} {name}: {int(dist.max())} bf16 steps apart"      # the suite's bar
            assert int(dist.max()) == 0, f"{w.name} {name}: same kernels, same order: expected identical bits"


def test_static_scratch_in_place_and_size_limit(libqknorm):
    S = 4
    w = W.Workload("noalloc_c", tokens=512, dq=2048, dk=512, shards=(S,), seed=43)
    d = device_shards(w, S)
    scratch = torch.empty((2 * S * w.tokens,), dtype=torch.float32, device="cuda")
    want_q, want_k = binding.qknorm_baseline_two_pass(d["q"], d["k"], d["gamma_q"], d["gamma_k"], w.eps, scratch=scratch)
    binding.qknorm_baseline_two_pass_static(d["q"], d["k"], d["gamma_q"], d["gamma_k"], w.eps, d["q"], d["k"])
    torch.cuda.synchronize()
    assert np.array_equal(bits(d["q"]), bits(want_q)) and np.array_equal(bits(d["k"]), bits(want_k))
    ref = oracle_bits(w)
    H.compare_output(bits(d["q"]), ref["q"], "in place, built-in scratch: q against the oracle")
    H.compare_output(bits(d["k"]), ref["k"], "in place, built-in scratch: k against the oracle")
    # one token more than the built-in array can serve: refused with its own status, nothing launched
    cap = binding.static_scratch_capacity()
    T = cap // (2 * S) + 1
    big = {n: [torch.zeros((T, 8), dtype=torch.bfloat16, device="cuda") for _ in range(S)] for n in ("q", "k")}
    g = [torch.ones((8,), dtype=torch.bfloat16, device="cuda") for _ in range(S)]
    n0 = binding.launch_count()
    with pytest.raises(binding.QKNormError, match="built-in scratch") as ei:
        binding.qknorm_baseline_two_pass_static(big["q"], big["k"], g, g, 1e-6, big["q"], big["k"])
    assert ei.value.status == binding.QKNORM_ERR_STATIC_LIMIT and binding.launch_count() == n0
    # exactly at the limit it runs
    T -= 1
    ok = {n: [t[:T] for t in big[n]] for n in ("q", "k")}
    binding.qknorm_baseline_two_pass_static(ok["q"], ok["k"], g, g, 1e-6, ok["q"], ok["k"])
    torch.cuda.synchronize()
