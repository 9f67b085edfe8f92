"""The token queue of the prefill kernel (one warp per token).

After its first two waves of tokens a warp takes its next token from a counter that belongs
to the launch's stream; the last warp to leave puts the counter back to zero.  These tests
check what could go wrong with that: a counter that is not back at zero when the next call
on the stream starts, calls on many streams at once (more streams than there are counters),
a launch captured into a CUDA graph (which gets no counter and keeps the fixed round-robin
schedule), and that the schedule never changes a result.  Every result is compared with the
CPU oracle."""
import os

import numpy as np
import pytest
import torch

from paper_2608_09160_b200 import binding
from paper_2608_09160_b200 import workloads as W
from tests import gpu_harness as H

pytestmark = pytest.mark.gpu
NTHREADS = max(1, min(16, os.cpu_count() or 1))


def shards_on_device(inp, S):
    return {n: [t.cuda() for t in W.shard_columns(inp[n], S)] for n in ("q", "k", "gamma_q", "gamma_k")}


def check(w, inp, oq, ok, what):
    ref = H.oracle_unsharded(inp, w.eps, nthreads=NTHREADS)
    H.compare_output(H.bits(W.unshard_columns([t.cpu() for t in oq])), ref["q"]["y"], f"{what} q")
    H.compare_output(H.bits(W.unshard_columns([t.cpu() for t in ok])), ref["k"]["y"], f"{what} k")


def test_calls_of_different_sizes_back_to_back_on_one_stream(libqknorm):
    """Each call must find the stream's counter at zero: if the previous call left anything in
    it, tokens of the next call would be skipped (their output rows keep the poison)."""
    S = 8
    sizes = [9000, 2500, 12001, 2305, 6000]
    outs = []
    for i, T in enumerate(sizes):
        w = W.Workload(f"queue_{T}", tokens=T, dq=5120, dk=1024, shards=(S,), seed=60 + i)
        inp = W.make_inputs(w)
        d = shards_on_device(inp, S)
        oq = [torch.full_like(t, float("nan")) for t in d["q"]]
        ok = [torch.full_like(t, float("nan")) for t in d["k"]]
        binding.qknorm_fwd_sharded(d["q"], d["k"], d["gamma_q"], d["gamma_k"], w.eps, oq, ok)   # no sync in between
        assert binding.last_variant() == "warp"
        outs.append((w, inp, oq, ok))
    torch.cuda.synchronize()
    for w, inp, oq, ok in outs:
        check(w, inp, oq, ok, w.name)
    assert binding.device_error_word() == 0


def test_queue_and_fixed_schedule_give_the_same_bits(libqknorm, monkeypatch):
    w = W.Workload("queue_ab", tokens=7001, dq=5120, dk=5120, shards=(4,), seed=71)
    inp = W.make_inputs(w)
    d = shards_on_device(inp, 4)
    got = {}
    for mode in ("1", "0"):
        monkeypatch.setenv("QKNORM_QUEUE", mode)
        oq, ok = binding.qknorm_fwd_sharded(d["q"], d["k"], d["gamma_q"], d["gamma_k"], w.eps)
        torch.cuda.synchronize()
        assert binding.last_variant() == "warp"
        got[mode] = (H.bits(W.unshard_columns([t.cpu() for t in oq])), H.bits(W.unshard_columns([t.cpu() for t in ok])))
    assert np.array_equal(got["1"][0], got["0"][0]) and np.array_equal(got["1"][1], got["0"][1])
    check(w, inp, oq, ok, "fixed schedule")


def test_more_streams_than_counters(libqknorm):
    """300 streams make one call each without any synchronisation in between, so many calls are in
    flight at once; the library has 256 counters per device, the streams beyond that keep the
    fixed schedule.  All calls work on the same inputs, so one oracle result checks them all."""
    w = W.Workload("queue_streams", tokens=2600, dq=4096, dk=1024, shards=(1,), seed=72)
    inp = W.make_inputs(w)
    q, k = inp["q"].cuda(), inp["k"].cuda()
    gq, gk = inp["gamma_q"].cuda(), inp["gamma_k"].cuda()
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream() for _ in range(300)]
    outs = []
    for st in streams:
        oq, ok = torch.empty_like(q), torch.empty_like(k)
        binding.qknorm_fwd(q, k, gq, gk, w.eps, oq, ok, stream=st)
        assert binding.last_variant() == "warp"
        outs.append((oq, ok))
    torch.cuda.synchronize()
    ref = H.oracle_unsharded(inp, w.eps, nthreads=NTHREADS)
    first_q, first_k = H.bits(outs[0][0]), H.bits(outs[0][1])
    H.compare_output(first_q, ref["q"]["y"], "stream 0 q")
    H.compare_output(first_k, ref["k"]["y"], "stream 0 k")
    for i, (oq, ok) in enumerate(outs[1:], 1):
        assert torch.equal(oq, outs[0][0]) and torch.equal(ok, outs[0][1]), f"stream {i} differs from stream 0"
    assert binding.device_error_word() == 0


def test_captured_prefill_call_replays_next_to_eager_calls(libqknorm):
    """A launch captured into a graph may later run next to anything, so it takes no counter.
    Replays of the graph on one stream and eager calls on the capture stream run at the same time."""
    w = W.Workload("queue_graph", tokens=4500, dq=5120, dk=1024, shards=(8,), seed=73)
    inp = W.make_inputs(w)
    d = shards_on_device(inp, 8)
    g_oq = [torch.empty_like(t) for t in d["q"]]
    g_ok = [torch.empty_like(t) for t in d["k"]]
    e_oq = [torch.empty_like(t) for t in d["q"]]
    e_ok = [torch.empty_like(t) for t in d["k"]]
    cap, other = torch.cuda.Stream(), torch.cuda.Stream()
    graph_call = binding.prepared(binding.qknorm_fwd_sharded, d["q"], d["k"], d["gamma_q"], d["gamma_k"], w.eps, g_oq, g_ok)
    eager_call = binding.prepared(binding.qknorm_fwd_sharded, d["q"], d["k"], d["gamma_q"], d["gamma_k"], w.eps, e_oq, e_ok)
    with torch.cuda.stream(cap):
        graph_call()                       # warm-up on the capture stream (takes that stream's counter)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=cap):
        graph_call()
    torch.cuda.synchronize()
    for t in g_oq + g_ok:
        t.zero_()
    torch.cuda.synchronize()
    for _ in range(20):
        with torch.cuda.stream(other):
            g.replay()
        with torch.cuda.stream(cap):
            eager_call()
    torch.cuda.synchronize()
    check(w, inp, g_oq, g_ok, "graph replay")
    check(w, inp, e_oq, e_ok, "eager next to the replay")
    assert binding.device_error_word() == 0


def test_per_thread_default_stream_handle_takes_no_counter(libqknorm):
    """cudaStreamPerThread is ONE handle value that names a different stream in every host thread, so a
    counter keyed by it could be shared by kernels that run at the same time: such launches keep the
    fixed schedule.  The result is the same as on an ordinary stream."""
    CUDA_STREAM_PER_THREAD = 2
    w = W.Workload("queue_ptds", tokens=3100, dq=5120, dk=1024, shards=(1,), seed=74)
    inp = W.make_inputs(w)
    q, k = inp["q"].cuda(), inp["k"].cuda()
    gq, gk = inp["gamma_q"].cuda(), inp["gamma_k"].cuda()
    torch.cuda.synchronize()
    a_q, a_k = binding.qknorm_fwd(q, k, gq, gk, w.eps)
    b_q, b_k = torch.empty_like(q), torch.empty_like(k)
    binding.qknorm_fwd(q, k, gq, gk, w.eps, b_q, b_k, stream=CUDA_STREAM_PER_THREAD)
    assert binding.last_variant() == "warp"
    torch.cuda.synchronize()
    assert torch.equal(a_q, b_q) and torch.equal(a_k, b_k)
    ref = H.oracle_unsharded(inp, w.eps, nthreads=NTHREADS)
    H.compare_output(H.bits(b_q), ref["q"]["y"], "per-thread default stream q")
    H.compare_output(H.bits(b_k), ref["k"]["y"], "per-thread default stream k")
