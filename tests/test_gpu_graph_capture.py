"""Calls of the library captured into a CUDA graph and replayed: the calls allocate nothing and
synchronise nothing, so a capture holds exactly the kernel launch, and every replay recomputes
the outputs from whatever the input buffers hold at that moment."""
import numpy as np
import pytest
import torch

from paper_2608_09160_b200 import binding
from paper_2608_09160_b200 import workloads as W
from tests import gpu_harness as H

pytestmark = pytest.mark.gpu

CASES = [("decode", 8, 4096, 4096, 1, "rows"), ("decode-sharded", 64, 4096, 4096, 4, "rows"),
         ("prefill-sharded", 2100, 5120, 1024, 8, "warp")]


@pytest.mark.parametrize("name,T,dq,dk,S,variant", CASES, ids=[c[0] for c in CASES])
def test_capture_and_replay_with_new_inputs(libqknorm, name, T, dq, dk, S, variant):
    w1 = W.Workload("graph_a", tokens=T, dq=dq, dk=dk, shards=(S,), seed=21)
    w2 = W.Workload("graph_b", tokens=T, dq=dq, dk=dk, shards=(S,), seed=22, sigma=3.0)
    a, b = W.make_inputs(w1), W.make_inputs(w2)
    qs = [t.cuda() for t in W.shard_columns(a["q"], S)]
    ks = [t.cuda() for t in W.shard_columns(a["k"], S)]
    gq = [t.cuda() for t in W.shard_columns(a["gamma_q"], S)]
    gk = [t.cuda() for t in W.shard_columns(a["gamma_k"], S)]
    call = binding.prepared(binding.qknorm_fwd_sharded, qs, ks, gq, gk, w1.eps)
    oq, ok = call.outputs
    call()                                  # every one-time set-up (attributes, caches) happens here
    torch.cuda.synchronize()
    assert binding.last_variant() == variant
    st = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(st):
        with torch.cuda.graph(graph, stream=st):
            call(st)
    for inp, w in ((a, w1), (b, w2), (a, w1)):
        for dst, src in zip(qs + ks + gq + gk,
                            W.shard_columns(inp["q"], S) + W.shard_columns(inp["k"], S)
                            + W.shard_columns(inp["gamma_q"], S) + W.shard_columns(inp["gamma_k"], S)):
            dst.copy_(src)
        for o in oq + ok:
            o.zero_()
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        ref = H.oracle_unsharded(inp, w.eps, nthreads=8)
        H.compare_output(H.bits(W.unshard_columns([t.cpu() for t in oq])), ref["q"]["y"], f"{name} replay q")
        H.compare_output(H.bits(W.unshard_columns([t.cpu() for t in ok])), ref["k"]["y"], f"{name} replay k")
    assert binding.device_error_word() == 0


@pytest.mark.parametrize("tokens,dq,dk,variant", [(48, 4096, 1024, "rows"), (4200, 5120, 1024, "warp"),
                                                  (9000, 1024, 128, "warp")])
def test_stream_order_is_kept_when_launches_overlap(libqknorm, tokens, dq, dk, variant):
    """Calls may begin their launch while the previous kernel of the stream still runs (decode-size
    rows kernel and the prefill kernel alike, the latter also with several tokens per warp).
    A chain of dependent work without any synchronisation in between -- another kernel rewrites the
    input, the call normalises it in place, the next call normalises that result again -- must still
    see every predecessor's writes."""
    w = W.Workload("chain", tokens=tokens, dq=dq, dk=dk, shards=(1,), seed=55, sigma=3.0)
    inp = W.make_inputs(w)
    q, k = inp["q"].cuda(), inp["k"].cuda()
    gq, gk = inp["gamma_q"].cuda(), inp["gamma_k"].cuda()
    src_q, src_k = q.clone(), k.clone()
    call = binding.prepared(binding.qknorm_fwd, q, k, gq, gk, w.eps, q, k)
    call()                             # one pass on its own, synchronised: what the second pass starts from
    torch.cuda.synchronize()
    once = {"q": q.cpu(), "k": k.cpu(), "gamma_q": inp["gamma_q"], "gamma_k": inp["gamma_k"]}
    H.compare_output(H.bits(q), H.oracle_unsharded(inp, w.eps)["q"]["y"], "first pass q")
    for i in range(40 if tokens < 1000 else 12):
        q.copy_(src_q)                 # a foreign kernel writes the input ...
        k.copy_(src_k)
        if i % 2:
            q.neg_()                   # ... a second one changes it again ...
        call()                         # ... and two library calls in a row consume it, the second the first's output
        call()
    torch.cuda.synchronize()
    assert binding.last_variant() == variant
    ref2 = H.oracle_unsharded(once, w.eps, nthreads=8)
    want_q = ref2["q"]["y"] ^ np.uint16(0x8000)          # the last round (odd i) negated q first
    H.compare_output(H.bits(q), want_q, "chained q")
    H.compare_output(H.bits(k), ref2["k"]["y"], "chained k")
