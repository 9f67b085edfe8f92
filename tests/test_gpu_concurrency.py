"""The library called from several host threads at once, each on its own stream.

The C ABI keeps per-thread diagnostics (last variant, launch count, last CUDA error) and
guards its per-device caches with mutexes; the kernels of different calls share nothing
but the device error word.  Two threads with different shapes, so that each one takes
another kernel variant, must therefore get the results they get alone."""
import threading

import pytest
import torch

from paper_2608_09160_b200 import binding
from paper_2608_09160_b200 import workloads as W
from tests import gpu_harness as H

pytestmark = pytest.mark.gpu

REPEATS = 200


def _worker(w, S, inp, barrier, out):
    try:
        torch.cuda.set_device(0)
        st = torch.cuda.Stream()
        with torch.cuda.stream(st):
            qs = [t.cuda() for t in W.shard_columns(inp["q"], S)]
            ks = [t.cuda() for t in W.shard_columns(inp["k"], S)]
            gq = [t.cuda() for t in W.shard_columns(inp["gamma_q"], S)]
            gk = [t.cuda() for t in W.shard_columns(inp["gamma_k"], S)]
            st.synchronize()
            call = binding.prepared(binding.qknorm_fwd_sharded, qs, ks, gq, gk, w.eps, stream=st)
            n0 = binding.launch_count()
            barrier.wait(timeout=60)
            for _ in range(REPEATS):
                call()
            st.synchronize()
            out["launches"] = binding.launch_count() - n0
            out["variant"] = binding.last_variant()
            oq, ok = call.outputs
            out["q"] = H.bits(W.unshard_columns([t.cpu() for t in oq]))
            out["k"] = H.bits(W.unshard_columns([t.cpu() for t in ok]))
    except BaseException as e:  # surfaced by the test below
        out["error"] = e


def test_two_threads_two_streams_two_variants(libqknorm):
    small = {w.name: w for w in W.small_parity_shapes()}
    jobs = [(small["s_prefill_gqa"], 8, "warp"), (small["s_149"], 1, "rows")]
    inputs = [W.make_inputs(w) for w, _, _ in jobs]
    barrier = threading.Barrier(len(jobs))
    outs = [dict() for _ in jobs]
    threads = [threading.Thread(target=_worker, args=(w, S, inp, barrier, o))
               for (w, S, _), inp, o in zip(jobs, inputs, outs)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=120)
        assert not t.is_alive()
    for (w, S, variant), inp, o in zip(jobs, inputs, outs):
        assert "error" not in o, repr(o.get("error"))
        assert o["launches"] == REPEATS          # the count is per thread
        assert o["variant"] == variant           # and so is the variant name
        ref = H.oracle_unsharded(inp, w.eps)
        H.compare_output(o["q"], ref["q"]["y"], f"threaded {w.name} q")
        H.compare_output(o["k"], ref["k"]["y"], f"threaded {w.name} k")
    assert binding.device_error_word() == 0
