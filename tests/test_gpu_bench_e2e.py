"""The benchmark's end-to-end leg (pinned host buffers in, chunked copies and calls, pinned host
buffers out) produces the right bits: every chunk's output, reassembled, against the oracle."""
import numpy as np
import pytest
import torch

import bench
from paper_2608_09160_b200 import workloads as W
from tests import gpu_harness as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("in_place", [True, False])
def test_chunked_host_to_host_step(libqknorm, in_place):
    S, chunks = 4, 5
    w = W.Workload("e2e", tokens=8192 + 37, dq=1024, dk=256, shards=(S,), seed=66, in_place=in_place)
    case = bench.DeviceCase(w, S, host=True)
    assert case.prepare_e2e(chunks) == chunks
    case.e2e_step()
    case.e2e_step()                       # a second step on the same staging buffers
    torch.cuda.synchronize()
    inp = W.make_inputs(bench.rank_workload(w, 0))
    ref = H.oracle_unsharded(inp, w.eps, nthreads=8)
    got = {"q": [], "k": []}
    for c in case.chunks:
        rows = c["h_out"].numel() // (w.dq + w.dk)
        off = 0
        for name, d in (("q", w.dq), ("k", w.dk)):
            slices = []
            for _ in range(S):
                n = rows * (d // S)
                slices.append(c["h_out"][off:off + n].view(rows, d // S))
                off += n
            got[name].append(torch.cat(slices, dim=1))
    for name in ("q", "k"):
        H.compare_output(W.bf16_bits(torch.cat(got[name], dim=0)), ref[name]["y"], f"e2e {name}")
    h2d, d2h = case.e2e_bytes()
    assert h2d == d2h == w.tokens * (w.dq + w.dk) * 2
