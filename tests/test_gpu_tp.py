"""The tensor-parallel path (Algorithm 1 with its scalar exchange) on ONE GPU: all N ranks'
buffers on the device, one cooperative launch serving every rank, the pushes and polls going
through the ranks' inboxes exactly as they would between GPUs.  Compared with the fp64 oracle
of the sharded method, element by element."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_09160_b200 import binding, tp
from paper_2608_09160_b200 import workloads as W
from tests import gpu_harness as H
from tests.util import e4m3_ordinal_distance

pytestmark = pytest.mark.gpu

# (name, tokens, dq, dk, ranks)
SHAPES = [
    ("gqa8", 700, 5120, 1024, 8),
    ("odd4", 1025, 640, 128, 4),
    ("wide2", 300, 8192, 1024, 2),
    ("n16", 257, 4096, 2048, 16),
    ("n3", 611, 1536, 384, 3),
    ("konly", 650, 0, 2048, 4),
    ("qonly", 90, 2048, 0, 2),
    ("n1", 64, 1024, 256, 1),
    ("t1", 1, 5120, 1024, 8),
]


def device_slices(inp, N):
    dev = {}
    for name in ("q", "k", "gamma_q", "gamma_k"):
        x = inp[name]
        dev[name] = [t.cuda() for t in W.shard_columns(x, N)] if x.shape[-1] > 0 else None
    return dev


def oracle_sharded(inp, N, eps):
    out = {}
    for name in ("q", "k"):
        if inp[name].shape[1] == 0:
            out[name] = None
            continue
        xs = [W.bf16_bits(t) for t in W.shard_columns(inp[name], N)]
        gs = [W.bf16_bits(t) for t in W.shard_columns(inp["gamma_" + name], N)]
        out[name] = oracle.rmsnorm_sharded(xs, gs, eps, nthreads=8)
    return out


def check_group(bufs, ref, what):
    for name in ("q", "k"):
        if ref[name] is None:
            continue
        rstd0 = None
        for b in bufs:
            y = getattr(b, "out_" + name)
            H.compare_output(H.bits(y), ref[name]["y"][b.rank], f"{what} rank {b.rank} {name}")
            r = getattr(b, "rstd_" + name)
            if r is not None:
                H.compare_stat(r, ref[name]["rstd"], f"{what} rank {b.rank} rstd_{name}")
                rb = r.cpu().numpy().view(np.uint32)
                rstd0 = rb if rstd0 is None else rstd0
                assert np.array_equal(rb, rstd0), "ranks disagree on RMS^-1 bits"
            p = getattr(b, "partial_" + name)
            if p is not None:
                H.compare_stat(p, ref[name]["partials"][b.rank], f"{what} rank {b.rank} partial_{name}")


@pytest.mark.parametrize("name,T,dq,dk,N", SHAPES, ids=[s[0] for s in SHAPES])
def test_emulated_group_matches_oracle(libqknorm, name, T, dq, dk, N):
    w = W.Workload("tp_" + name, tokens=T, dq=dq, dk=dk, shards=(N,), seed=40 + N)
    inp = W.make_inputs(w)
    dev = device_slices(inp, N)
    grp = tp.EmulatedGroup(N, token_capacity=max(T, 8))
    bufs = grp.buffers(dev["q"], dev["k"], dev["gamma_q"], dev["gamma_k"], stats=True)
    n0 = binding.launch_count()
    grp.forward(bufs, w.eps)
    torch.cuda.synchronize()
    assert binding.launch_count() == n0 + 1 and binding.last_variant() == "tp"
    check_group(bufs, oracle_sharded(inp, N, w.eps), name)
    for b in grp.inboxes:
        assert tp.status(b)["status"] == tp.STATUS_OK


def test_consecutive_calls_reuse_the_inboxes_without_clearing(libqknorm):
    """Epochs 1..5 on the same inboxes, token counts going down and up again, fresh data each
    time: a stale slot of an earlier call must never be taken for the current one."""
    N, cap = 4, 900
    grp = tp.EmulatedGroup(N, token_capacity=cap)
    for call, T in enumerate((900, 600, 10, 900, 333)):
        w = W.Workload(f"tp_seq{call}", tokens=T, dq=2048, dk=512, shards=(N,), seed=70 + call)
        inp = W.make_inputs(w)
        dev = device_slices(inp, N)
        bufs = grp.buffers(dev["q"], dev["k"], dev["gamma_q"], dev["gamma_k"], stats=True)
        e = grp.forward(bufs, w.eps)
        assert e == call + 1
        torch.cuda.synchronize()
        check_group(bufs, oracle_sharded(inp, N, w.eps), f"call {call}")


def test_in_place_strided_and_bitwise_repeatable(libqknorm):
    """Every rank's slices are column blocks of one fused [T, (dq+dk)/N] buffer, normalised in place;
    two groups fed the same data give the same bits."""
    N, T, dq, dk = 8, 1200, 8192, 1024
    w = W.Workload("tp_fused", tokens=T, dq=dq, dk=dk, shards=(N,), seed=91, sigma=2.0)
    inp = W.make_inputs(w)
    ref = oracle_sharded(inp, N, w.eps)
    results = []
    for _ in range(2):
        qs, ks = W.shard_columns(inp["q"], N), W.shard_columns(inp["k"], N)
        fused = [torch.cat([a, b], dim=1).cuda() for a, b in zip(qs, ks)]
        wq = dq // N
        qv, kv = [f[:, :wq] for f in fused], [f[:, wq:] for f in fused]
        gq = [t.cuda() for t in W.shard_columns(inp["gamma_q"], N)]
        gk = [t.cuda() for t in W.shard_columns(inp["gamma_k"], N)]
        grp = tp.EmulatedGroup(N, token_capacity=T)
        bufs = grp.buffers(qv, kv, gq, gk, out_q=qv, out_k=kv)
        grp.forward(bufs, w.eps)
        torch.cuda.synchronize()
        check_group(bufs, ref, "fused in place")
        results.append([H.bits(f) for f in fused])
    for a, b in zip(*results):
        assert np.array_equal(a, b)


def test_fp8_activations(libqknorm):
    N, T = 4, 800
    w = W.Workload("tp_e4m3", tokens=T, dq=4096, dk=1024, shards=(N,), seed=93)
    inp = W.make_inputs_e4m3(w)
    qs = [t.cuda() for t in W.shard_columns(inp["q"], N)]
    ks = [t.cuda() for t in W.shard_columns(inp["k"], N)]
    gq = [t.cuda() for t in W.shard_columns(inp["gamma_q"], N)]
    gk = [t.cuda() for t in W.shard_columns(inp["gamma_k"], N)]
    grp = tp.EmulatedGroup(N, token_capacity=T)
    bufs = grp.buffers(qs, ks, gq, gk, stats=True)
    grp.forward(bufs, w.eps)
    torch.cuda.synchronize()
    assert binding.last_variant() == "tp"
    for name, xs, gs in (("q", qs, gq), ("k", ks, gk)):
        ref = oracle.rmsnorm_e4m3([W.e4m3_bits(t.cpu()) for t in xs], [W.bf16_bits(t.cpu()) for t in gs], w.eps)
        for b in bufs:
            got = W.e4m3_bits(getattr(b, "out_" + name).cpu())
            want = ref["y"][b.rank]
            d = e4m3_ordinal_distance(got, want)     # at most one code apart, and rarely
            assert d.max() <= 1, (name, b.rank, int(d.max()))
            assert (d == 1).mean() < 2e-3
            H.compare_stat(getattr(b, "rstd_" + name), ref["rstd"], f"e4m3 rstd_{name}")


def test_a_missing_peer_ends_the_wait_with_a_status_not_a_hang(libqknorm):
    """Only rank 0 of two is launched, so nobody fills its inbox: every poll runs into its (short)
    limit, the kernel records who was missing and ends, and the same inboxes serve a complete
    call afterwards."""
    N, T = 2, 64
    w = W.Workload("tp_missing", tokens=T, dq=1024, dk=256, shards=(N,), seed=95)
    inp = W.make_inputs(w)
    dev = device_slices(inp, N)
    grp = tp.EmulatedGroup(N, token_capacity=T)
    alone = grp.buffers(dev["q"], dev["k"], dev["gamma_q"], dev["gamma_k"], ranks=[0])
    e = grp.epochs.next()
    tp.qknorm_fwd_tp(alone, N, T, w.eps, e, wait_limit_us=20000)
    torch.cuda.synchronize()
    st = tp.status(grp.inboxes[0])
    assert st["status"] == tp.STATUS_PEER_TIMEOUT and st["missing_rank"] == 1 and 0 <= st["token"] < T
    assert tp.status(grp.inboxes[1])["status"] == tp.STATUS_OK
    tp.clear_status(grp.inboxes[0])
    bufs = grp.buffers(dev["q"], dev["k"], dev["gamma_q"], dev["gamma_k"], stats=True)
    grp.forward(bufs, w.eps)
    torch.cuda.synchronize()
    assert tp.status(grp.inboxes[0])["status"] == tp.STATUS_OK
    check_group(bufs, oracle_sharded(inp, N, w.eps), "after the timeout")
    assert binding.device_error_word() == 0


def test_argument_errors_launch_nothing(libqknorm):
    N, T = 2, 16
    w = W.Workload("tp_args", tokens=T, dq=512, dk=128, shards=(N,), seed=96)
    dev = device_slices(W.make_inputs(w), N)
    grp = tp.EmulatedGroup(N, token_capacity=T)
    bufs = grp.buffers(dev["q"], dev["k"], dev["gamma_q"], dev["gamma_k"])
    n0 = binding.launch_count()
    for kwargs, code in ((dict(epoch=0), binding.QKNORM_ERR_SHAPE), (dict(cap=8), binding.QKNORM_ERR_SHAPE),
                         (dict(eps=-1.0), binding.QKNORM_ERR_EPS)):
        with pytest.raises(binding.QKNormError) as ei:
            tp.qknorm_fwd_tp(bufs, N, kwargs.get("cap", T), kwargs.get("eps", w.eps), kwargs.get("epoch", 1))
        assert ei.value.status == code
    twice = [bufs[0], bufs[0]]
    with pytest.raises(binding.QKNormError) as ei:
        tp.qknorm_fwd_tp(twice, N, T, w.eps, 1)
    assert ei.value.status == binding.QKNORM_ERR_SHARDS
    bufs[1].out_q = bufs[0].out_q          # two ranks writing the same buffer
    with pytest.raises(binding.QKNormError) as ei:
        tp.qknorm_fwd_tp(bufs, N, T, w.eps, 1)
    assert ei.value.status == binding.QKNORM_ERR_ALIAS
    assert binding.launch_count() == n0


def _random_tp_cases(n, seed):
    rng = np.random.default_rng(seed)
    cases = []
    for i in range(n):
        N = int(rng.choice([1, 2, 3, 4, 5, 8, 12, 16]))
        wq = int(rng.integers(1, 160)) * 8 if rng.integers(0, 6) else 0
        wk = int(rng.integers(1, 96)) * 8 if (wq == 0 or rng.integers(0, 5)) else 0
        while (wq + wk) * N > 20000 or wq * N > 65536:      # keep the oracle quick
            wq, wk = wq // 2 // 8 * 8, max(8, wk // 2 // 8 * 8)
        T = int(rng.integers(1, 3000))
        cases.append((i, N, T, wq, wk))
    return cases


RANDOM_TP = _random_tp_cases(16, seed=31)


@pytest.mark.parametrize("i,N,T,wq,wk", RANDOM_TP, ids=[f"tp{c[0]}-N{c[1]}-T{c[2]}-{c[3]}+{c[4]}" for c in RANDOM_TP])
def test_random_tensor_parallel_shapes(libqknorm, i, N, T, wq, wk):
    w = W.Workload(f"tp_rand{i}", tokens=T, dq=wq * N, dk=wk * N, shards=(N,), seed=7000 + i, sigma=(0.5, 2.0)[i % 2])
    inp = W.make_inputs(w)
    dev = device_slices(inp, N)
    grp = tp.EmulatedGroup(N, token_capacity=T + i)
    for _ in range(2):                     # two calls in a row on the same inboxes
        bufs = grp.buffers(dev["q"], dev["k"], dev["gamma_q"], dev["gamma_k"], stats=True)
        grp.forward(bufs, w.eps)
        torch.cuda.synchronize()
        check_group(bufs, oracle_sharded(inp, N, w.eps), f"random tp {i}")
    assert all(tp.status(b)["status"] == tp.STATUS_OK for b in grp.inboxes)
