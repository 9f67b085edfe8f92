"""GPU parity: libqknorm (through its C ABI) against the fp64 CPU oracle,
element by element, on the same seeded inputs."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2608_09160_b200 import binding
from paper_2608_09160_b200 import workloads as W
from tests import gpu_harness as H

pytestmark = pytest.mark.gpu

SMALL = W.small_parity_shapes()
NTHREADS = max(1, min(16, os.cpu_count() or 1))


def run_case(w: W.Workload, S: int, *, in_place: bool = False, skew: int = 0, stats: bool = True,
             force_general: bool = False, monkeypatch=None):
    """One call through the C ABI with guarded buffers; returns GPU bits and stats."""
    inp = W.make_inputs(w)
    T = w.tokens
    ar = H.arena_for(w, copies=3)
    dev = {}
    res = {}
    if force_general:
        monkeypatch.setenv("QKNORM_FORCE_VARIANT", "general")
    kw = dict(skew_elems=skew) if skew else {}
    has_q, has_k = w.dq > 0, w.dk > 0
    rq = torch.full((T,), float("nan"), device="cuda") if (stats and has_q) else None
    rk = torch.full((T,), float("nan"), device="cuda") if (stats and has_k) else None
    if S == 1:
        q = H.put(ar, inp["q"], **kw) if has_q else None
        k = H.put(ar, inp["k"], **kw) if has_k else None
        gq = H.put(ar, inp["gamma_q"], **kw) if has_q else None
        gk = H.put(ar, inp["gamma_k"], **kw) if has_k else None
        oq = q if in_place else (ar.take((T, w.dq), **kw) if has_q else None)
        ok = k if in_place else (ar.take((T, w.dk), **kw) if has_k else None)
        binding.qknorm_fwd(q, k, gq, gk, w.eps, oq, ok, rstd_q=rq, rstd_k=rk)
        torch.cuda.synchronize()
        res["q"] = H.bits(oq) if has_q else None
        res["k"] = H.bits(ok) if has_k else None
        res["pq"] = res["pk"] = None
    else:
        def side(x, g, present):
            if not present:
                return None, None, None
            xs = [H.put(ar, p, **kw) for p in W.shard_columns(x, S)]
            gs = [H.put(ar, p, **kw) for p in W.shard_columns(g, S)]
            outs = xs if in_place else [ar.take(tuple(p.shape), **kw) for p in xs]
            return xs, gs, outs
        qs, gqs, oqs = side(inp["q"], inp["gamma_q"], has_q)
        ks, gks, oks = side(inp["k"], inp["gamma_k"], has_k)
        pq = torch.full((S, T), float("nan"), device="cuda") if (stats and has_q) else None
        pk = torch.full((S, T), float("nan"), device="cuda") if (stats and has_k) else None
        binding.qknorm_fwd_sharded(qs, ks, gqs, gks, w.eps, oqs, oks, partials_q=pq, partials_k=pk,
                                   rstd_q=rq, rstd_k=rk)
        torch.cuda.synchronize()
        res["q"] = H.bits(W.unshard_columns([o.cpu() for o in oqs])) if has_q else None
        res["k"] = H.bits(W.unshard_columns([o.cpu() for o in oks])) if has_k else None
        res["pq"], res["pk"] = pq, pk
    res["rq"], res["rk"] = rq, rk
    res["variant"] = binding.last_variant()
    ar.check()
    res["inp"] = inp
    return res


def check_against_oracle(w, S, res):
    inp = res["inp"]
    ref = H.oracle_unsharded(inp, w.eps, nthreads=NTHREADS)
    report = {}
    for name, r, p in (("q", res["rq"], res["pq"]), ("k", res["rk"], res["pk"])):
        if ref[name] is None:
            continue
        report[name] = H.compare_output(res[name], ref[name]["y"], f"{w.name}/S={S}/{name}")
        if r is not None:
            H.compare_stat(r, ref[name]["rstd"], f"{w.name}/S={S}/rstd_{name}")
        if p is not None:
            xs = [W.bf16_bits(t) for t in W.shard_columns(inp[name], S)]
            gs = [W.bf16_bits(t) for t in W.shard_columns(inp["gamma_" + name], S)]
            sh = oracle.rmsnorm_sharded(xs, gs, w.eps, nthreads=NTHREADS)
            H.compare_stat(p, sh["partials"], f"{w.name}/S={S}/partials_{name}")
            # the oracle's own sharded form agrees with its unsharded form (same test inputs)
            assert np.array_equal(np.concatenate(sh["y"], axis=1), ref[name]["y"])
    return report


CASES = [(w, S) for w in SMALL for S in w.shards]


@pytest.mark.parametrize("w,S", CASES, ids=[f"{w.name}-S{S}" for w, S in CASES])
def test_small_shapes_match_oracle(libqknorm, w, S):
    res = run_case(w, S)
    check_against_oracle(w, S, res)


@pytest.mark.parametrize("w,S", CASES, ids=[f"{w.name}-S{S}" for w, S in CASES])
def test_small_shapes_in_place(libqknorm, w, S):
    res = run_case(w, S, in_place=True, stats=False)
    check_against_oracle(w, S, res)


@pytest.mark.parametrize("w,S", CASES[::2], ids=[f"{w.name}-S{S}" for w, S in CASES[::2]])
def test_general_kernel_matches_oracle(libqknorm, monkeypatch, w, S):
    res = run_case(w, S, force_general=True, monkeypatch=monkeypatch)
    assert res["variant"] == "general"
    check_against_oracle(w, S, res)


@pytest.mark.parametrize("skew", [1, 3, 4])
def test_unaligned_buffers_take_the_general_kernel(libqknorm, skew):
    w = W.Workload("skewed", tokens=19, dq=1024, dk=256, shards=(1, 4), seed=77)
    for S in w.shards:
        res = run_case(w, S, skew=skew)
        assert res["variant"] == "general"
        check_against_oracle(w, S, res)


@pytest.mark.parametrize("name,S,variant", [
    ("s_t1", 1, "rows"), ("s_149", 8, "rows"), ("s_gqa8", 8, "rows"), ("s_mid_gqa", 1, "rows"), ("s_mid_mha", 2, "rows"),          # few tokens: register-resident rows
    ("s_prefill_gqa", 8, "warp"), ("s_prefill_gqa", 1, "warp"), ("s_prefill_odd", 1, "warp"),
    ("s_2305", 1, "warp"), ("s_tile_gqa", 1, "warp"), ("s_tile_tiny", 1, "warp"), ("s_tile_konly", 1, "warp"),
    ("s_tile_qonly", 1, "warp"),                                               # short unsharded rows: several tokens side by side per warp
    ("s_prefill_s3", 3, "warp"), ("s_prefill_konly", 2, "warp"), ("s_2305", 4, "warp"),
    ("s_prefill_s16", 16, "warp"), ("s_prefill_s5", 5, "warp"),
    ("s_prefill_wide", 1, "ring"), ("s_prefill_wide", 4, "ring"),
    ("s_unaligned", 7, "general"), ("s_max", 1, "wide"),
])
def test_every_kernel_variant_is_exercised(libqknorm, name, S, variant):
    w = next(x for x in SMALL if x.name == name)
    res = run_case(w, S)
    assert res["variant"] == variant, (name, S, res["variant"])
    check_against_oracle(w, S, res)


@pytest.mark.parametrize("name", ["s_2305", "s_tile_gqa", "s_tile_tiny", "s_tile_konly", "s_tile_qonly", "s_prefill_odd"])
def test_three_stage_tiled_kernel_on_short_unsharded_rows(libqknorm, monkeypatch, name):
    """Short unsharded rows normally go to the warp-per-tile form of the prefill kernel; the three-stage
    tiled kernel (the tensor-parallel kernel with a single rank) still serves them when asked to."""
    monkeypatch.setenv("QKNORM_FORCE_VARIANT", "tile")
    w = next(x for x in SMALL if x.name == name)
    res = run_case(w, 1)
    assert res["variant"] == "tile"
    check_against_oracle(w, 1, res)
    res = run_case(w, 1, in_place=True, stats=False)
    check_against_oracle(w, 1, res)


def test_one_slice_through_the_sharded_entry_point_on_short_rows(libqknorm):
    """S = 1 through qknorm_fwd_sharded_ex on rows short enough for several tokens per warp: the
    slice's scalar is the row's sum of squares, one per token, whichever lane group served the token."""
    w = next(x for x in SMALL if x.name == "s_tile_gqa")
    inp = W.make_inputs(w)
    T = w.tokens
    dev = {k: [v.cuda()] for k, v in inp.items()}
    pq = torch.full((1, T), float("nan"), device="cuda")
    pk = torch.full((1, T), float("nan"), device="cuda")
    rq = torch.full((T,), float("nan"), device="cuda")
    rk = torch.full((T,), float("nan"), device="cuda")
    oq, ok = binding.qknorm_fwd_sharded(dev["q"], dev["k"], dev["gamma_q"], dev["gamma_k"], w.eps,
                                        partials_q=pq, partials_k=pk, rstd_q=rq, rstd_k=rk)
    torch.cuda.synchronize()
    assert binding.last_variant() == "warp"
    for nm, out, p, r in (("q", oq, pq, rq), ("k", ok, pk, rk)):
        sh = oracle.rmsnorm_sharded([W.bf16_bits(inp[nm])], [W.bf16_bits(inp["gamma_" + nm])], w.eps, nthreads=NTHREADS)
        H.compare_output(H.bits(out[0]), sh["y"][0], f"one slice {nm}")
        H.compare_stat(p, sh["partials"], f"one slice partials {nm}")
        H.compare_stat(r, sh["rstd"], f"one slice rstd {nm}")


def test_results_are_bitwise_reproducible(libqknorm):
    w = next(x for x in SMALL if x.name == "s_gqa8")
    a = run_case(w, 8)
    b = run_case(w, 8)
    assert np.array_equal(a["q"], b["q"]) and np.array_equal(a["k"], b["k"])
    assert torch.equal(a["rq"], b["rq"]) and torch.equal(a["pq"], b["pq"])


@pytest.mark.parametrize("S", [1, 4])
def test_prefill_kernel_is_bitwise_reproducible_with_its_token_queue(libqknorm, S):
    """The C3 shape at a prefill size (the warp-per-token kernel at 40 chunk slots per lane).
    Which warp takes which token is decided at run time by the launch's token queue, but a
    token's arithmetic does not depend on the warp that does it: two runs give the same bits."""
    w = W.scaled(W.WORKLOADS["C3"], 4099)
    a = run_case(w, S)
    assert binding.last_variant() == "warp"
    b = run_case(w, S)
    assert np.array_equal(a["q"], b["q"]) and np.array_equal(a["k"], b["k"])
    assert torch.equal(a["rq"], b["rq"]) and torch.equal(a["rk"], b["rk"])
    check_against_oracle(w, S, a)


def test_sharded_and_unsharded_agree_within_tolerance(libqknorm):
    w = W.scaled(W.WORKLOADS["C2"], 64)
    a = run_case(w, 1)
    b = run_case(w, 4)
    for name in ("q", "k"):
        from tests.util import ordinal_distance
        assert ordinal_distance(a[name], b[name]).max() <= 2   # each within 1 of the same oracle value
    check_against_oracle(w, 1, a)
    check_against_oracle(w, 4, b)


def test_closed_form_constant_rows_on_gpu(libqknorm):
    # y = gamma * c / sqrt(c^2 + eps) for a constant row: exact expectation, no oracle involved
    T, d = 5, 2048
    for c, g in ((1.0, 1.0), (-3.0, 0.5), (96.0, 1.25), (2.0 ** -10, -3.0)):
        q = torch.full((T, d), c, dtype=torch.bfloat16, device="cuda")
        gam = torch.full((d,), g, dtype=torch.bfloat16, device="cuda")
        oq, _ = binding.qknorm_fwd(q, None, gam, None, 1e-6)
        want = oracle.f64_to_bf16(g * c / np.sqrt(c * c + float(np.float32(1e-6))))
        got = H.bits(oq)
        from tests.util import ordinal_distance
        assert ordinal_distance(got, np.full_like(got, want)).max() <= 1


def test_zero_rows_nan_rows_and_eps_zero(libqknorm):
    w = W.Workload("special", tokens=6, dq=1024, dk=128, shards=(1, 4), seed=5)
    inp = W.make_inputs(w)
    inp["q"][1].zero_()                       # zero row: finite, signed zeros out
    inp["q"][2, 17] = float("nan")            # NaN poisons only its row
    inp["k"][3, 5] = float("inf")
    for S in w.shards:
        for eps in (1e-6, 0.0):
            dq = [t.cuda() for t in W.shard_columns(inp["q"], S)]
            dk = [t.cuda() for t in W.shard_columns(inp["k"], S)]
            gq = [t.cuda() for t in W.shard_columns(inp["gamma_q"], S)]
            gk = [t.cuda() for t in W.shard_columns(inp["gamma_k"], S)]
            oq, ok = binding.qknorm_fwd_sharded(dq, dk, gq, gk, eps)
            with np.errstate(all="ignore"):
                ref = H.oracle_unsharded(inp, eps)
            H.compare_output(H.bits(W.unshard_columns([o.cpu() for o in oq])), ref["q"]["y"], f"special q S={S} eps={eps}")
            H.compare_output(H.bits(W.unshard_columns([o.cpu() for o in ok])), ref["k"]["y"], f"special k S={S} eps={eps}")


def test_non_default_stream_and_empty_call(libqknorm):
    w = next(x for x in SMALL if x.name == "s_149")
    inp = W.make_inputs(w)
    q, k = inp["q"].cuda(), inp["k"].cuda()
    gq, gk = inp["gamma_q"].cuda(), inp["gamma_k"].cuda()
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(st):
        oq, ok = binding.qknorm_fwd(q, k, gq, gk, w.eps, stream=st)
    st.synchronize()
    ref = H.oracle_unsharded(inp, w.eps)
    H.compare_output(H.bits(oq), ref["q"]["y"], "stream q")
    H.compare_output(H.bits(ok), ref["k"]["y"], "stream k")
    n0 = binding.launch_count()
    e = torch.empty((0, 128), dtype=torch.bfloat16, device="cuda")
    g = torch.ones((128,), dtype=torch.bfloat16, device="cuda")
    binding.qknorm_fwd(e, e.clone(), g, g.clone(), 1e-6)
    assert binding.launch_count() == n0


def test_alias_is_rejected_on_real_buffers(libqknorm):
    buf = torch.zeros((3 * 64 * 128,), dtype=torch.bfloat16, device="cuda")
    q = buf[: 64 * 128].view(64, 128)
    out_overlapping = buf[128: 128 + 64 * 128].view(64, 128)
    g = torch.ones((128,), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.QKNormError) as ei:
        binding.qknorm_fwd(q, None, g, None, 1e-6, out_overlapping, None)
    assert ei.value.status == binding.QKNORM_ERR_ALIAS


def test_no_bounded_wait_ever_ran_out(libqknorm):
    """Every in-kernel mbarrier wait is bounded and reports through a device word; after all
    the TMA-fed launches this process made so far the word must still be clear."""
    w = next(x for x in SMALL if x.name == "s_prefill_gqa")
    run_case(w, 8)
    assert binding.device_error_word() == 0


def test_prepared_call_repeats_the_same_c_call(libqknorm):
    """binding.prepared marshals once; the object makes the identical call again and again."""
    w = next(x for x in SMALL if x.name == "s_prefill_gqa")
    inp = W.make_inputs(w)
    S = 8
    qs = [t.cuda() for t in W.shard_columns(inp["q"], S)]
    ks = [t.cuda() for t in W.shard_columns(inp["k"], S)]
    gq = [t.cuda() for t in W.shard_columns(inp["gamma_q"], S)]
    gk = [t.cuda() for t in W.shard_columns(inp["gamma_k"], S)]
    n0 = binding.launch_count()
    call = binding.prepared(binding.qknorm_fwd_sharded, qs, ks, gq, gk, w.eps)
    assert binding.launch_count() == n0                 # preparing launches nothing
    oq, ok = call.outputs
    call()
    call()
    torch.cuda.synchronize()
    assert binding.launch_count() == n0 + 2
    ref = H.oracle_unsharded(inp, w.eps)
    H.compare_output(H.bits(W.unshard_columns([t.cpu() for t in oq])), ref["q"]["y"], "prepared q")
    H.compare_output(H.bits(W.unshard_columns([t.cpu() for t in ok])), ref["k"]["y"], "prepared k")


@pytest.mark.parametrize("T", [6, 700])          # the decode kernel and the prefill kernel
def test_tiny_and_subnormal_inputs_are_not_flushed(libqknorm, T):
    """bf16 subnormals and values whose squares underflow in fp32: with eps > 0 the statistic is
    eps-dominated and the outputs (x * gamma / sqrt(eps)) must match the oracle; nothing may be
    flushed to zero on the way."""
    d = 1024
    gen = torch.Generator().manual_seed(3)
    x = torch.empty((T, d), dtype=torch.float32).normal_(0, 1, generator=gen)
    x[0] *= 1e-39          # bf16 subnormals
    x[1] *= 1e-30          # squares underflow in fp32
    x[2] *= 1e-19          # squares are fp32 subnormals
    x[3] *= 1e19           # large, still finite in fp32 after squaring and summing (1e38 * 1024 overflows? no: 1e38*... keep below)
    x[3] *= 1e-2
    xb = x.to(torch.bfloat16)
    g = torch.empty((d,), dtype=torch.float32).uniform_(0.5, 1.5, generator=gen).to(torch.bfloat16)
    oq, _ = binding.qknorm_fwd(xb.cuda(), None, g.cuda(), None, 1e-6)
    with np.errstate(all="ignore"):
        ref = oracle.rmsnorm(W.bf16_bits(xb), W.bf16_bits(g), 1e-6)["y"]
    got = H.bits(oq)
    H.compare_output(got, ref, f"tiny inputs T={T}")
    assert (got[0] & 0x7FFF).any(), "subnormal inputs were flushed to zero"


@pytest.mark.parametrize("T,S,variant", [(40, 1, "rows"), (2100, 4, "warp")])   # variant of the second (K) launch
def test_rows_too_wide_for_one_cta_take_one_launch_per_tensor(libqknorm, T, S, variant):
    """Q and K together beyond 32768 elements do not fit one CTA's registers; each fits alone, and the
    two statistics are independent, so the call is served by two launches of the vectorised kernels
    instead of the slow general one."""
    w = W.Workload("very_wide", tokens=T, dq=32768, dk=8192, shards=(S,), seed=321, sigma=0.5)
    n0 = binding.launch_count()
    res = run_case(w, S, in_place=True)
    assert binding.launch_count() == n0 + 2
    assert res["variant"] == variant
    check_against_oracle(w, S, res)


def test_wide_gqa_rows_in_eight_slices_take_one_launch_per_tensor(libqknorm):
    """Rows too wide for the warp kernel with K much narrower than Q and 8 slices: Q goes to the ring
    kernel and K to the warp kernel, two launches, same results (statistics, partials included)."""
    w = W.Workload("wide_gqa", tokens=2100, dq=16384, dk=2048, shards=(8,), seed=322)
    n0 = binding.launch_count()
    res = run_case(w, 8)
    assert binding.launch_count() == n0 + 2
    assert res["variant"] == "warp"          # of the second (K) launch
    check_against_oracle(w, 8, res)


@pytest.mark.parametrize("T,dq,dk,S,in_place", [(300, 49152, 0, 4, True), (700, 65536, 40960, 1, False), (33, 0, 65536, 16, True)])
def test_tensors_beyond_one_cta_take_the_vectorised_two_pass_kernel(libqknorm, T, dq, dk, S, in_place):
    w = W.Workload("wide", tokens=T, dq=dq, dk=dk, shards=(S,), seed=323, sigma=2.0)
    res = run_case(w, S, in_place=in_place)
    assert res["variant"] == "wide"
    check_against_oracle(w, S, res)
