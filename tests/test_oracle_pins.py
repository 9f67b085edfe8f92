"""Pins for the oracle's RMSNorm (CPU only): what Eq. 1 and arithmetic fix,
independently of the oracle's own code."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2608_09160_b200 import workloads as W
from tests.util import bf16_bits_to_f64, ordinal_distance

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "eq1_hand_rows.txt")


def bits_of(vals) -> np.ndarray:
    """bf16 bit patterns of values that are exactly representable in bf16."""
    t = torch.tensor(np.asarray(vals, dtype=np.float64), dtype=torch.float64)
    b = t.to(torch.bfloat16)
    assert torch.equal(b.to(torch.float64), t), "test value is not bf16-exact"
    return W.bf16_bits(b).copy()


def rand_bits(rng, shape, sigma=1.0):
    f = torch.from_numpy((rng.standard_normal(shape) * sigma).astype(np.float32))
    return W.bf16_bits(f.to(torch.bfloat16)).copy()


def rand_gamma(rng, n):
    f = torch.from_numpy(rng.uniform(0.5, 1.5, n).astype(np.float32))
    return W.bf16_bits(f.to(torch.bfloat16)).copy()


# ---- hand-computed rows (tests/golden) ----------------------------------------

def _golden_cases():
    cases = []
    with open(GOLDEN) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            h, eps, xs, gs, ys = [p.strip() for p in line.split("|")]
            cases.append((int(h), float(eps), [float(v) for v in xs.split()],
                          [float(v) for v in gs.split()], [int(v, 16) for v in ys.split()]))
    return cases


@pytest.mark.parametrize("case", _golden_cases())
def test_hand_computed_rows(case):
    h, eps, xs, gs, want = case
    assert len(xs) == h and len(gs) == h and len(want) == h
    res = oracle.rmsnorm(bits_of(xs)[None, :], bits_of(gs), eps)
    assert [int(v) for v in res["y"][0]] == want


def test_rows_and_columns_are_not_transposed():
    # two different hand rows in one call: row 0 = [3,4,0,0], row 1 = [1,-1,1,-1]
    x = bits_of([[3, 4, 0, 0], [1, -1, 1, -1]])
    g = bits_of([1, 2, 0.5, -1])
    y = oracle.rmsnorm(x, g, 0.0)["y"]
    assert [int(v) for v in y[0]] == [0x3F9A, 0x404D, 0x0000, 0x8000]
    assert [int(v) for v in y[1]] == [0x3F80, 0xC000, 0x3F00, 0x3F80]   # gamma * x
    assert np.allclose(oracle.rmsnorm(x, g, 0.0)["acc"], [25.0, 4.0], rtol=0, atol=0)


# ---- P1: constant row, closed form ---------------------------------------------

@pytest.mark.parametrize("c", [1.0, -3.0, 0.5, 2.0 ** -10, 96.0])
@pytest.mark.parametrize("g", [1.0, -3.0, 0.5, 1.25])
@pytest.mark.parametrize("H", [1, 8, 1000, 5120])
def test_constant_row_closed_form(c, g, H):
    eps32 = np.float32(1e-6)
    x = np.full((1, H), bits_of([c])[0], dtype=np.uint16)
    gam = np.full((H,), bits_of([g])[0], dtype=np.uint16)
    res = oracle.rmsnorm(x, gam, float(eps32), want_y64=True)
    want = g * c / math.sqrt(c * c + float(eps32))
    assert np.allclose(res["y64"], want, rtol=1e-14, atol=0)
    assert np.all(res["y"] == oracle.f64_to_bf16(want))
    assert math.isclose(res["rstd"][0], 1.0 / math.sqrt(c * c + float(eps32)), rel_tol=1e-15)
    assert res["acc"][0] == pytest.approx(H * c * c, rel=1e-15)


# ---- P2: scale invariance --------------------------------------------------------

def test_scale_invariance_is_bitwise_without_eps():
    rng = np.random.default_rng(1)
    x = rand_bits(rng, (6, 640))
    g = rand_gamma(rng, 640)
    base = oracle.rmsnorm(x, g, 0.0)["y"]
    for k in (-20, -3, 1, 7, 30):
        xs = bits_of(bf16_bits_to_f64(x) * 2.0 ** k)       # power-of-two scaling is exact in bf16
        assert np.array_equal(oracle.rmsnorm(xs, g, 0.0)["y"], base), k


def test_eps_sensitivity_matches_first_order_formula():
    # d/d(eps) of 1/sqrt(m+eps) -> relative change of y is -eps/(2m) to first order
    rng = np.random.default_rng(2)
    x = rand_bits(rng, (4, 512))
    g = rand_gamma(rng, 512)
    eps = float(np.float32(1e-3))
    a = oracle.rmsnorm(x, g, 0.0, want_y64=True)
    b = oracle.rmsnorm(x, g, eps, want_y64=True)
    m = a["acc"] / 512
    rel = (b["y64"] - a["y64"]) / a["y64"]
    assert np.allclose(rel, (-eps / (2 * m))[:, None], rtol=5e-3)
    assert np.all(np.abs(b["y64"]) < np.abs(a["y64"]))


# ---- P3: sharded == unsharded -----------------------------------------------------

@pytest.mark.parametrize("S", [1, 2, 4, 8, 5])
def test_sharded_equals_unsharded(S):
    rng = np.random.default_rng(3)
    T, H = 9, 640
    x = rand_bits(rng, (T, H), sigma=2.0)
    g = rand_gamma(rng, H)
    full = oracle.rmsnorm(x, g, 1e-6)
    w = H // S
    xs = [np.ascontiguousarray(x[:, s * w:(s + 1) * w]) for s in range(S)]
    gs = [np.ascontiguousarray(g[s * w:(s + 1) * w]) for s in range(S)]
    sh = oracle.rmsnorm_sharded(xs, gs, 1e-6)
    assert np.array_equal(np.concatenate(sh["y"], axis=1), full["y"])
    assert np.array_equal(sh["rstd"], full["rstd"])
    assert np.allclose(sh["partials"].sum(axis=0), full["acc"], rtol=1e-14, atol=0)
    # each partial is that slice's own sum of squares (exact rational arithmetic)
    for s in range(S):
        for t in (0, T - 1):
            exact = sum(Fraction(float(v)) ** 2 for v in bf16_bits_to_f64(xs[s][t]))
            assert abs(Fraction(float(sh["partials"][s, t])) - exact) <= exact * Fraction(1, 10 ** 14)


def test_sharded_divisor_is_full_width_not_shard_width():
    # two slices of a constant row: the statistic must be that of the gathered row
    H, S = 256, 4
    xs = [np.full((1, H // S), bits_of([2.0])[0], dtype=np.uint16) for _ in range(S)]
    gs = [np.full((H // S,), bits_of([1.0])[0], dtype=np.uint16) for _ in range(S)]
    sh = oracle.rmsnorm_sharded(xs, gs, 0.0)
    assert sh["rstd"][0] == 0.5
    assert np.all(np.concatenate(sh["y"], axis=1) == 0x3F80)
    assert np.all(sh["partials"] == 4.0 * (H // S))


def test_shard_order_is_rank_order():
    # a different constant in every slice, different gamma per slice
    S, w = 4, 8
    cs = [1.0, 2.0, 4.0, 8.0]
    gvals = [1.0, 0.5, 0.25, 0.125]
    xs = [np.full((1, w), bits_of([c])[0], dtype=np.uint16) for c in cs]
    gs = [np.full((w,), bits_of([g])[0], dtype=np.uint16) for g in gvals]
    sh = oracle.rmsnorm_sharded(xs, gs, 0.0)
    ms = sum(c * c for c in cs) / S
    for s in range(S):
        want = oracle.f64_to_bf16(cs[s] * gvals[s] / math.sqrt(ms))
        assert np.all(sh["y"][s] == want)
    assert list(sh["partials"][:, 0]) == [w * c * c for c in cs]


# ---- P5 / P6 / P7 / P8 ---------------------------------------------------------------

def test_unit_mean_square_when_gamma_is_one():
    rng = np.random.default_rng(5)
    H = 1000
    x = rand_bits(rng, (5, H), sigma=3.0)
    g = np.full((H,), 0x3F80, dtype=np.uint16)
    res = oracle.rmsnorm(x, g, 0.0, want_y64=True)
    assert np.allclose((res["y64"] ** 2).sum(axis=1), H, rtol=1e-13)
    yq = bf16_bits_to_f64(res["y"])
    assert np.allclose((yq ** 2).sum(axis=1), H, rtol=2.0 ** -8)


@pytest.mark.parametrize("a", [1.0, -8.0, 2.0 ** -20, 2.0 ** 60])
def test_one_hot_row_and_bound(a):
    H, i = 4096, 77
    x = np.zeros((1, H), dtype=np.uint16)
    x[0, i] = bits_of([a])[0]
    rng = np.random.default_rng(6)
    g = rand_gamma(rng, H)
    eps = float(np.float32(1e-6))
    res = oracle.rmsnorm(x, g, eps, want_y64=True)
    gi = float(bf16_bits_to_f64(g[i]))
    want = gi * math.copysign(1.0, a) * math.sqrt(H) / math.sqrt(1.0 + eps * H / (a * a))
    assert math.isclose(res["y64"][0, i], want, rel_tol=1e-14)
    others = np.delete(res["y64"][0], i)
    assert np.all(others == 0.0)
    # |y_j| <= |gamma_j| sqrt(H) for any row
    xr = rand_bits(rng, (3, H), sigma=5.0)
    yr = oracle.rmsnorm(xr, g, eps, want_y64=True)["y64"]
    assert np.all(np.abs(yr) <= np.abs(bf16_bits_to_f64(g))[None, :] * math.sqrt(H))


def test_zero_row_and_signed_zeros():
    x = np.array([[0x0000, 0x8000, 0x0000, 0x8000]], dtype=np.uint16)
    g = bits_of([1.0, 1.0, -1.0, -1.0])
    res = oracle.rmsnorm(x, g, 1e-6)
    assert [int(v) for v in res["y"][0]] == [0x0000, 0x8000, 0x8000, 0x0000]
    assert math.isclose(res["rstd"][0], 1.0 / math.sqrt(float(np.float32(1e-6))), rel_tol=1e-15)
    # eps == 0 on a zero row: 0 * inf = NaN everywhere (documented behaviour)
    with np.errstate(all="ignore"):
        res0 = oracle.rmsnorm(x, g, 0.0)
    assert np.all((res0["y"] & 0x7F80) == 0x7F80) and np.all((res0["y"] & 0x7F) != 0)


def test_odd_symmetry_and_column_permutation():
    rng = np.random.default_rng(8)
    H = 384
    x = rand_bits(rng, (4, H))
    g = rand_gamma(rng, H)
    y = oracle.rmsnorm(x, g, 1e-6)["y"]
    yneg = oracle.rmsnorm(x ^ 0x8000, g, 1e-6)["y"]
    assert np.array_equal(yneg, y ^ 0x8000)
    p = rng.permutation(H)
    yp = oracle.rmsnorm(np.ascontiguousarray(x[:, p]), np.ascontiguousarray(g[p]), 1e-6)["y"]
    # fp64 sums in a different order may differ in the last bit of acc; outputs agree to <= 1 ordinal
    assert ordinal_distance(yp, y[:, p]).max() <= 1
    assert (ordinal_distance(yp, y[:, p]) != 0).mean() < 1e-3


def test_nan_and_inf_propagate():
    x = bits_of([[1.0, 2.0, 3.0, 4.0], [1.0, 2.0, 3.0, 4.0]])
    x[0, 1] = 0x7FC0          # NaN poisons its whole row and only its row
    x[1, 2] = 0x7F80          # +inf: inf * (1/inf) -> NaN at that position, zeros elsewhere
    g = bits_of([1.0, 1.0, 1.0, 1.0])
    with np.errstate(all="ignore"):
        y = oracle.rmsnorm(x, g, 1e-6)["y"]
    isnan = ((y & 0x7F80) == 0x7F80) & ((y & 0x7F) != 0)
    assert isnan[0].all()
    assert list(isnan[1]) == [False, False, True, False]
    assert [int(v) for v in y[1][[0, 1, 3]]] == [0, 0, 0]


# ---- P9: torch's fp64 rms_norm is the same definition --------------------------------

@pytest.mark.parametrize("shape", [(7, 1000), (3, 8192), (33, 136)])
def test_against_torch_rms_norm_fp64(shape):
    rng = np.random.default_rng(9)
    T, H = shape
    x = rand_bits(rng, (T, H), sigma=2.0)
    g = rand_gamma(rng, H)
    eps = float(np.float32(1e-6))
    res = oracle.rmsnorm(x, g, eps, want_y64=True)
    xt = W.from_bf16_bits(x).to(torch.float64)
    gt = W.from_bf16_bits(g).to(torch.float64)
    ref = torch.nn.functional.rms_norm(xt, (H,), gt, eps).numpy()
    assert np.allclose(res["y64"], ref, rtol=1e-12, atol=0)
    ref_bits = oracle.f64_to_bf16(ref)
    assert ordinal_distance(res["y"], ref_bits).max() <= 1
    assert (res["y"] != ref_bits).mean() < 1e-4
    assert np.allclose(res["rstd"], torch.rsqrt(xt.pow(2).mean(-1) + eps).numpy(), rtol=1e-14)


# ---- P10: the fp64 accumulator is the true sum -------------------------------------------

def test_accumulator_is_exact_on_workload_like_rows():
    rng = np.random.default_rng(10)
    for H, sigma in ((4096, 1.0), (8192, 2.0), (5120, 1.0)):
        x = rand_bits(rng, (2, H), sigma=sigma)
        g = rand_gamma(rng, H)
        acc = oracle.rmsnorm(x, g, 1e-6)["acc"]
        for t in range(2):
            exact = sum(Fraction(float(v)) ** 2 for v in bf16_bits_to_f64(x[t]))
            err = abs(Fraction(float(acc[t])) - exact) / exact
            assert err < Fraction(1, 10 ** 13)


# ---- in-place and threading do not change the answer ---------------------------------------

def test_in_place_and_threads_give_identical_bits():
    rng = np.random.default_rng(11)
    x = rand_bits(rng, (37, 1280))
    g = rand_gamma(rng, 1280)
    ref = oracle.rmsnorm(x, g, 1e-6)
    buf = x.copy()
    oracle.rmsnorm(buf, g, 1e-6, out=buf)
    assert np.array_equal(buf, ref["y"])
    thr = oracle.rmsnorm(x, g, 1e-6, nthreads=4)
    assert np.array_equal(thr["y"], ref["y"]) and np.array_equal(thr["rstd"], ref["rstd"])


# ---- the input generator -----------------------------------------------------------------

def test_workload_generator_is_seeded_and_shaped():
    w = W.scaled(W.WORKLOADS["C3"], 64)
    a, b = W.make_inputs(w), W.make_inputs(w)
    for key in ("q", "k", "gamma_q", "gamma_k"):
        assert torch.equal(a[key], b[key])
    assert a["q"].shape == (64, 5120) and a["k"].shape == (64, 5120)
    g = a["gamma_q"].float()
    assert 0.5 <= float(g.min()) and float(g.max()) <= 1.5
    col_rms = a["q"].float().pow(2).mean(0).sqrt()
    assert int((col_rms > 8).sum()) == 51          # 1 % of 5120 channels scaled x20
    parts = W.shard_columns(a["q"], 4)
    assert all(p.shape == (64, 1280) and p.is_contiguous() for p in parts)
    assert torch.equal(W.unshard_columns(parts), a["q"])
    assert W.WORKLOADS["C5"].algorithmic_bytes == 2415937536
    assert W.WORKLOADS["C1"].algorithmic_bytes == 278528
