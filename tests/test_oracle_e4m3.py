"""Pins for the oracle's FP8-E4M3 form (CPU only): the codec against the format's
definition and torch's float8_e4m3fn, the norm against closed forms and the bf16 oracle."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2608_09160_b200 import workloads as W
from tests.util import bf16_bits_to_f64, e4m3_ordinal_distance

ALL = np.arange(256, dtype=np.uint8)


def bf16_bits_of(vals):
    t = torch.tensor(np.asarray(vals, dtype=np.float64)).to(torch.bfloat16)
    return W.bf16_bits(t).copy()


def test_known_values():
    known = {0x00: 0.0, 0x80: -0.0, 0x38: 1.0, 0x40: 2.0, 0xC4: -3.0, 0x30: 0.5, 0x7E: 448.0, 0xFE: -448.0,
             0x01: 2.0 ** -9, 0x07: 7 * 2.0 ** -9, 0x08: 2.0 ** -6, 0x3C: 1.5, 0x39: 1.125, 0x77: 240.0}
    for bits, val in known.items():
        assert float(oracle.e4m3_to_f64(np.uint8(bits))) == val, hex(bits)
        assert int(oracle.f64_to_e4m3(val)) == bits, hex(bits)
    assert np.isnan(oracle.e4m3_to_f64(np.uint8(0x7F))) and np.isnan(oracle.e4m3_to_f64(np.uint8(0xFF)))
    assert int(oracle.f64_to_e4m3(float("nan"))) & 0x7F == 0x7F


def test_decode_matches_torch_for_every_pattern():
    ours = oracle.e4m3_to_f64(ALL)
    theirs = torch.from_numpy(ALL.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    nan = np.isnan(theirs)
    assert nan.sum() == 2 and np.array_equal(np.isnan(ours), nan)
    assert np.array_equal(ours[~nan], theirs[~nan]) and np.array_equal(np.signbit(ours[~nan]), np.signbit(theirs[~nan]))


def test_roundtrip_ties_and_saturation():
    vals = oracle.e4m3_to_f64(ALL)
    nan = np.isnan(vals)
    assert np.array_equal(oracle.f64_to_e4m3(vals)[~nan], ALL[~nan])
    lo_bits = np.arange(0x00, 0x7E, dtype=np.uint8)         # adjacent non-negative finite pairs
    hi_bits = lo_bits + 1
    lo, hi = oracle.e4m3_to_f64(lo_bits), oracle.e4m3_to_f64(hi_bits)
    mid = (lo + hi) / 2
    even = np.where((lo_bits & 1) == 0, lo_bits, hi_bits)
    assert np.array_equal(oracle.f64_to_e4m3(mid), even)
    assert np.array_equal(oracle.f64_to_e4m3(np.nextafter(mid, lo)), lo_bits)
    assert np.array_equal(oracle.f64_to_e4m3(np.nextafter(mid, hi)), hi_bits)
    assert np.array_equal(oracle.f64_to_e4m3(-mid), even | 0x80)
    # beyond the largest finite value: saturate, never NaN or a wrapped exponent
    for v in (449.0, 464.0, 480.0, 1e4, 1e300, float("inf")):
        assert int(oracle.f64_to_e4m3(v)) == 0x7E and int(oracle.f64_to_e4m3(-v)) == 0xFE
    assert int(oracle.f64_to_e4m3(2.0 ** -10)) == 0x00       # tie between 0 and the smallest subnormal
    assert int(oracle.f64_to_e4m3(np.nextafter(2.0 ** -10, 1))) == 0x01


def test_encode_matches_torch_inside_the_finite_range():
    rng = np.random.default_rng(3)
    f = np.concatenate([rng.standard_normal(20000) * s for s in (1.0, 30.0, 0.01)]).astype(np.float32)
    f = f[np.abs(f) <= 448.0]
    want = torch.from_numpy(f).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = oracle.f64_to_e4m3(f.astype(np.float64))
    assert np.array_equal(got, want)


def rand_e4m3(rng, shape, sigma=1.0):
    f = torch.from_numpy((rng.standard_normal(shape) * sigma).astype(np.float32)).clamp_(-448, 448)
    return W.e4m3_bits(f.to(torch.float8_e4m3fn)).copy()


def rand_gamma(rng, n):
    f = torch.from_numpy(rng.uniform(0.5, 1.5, n).astype(np.float32))
    return W.bf16_bits(f.to(torch.bfloat16)).copy()


@pytest.mark.parametrize("c", [1.0, -3.0, 0.5, 2.0 ** -9, 240.0])
@pytest.mark.parametrize("g", [1.0, -0.5, 1.25])
def test_constant_row_closed_form(c, g):
    H = 640
    eps = float(np.float32(1e-6))
    x = np.full((1, H), oracle.f64_to_e4m3(c), dtype=np.uint8)
    assert float(oracle.e4m3_to_f64(x[0, 0])) == c
    res = oracle.rmsnorm_e4m3([x], [np.full((H,), bf16_bits_of([g])[0], dtype=np.uint16)], eps, want_y64=True)
    want = g * c / math.sqrt(c * c + eps)
    assert np.allclose(res["y64"], want, rtol=1e-14, atol=0)
    assert np.all(res["y"][0] == oracle.f64_to_e4m3(want))
    assert res["acc"][0] == pytest.approx(H * c * c, rel=1e-15)


def test_hand_rows():
    # [3,4,0,0], eps = 0: x/rms = [1.2, 1.6, 0, 0]; gamma [1,2,0.5,-1] -> [1.2, 3.2, 0, -0]
    # E4M3 neighbours of 1.2 are 1.125 (0x39) and 1.25 (0x3A): 1.2 is nearer 1.25.  3.2: 3.0 (0x44), 3.25 (0x45) -> 3.25.
    x = oracle.f64_to_e4m3([[3, 4, 0, 0]])
    y = oracle.rmsnorm_e4m3([x], [bf16_bits_of([1, 2, 0.5, -1])], 0.0)["y"][0][0]
    assert [int(v) for v in y] == [0x3A, 0x45, 0x00, 0x80]


def test_agrees_with_the_bf16_oracle_before_rounding():
    # every E4M3 value is also a bf16 value: the two oracles must give the same fp64 result
    rng = np.random.default_rng(5)
    x8 = rand_e4m3(rng, (6, 1024), sigma=2.0)
    g = rand_gamma(rng, 1024)
    x16 = W.bf16_bits(torch.from_numpy(oracle.e4m3_to_f64(x8)).to(torch.bfloat16)).copy()
    assert np.array_equal(bf16_bits_to_f64(x16), oracle.e4m3_to_f64(x8))
    a = oracle.rmsnorm_e4m3([x8], [g], 1e-6, want_y64=True)
    b = oracle.rmsnorm(x16, g, 1e-6, want_y64=True)
    assert np.array_equal(a["y64"], b["y64"]) and np.array_equal(a["rstd"], b["rstd"])
    assert np.array_equal(a["y"][0], oracle.f64_to_e4m3(b["y64"]))


@pytest.mark.parametrize("S", [2, 4, 8])
def test_sharded_equals_unsharded(S):
    rng = np.random.default_rng(7)
    T, H = 5, 1024
    x = rand_e4m3(rng, (T, H), sigma=3.0)
    g = rand_gamma(rng, H)
    full = oracle.rmsnorm_e4m3([x], [g], 1e-6)
    w = H // S
    sh = oracle.rmsnorm_e4m3([np.ascontiguousarray(x[:, s * w:(s + 1) * w]) for s in range(S)],
                             [np.ascontiguousarray(g[s * w:(s + 1) * w]) for s in range(S)], 1e-6)
    assert np.array_equal(np.concatenate(sh["y"], axis=1), full["y"][0])
    assert np.array_equal(sh["rstd"], full["rstd"])
    assert np.allclose(sh["partials"].sum(axis=0), full["acc"], rtol=1e-14)
    assert np.allclose(sh["partials"][1], (oracle.e4m3_to_f64(x[:, w:2 * w]) ** 2).sum(axis=1), rtol=1e-14)


def test_saturation_and_nan_in_the_norm():
    H = 16
    x = np.zeros((2, H), dtype=np.uint8)
    x[0, 3] = 0x38                                     # one-hot 1.0: y_3 = gamma * sqrt(16) = 4 * gamma
    x[1, 0] = 0x7F                                     # NaN poisons its row
    g = np.full((H,), bf16_bits_of([200.0])[0], dtype=np.uint16)   # 800 > 448: saturates
    with np.errstate(all="ignore"):
        y = oracle.rmsnorm_e4m3([x], [g], 0.0)["y"][0]
    assert int(y[0, 3]) == 0x7E and np.all(np.delete(y[0], 3) == 0x00)
    assert np.all((y[1] & 0x7F) == 0x7F)
    assert e4m3_ordinal_distance(y[0], y[0]).max() == 0
