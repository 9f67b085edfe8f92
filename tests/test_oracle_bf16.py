"""Pins for the oracle's bf16 codec (CPU only)."""
import numpy as np
import torch

import oracle


ALL = np.arange(65536, dtype=np.uint16)


def _finite_mask(bits):
    return (bits & 0x7F80) != 0x7F80


def test_known_values():
    known = {
        0x3F80: 1.0, 0x4000: 2.0, 0xC040: -3.0, 0x3F00: 0.5, 0x42C0: 96.0,
        0x3DCD: 0.10009765625, 0x0001: 2.0 ** -133, 0x0080: 2.0 ** -126,
        0x7F7F: (2.0 - 2.0 ** -7) * 2.0 ** 127, 0x8000: -0.0, 0x0000: 0.0,
        0x3A80: 2.0 ** -10, 0x3F81: 1.0 + 2.0 ** -7,
    }
    for bits, val in known.items():
        got = float(oracle.bf16_to_f64(np.uint16(bits)))
        assert got == val, (hex(bits), got, val)
        assert int(oracle.f64_to_bf16(val)) == bits, hex(bits)
    assert np.signbit(oracle.bf16_to_f64(np.uint16(0x8000)))
    assert np.isposinf(oracle.bf16_to_f64(np.uint16(0x7F80)))
    assert np.isneginf(oracle.bf16_to_f64(np.uint16(0xFF80)))
    assert np.isnan(oracle.bf16_to_f64(np.uint16(0x7FC1)))


def test_widening_matches_torch_for_every_pattern():
    ours = oracle.bf16_to_f64(ALL)
    theirs = torch.from_numpy(ALL.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    nan = np.isnan(theirs)
    assert np.array_equal(np.isnan(ours), nan)
    assert np.array_equal(ours[~nan], theirs[~nan])
    assert np.array_equal(np.signbit(ours[~nan]), np.signbit(theirs[~nan]))


def test_roundtrip_every_pattern():
    vals = oracle.bf16_to_f64(ALL)
    back = oracle.f64_to_bf16(vals)
    nan = np.isnan(vals)
    assert np.array_equal(back[~nan], ALL[~nan])
    # NaN stays NaN
    assert np.all((back[nan] & 0x7F80) == 0x7F80) and np.all((back[nan] & 0x7F) != 0)


def test_ties_go_to_even_and_neighbours_go_home():
    # every pair of adjacent non-negative finite bf16 values (subnormals included)
    lo_bits = np.arange(0x0000, 0x7F7F, dtype=np.uint16)
    hi_bits = lo_bits + 1
    lo = oracle.bf16_to_f64(lo_bits)
    hi = oracle.bf16_to_f64(hi_bits)
    mid = (lo + hi) / 2.0                   # exact in fp64
    assert np.all((mid > lo) & (mid < hi))
    even = np.where((lo_bits & 1) == 0, lo_bits, hi_bits)
    assert np.array_equal(oracle.f64_to_bf16(mid), even)
    assert np.array_equal(oracle.f64_to_bf16(np.nextafter(mid, lo)), lo_bits)
    assert np.array_equal(oracle.f64_to_bf16(np.nextafter(mid, hi)), hi_bits)
    # sign symmetry
    neg_even = even | 0x8000
    assert np.array_equal(oracle.f64_to_bf16(-mid), neg_even)


def test_overflow_and_underflow_edges():
    big = float(oracle.bf16_to_f64(np.uint16(0x7F7F)))
    half_ulp = 2.0 ** (127 - 8)
    assert int(oracle.f64_to_bf16(big + half_ulp)) == 0x7F80        # tie -> even -> inf
    assert int(oracle.f64_to_bf16(np.nextafter(big + half_ulp, 0))) == 0x7F7F
    assert int(oracle.f64_to_bf16(1e300)) == 0x7F80
    assert int(oracle.f64_to_bf16(-1e300)) == 0xFF80
    tiny = 2.0 ** -133
    assert int(oracle.f64_to_bf16(tiny / 2)) == 0x0000               # tie -> even -> 0
    assert int(oracle.f64_to_bf16(np.nextafter(tiny / 2, 1))) == 0x0001
    assert int(oracle.f64_to_bf16(-tiny / 2)) == 0x8000
    assert int(oracle.f64_to_bf16(1e-300)) == 0x0000


def test_single_rounding_witness():
    # Slightly above the midpoint of 1 and 1+2^-7.  Rounding to fp32 first lands
    # exactly ON the midpoint and the tie would then fall to 1.0: a one-step
    # rounding must give 1+2^-7.
    v = 1.0 + 2.0 ** -8 + 2.0 ** -30
    assert np.float32(v) == np.float32(1.0 + 2.0 ** -8)
    assert int(oracle.f64_to_bf16(v)) == 0x3F81


def test_narrowing_matches_torch_on_fp32_values():
    # For values that are exactly fp32 numbers, torch's fp32 -> bf16 cast is a
    # single round-to-nearest-even and must agree with the oracle's.
    rng = np.random.default_rng(7)
    f = np.concatenate([
        rng.standard_normal(20000).astype(np.float32),
        (rng.standard_normal(5000) * 1e-38).astype(np.float32),      # subnormal bf16 range
        (rng.standard_normal(5000) * 1e38).astype(np.float32),
        np.array([0.0, -0.0, 3.3895314e38, -3.3895314e38, np.inf, -np.inf], dtype=np.float32),
    ])
    want = torch.from_numpy(f).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = oracle.f64_to_bf16(f.astype(np.float64))
    assert np.array_equal(got, want)
