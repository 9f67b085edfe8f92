"""Pins for the oracle's headwise form (CPU only)."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2608_09160_b200 import workloads as W
from tests.test_oracle_pins import bits_of, rand_bits, rand_gamma
from tests.util import ordinal_distance


def test_one_head_is_the_layerwise_norm():
    rng = np.random.default_rng(1)
    x, g = rand_bits(rng, (5, 512)), rand_gamma(rng, 512)
    a = oracle.rmsnorm_headwise(x, g, 512, 1e-6, want_y64=True)
    b = oracle.rmsnorm(x, g, 1e-6, want_y64=True)
    assert np.array_equal(a["y"], b["y"]) and np.array_equal(a["y64"], b["y64"])
    assert np.array_equal(a["rstd"][:, 0], b["rstd"])


@pytest.mark.parametrize("hd", [8, 64, 128])
def test_every_head_is_its_own_row(hd):
    rng = np.random.default_rng(2)
    T, H = 4, 1024
    x, g = rand_bits(rng, (T, H), sigma=2.0), rand_gamma(rng, H)
    hw = oracle.rmsnorm_headwise(x, g, hd, 1e-6)
    for h in (0, 1, H // hd - 1):
        sl = slice(h * hd, (h + 1) * hd)
        ref = oracle.rmsnorm(np.ascontiguousarray(x[:, sl]), np.ascontiguousarray(g[sl]), 1e-6)
        assert np.array_equal(hw["y"][:, sl], ref["y"])
        assert np.array_equal(hw["rstd"][:, h], ref["rstd"])


def test_heads_with_different_constants_closed_form():
    hd, consts, gam = 16, [1.0, -3.0, 0.5, 96.0], [1.0, 0.5, -2.0, 1.25]
    x = np.concatenate([np.full((1, hd), bits_of([c])[0], dtype=np.uint16) for c in consts], axis=1)
    g = np.concatenate([np.full((hd,), bits_of([v])[0], dtype=np.uint16) for v in gam])
    eps = float(np.float32(1e-6))
    res = oracle.rmsnorm_headwise(x, g, hd, eps, want_y64=True)
    for h, (c, v) in enumerate(zip(consts, gam)):
        want = v * c / math.sqrt(c * c + eps)
        assert np.allclose(res["y64"][0, h * hd:(h + 1) * hd], want, rtol=1e-14, atol=0)
        assert math.isclose(res["rstd"][0, h], 1 / math.sqrt(c * c + eps), rel_tol=1e-15)
    # a layerwise norm of the same row would mix the heads: the two must differ
    lw = oracle.rmsnorm(x, g, eps)["y"]
    assert not np.array_equal(lw, res["y"])


def test_against_torch_rms_norm_on_the_head_axis():
    rng = np.random.default_rng(3)
    T, nh, hd = 6, 40, 128
    x, g = rand_bits(rng, (T, nh * hd)), rand_gamma(rng, nh * hd)
    res = oracle.rmsnorm_headwise(x, g, hd, 1e-6, want_y64=True)
    xt = W.from_bf16_bits(x).to(torch.float64).view(T, nh, hd)
    gt = W.from_bf16_bits(g).to(torch.float64).view(nh, hd)
    eps = float(np.float32(1e-6))
    ref = (xt * torch.rsqrt(xt.pow(2).mean(-1, keepdim=True) + eps) * gt).reshape(T, nh * hd).numpy()
    lib = torch.nn.functional.rms_norm(xt, (hd,), None, eps) * gt
    assert np.allclose(res["y64"], ref, rtol=1e-12, atol=0)
    assert np.allclose(res["y64"], lib.reshape(T, nh * hd).numpy(), rtol=1e-12, atol=0)
    assert ordinal_distance(res["y"], oracle.f64_to_bf16(ref)).max() <= 1


def test_e4m3_headwise_matches_the_e4m3_row_oracle():
    rng = np.random.default_rng(4)
    f = torch.from_numpy((rng.standard_normal((3, 512)) * 2).astype(np.float32)).clamp_(-448, 448)
    x8 = W.e4m3_bits(f.to(torch.float8_e4m3fn)).copy()
    g = rand_gamma(rng, 512)
    hw = oracle.rmsnorm_headwise(x8, g, 128, 1e-6)
    for h in range(4):
        sl = slice(h * 128, (h + 1) * 128)
        ref = oracle.rmsnorm_e4m3([np.ascontiguousarray(x8[:, sl])], [np.ascontiguousarray(g[sl])], 1e-6)
        assert np.array_equal(hw["y"][:, sl], ref["y"][0]) and np.array_equal(hw["rstd"][:, h], ref["rstd"])


def test_bad_head_dim_is_rejected():
    x, g = np.zeros((1, 24), dtype=np.uint16), np.zeros((24,), dtype=np.uint16)
    with pytest.raises(ValueError):
        oracle.rmsnorm_headwise(x, g, 16, 1e-6)
