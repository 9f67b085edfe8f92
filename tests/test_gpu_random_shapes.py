"""Seeded random shapes through the main entry points against the oracle: token counts on both
sides of every dispatch boundary, widths that are and are not multiples of 8, every slice count
that divides them, in place and not.  What a hand-picked list of shapes can miss."""
import numpy as np
import pytest
import torch

from paper_2608_09160_b200 import binding
from paper_2608_09160_b200 import workloads as W
from tests import gpu_harness as H
from tests.test_gpu_parity import check_against_oracle, run_case

pytestmark = pytest.mark.gpu

BOUNDARIES = [591, 592, 593, 1280, 1281, 2048, 2049]


def random_cases(n, seed):
    rng = np.random.default_rng(seed)
    cases = []
    for i in range(n):
        kind = rng.integers(0, 4)
        if kind == 0:      # vector-friendly GQA-like
            dk = int(rng.choice([128, 256, 512, 1024]))
            dq = dk * int(rng.choice([1, 2, 4, 8]))
        elif kind == 1:    # multiples of 8, nothing else nice
            dq, dk = int(rng.integers(1, 700)) * 8, int(rng.integers(1, 300)) * 8
        elif kind == 2:    # one tensor only
            dq, dk = (int(rng.integers(1, 600)) * 8, 0) if rng.integers(0, 2) else (0, int(rng.integers(1, 600)) * 8)
        else:              # arbitrary widths: the general kernel
            dq, dk = int(rng.integers(1, 3000)), int(rng.integers(1, 900))
        T = int(rng.choice(BOUNDARIES)) if rng.integers(0, 3) == 0 else int(rng.integers(1, 4500))
        divisors = [s for s in range(1, 17) if dq % s == 0 and dk % s == 0]
        S = int(rng.choice(divisors))
        cases.append((i, T, dq, dk, S, bool(rng.integers(0, 2))))
    return cases


CASES = random_cases(40, seed=20261125)


@pytest.mark.parametrize("i,T,dq,dk,S,in_place", CASES, ids=[f"r{c[0]}-T{c[1]}-{c[2]}x{c[3]}-S{c[4]}" for c in CASES])
def test_random_shape(libqknorm, i, T, dq, dk, S, in_place):
    w = W.Workload(f"rand{i}", tokens=T, dq=dq, dk=dk, shards=(S,), seed=9000 + i, sigma=(0.5, 1.0, 4.0)[i % 3],
                   outlier_frac=0.02 if i % 4 == 0 else 0.0)
    res = run_case(w, S, in_place=in_place)
    check_against_oracle(w, S, res)
    assert binding.device_error_word() == 0
