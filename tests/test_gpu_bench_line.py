"""The JSON line bench.py prints on a GPU: contract keys, the kernel named for the timed
launches (not for whatever ran last), the per-config summary inside `roofline`, the source
file of the ncu traffic figure, and the tensor-parallel mode on one rank."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_bench(*flags, timeout=900):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *flags], capture_output=True, text=True,
                         timeout=timeout, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1, "exactly one JSON line on stdout"
    return json.loads(lines[0])


def test_headline_line_names_the_timed_kernel_and_carries_all_configs(libqknorm):
    d = run_bench("--steps", "5", "--warmup", "3", "--no-cpu", "--table-scope", "configs")
    assert d["metric"] == "qknorm_prefill_GBps" and d["unit"] == "GB/s" and d["n_gpus"] == 1
    assert d["dtype"] == "f32" and d["storage_dtype"] == "bf16" and d["accum_dtype"] == "f32"
    assert d["gpu_launches"] == 5 and d["value"] > 0
    assert d["config"]["workload"].startswith("C5") and d["config"]["kernel_variant"] == "warp"
    assert d["e2e"]["kernel_variant"] in ("rows", "warp") and d["e2e"]["h2d_bytes_per_step"] > 0
    r = d["roofline"]
    assert r["kernel_variant"] == "warp" and r["bound"] == "hbm"
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-3
    if r["traffic"] is not None:
        assert os.path.isfile(os.path.join(ROOT, r["traffic_source"]))
        assert 0.9 < r["traffic"] / r["algorithmic_bytes_per_launch"] < 1.1
    rows = r["per_config"]
    assert sorted(rows) == ["C1/S1", "C2/S1", "C2/S4", "C3/S1", "C3/S4", "C4/S8", "C5/S8"]
    for key, row in rows.items():
        assert row["us_median"] > 0 and row["us_back_to_back"] > 0 and isinstance(row["variant"], str)
        if key.startswith(("C1", "C2")):
            assert row["variant"] == "rows" and row["us_graph_replay"] > 0 and row["us_graph_replay_l2_cold"] > 0
        else:
            assert row["variant"] == "warp" and 0 < row["frac"] < 1.2 and row["GBps"] > 0


def test_tensor_parallel_mode_on_one_rank(libqknorm):
    d = run_bench("--parallelism", "tp", "--gpus", "1", "--workload", "C4", "--tokens", "4096", "--steps", "3",
                  "--warmup", "3")
    assert d["config"]["parallelism"] == "tensor-parallel x1, scalar exchange" and d["scaling"] == "strong"
    assert d["gpu_launches"] == 3 and d["value"] > 0 and d["roofline"]["all_waits_completed"] is True
    assert d["e2e"]["h2d_bytes_per_step"] == 4096 * (5120 + 1024) * 2
