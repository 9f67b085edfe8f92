"""The C ABI used from C: tests/c_client/client.c is compiled with gcc against include/qknorm.h,
linked to libqknorm.so and the CUDA runtime, and run; it checks closed-form results itself."""
import os
import shutil
import subprocess

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_c_client_builds_and_runs(libqknorm, tmp_path):
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    if not (shutil.which("gcc") and os.path.isdir(os.path.join(cuda, "include"))):
        pytest.skip("needs gcc and the CUDA runtime headers")
    pkg = os.path.join(ROOT, "paper_2608_09160_b200")
    exe = str(tmp_path / "client")
    cmd = ["gcc", "-O1", "-std=c11", os.path.join(ROOT, "tests", "c_client", "client.c"), "-o", exe,
           "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
           "-L", pkg, "-lqknorm", "-L", os.path.join(cuda, "lib64"), "-lcudart", "-lm",
           f"-Wl,-rpath,{pkg}", f"-Wl,-rpath,{os.path.join(cuda, 'lib64')}"]
    subprocess.run(cmd, check=True, capture_output=True, text=True)
    out = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert out.returncode == 0, out.stdout + out.stderr
    assert "qknorm_fwd: variant warp" in out.stdout and out.stdout.strip().endswith("ok")
