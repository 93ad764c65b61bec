"""The C ABI without Python in between: the example program is compiled with gcc as C99, linked against the
library and the CUDA runtime, and run; it validates three candidates it built itself and checks what it gets."""
import os
import shutil
import subprocess

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")


def test_c_example_builds_and_runs(tmp_path):
    from paper_2510_03760_b200 import build
    lib = build.build()
    if shutil.which("gcc") is None or not os.path.exists(os.path.join(CUDA, "include", "cuda_runtime_api.h")):
        pytest.skip("needs gcc and the CUDA toolkit headers")
    exe = str(tmp_path / "validate_example")
    libdir = os.path.dirname(lib)
    cmd = ["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-I", os.path.join(ROOT, "include"), "-I", os.path.join(CUDA, "include"),
           os.path.join(ROOT, "paper_2510_03760_b200", "examples", "validate_example.c"), "-L", libdir, "-levo",
           "-L", os.path.join(CUDA, "lib64"), "-lcudart", "-Wl,-rpath," + libdir, "-Wl,-rpath," + os.path.join(CUDA, "lib64"),
           "-o", exe]
    p = subprocess.run(cmd, capture_output=True, text=True)
    assert p.returncode == 0, p.stderr
    r = subprocess.run([exe], capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stdout + r.stderr
    lines = r.stdout.strip().splitlines()
    assert lines[-1] == "ok" and len(lines) == 4
    assert lines[1].startswith("cand 1 n_mismatch 5 ") and " pass 0 " in lines[1]
