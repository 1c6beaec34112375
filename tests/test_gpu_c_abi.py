"""A plain C program (tests/c/use_kb_gpu.c) uses the library through include/kb.h and the CUDA
runtime's C API: no Python, no torch on that path."""
import os
import subprocess

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_c_program_screens_three_candidates(tmp_path):
    from paper_2608_02611_b200 import build
    lib_path = build.build()
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    exe = tmp_path / "use_kb_gpu"
    cmd = ["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"),
           "-I", os.path.join(cuda, "include"), os.path.join(ROOT, "tests", "c", "use_kb_gpu.c"),
           lib_path, "-L", os.path.join(cuda, "lib64"), "-lcudart", "-lm", "-o", str(exe),
           "-Wl,-rpath," + os.path.dirname(lib_path), "-Wl,-rpath," + os.path.join(cuda, "lib64")]
    done = subprocess.run(cmd, capture_output=True, text=True)
    assert done.returncode == 0, done.stderr
    run = subprocess.run([str(exe)], capture_output=True, text=True, timeout=120)
    assert run.returncode == 0 and run.stdout.strip() == "ok", (run.returncode, run.stdout, run.stderr)
