"""The C ABI from plain C (no Python, no torch in the program under test): compiled with gcc against include/catekv.h
and libcatekv.so; linked here on any machine, run where there is a GPU."""
import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")


def _build(tmp_path):
    import paper_2608_30295_b200.build as b
    lib = b.build()
    exe = str(tmp_path / "c_abi_smoke")
    cmd = ["gcc", "-std=c11", "-O1", "-I", os.path.join(ROOT, "include"), "-I", os.path.join(CUDA, "include"),
           os.path.join(ROOT, "tests", "c_abi", "smoke.c"), "-L", os.path.dirname(lib), "-lcatekv",
           "-L", os.path.join(CUDA, "lib64"), "-lcudart", "-lm", "-Wl,-rpath," + os.path.dirname(lib),
           "-Wl,-rpath," + os.path.join(CUDA, "lib64"), "-o", exe]
    subprocess.run(cmd, check=True, capture_output=True, text=True)
    return exe


@pytest.mark.skipif(shutil.which("gcc") is None, reason="no C compiler")
def test_c_program_compiles_and_links_against_the_header_and_library(tmp_path):
    assert os.path.exists(_build(tmp_path))


@pytest.mark.gpu
@pytest.mark.skipif(shutil.which("gcc") is None, reason="no C compiler")
def test_c_program_runs_append_plan_and_attention(tmp_path):
    r = subprocess.run([_build(tmp_path)], capture_output=True, text=True, timeout=120)
    assert r.returncode == 0, (r.stdout, r.stderr)
    assert "c abi smoke: rel-L2" in r.stdout
