"""The C ABI driven from a plain C program on the GPU: tests/c_abi/gpu_parity.c uses the CUDA
runtime, libdesloc.so and -- being a test -- the oracle library, and nothing of Python or torch
at run time.  It checks nine DES-LOC-Adam steps of three workers against the oracle itself."""
import os
import subprocess

import pytest

import oracle

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _cuda_home():
    for cand in (os.environ.get("CUDA_HOME"), "/usr/local/cuda"):
        if cand and os.path.exists(os.path.join(cand, "include", "cuda_runtime_api.h")):
            return cand
    pytest.skip("CUDA toolkit headers not found")


def test_c_program_steps_on_the_gpu_and_matches_the_oracle(tmp_path):
    from paper_2505_22549_b200 import binding
    cuda = _cuda_home()
    libdir = os.path.dirname(binding.LIB_PATH)
    olib = oracle.build()
    odir = os.path.dirname(olib)
    src = os.path.join(ROOT, "tests", "c_abi", "gpu_parity.c")
    exe = str(tmp_path / "gpu_parity")
    subprocess.check_call(
        ["gcc", "-std=c99", "-O1", "-Wall", "-Wextra", "-Werror", "-I", os.path.join(ROOT, "include"),
         "-I", os.path.join(cuda, "include"), src, "-o", exe,
         "-L", libdir, "-ldesloc", "-L", odir, "-l:" + os.path.basename(olib),
         "-L", os.path.join(cuda, "lib64"), "-lcudart", "-lm",
         f"-Wl,-rpath,{libdir}", f"-Wl,-rpath,{odir}", f"-Wl,-rpath,{os.path.join(cuda, 'lib64')}"])
    r = subprocess.run([exe], capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "gpu_parity: ok" in r.stdout
    print(r.stdout)
