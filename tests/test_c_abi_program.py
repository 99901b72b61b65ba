"""The C ABI used from plain C: compile tests/c_abi/c_abi_check.c against include/equarx.h,
link it with the CUDA library and the C oracle, and run it on the GPU."""
import os
import shutil
import subprocess

import pytest

import oracle
import paper_2506_17615_b200 as eq

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "tests", "c_abi", "c_abi_check.c")


def cuda_home():
    for cand in (os.environ.get("CUDA_HOME"), "/usr/local/cuda"):
        if cand and os.path.exists(os.path.join(cand, "include", "cuda_runtime_api.h")):
            return cand
    return None


def compile_program(tmpdir):
    cuda = cuda_home()
    if cuda is None or shutil.which("gcc") is None:
        pytest.skip("no CUDA headers or no gcc")
    oracle.build()
    exe = os.path.join(tmpdir, "c_abi_check")
    libdir, olibdir = os.path.dirname(eq.LIB_PATH), os.path.dirname(oracle.lib_path())
    cmd = ["gcc", "-std=c11", "-O1", "-Wall", "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
           SRC, "-o", exe, "-L", libdir, "-lequarx", "-L", olibdir, "-lequarx_oracle",
           "-L", os.path.join(cuda, "lib64"), "-lcudart", "-lm",
           f"-Wl,-rpath,{libdir}", f"-Wl,-rpath,{olibdir}", f"-Wl,-rpath,{os.path.join(cuda, 'lib64')}"]
    subprocess.run(cmd, check=True)
    return exe


def test_c_program_compiles_against_the_header(tmp_path):
    """No GPU needed: the header is valid C11 and the library resolves every symbol the program uses."""
    compile_program(str(tmp_path))


@pytest.mark.gpu
def test_c_program_matches_the_oracle_on_the_gpu(tmp_path):
    exe = compile_program(str(tmp_path))
    out = subprocess.run([exe], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr + out.stdout
    assert "c abi ok" in out.stdout
