"""A plain C program against the C ABI: the headers compile as C99 and link (CPU), and on a GPU the program's
result matches the oracle (it links the oracle itself: test infrastructure)."""
import os
import subprocess
import sys

import pytest

from oracle import hg_oracle
from paper_2604_18529_b200 import binding, build as hgbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "tests", "c_abi", "c_parity.c")
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")


def compile_program(out_path):
    hgbuild.build()
    lib = binding.lib_path()
    ora = hg_oracle.build()
    cmd = ["gcc", "-std=c99", "-Wall", "-Werror", "-O1", SRC, "-o", out_path,
           "-I", os.path.join(ROOT, "include"), "-I", os.path.join(CUDA, "include"),
           lib, ora, "-L", os.path.join(CUDA, "lib64"), "-lcudart", "-lm",
           "-Wl,-rpath," + os.path.dirname(lib), "-Wl,-rpath," + os.path.dirname(ora),
           "-Wl,-rpath," + os.path.join(CUDA, "lib64")]
    subprocess.check_call(cmd)
    return out_path


def test_c_program_compiles_and_links_against_the_headers(tmp_path):
    exe = compile_program(str(tmp_path / "c_parity"))
    assert os.path.exists(exe)
    # both public headers are valid C on their own
    for header in ("hybridgen_attn.h", "hybridgen_host.h"):
        src = tmp_path / (header + ".c")
        src.write_text(f'#include "{header}"\nint main(void) {{ return 0; }}\n')
        subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-fsyntax-only", "-I", os.path.join(ROOT, "include"), str(src)])


@pytest.mark.gpu
def test_c_program_matches_the_oracle_on_the_gpu(tmp_path):
    exe = compile_program(str(tmp_path / "c_parity"))
    run = subprocess.run([exe], capture_output=True, text=True, timeout=300)
    sys.stdout.write(run.stdout)
    sys.stderr.write(run.stderr)
    assert run.returncode == 0, run.stderr
    assert "C ABI parity OK" in run.stdout
