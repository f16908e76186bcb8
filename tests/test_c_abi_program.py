"""The C ABI used from plain C: a C program that owns its device memory (cudaMalloc), links libaafkv.so
and checks a fork / append / compose round byte by byte, without Python or PyTorch in the process."""
from __future__ import annotations

import os
import subprocess

import pytest

import __graft_entry__ as entry
from paper_2607_10987_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")


def build_program(tmp_path) -> str:
    entry.build()
    exe = str(tmp_path / "c_abi_program")
    libdir = os.path.dirname(binding.LIB_PATH)
    subprocess.check_call(["gcc", "-std=c11", "-O1", "-Wall", "-I", os.path.join(ROOT, "include"), "-I",
                           os.path.join(CUDA, "include"), os.path.join(ROOT, "tests", "c_abi_program.c"), "-o", exe,
                           "-L", libdir, "-laafkv", "-L", os.path.join(CUDA, "lib64"), "-lcudart",
                           f"-Wl,-rpath,{libdir}", f"-Wl,-rpath,{os.path.join(CUDA, 'lib64')}"])
    return exe


def test_c_program_compiles_against_the_header(tmp_path):
    assert os.path.exists(build_program(tmp_path))


@pytest.mark.gpu
def test_c_program_runs_the_operators(tmp_path):
    out = subprocess.run([build_program(tmp_path)], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, (out.returncode, out.stderr[-1000:])
    assert "c abi ok" in out.stdout
