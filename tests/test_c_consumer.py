"""The C ABI used from plain C: tests/c_consumer/abi_consumer.c is compiled with gcc against include/kop.h,
libkop.so and the CUDA runtime (CPU test: it builds and links), and run on the GPU (gpu test: it exits 0)."""
import os
import shutil
import subprocess

import pytest

from paper_2609_30059_b200 import build as kbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "tests", "c_consumer", "abi_consumer.c")
EXE = os.path.join(ROOT, "tests", "c_consumer", "abi_consumer")


def cuda_home():
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    return os.path.dirname(os.path.dirname(os.path.realpath(nvcc)))


def build_consumer():
    kbuild.build()
    libdir = os.path.join(ROOT, "paper_2609_30059_b200")
    cuda = cuda_home()
    cmd = ["gcc", "-std=c11", "-O1", "-Wall", "-Werror", SRC, "-o", EXE, "-I" + os.path.join(ROOT, "include"),
           "-I" + os.path.join(cuda, "include"), "-L" + libdir, "-lkop", "-L" + os.path.join(cuda, "lib64"),
           "-lcudart", "-lcublas", "-lm", "-Wl,-rpath," + libdir, "-Wl,-rpath," + os.path.join(cuda, "lib64")]
    res = subprocess.run(cmd, capture_output=True, text=True)
    assert res.returncode == 0, res.stderr
    return EXE


def test_c_consumer_compiles_and_links_as_c11():
    assert os.path.exists(build_consumer())


@pytest.mark.gpu
def test_c_consumer_runs():
    exe = build_consumer()
    res = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert res.returncode == 0, res.stdout + res.stderr
    assert "abi consumer ok" in res.stdout
