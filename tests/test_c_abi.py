"""The C ABI from plain C: the header must compile as C99 and as C++ on its own, and a C program that links the
library and the CUDA runtime (no Python, no torch on its path) must round-trip a buffer and see tampering."""
import os
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
INCLUDE = os.path.join(ROOT, "include")
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")


@pytest.mark.parametrize("compiler,std", [("gcc", "-std=c99"), ("gcc", "-std=c11"), ("g++", "-std=c++11"), ("g++", "-std=c++17")])
def test_header_compiles_on_its_own(tmp_path, compiler, std):
    src = tmp_path / ("use.c" if compiler == "gcc" else "use.cpp")
    src.write_text('#include "fastrack.h"\n#include "fastrack.h"\n'
                   "int use(fastrack_ctx* c) { return (int)fastrack_num_chunks(c, FASTRACK_MAX_CHUNK_BYTES) + FASTRACK_OK; }\n")
    subprocess.check_call([compiler, std, "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", INCLUDE, "-c", str(src), "-o",
                           str(tmp_path / "use.o")])


def _build_roundtrip(tmp_path):
    from paper_2410_15240_b200 import build as lib_build
    lib = lib_build.build()
    exe = tmp_path / "roundtrip"
    subprocess.check_call(["gcc", "-std=c99", "-O1", "-Wall", "-Wextra", "-I", INCLUDE, "-I", os.path.join(CUDA, "include"),
                           os.path.join(ROOT, "tests", "c_abi", "roundtrip.c"), "-o", str(exe), lib,
                           "-L", os.path.join(CUDA, "lib64"), "-lcudart", "-Wl,-rpath," + os.path.dirname(lib),
                           "-Wl,-rpath," + os.path.join(CUDA, "lib64")])
    return exe


def test_c_program_links_against_the_library(tmp_path):
    _build_roundtrip(tmp_path)


@pytest.mark.gpu
@pytest.mark.parametrize("chunk,length", [(65536, (3 << 20) + 4099), (1 << 20, 64 << 20), (256, (1 << 20) + 17), (16, 4096 * 16)])
def test_c_program_round_trip(tmp_path, chunk, length):
    exe = _build_roundtrip(tmp_path)
    out = subprocess.run([str(exe), str(chunk), str(length)], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    assert out.stdout.startswith("ok ") and "rejected=2" in out.stdout
