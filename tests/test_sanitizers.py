"""Host code under AddressSanitizer and UndefinedBehaviorSanitizer: the library's host half
(encoder, validator, unpack / pack, statistics, storage form, FIFO model -- damaged inputs included)
and the oracle, each driven by a small program in tests/sanitize/.  No GPU involved."""
import os
import shutil
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SAN = ["-fsanitize=address,undefined", "-fno-sanitize-recover=all", "-fno-omit-frame-pointer", "-g", "-O1"]


def _run(cmd, **kw):
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600, **kw)
    assert r.returncode == 0, " ".join(cmd) + "\n" + r.stdout + r.stderr
    return r.stdout


@pytest.fixture(scope="module")
def compilers():
    if not shutil.which("gcc") or not shutil.which("g++"):
        pytest.skip("gcc / g++ not found")


def test_host_library_under_asan_and_ubsan(tmp_path, compilers):
    exe = str(tmp_path / "host_san")
    _run(["g++", "-std=c++17", *SAN, "-fopenmp", "-I", os.path.join(ROOT, "include"),
          "-I", os.path.join(ROOT, "paper_1905_10138_b200", "csrc"),
          os.path.join(ROOT, "paper_1905_10138_b200", "csrc", "sqnn_host.cpp"),
          os.path.join(ROOT, "tests", "sanitize", "host_san.cpp"), "-o", exe])
    out = _run([exe], env=dict(os.environ, ASAN_OPTIONS="detect_leaks=1", OMP_NUM_THREADS="4"))
    assert "host_san ok" in out


def test_oracle_under_asan_and_ubsan(tmp_path, compilers):
    exe = str(tmp_path / "oracle_san")
    _run(["gcc", "-std=c11", *SAN, "-fopenmp", os.path.join(ROOT, "oracle", "sqnn_oracle.c"),
          os.path.join(ROOT, "tests", "sanitize", "oracle_san.c"), "-lm", "-o", exe])
    out = _run([exe], env=dict(os.environ, ASAN_OPTIONS="detect_leaks=1", OMP_NUM_THREADS="4"))
    assert "oracle_san ok" in out
