"""Sanitizer runs on the host (compute-sanitizer is not available for the device side): the
CPU oracles and the library's host-only entry points under AddressSanitizer and
UndefinedBehaviorSanitizer.  No GPU is needed: nothing here reaches a device call that could
succeed, and the library's layout arithmetic and argument checks run before any device use."""
import os
import shutil
import subprocess

import pytest

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
SAN = ["-fsanitize=address,undefined", "-fno-sanitize-recover=all", "-fno-omit-frame-pointer", "-g", "-O1"]
ENV = dict(os.environ, ASAN_OPTIONS="detect_leaks=1:abort_on_error=0:protect_shadow_gap=0",
           UBSAN_OPTIONS="print_stacktrace=1")


def _run(exe, env=ENV):
    res = subprocess.run([exe], capture_output=True, text=True, env=env, timeout=300)
    assert res.returncode == 0, res.stdout + res.stderr
    assert res.stdout.strip().endswith("ok")
    assert "Sanitizer" not in res.stderr and "runtime error" not in res.stderr, res.stderr


def test_oracles_under_asan_and_ubsan(tmp_path):
    exe = str(tmp_path / "oracle_sanitize")
    subprocess.run(["g++", "-std=c++17", "-ffp-contract=off"] + SAN + ["-o", exe,
                    os.path.join(HERE, "c_abi", "oracle_sanitize_driver.cpp"),
                    os.path.join(ROOT, "oracle", "ef_oracle.cpp"),
                    os.path.join(ROOT, "oracle", "vote_topk_oracle.cpp")], check=True)
    _run(exe)


def test_library_host_code_under_asan_and_ubsan(tmp_path):
    """The host half of libef (argument checks, workspace layout) compiled by nvcc with the
    sanitizers passed to the host compiler; the driver calls only what needs no GPU."""
    nvcc = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    if not os.path.exists(nvcc) and shutil.which("nvcc") is None:
        pytest.skip("nvcc not found")
    csrc = os.path.join(ROOT, "paper_1905_10936_b200", "csrc")
    exe = str(tmp_path / "ef_host_sanitize")
    host_flags = []
    for f in ["-fsanitize=address", "-fsanitize=undefined"] + SAN[1:]:
        host_flags += ["-Xcompiler", f]
    subprocess.run([nvcc, "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-fmad=false"]
                   + host_flags + ["-o", exe, "-I", os.path.join(ROOT, "include"),
                    "-x", "cu", os.path.join(HERE, "c_abi", "ef_host_sanitize_driver.c"),
                    os.path.join(csrc, "ef_lib.cu"), os.path.join(csrc, "ef_vote.cu"),
                    os.path.join(csrc, "ef_topk.cu"), "-lasan", "-lubsan"], check=True)
    # the CUDA runtime allocates and keeps process-lifetime objects: leak checking is for our code
    # in the oracle test above; here only memory errors and undefined behaviour count
    _run(exe, dict(ENV, ASAN_OPTIONS="detect_leaks=0:protect_shadow_gap=0"))
