"""Every call of the interface that enqueues work opens an NVTX range named after itself, so that
an attached profiler can group or filter the kernels by call.  Checked without a GPU: a minimal
NVTX tool (tests/c_abi/nvtx_recorder.c, loaded through NVTX_INJECTION64_PATH) records the ranges
while the calls are made with arguments they refuse."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CUDA_INC = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "include")

CHILD = r"""
import ctypes, sys
lib = ctypes.CDLL(sys.argv[1])
n = None
lib.ef_init(n, 0, 0, n, 0, ctypes.c_float(0), ctypes.c_float(0), 0, n, 0, n)
lib.ef_worker_step(n, 0, n)
lib.ef_worker_step_all(n, n, 0)
lib.ef_worker_step_push(n, 0, n, n)
lib.ef_server_step(n)
lib.ef_server_step_range(n, 0, 0, n, 0)
lib.ef_apply_update(n, 0, 0, n)
lib.ef_pack_message(n, 0, 0, 0, n)
lib.ef_vote_worker_step(n, 0, n)
lib.ef_vote_server_step(n)
lib.ef_topk_compress(n, 0, 0, n, n, n, n, 0, n)
"""


@pytest.mark.skipif(not os.path.exists(os.path.join(CUDA_INC, "nvtx3", "nvToolsExt.h")),
                    reason="NVTX headers not found")
def test_calls_open_and_close_a_range_named_after_themselves(tmp_path):
    from paper_1905_10936_b200 import build
    lib = build.build_library()
    tool = str(tmp_path / "nvtx_recorder.so")
    subprocess.run(["gcc", "-shared", "-fPIC", "-O1", "-I", CUDA_INC, "-o", tool,
                    os.path.join(ROOT, "tests", "c_abi", "nvtx_recorder.c")], check=True)
    log = str(tmp_path / "ranges.log")
    env = dict(os.environ, NVTX_INJECTION64_PATH=tool, EF_NVTX_LOG=log)
    subprocess.run([sys.executable, "-c", CHILD, lib], check=True, env=env, cwd=ROOT)
    lines = open(log).read().split()
    names, depth = [], 0
    for ln in lines:
        if ln == "pop":
            depth -= 1
        else:
            names.append(ln)
            depth += 1
        assert 0 <= depth <= 2
    assert depth == 0                                  # every range is closed, also on the error returns
    assert names == ["ef_init", "ef_worker_step", "ef_worker_step_all", "ef_worker_step_push",
                     "ef_server_step", "ef_server_step_range", "ef_apply_update",
                     "ef_push_message",                # ef_pack_message is ef_push_message with one target
                     "ef_vote_worker_step", "ef_vote_server_step", "ef_topk_compress"]


def test_without_a_tool_the_ranges_are_inert():
    from paper_1905_10936_b200 import build
    lib = build.build_library()
    env = {k: v for k, v in os.environ.items() if k != "NVTX_INJECTION64_PATH"}
    subprocess.run([sys.executable, "-c", CHILD, lib], check=True, env=env, cwd=ROOT)
