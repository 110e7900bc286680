"""The C ABI used from plain C: a small driver program (tests/c_abi/ef_c_driver.c) linked
against libef.so runs the hand-worked case of Algorithm 4 on the GPU; its printed outputs must
equal the pencil-and-paper table in tests/golden/alg4_hand_case_e1.txt exactly."""
import os
import subprocess

import pytest

from paper_1905_10936_b200 import binding as ef
from paper_1905_10936_b200 import build as efbuild
from test_oracle_pins import parse_hand_case

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
SRC = os.path.join(HERE, "c_abi", "ef_c_driver.c")


def _build(tmp_path):
    efbuild.build_library()            # no-op when libef.so is up to date
    exe = str(tmp_path / "ef_c_driver")
    nvcc = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    libdir = os.path.dirname(ef.LIB_PATH)
    subprocess.run([nvcc, "-O1", "-o", exe, SRC, "-I", os.path.join(ROOT, "include"),
                    "-L", libdir, "-lef", "-Xlinker", f"-rpath={libdir}"], check=True)
    return exe


def test_driver_compiles_against_the_header(tmp_path):
    """No GPU needed: the header is valid C and the library links from C."""
    assert os.path.exists(_build(tmp_path))


@pytest.mark.gpu
def test_hand_case_through_the_c_abi_from_c(tmp_path):
    cfg, grads, rows = parse_hand_case(os.path.join(HERE, "golden", "alg4_hand_case_e1.txt"))
    exe = _build(tmp_path)
    d, M, steps, off = cfg["d"], cfg["M"], cfg["steps"], cfg["offsets"]
    text = [f"{d} {len(off) - 1}", " ".join(map(str, off)), f"{M} {cfg['mu']} {cfg['eta']} {steps}"]
    for t in range(steps):
        for i in range(M):
            text.append(" ".join(repr(v) for v in grads[(t, i)]))
    out = subprocess.run([exe], input="\n".join(text) + "\n", capture_output=True, text=True, check=True)
    lines = [l for l in out.stdout.splitlines() if l]
    assert lines[-1] == f"T {steps}"
    parsed = {}
    for l in lines[:-1]:
        head, *cols = [c.strip() for c in l.split(":")]
        parsed[tuple(head.split())] = [[float(v) for v in c.split()] for c in cols]
    for kind, head, cols in rows:
        if kind == "worker":
            t, i = head
            m, p, scales, bits, words, resid = cols
            got = parsed[("W", str(t), str(i))]
            assert got[0] == words and got[1] == scales and got[2] == resid
        else:
            (t,) = head
            p, scales, bits, words, resid, x = cols
            got = parsed[("S", str(t))]
            assert got[0] == words and got[1] == scales and got[2] == resid and got[3] == x
