"""The C boundary from a plain C program: tests/c_client/five_calls.c is compiled with gcc against
include/eakv.h and the in-tree library, runs one agent turn with the five calls (no Python and no
torch in that process), and its printed results are compared with the CPU oracle."""
import os
import subprocess

import numpy as np
import pytest

from oracle import hash as ohash

from gpu_util import require_gpu

pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
PKG = os.path.join(ROOT, "paper_2609_33762_b200")
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")


def build_client(out_dir):
    exe = os.path.join(str(out_dir), "five_calls")
    cmd = ["gcc", "-std=c99", "-Wall", "-Werror", "-O1", os.path.join(HERE, "c_client", "five_calls.c"),
           "-I" + os.path.join(ROOT, "include"), "-I" + os.path.join(CUDA, "include"),
           "-L" + PKG, "-leakv", "-L" + os.path.join(CUDA, "lib64"), "-lcudart",
           "-Wl,-rpath," + PKG, "-Wl,-rpath," + os.path.join(CUDA, "lib64"), "-o", exe]
    subprocess.run(cmd, check=True, capture_output=True, text=True)
    return exe


def test_plain_c_client_runs_the_five_calls(tmp_path):
    require_gpu()
    exe = build_client(tmp_path)
    run = subprocess.run([exe], capture_output=True, text=True, timeout=300)
    assert run.returncode == 0, run.stdout + run.stderr
    lines = dict(l.split(" ", 1) for l in run.stdout.strip().splitlines())
    # the client's prompt, restated here: 100 tokens, block 16 -> 6 full blocks
    tokens = [(i * 2654435761 % (1 << 32)) % 50000 for i in range(100)]
    want = ohash.hash_blocks(tokens, 16)
    got = [int(x, 16) for x in lines["keys"].split()]
    assert got == [int(k) for k in want]
    assert lines["match1"] == "0 0"
    assert lines["step"] == "admitted=6 slots=0,1,2,3,4,5"       # empty tier: slots in ascending order
    assert lines["match2"] == "0 6"                              # every block is now a host hit
    assert lines["roundtrip"] == "ok" and lines["untouched"] == "ok"
    assert lines["stats"] == "stored=6 loaded=6"
