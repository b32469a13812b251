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


def build_client(out_dir, name="five_calls"):
    exe = os.path.join(str(out_dir), name)
    cmd = ["gcc", "-std=c99", "-Wall", "-Werror", "-O1", os.path.join(HERE, "c_client", name + ".c"),
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


def test_plain_c_client_runs_the_turn_engine(tmp_path):
    """tests/c_client/turn_calls.c: three turns through eakv_turn_begin / eakv_turn_end, the third
    one restored from the host tier inside the library; the view it prints is what the paper's
    definitions give for those prompts, and the new block's key is the oracle's."""
    require_gpu()
    exe = build_client(tmp_path, "turn_calls")
    run = subprocess.run([exe], capture_output=True, text=True, timeout=300)
    assert run.returncode == 0, run.stdout + run.stderr
    lines = dict(l.split(" ", 1) for l in run.stdout.strip().splitlines())
    # 6 blocks + 4 tokens, nothing cached; then 8 other blocks fill the 8-block GPU tier; then the
    # first prompt with 7 full blocks: 6 from the host, one new
    assert lines["turn1"] == "blocks=6 G=0 H=0 restore=0..0 fresh=100 fill=6 store=6 tail=1"
    assert lines["turn2"] == "blocks=8 G=0 H=0 restore=0..0 fresh=128 fill=8 store=8 tail=0"
    assert lines["turn3"] == "blocks=7 G=0 H=6 restore=0..6 fresh=16 fill=1 store=1 tail=0"
    assert lines["restored"] == "ok"
    tokens = [(i * 2246822519 % (1 << 32)) % 40000 for i in range(7 * 16)]
    assert int(lines["key7"], 16) == int(ohash.hash_blocks(tokens, 16)[6])
