"""The C-ABI library loads without a GPU, exports every symbol include/eakv.h declares,
and refuses to create a context when no CUDA device is present (no CPU fallback)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_33762_b200 import build, eakv
    build.build()
    return eakv.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "eakv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(eakv_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2609_33762_b200 import eakv
    names = declared_symbols()
    assert len(names) >= 18
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(eakv.EXPORTS) == names


def test_config_defaults_and_layout(lib):
    from paper_2609_33762_b200 import eakv
    cfg = eakv.Config()
    assert lib.eakv_config_init(C.byref(cfg)) == 0
    # controller defaults of the paper's parameter table
    assert (cfg.theta_percent, cfg.window_ms, cfg.len_window, cfg.kappa_blocks) == (95, 60000, 256, 8)
    assert cfg.policy == eakv.POLICY_WRITE_ALL and cfg.elem_bytes == 2
    assert cfg.link_strategy == eakv.LINK_STAGED and cfg.copy_path == eakv.COPY_BULK
    assert lib.eakv_config_init(None) == eakv.E_INVAL


def test_binding_structs_have_the_layout_of_the_header(tmp_path):
    """include/eakv.h compiles as plain C, and the ctypes mirrors of its structs have the same
    sizes and field offsets as a C compiler gives them."""
    import subprocess
    from paper_2609_33762_b200 import eakv
    src = tmp_path / "layout.c"
    src.write_text(
        '#include <stdio.h>\n#include <stddef.h>\n#include "eakv.h"\n'
        'int main(void) {\n'
        '  printf("%zu %zu %zu %zu\\n", sizeof(eakv_config), sizeof(eakv_stats), sizeof(eakv_step_info), sizeof(eakv_turn_view));\n'
        '  printf("%zu %zu %zu %zu %zu\\n", offsetof(eakv_config, kv_base), offsetof(eakv_config, window_ms),\n'
        '         offsetof(eakv_config, tier_memory), offsetof(eakv_config, telemetry_period_ms),\n'
        '         offsetof(eakv_turn_view, keys));\n'
        '  return 0;\n}\n')
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)],
                   check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True, check=True).stdout.split()
    sizes, offsets = [int(x) for x in out[:4]], [int(x) for x in out[4:]]
    assert sizes == [C.sizeof(eakv.Config), C.sizeof(eakv.Stats), C.sizeof(eakv.StepInfo), C.sizeof(eakv.TurnView)]
    assert offsets == [eakv.Config.kv_base.offset, eakv.Config.window_ms.offset, eakv.Config.tier_memory.offset,
                       eakv.Config.telemetry_period_ms.offset, eakv.TurnView.keys.offset]


def test_strerror(lib):
    assert lib.eakv_strerror(0) == b"ok"
    for code in range(-7, 0):
        assert lib.eakv_strerror(code) not in (b"ok", b"unknown error")
    assert lib.eakv_strerror(-99) == b"unknown error"


def test_create_rejects_bad_config_before_touching_cuda(lib):
    from paper_2609_33762_b200 import eakv
    cfg = eakv.Config()
    lib.eakv_config_init(C.byref(cfg))
    h = C.c_void_p()
    assert lib.eakv_create(C.byref(cfg), C.byref(h)) == eakv.E_INVAL      # empty shape
    assert lib.eakv_create(None, C.byref(h)) == eakv.E_INVAL
    assert not h.value
    # sizes beyond 32-bit ids are refused, also where host_blocks * chunk_blocks would wrap around
    for hb, cb in ((1 << 31, 1), (1 << 62, 4), ((1 << 31) // 64 + 1, 64)):
        cfg = eakv.Config()
        lib.eakv_config_init(C.byref(cfg))
        cfg.num_layers, cfg.kv_heads, cfg.head_dim, cfg.block_size = 1, 1, 8, 16
        cfg.gpu_blocks, cfg.host_blocks, cfg.chunk_blocks, cfg.control_plane_only = 4, hb, cb, 1
        assert lib.eakv_create(C.byref(cfg), C.byref(h)) == eakv.E_INVAL and not h.value


def test_no_cpu_fallback_without_a_gpu(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2609_33762_b200 import eakv
    ptrs = [16 * (i + 1) for i in range(8)]
    with pytest.raises(eakv.EakvError) as ei:
        eakv.Context(num_layers=4, kv_heads=2, head_dim=64, block_size=16, gpu_blocks=8,
                     host_blocks=8, kv_base=ptrs)
    assert ei.value.code == eakv.E_CUDA


def test_a_plain_c_client_compiles_and_links(tmp_path):
    """The header is a C99 header and the library resolves every call a C client makes
    (tests/c_client/five_calls.c and turn_calls.c; they are run on a GPU by tests/test_gpu_c_client.py)."""
    import shutil
    import subprocess
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    if shutil.which("gcc") is None or not os.path.exists(os.path.join(cuda, "include", "cuda_runtime_api.h")):
        pytest.skip("gcc or the CUDA headers are missing")
    here = os.path.dirname(os.path.abspath(__file__))
    root = os.path.dirname(here)
    pkg = os.path.join(root, "paper_2609_33762_b200")
    for name in ("five_calls", "turn_calls"):
        exe = os.path.join(str(tmp_path), name)
        cmd = ["gcc", "-std=c99", "-Wall", "-Werror", "-O1", os.path.join(here, "c_client", name + ".c"),
               "-I" + os.path.join(root, "include"), "-I" + os.path.join(cuda, "include"),
               "-L" + pkg, "-leakv", "-L" + os.path.join(cuda, "lib64"), "-lcudart", "-Wl,-rpath," + pkg, "-o", exe]
        run = subprocess.run(cmd, capture_output=True, text=True)
        assert run.returncode == 0, run.stderr
        assert os.path.exists(exe)
