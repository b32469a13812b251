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
    assert C.sizeof(eakv.Config) == 176 and C.sizeof(eakv.Stats) == 128
    assert lib.eakv_config_init(None) == eakv.E_INVAL


def test_strerror(lib):
    assert lib.eakv_strerror(0) == b"ok"
    for code in range(-6, 0):
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
