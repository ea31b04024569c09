"""Host-side checks that need no GPU: the C-ABI library builds, loads and exports what include/foe.h declares,
and its pure host paths (status strings, argument validation before any device work) behave."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    import __graft_entry__ as g
    g.build()
    from paper_2605_06206_b200 import binding
    return binding.load_library()


def test_every_declared_symbol_is_exported(lib):
    from paper_2605_06206_b200 import binding
    hdr = open(os.path.join(ROOT, "include", "foe.h")).read()
    declared = set(re.findall(r"\b(foe_[a-z_]+)\s*\(", hdr))
    assert declared, "no declarations found"
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    seen = set()
    for code in range(0, -9, -1):
        s = lib.foe_status_string(code).decode()
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 9
    assert lib.foe_status_string(5).decode() == "unknown status"


def test_struct_layouts_match_header():
    from paper_2605_06206_b200 import binding
    assert ctypes.sizeof(binding.FoeConfig) == 16 * 4
    assert ctypes.sizeof(binding.FoeWeights) == 11 * 8
    assert ctypes.sizeof(binding.FoeKvCache) == 5 * 8 + 5 * 4 + 4     # 4 bytes of tail padding
    assert ctypes.sizeof(binding.FoeAux) == 8 + 11 * 8


def test_null_and_config_errors_need_no_device(lib):
    from paper_2605_06206_b200 import binding
    h = ctypes.c_void_p()
    assert lib.foe_layer_create(None, None, ctypes.byref(h)) == -1
    cfg = binding.FoeConfig(256, 8, 4, 4, 32, 8, 2, 128, 64, 8, 1, 64, 1e4, 1e-6, 0, 0)   # head_dim 32: invalid
    w = binding.FoeWeights()
    assert lib.foe_layer_create(ctypes.byref(cfg), ctypes.byref(w), ctypes.byref(h)) == -2
    cfg.head_dim = 64
    cfg.top_k_per_cluster = 9                                                              # k_c > E_c
    assert lib.foe_layer_create(ctypes.byref(cfg), ctypes.byref(w), ctypes.byref(h)) == -2
    cfg.top_k_per_cluster = 2
    assert lib.foe_layer_create(ctypes.byref(cfg), ctypes.byref(w), ctypes.byref(h)) == -1  # weights are NULL
    assert lib.foe_layer_destroy(None) == 0
    assert lib.foe_prefill(None, None, None, None, None) == -1
    assert lib.foe_last_launch_count(None) == 0
    assert lib.foe_num_stages() == 9 and lib.foe_stage_name(6).decode() == "expert_gemm1_swiglu"


def test_product_path_fails_loudly_without_a_gpu():
    import torch
    from paper_2605_06206_b200 import binding, synth
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    shape, _ = synth.workload(1)
    with pytest.raises(RuntimeError):
        binding.FoeLayer(shape, {}, 8, 1, 64)
