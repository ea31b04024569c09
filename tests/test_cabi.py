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


def test_split_k_partial_scores_fit_their_buffer_at_every_call_size(lib):
    """The fp32 score kernels write [k_splits][n_tokens][E] partial scores into a workspace buffer whose size is fixed
    when the handle is created: for every call size up to the largest that splits, on the five workloads' layer
    shapes (and the widest layer the configuration rules allow) and several max_tokens, what a call writes must fit.
    Without the clamp on the number of splits this fails (e.g. E = 128, d = 4096, 1025..1152 tokens: 16 splits)."""
    from paper_2605_06206_b200 import synth
    shapes = [(synth.workload(i)[0].hidden, synth.workload(i)[0].n_experts) for i in range(1, 6)]
    shapes += [(4096, 128), (2048, 1024), (8192, 1024), (128, 1)]
    worst = 0.0
    for d, E in shapes:
        for max_tokens in (1, 64, 300, 2047, 8192, 16384, 32768):
            cap = lib.foe_route_partial_capacity(max_tokens, 64, E)
            assert cap >= max(max_tokens, 64) * E
            for n in range(1, min(max_tokens, 2047) + 1):
                wrote = lib.foe_route_partial_floats(d, E, n, 148, cap)
                assert n * E <= wrote <= cap, (d, E, max_tokens, n, wrote, cap)
                worst = max(worst, wrote / cap)
    assert worst > 0.5          # the sweep does reach cases where the clamp is what keeps the call inside
    assert lib.foe_route_partial_floats(2048, 64, 0, 148, 1 << 21) == 0
    # the tensor-core score kernel (2048 tokens and more) writes one slice
    assert lib.foe_route_partial_floats(2048, 64, 16384, 148, 1 << 21) == 16384 * 64


def test_product_path_fails_loudly_without_a_gpu():
    import torch
    from paper_2605_06206_b200 import binding, synth
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    shape, _ = synth.workload(1)
    with pytest.raises(RuntimeError):
        binding.FoeLayer(shape, {}, 8, 1, 64)
