"""Host side of the cluster-per-GPU group, without a GPU: the library exports what include/foe_shard.h declares,
the description checks and buffer sizes, the per-cluster slicing of shapes and weights, and the handle exchange
that forms a group -- run as two gloo ranks on CPU with stand-ins for the device buffers."""
import ctypes
import json
import os
import re
import socket
import subprocess
import sys
import textwrap

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    import __graft_entry__ as g
    g.build()
    from paper_2605_06206_b200 import shard
    return shard.load_library()


def test_every_symbol_of_the_shard_header_is_exported(lib):
    from paper_2605_06206_b200 import shard
    hdr = open(os.path.join(ROOT, "include", "foe_shard.h")).read()
    declared = set(re.findall(r"\b(foe_shard_[a-z_]+)\s*\(", hdr))
    assert declared == set(shard.SHARD_EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_description_checks_and_buffer_size(lib):
    from paper_2605_06206_b200 import shard
    assert ctypes.sizeof(shard.FoeShardConfig) == 20
    ok = shard.FoeShardConfig(2, 8, 4096, 16384, 0)
    # header (8 gather counters, then slot counters [2 parities][8 sources][64 blocks of 256 rows], rounded up to 1 KB)
    # + slots [2][8][16384][512] + gather [2][16384][4096], bf16
    header = -(-(128 + 2 * 8 * (16384 // 256) * 4) // 1024) * 1024
    assert header == 5120
    assert lib.foe_shard_buffer_bytes(ctypes.byref(ok)) == header + 2 * (2 * 16384 * 4096 * 2)
    for bad in [shard.FoeShardConfig(8, 8, 4096, 16, 0),      # rank out of range
                shard.FoeShardConfig(0, 9, 4608, 16, 0),      # more than 8 ranks
                shard.FoeShardConfig(0, 8, 4096 + 128, 16, 0),  # hidden not a multiple of 32 * ranks
                shard.FoeShardConfig(0, 4, 256, 0, 0),        # no tokens
                shard.FoeShardConfig(0, 4, 256, 16, -1)]:
        assert lib.foe_shard_buffer_bytes(ctypes.byref(bad)) == 0
        p = ctypes.c_void_p()
        assert lib.foe_shard_buffer_alloc(ctypes.byref(bad), ctypes.byref(p)) == -2
        tbl = (ctypes.c_void_p * 8)(*([1] * 8))
        assert lib.foe_shard_create(ctypes.byref(bad), tbl, ctypes.byref(p)) == -2
    h = ctypes.c_void_p()
    assert lib.foe_shard_create(None, None, ctypes.byref(h)) == -1
    tbl = (ctypes.c_void_p * 8)(*([1] * 7 + [None]))
    assert lib.foe_shard_create(ctypes.byref(ok), tbl, ctypes.byref(h)) == -1        # a missing buffer
    assert lib.foe_shard_destroy(None) == 0 and lib.foe_shard_buffer_free(None) == 0
    assert lib.foe_shard_push(None, None, 0, 1.0, None) == -1
    assert lib.foe_shard_attend(None, None, None, None, 0, None) == -1


def test_cluster_slices_of_shape_and_weights():
    from paper_2605_06206_b200 import shard, synth
    s = synth.LayerShape(256, 8, 4, 4, 64, 8, 2, 128, position="first", sync="sum")
    W = synth.make_weights(s, 3, "cpu")
    W["router_b"] = torch.arange(s.n_experts, dtype=torch.float32)
    for h in range(4):
        sh = shard.cluster_shape(s, h)
        assert (sh.n_clusters, sh.n_q_heads, sh.n_kv_heads, sh.experts_per_cluster, sh.top_k_per_cluster) == (1, 2, 1, 8, 2)
        assert (sh.position, sh.sync, sh.hidden, sh.head_dim) == ("first", "sum", 256, 64)
        w = shard.cluster_weights(s, W, h)
        assert all(t.is_contiguous() for t in w.values())
        assert w["wq"].shape == (1, 256, 128) and torch.equal(w["wq"][0], W["wq"][h])
        assert w["wk"].shape == (1, 256, 64) and torch.equal(w["wv"][0], W["wv"][h])
        assert w["wo"].shape == (128, 256) and torch.equal(w["wo"], W["wo"][h * 128:(h + 1) * 128])
        assert torch.equal(w["w_down"], W["w_down"][h * 8:(h + 1) * 8]) and w["w_gate"].shape == (8, 256, 128)
        assert torch.equal(w["router_w"], W["router_w"][h * 8:(h + 1) * 8])
        assert w["router_b"].tolist() == list(range(h * 8, h * 8 + 8))
        assert w["attn_norm_g"] is W["attn_norm_g"] and w["ffn_norm_g"] is W["ffn_norm_g"]
        # views, not copies
        assert w["w_up"].data_ptr() == W["w_up"][h * 8].data_ptr()
    with pytest.raises(ValueError):                 # 1 query head of width 64 per cluster: no 128-wide O-proj block
        shard.cluster_shape(synth.LayerShape(256, 4, 4, 4, 64, 8, 2, 128), 0)
    cfg = shard.exchange_config(s, 3, 77, 5)
    assert (cfg.rank, cfg.n_ranks, cfg.hidden, cfg.max_tokens, cfg.wait_limit_ms) == (3, 4, 256, 77, 5)


CHILD = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    import torch, torch.distributed as dist
    from paper_2605_06206_b200 import shard, synth
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mode = sys.argv[1]

    class FakeBuffer:                       # stands in for device memory and its IPC handle
        def __init__(self, cfg, imported_from=None):
            if imported_from is None:
                self.ptr = 0x1000 * (cfg.rank + 1)
                self.owner = cfg.rank
            else:
                assert imported_from[1:] == bytes(63)
                self.owner = imported_from[0]
                self.ptr = 0x900000 + 0x1000 * (self.owner + 1)       # a mapping of the owner's buffer
            self.imported = imported_from is not None
        def export(self):
            return bytes([self.owner]) + bytes(63)

    class FakeExchange:
        def __init__(self, cfg, ptrs):
            self.cfg, self.ptrs = cfg, list(ptrs)

    shape = synth.LayerShape(256, 4, 2, world, 64, 8, 2, 128)
    max_tokens = 64 if (mode == "ok" or rank == 0) else 65        # "mismatch": rank 1 sizes its buffers differently
    try:
        ex, bufs = shard.connect(shape, max_tokens, make_buffer=FakeBuffer, make_exchange=FakeExchange)
        print(json.dumps(dict(rank=rank, ptrs=ex.ptrs, owners=[b.owner for b in bufs], imported=[b.imported for b in bufs],
                              cfg=[ex.cfg.rank, ex.cfg.n_ranks, ex.cfg.hidden, ex.cfg.max_tokens])))
    except RuntimeError as e:
        print(json.dumps(dict(rank=rank, error=str(e))))
    dist.destroy_process_group()
""") % ROOT


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _run_two(mode):
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", LOCAL_RANK=str(r), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD, mode], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        o, e = p.communicate(timeout=180)
        assert p.returncode == 0, e
        outs.append(json.loads(o.strip().splitlines()[-1]))
    return sorted(outs, key=lambda d: d["rank"])


def test_two_ranks_form_a_group_over_gloo():
    a, b = _run_two("ok")
    # entry r of every table is rank r's buffer: the rank's own allocation at its own index, a mapping elsewhere
    assert a["ptrs"] == [0x1000, 0x900000 + 0x2000] and b["ptrs"] == [0x900000 + 0x1000, 0x2000]
    assert a["owners"] == [0, 1] and b["owners"] == [0, 1]
    assert a["imported"] == [False, True] and b["imported"] == [True, False]
    assert a["cfg"] == [0, 2, 256, 64] and b["cfg"] == [1, 2, 256, 64]


def test_ranks_that_disagree_on_the_exchange_description_fail_on_both_sides():
    a, b = _run_two("mismatch")
    assert "describes the exchange" in a["error"] and "describes the exchange" in b["error"]


def test_gather_handles_rejects_duplicates_and_wrong_counts():
    from paper_2605_06206_b200 import shard
    h = bytes(range(64))

    def echo_twice(t):
        return [t.clone(), t.clone()]                 # both "ranks" claim to be rank 0

    with pytest.raises(RuntimeError, match="duplicate"):
        shard.gather_handles(h, (2, 256, 64), 0, 2, echo_twice)
    with pytest.raises(RuntimeError, match="expected 2"):
        shard.gather_handles(h, (2, 256, 64), 0, 2, lambda t: [t])
    assert shard.gather_handles(h, (1, 256, 64), 0, 1, lambda t: [t]) == [h]
