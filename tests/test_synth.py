"""Seeded input generator: hash restatement, determinism, distribution, paging helpers."""
import numpy as np
import torch

from paper_2605_06206_b200 import synth


def test_hash_matches_python_restatement():
    idx = torch.tensor([0, 1, 2, 12345, 2**31 + 7, 2**40 + 3], dtype=torch.int64)
    for seed, tid in ((0, 1), (3, 20), (5, 1009)):
        got = synth.hash16(seed, tid, idx).tolist()
        want = [synth.hash16_scalar(seed, tid, int(i)) for i in idx]
        assert got == want
        assert all(0 <= g < 65536 for g in got)


def test_normal_is_deterministic_chunk_independent_and_gaussian():
    a = synth.normal_bf16(7, 20, (1000, 64))
    b = synth.normal_bf16(7, 20, (1000, 64), chunk=777)
    assert torch.equal(a, b)
    tail = synth.normal_bf16(7, 20, (500, 64), start=500 * 64)
    assert torch.equal(a[500:], tail)
    c = synth.normal_bf16(8, 20, (1000, 64))
    assert not torch.equal(a, c)
    f = a.float()
    assert abs(float(f.mean())) < 0.02 and abs(float(f.std()) - 1.0) < 0.02
    g = synth.normal_bf16(7, 1, (4096,), 0.02, 1.0).float()
    assert abs(float(g.mean()) - 1.0) < 5e-3 and abs(float(g.std()) - 0.02) < 5e-3


def test_workloads_and_paging_roundtrip():
    s, info = synth.workload(3)
    assert len(info["context_lens"]) == 64
    assert min(info["context_lens"]) >= 4096 and max(info["context_lens"]) <= 16384
    s1, i1 = synth.workload(1)
    ctx, ql = [70, 0, 129], [1, 5, 3]
    kv = synth.make_paged_cache(s1, 11, ctx, ql)
    used = []
    for b in range(3):
        n = (ctx[b] + ql[b] + 63) // 64
        used += kv.block_table[b, :n].tolist()
    assert sorted(used) == list(range(kv.k_pages.shape[0]))       # every page used exactly once
    k, v = synth.gather_logical_cache(kv, 2, 129, 64)
    assert k.shape == (129, s1.n_kv_heads, s1.head_dim)
    page, off = int(kv.block_table[2, 2]), 0                      # logical position 128
    assert torch.equal(k[128], kv.k_pages[page, :, off, :])
    p = synth.permutation(1, 42, 100)
    assert sorted(p.tolist()) == list(range(100))


def test_zipf_bias_shape_and_dead_experts():
    s, _ = synth.workload(4)
    b = synth.zipf_router_bias(s, 4, 1.0, 1.2, dead_per_cluster=2)
    assert b.shape == (s.n_experts,)
    per = b.view(s.n_clusters, s.experts_per_cluster)
    assert int((per < -1e29).sum()) == 2 * s.n_clusters
    live = per[per > -1e29]
    assert float(live.max()) < 0.0
