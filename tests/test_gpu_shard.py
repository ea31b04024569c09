"""One cluster per rank (include/foe_shard.h), all ranks emulated on one device: H layer handles built from the
per-cluster slices of the weights, H exchange buffers, the three phases issued rank by rank.  The group's result is
checked against the same oracle as the one-device block (which knows nothing about ranks), the exchange alone
against its rounding model bit for bit."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import adapter
from paper_2605_06206_b200 import binding, shard, synth

from parity import assert_close, compare_with_oracle, scaled_weights

pytestmark = pytest.mark.gpu


def run_group(shape, seed, q_lens, ctx_lens, decode=False, wscale=1.0, also_one_device=False):
    dev = "cuda"
    H = shape.n_clusters
    W = scaled_weights(shape, seed, dev, wscale)
    S = sum(q_lens)
    x = synth.make_x(shape, seed, S, dev)
    kv = synth.make_paged_cache(shape, seed, ctx_lens, q_lens, dev)
    cache = adapter.logical_cache(kv.k_pages, kv.v_pages, kv.block_table, ctx_lens, 64)
    kvs = [shard.split_cache(shape, kv, h) for h in range(H)]
    max_ctx = max(c + q for c, q in zip(ctx_lens, q_lens))
    group = shard.LocalGroup(shape, max_tokens=S)
    layers = group.make_layer(shape, W, S, len(q_lens), max_ctx)
    out = group.forward(layers, x, kvs, decode)
    assert group.poll_status() == 0
    assert all(l.layer.poll_status() == 0 for l in layers)
    auxs = [l.layer.aux() for l in layers]
    for a in auxs[1:]:                       # every rank holds the same synced residual and expert input
        assert torch.equal(a["r_full"], auxs[0]["r_full"]) and torch.equal(a["u"], auxs[0]["u"])
    Ec = shape.experts_per_cluster
    aux = dict(q=torch.cat([a["q"] for a in auxs], 1), attn_o=torch.cat([a["attn_o"] for a in auxs], 1),
               r_full=auxs[0]["r_full"], u=auxs[0]["u"],
               topk_idx=torch.cat([a["topk_idx"] + h * Ec for h, a in enumerate(auxs)], 1),
               topk_w=torch.cat([a["topk_w"] for a in auxs], 1))
    kv_all = dataclasses.replace(kv, k_pages=torch.cat([k.k_pages for k in kvs], 1), v_pages=torch.cat([k.v_pages for k in kvs], 1))
    res = compare_with_oracle(shape, W, x, q_lens, ctx_lens, cache, kv_all, out, aux, stress=(wscale != 1.0),
                              cluster_maps=auxs)
    launches = [l.layer.last_launch_count() for l in layers]
    for l in layers:
        l.close()
    group.close()
    if also_one_device:
        kv1 = synth.make_paged_cache(shape, seed, ctx_lens, q_lens, dev)
        one = binding.FoeLayer(shape, W, S, len(q_lens), max_ctx)
        ref = one.decode(x, kv1) if decode else one.prefill(x, kv1)
        idx_one = one.aux()["topk_idx"]
        one.close()
        same = (torch.sort(idx_one, -1).values == torch.sort(aux["topk_idx"], -1).values).all(-1).all(-1)   # tokens routed alike
        assert same.float().mean() > 0.7            # (bf16 partials move a few near-ties)
        a = out[:, same] if shape.grouped_output else out[same]
        b = ref[:, same] if shape.grouped_output else ref[same]
        assert_close(a.float().cpu().numpy(), b.float().cpu().numpy(), "group against the one-device block", 2e-2, 4e-3)
    res["launches"] = launches
    return res


def shape_small(**kw):
    base = dict(hidden=256, n_q_heads=8, n_kv_heads=4, n_clusters=4, head_dim=64, experts_per_cluster=8,
                top_k_per_cluster=2, ffn_inter=128)
    base.update(kw)
    return synth.LayerShape(**base)


@pytest.mark.parametrize("position,sync", [("middle", "mean"), ("middle", "sum"), ("first", "mean"), ("last", "mean"),
                                            ("single", "mean")])
def test_group_prefill_positions_and_sync_modes(position, sync):
    run_group(shape_small(position=position, sync=sync), 11, [130, 203], [0, 64], also_one_device=(position == "middle"))


@pytest.mark.parametrize("position", ["middle", "first", "last"])
def test_group_decode(position):
    res = run_group(shape_small(position=position), 12, [1] * 9, [5, 64, 127, 128, 300, 1, 77, 640, 63], decode=True,
                    also_one_device=(position == "middle"))
    # QKV, attention, O-proj, push | gather | two route launches, two expert GEMMs, combine
    assert all(n == 10 for n in res["launches"])


def test_group_decode_pushes_from_the_projection_epilogue_when_the_owner_span_allows():
    """hidden 1024 over 4 ranks: 256 columns per owner, a whole number of the decode O-projection's 128-row weight slabs,
    so the projection stores its result straight into the owners' slots (no push launch: nine launches per rank), over
    several row blocks' worth of exchanges of different sizes (a prefill first, then decode steps on what it cached)."""
    s = synth.LayerShape(1024, 8, 4, 4, 128, 4, 2, 128)
    res = run_group(s, 17, [1] * 70, [3 + 7 * i for i in range(70)], decode=True, also_one_device=True)
    assert all(n == 9 for n in res["launches"])
    run_group(s, 18, [300, 41], [0, 0])
    res = run_group(s, 19, [1] * 3, [64, 5, 600], decode=True)
    assert all(n == 9 for n in res["launches"])


def test_group_several_tiles_ragged_tail_head_dim_128():
    # 8 clusters x (2 query heads, 1 KV head) of width 128, hidden 2048: 256 columns per owner, rows spanning three
    # 256-row tile pairs with a ragged tail
    s = synth.LayerShape(2048, 16, 8, 8, 128, 8, 2, 256)
    run_group(s, 13, [517, 100], [0, 0], also_one_device=True)


def test_group_owner_span_not_a_multiple_of_the_tile():
    # hidden 768 over 8 ranks: 96 columns per owner, so one 256-column accumulator tile feeds three or four owners
    s = synth.LayerShape(768, 16, 8, 8, 64, 4, 1, 128)
    run_group(s, 14, [300], [0])
    run_group(s, 15, [1] * 5, [10, 200, 64, 65, 1], decode=True)


def test_group_with_scaled_weights():
    run_group(shape_small(), 16, [257], [0], wscale=4.0)


def exchange_model(tensors, scale):
    """What the exchange computes, rounding by rounding: bf16(scale * t_h), fp32 sum in rank order, bf16."""
    acc = torch.zeros_like(tensors[0], dtype=torch.float32)
    for t in tensors:
        acc = acc + (t.float() * scale).to(torch.bfloat16).float()
    return acc.to(torch.bfloat16)


@pytest.mark.parametrize("H,d", [(4, 256), (8, 768), (1, 128), (3, 96 * 3)])
def test_exchange_is_bit_exact_against_its_rounding_model_over_many_rounds(H, d):
    s = synth.LayerShape(d, H, H, H, 64, 4, 1, 128)
    group = shard.LocalGroup(s, max_tokens=300)
    g = torch.Generator(device="cuda").manual_seed(5)
    for n, scale in [(77, 0.25), (300, 1.0), (1, 1.0 / H), (16, 3.0), (299, 0.5), (0, 1.0), (33, 1.0)]:   # both buffer halves, ragged blocks
        ts = [torch.randn(n, d, device="cuda", generator=g).to(torch.bfloat16) for _ in range(H)]
        got = group.allreduce(ts, scale)
        want = exchange_model(ts, scale)
        for r in got:
            assert torch.equal(r, want)
    assert group.poll_status() == 0
    group.close()


def test_exchange_rejects_calls_out_of_order_and_oversized_tensors():
    s = shape_small()
    group = shard.LocalGroup(s, max_tokens=32)
    ex = group.exchanges[0]
    t = torch.zeros(8, s.hidden, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.FoeError) as e:
        ex.reduce()
    assert e.value.code == -4
    with pytest.raises(binding.FoeError) as e:
        ex.push(torch.zeros(33, s.hidden, dtype=torch.bfloat16, device="cuda"))
    assert e.value.code == -3
    group.allreduce([t] * 4)
    for x in group.exchanges:
        x.push(t)
    with pytest.raises(binding.FoeError) as e:
        ex.push(t)                                     # the previous exchange is still open
    assert e.value.code == -4
    for x in group.exchanges:
        x.reduce()
    for x in group.exchanges:
        x.gather()
    assert group.poll_status() == 0
    group.close()


def test_a_wait_that_nothing_satisfies_runs_out_and_is_reported():
    # rank 0 pushes and reduces, the other ranks never push: the owner's wait is bounded (20 ms here), the kernel
    # returns, the status word says so and the device stays usable
    s = shape_small()
    group = shard.LocalGroup(s, max_tokens=16, wait_limit_ms=20)
    ex = group.exchanges[0]
    ex.push(torch.ones(16, s.hidden, dtype=torch.bfloat16, device="cuda"))
    ex.reduce()
    assert ex.poll_status() == -7
    assert ex.poll_status() == 0                        # reading resets the word
    group.close()
    y = torch.ones(4, device="cuda") * 2
    assert float(y.sum()) == 8.0


def test_group_stack_prefill_then_decode_on_per_cluster_caches():
    """Three layers (first, middle, last), a prefill and two decode steps: every layer runs once on one device and once
    as a group of ranks with per-cluster caches, both fed the one-device path's input to that layer.  The decode steps
    read what the group's own prefill wrote into the per-cluster pages."""
    base, L, q_lens, steps = shape_small(), 3, [70, 130], 2
    H, Ec, S, n_seqs = base.n_clusters, base.experts_per_cluster, sum(q_lens), len(q_lens)
    max_ctx = max(q_lens) + steps
    group = shard.LocalGroup(base, max_tokens=S)
    ones, groups, kv_one, kv_grp = [], [], [], []
    total = [q + steps for q in q_lens]
    for l in range(L):
        sh = dataclasses.replace(base, position=("first", "middle", "last")[l])
        W = scaled_weights(sh, 21, "cuda", layer=l + 1)
        ones.append(binding.FoeLayer(sh, W, S, n_seqs, max_ctx))
        groups.append(group.make_layer(sh, W, S, n_seqs, max_ctx))
        kv = synth.make_paged_cache(base, 21, [0] * n_seqs, total, "cuda", fill_random=False)
        kv_one.append(kv)
        kv_grp.append([shard.split_cache(base, kv, h) for h in range(H)])

    def run_all(x, ctx, decode):
        ctx_t = torch.tensor(ctx, dtype=torch.int32, device="cuda")
        q_t = torch.tensor([1] * n_seqs if decode else q_lens, dtype=torch.int32, device="cuda")
        h_in = x
        for l in range(L):
            for kv in [kv_one[l]] + kv_grp[l]:
                kv.context_lens, kv.q_lens = ctx_t, q_t
            ref = ones[l].decode(h_in, kv_one[l]) if decode else ones[l].prefill(h_in, kv_one[l])
            got = group.forward(groups[l], h_in, kv_grp[l], decode)
            idx_one = ones[l].aux()["topk_idx"]
            idx_grp = torch.cat([r.layer.aux()["topk_idx"] + h * Ec for h, r in enumerate(groups[l])], 1)
            same = (torch.sort(idx_one, -1).values == torch.sort(idx_grp, -1).values).all(-1).all(-1)
            assert same.float().mean() > 0.7
            grouped = ones[l].shape.grouped_output
            a = got[:, same] if grouped else got[same]
            b = ref[:, same] if grouped else ref[same]
            assert_close(a.float().cpu().numpy(), b.float().cpu().numpy(), f"layer {l} ({'decode' if decode else 'prefill'})", 2e-2, 4e-3)
            h_in = ref
        return h_in

    run_all(synth.make_x(dataclasses.replace(base, position="first"), 21, S, "cuda"), [0] * n_seqs, False)
    for s in range(steps):
        run_all(synth.make_x(dataclasses.replace(base, position="first"), 21, n_seqs, "cuda", tid=synth.TID["x_step"] + s),
                [q + s for q in q_lens], True)
    # the per-cluster pages hold what the one-device cache holds for the cluster's KV heads
    c = base.kv_per_cluster
    for l in range(L):
        for h in range(H):
            ref_k = kv_one[l].k_pages[:, h * c:(h + 1) * c].float()
            assert_close(kv_grp[l][h].k_pages.float().cpu().numpy(), ref_k.cpu().numpy(), f"K pages, layer {l}, cluster {h}", 3e-2, 1.5e-2)
    assert group.poll_status() == 0
    for l in range(L):
        ones[l].close()
        for r in groups[l]:
            r.close()
    group.close()
