"""GPU parity tests: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs.  Small cases are compared element by element; the full-size workloads on sampled tokens."""
import numpy as np
import pytest
import torch

from oracle import adapter
from oracle import foe_oracle as orc
from paper_2605_06206_b200 import binding, synth

from parity import (assert_close, check_every_row, check_maps, check_routing, run_block_parity, scaled_weights)

pytestmark = pytest.mark.gpu


def shape_small(**kw):
    base = dict(hidden=256, n_q_heads=8, n_kv_heads=4, n_clusters=4, head_dim=64, experts_per_cluster=8,
                top_k_per_cluster=2, ffn_inter=128)
    base.update(kw)
    return synth.LayerShape(**base)


# ------------------------------------------------------------------------------------------ routing
# 2048 tokens and more take the tensor-core score kernel (workload 1: 32 experts, padded to its 64-wide tile)
@pytest.mark.parametrize("wl,n_tok,zipf", [(1, 128, False), (1, 2111, False), (2, 3000, False), (4, 2500, True), (4, 64, True)])
def test_route_bit_exact(wl, n_tok, zipf):
    shape, info = synth.workload(wl)
    dev = "cuda"
    W = synth.make_weights(shape, info["seed"], dev)
    if zipf:
        W["router_b"] = synth.zipf_router_bias(shape, info["seed"], 1.0, 1.2, dead_per_cluster=2).to(dev)
    h = synth.normal_bf16(info["seed"], 77, (n_tok, shape.hidden), 1.5, 0.0, dev)
    layer = binding.FoeLayer(shape, W, max_tokens=n_tok, max_seqs=1, max_context=64)
    idx, w = layer.route(h)
    assert layer.poll_status() == 0
    aux = layer.aux()
    layer.close()
    cfg = adapter.cfg_from_shape(shape)
    Wn = {k: adapter.to_np(W[k]) for k in ("ffn_norm_g", "router_w", "router_b")}
    rt = orc.route(cfg, Wn, adapter.to_np(h))
    idx_g, w_g = idx.cpu().numpy(), w.cpu().numpy().astype(np.float64)
    exempt = check_routing(shape, idx_g, w_g, rt["logits"], rt["idx"], rt["w"])
    assert exempt <= max(2, n_tok // 200)
    # list order: descending score inside every (token, cluster)
    lg = np.take_along_axis(rt["logits"], idx_g.reshape(n_tok, -1).astype(np.int64), 1).reshape(idx_g.shape)
    assert (np.diff(lg, axis=-1) <= 1e-5).all()
    assert np.abs(adapter.to_np(aux["logits"]) - rt["logits"]).max() <= 2e-5 * max(1.0, np.abs(rt["logits"][rt["logits"] > -1e29]).max())
    mp = check_maps(shape, aux, idx_g)
    if zipf:
        dead = adapter.to_np(W["router_b"]) < -1e29
        assert dead.sum() == 2 * shape.n_clusters and (mp["counts"][dead] == 0).all()      # guaranteed-empty experts
        live = mp["counts"][~dead]
        assert live.max() > 4 * max(1, live.min())                                          # skewed load


def test_route_bit_exact_tensor_core_scores_odd_k_blocks():
    """The tensor-core score kernel spreads the k-blocks over eight accumulators; hidden 768 gives 12 k-blocks (an
    uneven spread), 8 experts per cluster the narrowest register top-k."""
    shape = synth.LayerShape(768, 8, 8, 8, 96, 8, 1, 384)
    W = synth.make_weights(shape, 41, "cuda")
    n_tok = 2304
    h = synth.normal_bf16(41, 77, (n_tok, shape.hidden), 1.5, 0.0, "cuda")
    layer = binding.FoeLayer(shape, W, max_tokens=n_tok, max_seqs=1, max_context=64)
    idx, w = layer.route(h)
    assert layer.poll_status() == 0
    aux = layer.aux()
    layer.close()
    cfg = adapter.cfg_from_shape(shape)
    Wn = {k: adapter.to_np(W[k]) for k in ("ffn_norm_g", "router_w", "router_b")}
    rt = orc.route(cfg, Wn, adapter.to_np(h))
    exempt = check_routing(shape, idx.cpu().numpy(), w.cpu().numpy().astype(np.float64), rt["logits"], rt["idx"], rt["w"])
    assert exempt <= n_tok // 200
    assert np.abs(adapter.to_np(aux["logits"]) - rt["logits"]).max() <= 2e-5 * max(1.0, np.abs(rt["logits"]).max())
    check_maps(shape, aux, idx.cpu().numpy())


@pytest.mark.parametrize("H,Ec,kc", [(1, 100, 8), (2, 96, 4), (5, 64, 2), (2, 128, 16), (4, 24, 3)])
def test_route_tensor_core_scores_with_padded_expert_counts(H, Ec, kc):
    """The tensor-core score kernel pads the expert count to a multiple of 64 and gives a CTA 128 experts when the
    padded count is a multiple of 128, 64 otherwise: 100 -> 128 (one CTA column of 128, 28 of them padding),
    192 and 320 (columns of 64), 256 (two columns of 128), 96 -> 128."""
    shape = synth.LayerShape(512, 2 * H, H, H, 64, Ec, kc, 128)
    seed = 1500 + H * Ec
    W = dict(ffn_norm_g=synth.normal_bf16(seed, synth.TID["ffn_norm_g"], (shape.hidden,), 0.02, 1.0, "cuda"),
             router_w=synth.normal_bf16(seed, synth.TID["router_w"], (shape.n_experts, shape.hidden), 0.02, 0.0, "cuda").float())
    n_tok = 2100
    h = synth.normal_bf16(seed, 77, (n_tok, shape.hidden), 1.5, 0.0, "cuda")
    layer = binding.FoeLayer(shape, _route_only_weights(shape, W), max_tokens=n_tok, max_seqs=1, max_context=64)
    idx, w = layer.route(h)
    assert layer.poll_status() == 0
    aux = layer.aux()
    layer.close()
    cfg = adapter.cfg_from_shape(shape)
    Wn = {k: adapter.to_np(W[k]) for k in ("ffn_norm_g", "router_w")}
    Wn["router_b"] = None
    rt = orc.route(cfg, Wn, adapter.to_np(h))
    exempt = check_routing(shape, idx.cpu().numpy(), w.cpu().numpy().astype(np.float64), rt["logits"], rt["idx"], rt["w"])
    assert exempt <= max(2, n_tok // 200)
    assert np.abs(adapter.to_np(aux["logits"]) - rt["logits"]).max() <= 2e-5 * max(1.0, np.abs(rt["logits"]).max())
    check_maps(shape, aux, idx.cpu().numpy())


@pytest.mark.parametrize("wl,n_tok,max_tokens", [(5, 1088, 1088), (5, 1100, 16384), (4, 560, 8192), (4, 1152, 4096)])
def test_route_bit_exact_where_split_k_partials_would_outgrow_their_buffer(wl, n_tok, max_tokens):
    """Call sizes at which the fp32 score kernel would like 16 slices of the hidden dimension while the partial-score
    buffer of the handle holds fewer: the number of slices is reduced, the scores still agree with the oracle's."""
    shape, info = synth.workload(wl)
    W = dict(ffn_norm_g=synth.normal_bf16(info["seed"], synth.TID["ffn_norm_g"], (shape.hidden,), 0.02, 1.0, "cuda"),
             router_w=synth.normal_bf16(info["seed"], synth.TID["router_w"], (shape.n_experts, shape.hidden), 0.02, 0.0, "cuda").float())
    h = synth.normal_bf16(info["seed"], 77, (n_tok, shape.hidden), 1.5, 0.0, "cuda")
    lib = binding.load_library()
    cap = lib.foe_route_partial_capacity(max_tokens, 1, shape.n_experts)
    assert 16 * n_tok * shape.n_experts > cap                                       # the case is the one meant
    layer = binding.FoeLayer(shape, _route_only_weights(shape, W), max_tokens=max_tokens, max_seqs=1, max_context=64)
    idx, w = layer.route(h)
    assert layer.poll_status() == 0
    aux = layer.aux()
    layer.close()
    cfg = adapter.cfg_from_shape(shape)
    Wn = {k: adapter.to_np(W[k]) for k in ("ffn_norm_g", "router_w")}
    Wn["router_b"] = None
    rt = orc.route(cfg, Wn, adapter.to_np(h))
    exempt = check_routing(shape, idx.cpu().numpy(), w.cpu().numpy().astype(np.float64), rt["logits"], rt["idx"], rt["w"])
    assert exempt <= max(2, n_tok // 200)
    assert np.abs(adapter.to_np(aux["logits"]) - rt["logits"]).max() <= 2e-5 * max(1.0, np.abs(rt["logits"]).max())
    check_maps(shape, aux, idx.cpu().numpy())


@pytest.mark.parametrize("H,Ec,kc,n_tok,ties", [(1, 128, 16, 2, False), (1, 128, 32, 200, False), (2, 100, 31, 33, False),
                                                (4, 24, 24, 256, False), (8, 64, 7, 65, False), (1, 3, 3, 5, False),
                                                (2, 96, 20, 40, True), (1, 33, 32, 3, True)])
def test_route_of_a_decode_step_with_wide_or_odd_expert_sets(H, Ec, kc, n_tok, ties):
    """Calls of at most 256 tokens select inside the map kernel; cluster sizes other than 4, 8, 16 and 32 take its
    one-warp-per-(token, cluster) selection.  With `ties` the router weights are zero and the bias repeats each value
    four times, so that every selection is decided by the lower-expert-id rule."""
    shape = synth.LayerShape(512, 2 * H, H, H, 64, Ec, kc, 128)
    seed = 1300 + Ec + kc
    W = dict(ffn_norm_g=synth.normal_bf16(seed, synth.TID["ffn_norm_g"], (shape.hidden,), 0.02, 1.0, "cuda"),
             router_w=synth.normal_bf16(seed, synth.TID["router_w"], (shape.n_experts, shape.hidden), 0.02, 0.0, "cuda").float())
    full = _route_only_weights(shape, W)
    if ties:
        W["router_w"] = torch.zeros_like(W["router_w"])
        full["router_w"] = W["router_w"]
        b = torch.tensor([float((7 * (e // 4)) % 11) for e in range(shape.n_experts)], dtype=torch.float32, device="cuda")
        W["router_b"] = full["router_b"] = b
    h = synth.normal_bf16(seed, 77, (n_tok, shape.hidden), 1.5, 0.0, "cuda")
    layer = binding.FoeLayer(shape, full, max_tokens=256, max_seqs=1, max_context=64)
    idx, w = layer.route(h)
    assert layer.poll_status() == 0
    aux = layer.aux()
    layer.close()
    cfg = adapter.cfg_from_shape(shape)
    Wn = {k: adapter.to_np(W[k]) for k in ("ffn_norm_g", "router_w")}
    Wn["router_b"] = adapter.to_np(W["router_b"]) if ties else None
    rt = orc.route(cfg, Wn, adapter.to_np(h))
    idx_g, w_g = idx.cpu().numpy(), w.cpu().numpy().astype(np.float64)
    if ties:
        assert np.array_equal(idx_g.reshape(rt["idx"].shape), rt["idx"])            # exact scores: no exemptions
        assert np.abs(w_g.reshape(rt["w"].shape) - rt["w"]).max() <= 1e-6
    else:
        exempt = check_routing(shape, idx_g, w_g, rt["logits"], rt["idx"], rt["w"])
        assert exempt <= 2
        lg = np.take_along_axis(rt["logits"], idx_g.reshape(n_tok, -1).astype(np.int64), 1).reshape(idx_g.shape)
        assert (np.diff(lg, axis=-1) <= 1e-5).all()
    check_maps(shape, aux, idx_g)


def _route_only_weights(shape, W):
    """A full weight set for foe_layer_create in which everything but the router and the FFN-norm gain is a small
    shared zero buffer of the right size class (routing reads nothing else)."""
    s = shape
    dev = "cuda"
    H, g, c, dh, d, I, E = s.n_clusters, s.n_q_heads // s.n_clusters, s.n_kv_heads // s.n_clusters, s.head_dim, s.hidden, s.ffn_inter, s.n_experts
    z = lambda *shp: torch.zeros(shp, dtype=torch.bfloat16, device=dev)
    return dict(attn_norm_g=z(d), wq=z(H, d, g * dh), wk=z(H, d, c * dh), wv=z(H, d, c * dh), wo=z(s.n_q_heads * dh, d),
                ffn_norm_g=W["ffn_norm_g"], w_gate=z(E, d, I), w_up=z(E, d, I), w_down=z(E, I, d),
                router_w=W["router_w"], router_b=None)


def test_route_is_deterministic():
    shape, info = synth.workload(1)
    W = synth.make_weights(shape, 0, "cuda")
    h = synth.normal_bf16(0, 78, (500, shape.hidden), 1.0, 0.0, "cuda")
    layer = binding.FoeLayer(shape, W, max_tokens=500, max_seqs=1, max_context=64)
    a = layer.route(h)
    auxa = layer.aux()
    b = layer.route(h)
    auxb = layer.aux()
    layer.close()
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    for k in ("perm", "inv", "counts", "offsets"):
        assert torch.equal(auxa[k], auxb[k])


# ------------------------------------------------------------------------------------------ small blocks
def test_workload1_prefill_elementwise():
    shape, info = synth.workload(1)
    r = run_block_parity(shape, info["seed"], info["q_lens"], info["context_lens"])
    assert r["launches"] > 0


@pytest.mark.parametrize("position,sync", [("middle", "mean"), ("middle", "sum"), ("first", "mean"),
                                           ("last", "mean"), ("single", "mean"), ("last", "sum")])
def test_positions_and_sync_modes(position, sync):
    shape = shape_small(position=position, sync=sync)
    run_block_parity(shape, 11, [100, 29, 1, 200], [0, 0, 0, 0], wscale=4.0)


def test_one_cluster_baseline_and_wide_topk():
    shape = shape_small(n_clusters=1, experts_per_cluster=32, top_k_per_cluster=8)
    run_block_parity(shape, 12, [150, 70], [0, 0], wscale=4.0)
    shape = shape_small(n_clusters=2, n_kv_heads=4, experts_per_cluster=128, top_k_per_cluster=16)
    run_block_parity(shape, 13, [90], [0], wscale=4.0)


@pytest.mark.parametrize("H", [3, 6])
def test_cluster_counts_that_are_not_powers_of_two(H):
    # (the pre-attention statistics kernel sums the H residual streams with H as a template parameter)
    shape = synth.LayerShape(384, 2 * H, H, H, 64, 4, 2, 128)
    run_block_parity(shape, 40 + H, [300, 117], [0, 64], wscale=4.0)
    run_block_parity(shape, 50 + H, [1] * 5, [3, 64, 200, 65, 130], decode=True, wscale=4.0)


def test_head_dim_128_and_ragged_tiles():
    shape = synth.LayerShape(512, 8, 2, 2, 128, 4, 2, 256)
    run_block_parity(shape, 14, [130, 300, 63, 65], [0, 0, 0, 0], wscale=4.0)       # several 128-row tiles + tails


def test_head_dim_96_prefill_and_decode():
    """head_dim 96 (the paper's 1B model): the attention kernels work on heads zero-padded to 128, the projection
    epilogues on 32-column passes."""
    shape = synth.LayerShape(256, 4, 2, 2, 96, 4, 2, 128)
    run_block_parity(shape, 31, [130, 70, 1, 200], [0, 64, 300, 0], wscale=4.0)
    run_block_parity(shape, 32, [1] * 5, [0, 63, 64, 200, 1500], decode=True, wscale=4.0)
    for position in ("first", "last"):
        sh = synth.LayerShape(256, 4, 2, 2, 96, 4, 2, 128, position=position)
        run_block_parity(sh, 33, [90, 41], [0, 10], wscale=4.0)


def test_paper_1b_layer_shape_prefill_and_decode():
    """Layer shape of the paper's 1B model (Table 8): hidden 768, 8 query / 8 KV heads of 96, 8 groups x 8 experts
    top-1, intermediate 384, rope theta 5e5.  One query and one KV head per group: 288 projection columns per group,
    not a multiple of the 64-row slabs and 64-column passes used elsewhere."""
    shape = synth.LayerShape(768, 8, 8, 8, 96, 8, 1, 384, rope_theta=5.0e5)
    r = run_block_parity(shape, 34, [700, 333, 129], [0, 0, 64])
    print("1B shape prefill:", {k: r[k] for k in ("max_abs", "rel_l1", "flips")})
    r = run_block_parity(shape, 35, [1] * 6, [0, 100, 1000, 2047, 2048, 3000], decode=True)
    print("1B shape decode:", {k: r[k] for k in ("max_abs", "rel_l1", "flips")})


def test_chunked_prefill_over_cached_context():
    shape = shape_small()
    run_block_parity(shape, 15, [40, 17, 130], [100, 64, 1], wscale=4.0)


def test_prefill_call_with_more_sequences_than_the_token_map_scans_in_one_block():
    """Up to 1024 sequences the token-map kernel builds the prefix sums of q_lens itself, beyond that a separate kernel
    does; 1030 sequences of one or two tokens (and, in the same test, 1024 exactly) over short cached contexts."""
    shape = shape_small()
    for n in (1030, 1024):
        q = [1 + (i % 3 == 0) for i in range(n)]
        ctx = [(7 * i) % 40 for i in range(n)]
        run_block_parity(shape, 33, q, ctx, decode=False, wscale=4.0)


def test_mixed_batch_of_prefill_chunks_and_decode_tokens():
    """One prefill call carrying fresh prompts, a chunk of a longer prompt and single decode tokens of running
    sequences (q_len 1 over a long cached context): the serving batch shape of Section 4's engine."""
    shape = shape_small()
    run_block_parity(shape, 18, [1, 200, 1, 64, 1], [300, 0, 1000, 64, 63], wscale=4.0)


@pytest.mark.parametrize("dh,group", [(128, 2), (64, 4), (128, 1), (64, 3)])
def test_prefill_attention_step_counts_and_mask_positions(dh, group):
    """The prefill attention hands the 64-key steps of a query block alternately to two threads per row, so the cases
    that matter are the number of steps of a block (one, two, odd, even), where the causal mask starts (an even or an
    odd step, at a page boundary or inside a page) and a last block with few rows: new-token counts around 64, 128 and
    192 on cached contexts around the page size.  One or two query heads per CTA (odd group sizes take one)."""
    n_kv = 2
    shape = synth.LayerShape(512, n_kv * group, n_kv, 2, dh, 4, 2, 128)
    q_lens = [1, 63, 64, 65, 127, 128, 129, 191, 192, 193, 257, 5]
    ctx = [0, 1, 64, 63, 130, 0, 62, 65, 128, 1, 191, 700]
    run_block_parity(shape, 60 + dh + group, q_lens, ctx, wscale=2.0)


def test_empty_and_single_token_calls():
    shape = shape_small()
    W = synth.make_weights(shape, 16, "cuda")
    layer = binding.FoeLayer(shape, W, max_tokens=8, max_seqs=2, max_context=128)
    kv = synth.make_paged_cache(shape, 16, [0], [0], "cuda")
    x = torch.empty((4, 0, 256), dtype=torch.bfloat16, device="cuda")
    out = layer.prefill(x, kv, n_tokens=0, max_q_len=0)
    assert out.shape == (4, 0, 256) and layer.last_launch_count() == 0
    layer.close()
    run_block_parity(shape, 16, [1], [0], wscale=4.0)


def test_skewed_router_bias_small():
    shape = shape_small(experts_per_cluster=16, top_k_per_cluster=4)
    bias = synth.zipf_router_bias(shape, 17, 1.0, 1.2, dead_per_cluster=3)
    r = run_block_parity(shape, 17, [300, 212], [0, 0], wscale=4.0, router_bias=bias)
    assert (r["counts"] == 0).sum() >= 12                                         # dead experts stay empty


def test_small_prefill_with_skewed_routing_streams_experts_in_several_passes():
    # 120 tokens, 16 experts per cluster, top-1: few enough rows per expert on average for the weight-streaming
    # expert kernels, but the skewed bias sends dozens of rows to single experts (several 16-row passes) and none to others
    shape = shape_small(experts_per_cluster=16, top_k_per_cluster=1)
    bias = synth.zipf_router_bias(shape, 19, 1.5, 1.2, dead_per_cluster=4)
    r = run_block_parity(shape, 19, [70, 50], [0, 33], wscale=4.0, router_bias=bias)
    assert r["counts"].max() > 16 and (r["counts"] == 0).sum() >= 16


# ------------------------------------------------------------------------------------------ decode
def test_decode_small_elementwise():
    shape = shape_small()
    run_block_parity(shape, 21, [1] * 7, [0, 1, 63, 64, 65, 200, 1500], decode=True, wscale=4.0)


def test_decode_head_dim_128_many_splits():
    shape = synth.LayerShape(512, 8, 2, 2, 128, 4, 2, 256)
    run_block_parity(shape, 22, [1] * 4, [10, 1030, 2100, 5000], decode=True, wscale=4.0)


@pytest.mark.parametrize("dh,n_seqs,spread", [(128, 40, 5200), (64, 45, 3000), (128, 33, 9000), (64, 3, 700)])
def test_decode_attention_page_partition_across_sequences(dh, n_seqs, spread):
    """The decode attention kernel cuts the list of all (sequence, KV head, page) entries into equal ranges, one per
    CTA: with a few thousand pages in the call the ranges are longer than the minimum, start and end anywhere inside
    a pair, and a range may hold the tail of one sequence, whole short sequences and the head of the next.  Contexts
    on and around page boundaries, one-page sequences, more than 32 sequences (the range search walks them in chunks
    of 32)."""
    if dh == 64:
        shape = shape_small()
    else:
        shape = synth.LayerShape(512, 8, 2, 2, 128, 4, 2, 256)
    ctx = [(613 * i * i + 97 * i) % spread for i in range(n_seqs)]
    for i, v in enumerate([0, 63, 64, 65, 127, 128, 1, 511, 512]):
        if 2 * i + 1 < n_seqs:
            ctx[2 * i + 1] = v
    run_block_parity(shape, 31, [1] * n_seqs, ctx, decode=True, wscale=4.0)


@pytest.mark.parametrize("dh,position,n_seqs", [(64, "middle", 130), (128, "middle", 200), (64, "first", 65), (128, "last", 256)])
def test_decode_more_sequences_than_one_token_tile(dh, position, n_seqs):
    # the decode projections take 64 tokens per CTA: several token tiles, the last one ragged (or exactly full)
    if dh == 64:
        shape = shape_small(position=position)
    else:
        shape = synth.LayerShape(512, 8, 2, 2, 128, 4, 2, 256, position=position)
    ctx = [(37 * i) % 300 for i in range(n_seqs)]
    run_block_parity(shape, 29, [1] * n_seqs, ctx, decode=True, wscale=4.0)


@pytest.mark.timeout(300)
@pytest.mark.parametrize("H,n_seqs", [(5, 150), (4, 150), (8, 250)])
def test_decode_head_dim_96_with_more_projection_tasks_than_resident_ctas(H, n_seqs):
    """Heads of width 96 take the weight-streaming QKV projection; with 150 and more sequences it has more
    (cluster, slab, 16-token chunk) tasks than the 2 x 148 CTAs of its grid, so CTAs run a second task, and the last
    chunk of every cluster is ragged (150 = 9 x 16 + 6)."""
    shape = synth.LayerShape(1024, 4 * H, H, H, 96, 2, 1, 256, position="single")
    ctx = [(37 * i) % 300 for i in range(n_seqs)]
    run_block_parity(shape, 34, [1] * n_seqs, ctx, decode=True)


@pytest.mark.parametrize("position", ["first", "last"])
def test_decode_boundary_layers(position):
    shape = shape_small(position=position)
    run_block_parity(shape, 23, [1] * 3, [5, 70, 300], decode=True, wscale=4.0)


def test_physical_page_order_does_not_matter():
    shape = shape_small()
    a = run_block_parity(shape, 24, [1] * 3, [100, 257, 640], decode=True, wscale=4.0, shuffle_pages=True,
                         return_all=True)
    # same logical cache laid out in identity page order
    kv_a = a["kv"]
    ctx = [100, 257, 640]
    kv_b = synth.make_paged_cache(shape, 24, ctx, [1] * 3, "cuda", fill_random=False, shuffle=False)
    for s in range(3):
        npg = (ctx[s] + 1 + 63) // 64
        kv_b.k_pages[kv_b.block_table[s, :npg].long()] = kv_a.k_pages[kv_a.block_table[s, :npg].long()]
        kv_b.v_pages[kv_b.block_table[s, :npg].long()] = kv_a.v_pages[kv_a.block_table[s, :npg].long()]
    layer = binding.FoeLayer(shape, a["W"], max_tokens=1, max_seqs=3, max_context=700)
    out_b = layer.decode(a["x"], kv_b)
    assert layer.poll_status() == 0
    layer.close()
    assert torch.equal(out_b, a["out"])                                            # bit-identical


def test_prefill_then_decode_matches_longer_prefill():
    shape = shape_small()
    T = 150
    W = scaled_weights(shape, 25, "cuda", 4.0)
    x = synth.make_x(shape, 25, T + 1, "cuda")
    kv = synth.make_paged_cache(shape, 25, [0], [T + 1], "cuda", fill_random=False)
    layer = binding.FoeLayer(shape, W, max_tokens=T + 1, max_seqs=1, max_context=T + 1)
    full = layer.prefill(x, kv)
    kv2 = synth.make_paged_cache(shape, 25, [0], [T + 1], "cuda", fill_random=False)
    kv2.q_lens = torch.tensor([T], dtype=torch.int32, device="cuda")
    layer.prefill(x[:, :T].contiguous(), kv2)
    kv2.context_lens = torch.tensor([T], dtype=torch.int32, device="cuda")
    step = layer.decode(x[:, T:].contiguous(), kv2)
    assert layer.poll_status() == 0
    layer.close()
    assert_close(adapter.to_np(step[:, 0]), adapter.to_np(full[:, T]).astype(np.float64), "decode vs prefill row")
    # the first T tokens went through the same kernels; the last one through the decode projection
    assert_close(adapter.to_np(kv2.k_pages), adapter.to_np(kv.k_pages).astype(np.float64), "K pages", 1e-2, 1e-3)
    assert_close(adapter.to_np(kv2.v_pages), adapter.to_np(kv.v_pages).astype(np.float64), "V pages", 1e-2, 1e-3)


def test_same_inputs_give_bit_identical_outputs():
    shape = shape_small()
    W = scaled_weights(shape, 26, "cuda", 4.0)
    x = synth.make_x(shape, 26, 333, "cuda")
    layer = binding.FoeLayer(shape, W, max_tokens=333, max_seqs=2, max_context=256)
    outs = []
    for _ in range(2):
        kv = synth.make_paged_cache(shape, 26, [0, 0], [200, 133], "cuda", fill_random=False)
        outs.append(layer.prefill(x, kv).clone())
    layer.close()
    assert torch.equal(outs[0], outs[1])


@pytest.mark.parametrize("dh,q_lens,ctx", [(128, [130, 300, 63, 65], [0, 0, 0, 0]), (64, [700, 333, 129], [64, 0, 130])])
def test_repeated_prefill_is_bit_stable_under_timing_noise(dh, q_lens, ctx):
    """The same call repeated many times, with the L2 flushed at irregular intervals, must give the same bits every
    time: a warp that runs a pipeline phase ahead of its neighbours may not change what it reads."""
    shape = synth.LayerShape(512, 8, 2, 2, 128, 4, 2, 256) if dh == 128 else synth.LayerShape(256, 8, 4, 4, 64, 8, 2, 128)
    W = scaled_weights(shape, 14, "cuda", 4.0)
    S = sum(q_lens)
    x = synth.make_x(shape, 14, S, "cuda")
    layer = binding.FoeLayer(shape, W, max_tokens=S, max_seqs=len(q_lens), max_context=max(c + q for c, q in zip(ctx, q_lens)))
    first = None
    for it in range(120):
        kv = synth.make_paged_cache(shape, 14, ctx, q_lens, "cuda")
        if it % 3 == 1:
            torch.empty(192 << 20, dtype=torch.uint8, device="cuda").fill_(1)
        out = layer.prefill(x, kv)
        assert layer.poll_status() == 0
        cur = (out.clone(), layer.aux()["attn_o"].clone(), kv.k_pages.clone(), kv.v_pages.clone())
        if first is None:
            first = cur
        else:
            for a, b, name in zip(first, cur, ("out", "attn_o", "k_pages", "v_pages")):
                assert torch.equal(a, b), f"repeat {it}: {name} changed"
    layer.close()


@pytest.mark.parametrize("decode,n", [(True, 64), (True, 9), (False, 100), (False, 1)])
def test_repeated_small_calls_are_bit_stable_with_overlapping_launches(decode, n):
    """Decode steps and small prefill calls launch every kernel so that it may start while its predecessor drains
    (a kernel waits for the predecessor only where it first touches its results).  Back-to-back repeats without any
    host synchronisation in between, partly with other work queued on the device first, must give the same bits."""
    shape = synth.LayerShape(512, 8, 2, 2, 128, 4, 2, 256)
    W = scaled_weights(shape, 31, "cuda", 4.0)
    if decode:
        q_lens, ctx = [1] * n, [(53 * i) % 700 + 1 for i in range(n)]
    else:
        q_lens, ctx = [n], [70]
    S = sum(q_lens)
    x = synth.make_x(shape, 31, S, "cuda")
    layer = binding.FoeLayer(shape, W, max_tokens=S, max_seqs=len(q_lens), max_context=max(c + q for c, q in zip(ctx, q_lens)))
    kv = synth.make_paged_cache(shape, 31, ctx, q_lens, "cuda")
    run = (lambda: layer.decode(x, kv)) if decode else (lambda: layer.prefill(x, kv))
    first = run().clone()
    first_aux = layer.aux()
    k0, v0 = kv.k_pages.clone(), kv.v_pages.clone()
    outs = []
    for it in range(150):
        if it % 7 == 3:
            torch.empty(160 << 20, dtype=torch.uint8, device="cuda").fill_(1)     # something else in the queue, L2 flushed
        outs.append(run().clone())                   # (the call rewrites the same K/V slots with the same values)
    torch.cuda.synchronize()
    assert layer.poll_status() == 0
    for it, o in enumerate(outs):
        assert torch.equal(o, first), f"repeat {it} differs"
    aux = layer.aux()
    for k in ("r_full", "topk_idx", "attn_o", "perm"):
        assert torch.equal(aux[k], first_aux[k]), k
    assert torch.equal(kv.k_pages, k0) and torch.equal(kv.v_pages, v0)
    layer.close()


@pytest.mark.parametrize("decode", [True, False])
def test_calls_can_be_captured_into_a_cuda_graph(decode):
    """After one ordinary call (which does the one-time kernel configuration) a call only launches kernels on the
    given stream, so it can be captured; replays give the direct call's bits."""
    shape = synth.LayerShape(512, 8, 2, 2, 128, 4, 2, 256)
    W = scaled_weights(shape, 33, "cuda", 4.0)
    if decode:
        q_lens, ctx = [1] * 20, [(41 * i) % 500 + 3 for i in range(20)]
    else:
        q_lens, ctx = [300, 41], [0, 100]
    S = sum(q_lens)
    x = synth.make_x(shape, 33, S, "cuda")
    kv = synth.make_paged_cache(shape, 33, ctx, q_lens, "cuda")
    layer = binding.FoeLayer(shape, W, max_tokens=S, max_seqs=len(q_lens), max_context=max(c + q for c, q in zip(ctx, q_lens)))
    out = torch.empty_like(x)
    mq = max(q_lens)
    run = (lambda: layer.decode(x, kv, out=out)) if decode else (lambda: layer.prefill(x, kv, n_tokens=S, max_q_len=mq, out=out))
    run()
    torch.cuda.synchronize()
    ref = out.clone()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        run()
    for _ in range(3):
        out.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, ref)
    assert layer.poll_status() == 0
    layer.close()


# ------------------------------------------------------------------------------------------ error paths (host side)
def test_host_side_argument_errors():
    shape = shape_small()
    W = synth.make_weights(shape, 27, "cuda")
    bad = shape_small(head_dim=32)
    with pytest.raises(binding.FoeError) as e:
        binding.FoeLayer(bad, W, 8, 1, 64)
    assert e.value.code == -2
    layer = binding.FoeLayer(shape, W, max_tokens=8, max_seqs=1, max_context=64)
    kv = synth.make_paged_cache(shape, 27, [0], [16], "cuda")
    x = synth.make_x(shape, 27, 16, "cuda")
    with pytest.raises(binding.FoeError) as e:
        layer.prefill(x, kv)                                                       # 16 tokens > max_tokens
    assert e.value.code == -3
    # a block-table entry outside the pool is reported through the device status word, nothing faults
    kv = synth.make_paged_cache(shape, 27, [0], [8], "cuda")
    kv.block_table[0, 0] = 10_000
    layer.prefill(synth.make_x(shape, 27, 8, "cuda"), kv)
    assert layer.poll_status() == -8
    assert layer.poll_status() == 0
    # the same in a decode step, where position and slot are looked up inside the QKV projection
    kv = synth.make_paged_cache(shape, 27, [20], [1], "cuda")
    kv.block_table[0, 0] = -3
    layer.decode(synth.make_x(shape, 27, 1, "cuda"), kv)
    assert layer.poll_status() == -8
    kv = synth.make_paged_cache(shape, 27, [63], [1], "cuda")          # position 63 is fine, position 64 = max_context is not
    layer.decode(synth.make_x(shape, 27, 1, "cuda"), kv)
    assert layer.poll_status() == 0
    kv = synth.make_paged_cache(shape, 27, [64], [1], "cuda")
    layer.decode(synth.make_x(shape, 27, 1, "cuda"), kv)
    assert layer.poll_status() == -8
    kv.context_lens[0] = -5                                            # a negative context length never reaches the block table
    layer.decode(synth.make_x(shape, 27, 1, "cuda"), kv)
    assert layer.poll_status() == -8
    # prefill: context + new tokens one past max_context (the rotary table ends there), reported, nothing faults
    kv = synth.make_paged_cache(shape, 27, [57], [8], "cuda")          # positions 57..64
    x8 = synth.make_x(shape, 27, 8, "cuda")
    layer.prefill(x8, kv)
    assert layer.poll_status() == -8
    kv = synth.make_paged_cache(shape, 27, [56], [8], "cuda")          # positions 56..63: fine
    layer.prefill(x8, kv)
    assert layer.poll_status() == 0
    kv.context_lens[0] = -60
    layer.prefill(x8, kv)
    assert layer.poll_status() == -8
    # q_lens that do not add up to the call's token count, or exceed the stated bound
    kv = synth.make_paged_cache(shape, 27, [0], [8], "cuda")
    kv.q_lens[0] = 5
    layer.prefill(x8, kv, n_tokens=8, max_q_len=8)
    assert layer.poll_status() == -8
    kv.q_lens[0] = 8
    layer.prefill(x8, kv, n_tokens=8, max_q_len=4)
    assert layer.poll_status() == -8
    layer.prefill(x8, kv, n_tokens=8, max_q_len=8)                     # and the handle is fine afterwards
    assert layer.poll_status() == 0
    # views that start 2 bytes off a 16-byte boundary (contiguous, right type): refused before any launch
    def off_by_one(t):
        flat = torch.empty(t.numel() + 8, dtype=t.dtype, device=t.device)
        v = flat[1:1 + t.numel()].view(t.shape)
        v.copy_(t)
        assert v.is_contiguous() and v.data_ptr() % 16 != 0
        return v
    for call in (lambda: layer.prefill(off_by_one(x8), kv, n_tokens=8, max_q_len=8),
                 lambda: layer.prefill(x8, kv, n_tokens=8, max_q_len=8, out=off_by_one(torch.empty_like(x8))),
                 lambda: layer.route(off_by_one(synth.normal_bf16(27, 77, (8, shape.hidden), 1.0, 0.0, "cuda")))):
        with pytest.raises(binding.FoeError) as e:
            call()
        assert e.value.code == -3
    kv1 = synth.make_paged_cache(shape, 27, [20], [1], "cuda")
    with pytest.raises(binding.FoeError) as e:
        layer.decode(off_by_one(synth.make_x(shape, 27, 1, "cuda")), kv1)
    assert e.value.code == -3
    kv1.k_pages = off_by_one(kv1.k_pages)
    with pytest.raises(binding.FoeError) as e:
        layer.decode(synth.make_x(shape, 27, 1, "cuda"), kv1)
    assert e.value.code == -3
    assert layer.poll_status() == 0
    layer.prefill(x8, kv, n_tokens=8, max_q_len=8)
    assert layer.poll_status() == 0
    W2 = dict(W)
    W2["wq"] = off_by_one(W["wq"])
    with pytest.raises(binding.FoeError) as e:
        binding.FoeLayer(shape, W2, 8, 1, 64)
    assert e.value.code == -3
    layer.close()


# ------------------------------------------------------------------------------------------ full-size workloads
def _sample_rows(q_lens, per_seq, seed):
    rows, at = [], 0
    for b, T in enumerate(q_lens):
        pick = synth.uniform_int(seed, 500 + b, per_seq, 0, T - 1).tolist()
        pick += [0, T - 1, 63, 64, 127, 128]
        rows += sorted({at + p for p in pick if p < T})
        at += T
    return np.array(rows, dtype=np.int64)


def test_workload2_full_size_prefill_sampled_end_to_end_and_every_row_per_stage():
    """End to end (every stage chained) on sampled tokens; then the experts stage over all 16,384 tokens and the
    attention stage over every row of the last sequence, each against the oracle fed the GPU's own stage input."""
    shape, info = synth.workload(2)
    rows = _sample_rows(info["q_lens"], 40, 2)
    r = run_block_parity(shape, info["seed"], info["q_lens"], info["context_lens"], rows=rows, return_all=True)
    print("workload 2:", {k: r[k] for k in ("max_abs", "rel_l1", "flips", "launches")})
    c = r["counts"]
    assert c.min() > 1500 and c.max() < 2700                                       # near-uniform load, ~2048 rows/expert
    e = check_every_row(shape, r["W"], r["out"], r["aux"], r["kv"], info["q_lens"], info["context_lens"], attn_seqs=[3])
    print("workload 2, every row:", e)


def test_workload3_full_size_decode_all_tokens():
    shape, info = synth.workload(3)
    r = run_block_parity(shape, info["seed"], info["q_lens"], info["context_lens"], decode=True)
    print("workload 3:", {k: r[k] for k in ("max_abs", "rel_l1", "flips", "launches")})


def test_workload4_skewed_routing_sampled_end_to_end_and_every_row_per_stage():
    shape, info = synth.workload(4)
    dev = "cuda"
    W = synth.make_weights(shape, info["seed"], dev)
    # spread of the unbiased scores, measured with the library on a sample, sets the bias scale
    h = synth.normal_bf16(info["seed"], 79, (2048, shape.hidden), 1.0, 0.0, dev)
    layer = binding.FoeLayer(shape, W, max_tokens=2048, max_seqs=1, max_context=64)
    layer.route(h)
    sigma = float(layer.aux()["logits"].std())
    layer.close()
    bias = synth.zipf_router_bias(shape, info["seed"], sigma, info["zipf"], dead_per_cluster=2)
    rows = _sample_rows(info["q_lens"], 12, 4)
    r = run_block_parity(shape, info["seed"], info["q_lens"], info["context_lens"], rows=rows, router_bias=bias,
                         weights=W, return_all=True)
    c = r["counts"].reshape(shape.n_clusters, shape.experts_per_cluster)
    print("workload 4:", {k: r[k] for k in ("max_abs", "rel_l1", "flips")}, "max/mean rows", c.max() / c.mean())
    assert (c == 0).sum() >= 2 * shape.n_clusters and c.max() > 3 * c.mean()       # empty and overfull experts
    # every row of every expert's tiles (the hottest expert's ~13 k rows and the empty ones included), and every
    # query block of the first and the last sequence
    e = check_every_row(shape, r["W"], r["out"], r["aux"], r["kv"], info["q_lens"], info["context_lens"], attn_seqs=[0, 7])
    print("workload 4, every row:", e, "hottest expert rows", int(c.max()))


# ------------------------------------------------------------------------------------------ the paper's own model shape
def test_paper_7b_layer_shape_prefill_and_decode():
    """The "Full" model of the paper's training-configuration table: hidden 2048, 16 query / 8 KV heads of 128,
    64 experts, top-8, 8 groups (so 8 experts and top-1 per group), expert FFN multiplier 1/2 (inter 1024),
    RoPE base 500,000."""
    shape = synth.LayerShape(2048, 16, 8, 8, 128, 8, 1, 1024, rope_theta=5.0e5)
    rows = _sample_rows([1024, 3000], 10, 7)
    r = run_block_parity(shape, 70, [1024, 3000], [0, 0], rows=rows)
    print("paper 7B layer, prefill:", {k: r[k] for k in ("max_abs", "rel_l1", "flips")})
    r = run_block_parity(shape, 71, [1] * 12, [17, 900, 2048, 5000, 63, 64, 4095, 4096, 30000, 1, 777, 12000], decode=True)
    print("paper 7B layer, decode:", {k: r[k] for k in ("max_abs", "rel_l1", "flips")})
