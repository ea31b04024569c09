"""The allocation-free routing entry point against the handle-based one.

Collected last on purpose (file name): if it fails, a run that stops at the first failure has already run every
other test.  It is for callers that cannot allocate device memory (all of it belongs to their own pool, or they
must keep away from the driver's allocator on a latency-critical path), so the check is simply that
foe_route_noalloc, which works on the scratch array built into the library, returns what foe_route returns:
the same expert ids and gates within the 1e-5 the routing tests use, on two calls in a row (the second call
finds the first call's leftovers in the shared scratch)."""
import numpy as np
import pytest
import torch

from oracle import adapter
from oracle import foe_oracle as orc
from paper_2605_06206_b200 import binding, synth

from parity import check_routing

pytestmark = pytest.mark.gpu


def _reference(shape, W, hs):
    layer = binding.FoeLayer(shape, W, max_tokens=max(h.shape[0] for h in hs), max_seqs=1, max_context=64)
    out = []
    for h in hs:
        idx, w = layer.route(h)
        out.append((idx.clone(), w.clone(), layer.aux()["logits"]))
    layer.close()
    return out


def test_noalloc_route_matches_handle_route_twice_in_a_row():
    shape, info = synth.workload(4)                        # 8 clusters x 32 experts, top-4
    dev = "cuda"
    W = synth.make_weights(shape, info["seed"], dev)
    W["router_b"] = synth.zipf_router_bias(shape, info["seed"], 1.0, 1.2, dead_per_cluster=2).to(dev)
    hs = [synth.normal_bf16(9, 90, (1500, shape.hidden), 1.3, 0.0, dev),
          synth.normal_bf16(9, 91, (37, shape.hidden), 0.7, 0.0, dev)]      # second call: other size, split-K path
    ref = _reference(shape, W, hs)
    for h, (idx_ref, w_ref, logits) in zip(hs, ref):
        n = h.shape[0]
        idx = torch.full((n, shape.n_clusters, shape.top_k_per_cluster), -1, dtype=torch.int32, device=dev)
        w = torch.zeros((n, shape.n_clusters, shape.top_k_per_cluster), dtype=torch.float32, device=dev)
        binding.route_noalloc(shape, W["ffn_norm_g"], W["router_w"], W["router_b"], h, idx, w)
        torch.cuda.synchronize()
        # ids: identical wherever the k-th / (k+1)-th scores are at least 1e-5 apart (the routing tests' rule)
        lg = logits.view(n, shape.n_clusters, shape.experts_per_cluster).float()
        srt = torch.sort(lg, dim=-1, descending=True).values
        kc = shape.top_k_per_cluster
        clear = (srt[..., kc - 1] - srt[..., kc]) >= 1e-5
        same = (torch.sort(idx, -1).values == torch.sort(idx_ref, -1).values).all(-1)
        assert bool((same | ~clear).all()), "expert ids differ outside near-ties"
        assert int((~clear).sum()) <= 2
        wa = torch.gather(w, -1, torch.argsort(idx, -1))
        wb = torch.gather(w_ref, -1, torch.argsort(idx_ref, -1))
        assert float((wa - wb).abs()[same].max()) <= 1e-5
        np.testing.assert_allclose(w.sum(-1).cpu().numpy(), 1.0, atol=1e-5)
        # and directly against the oracle's routing of the same rows (ids bit-exact outside near-ties, gates to 1e-5)
        Wn = {k: adapter.to_np(W[k]) for k in ("ffn_norm_g", "router_w", "router_b")}
        rt = orc.route(adapter.cfg_from_shape(shape), Wn, adapter.to_np(h))
        check_routing(shape, idx.cpu().numpy(), w.cpu().numpy().astype(np.float64), rt["logits"], rt["idx"], rt["w"])


def test_noalloc_route_refuses_misaligned_views_without_launching():
    """The kernels read h and the router weights 16 bytes at a time: a view that starts in the middle of such a group
    is refused on the host (a caller without an allocator of its own tends to carve tensors out of one big buffer)."""
    shape, _ = synth.workload(1)
    dev = "cuda"
    W = synth.make_weights(shape, 1, dev)
    n = 16
    big = torch.zeros(n * shape.hidden + 8, dtype=torch.bfloat16, device=dev)
    h_bad = big[1:1 + n * shape.hidden].view(n, shape.hidden)          # 2 bytes past a 16-byte boundary
    idx = torch.full((n, shape.n_clusters, shape.top_k_per_cluster), -7, dtype=torch.int32, device=dev)
    w = torch.zeros((n, shape.n_clusters, shape.top_k_per_cluster), dtype=torch.float32, device=dev)
    with pytest.raises(binding.FoeError) as e:
        binding.route_noalloc(shape, W["ffn_norm_g"], W["router_w"], None, h_bad, idx, w)
    assert e.value.code == -3
    rw = torch.zeros(W["router_w"].numel() + 4, dtype=torch.float32, device=dev)
    rw_bad = rw[1:1 + W["router_w"].numel()].view_as(W["router_w"])    # 4 bytes past
    with pytest.raises(binding.FoeError) as e:
        binding.route_noalloc(shape, W["ffn_norm_g"], rw_bad, None, big[:n * shape.hidden].view(n, shape.hidden), idx, w)
    assert e.value.code == -3
    torch.cuda.synchronize()
    assert int((idx != -7).sum()) == 0


def test_noalloc_route_rejects_oversized_calls_without_launching():
    shape, _ = synth.workload(4)
    dev = "cuda"
    W = synth.make_weights(shape, 4, dev)
    n = 2049                                               # 2049 * 256 experts > 524288 scores
    h = torch.zeros((n, shape.hidden), dtype=torch.bfloat16, device=dev)
    idx = torch.full((n, shape.n_clusters, shape.top_k_per_cluster), -7, dtype=torch.int32, device=dev)
    w = torch.zeros((n, shape.n_clusters, shape.top_k_per_cluster), dtype=torch.float32, device=dev)
    with pytest.raises(binding.FoeError) as e:
        binding.route_noalloc(shape, W["ffn_norm_g"], W["router_w"], None, h, idx, w)
    assert e.value.code == -3
    torch.cuda.synchronize()
    assert int((idx != -7).sum()) == 0                     # outputs untouched
