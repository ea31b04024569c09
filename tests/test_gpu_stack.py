"""Stacks of FoE layers through the C ABI: first / middle / last boundary forms feeding each other, one shared
workspace, prefill followed by decode steps on per-layer paged caches.

The small stack is checked end to end; the full 16-layer workload (hidden 4096, 8 clusters x 16 experts, 2 x 16384
prompt tokens, 128 decode steps, and its one-cluster equal-size MoE twin) is checked layer by layer with teacher
forcing: the oracle gets the GPU's own input to a layer, so depth error is not conflated with kernel error."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import adapter
from oracle import foe_oracle as orc
from paper_2605_06206_b200 import binding, synth

from parity import assert_close, compare_with_oracle, scaled_weights

pytestmark = pytest.mark.gpu


class Stack:
    """n_layers FoE layers (first, middle..., last) sharing one workspace, each with its own paged cache."""

    def __init__(self, base, n_layers, seed, q_lens, extra_tokens, wscale=1.0, keep_weights=()):
        self.base, self.n_layers, self.seed = base, n_layers, seed
        self.n_seqs = len(q_lens)
        S = sum(q_lens)
        self.max_context = max(q_lens) + extra_tokens
        self.layers, self.shapes, self.kept = [], [], {}
        for l in range(n_layers):
            pos = "first" if l == 0 else ("last" if l == n_layers - 1 else "middle")
            if n_layers == 1:
                pos = "single"
            sh = dataclasses.replace(base, position=pos)
            W = scaled_weights(sh, seed, "cuda", wscale, layer=l + 1)
            self.layers.append(binding.FoeLayer(sh, W, max_tokens=S, max_seqs=self.n_seqs, max_context=self.max_context,
                                                share_workspace_with=self.layers[0] if self.layers else None))
            self.shapes.append(sh)
            if l in keep_weights:
                self.kept[l] = {k: v.cpu() for k, v in W.items()}
            del W
        torch.cuda.empty_cache()
        total = [q + extra_tokens for q in q_lens]
        self.kvs = [synth.make_paged_cache(base, seed, [0] * self.n_seqs, total, "cuda", fill_random=False)
                    for _ in range(n_layers)]
        for kv in self.kvs:
            kv.q_lens = torch.tensor(q_lens, dtype=torch.int32, device="cuda")

    def forward(self, x, context_lens, decode, capture=()):
        """Runs all layers; returns the final output and, for the layer indices in `capture`, a record of the
        layer's input, output, intermediates and the logical cache from before the call."""
        rec = {}
        ctx_t = torch.tensor(context_lens, dtype=torch.int32, device="cuda")
        h = x
        for l, layer in enumerate(self.layers):
            kv = self.kvs[l]
            kv.context_lens = ctx_t
            before = None
            if l in capture:
                before = adapter.logical_cache(kv.k_pages, kv.v_pages, kv.block_table, context_lens, 64)
            out = layer.decode(h, kv) if decode else layer.prefill(h, kv)
            if l in capture:
                rec[l] = dict(x=h.clone(), out=out.clone(), aux=layer.aux(), cache=before)
            h = out
        assert self.layers[0].poll_status() == 0
        return h, rec

    def close(self):
        for layer in self.layers:
            layer.close()


def _rows(q_lens, per_seq, seed):
    rows, at = [], 0
    for b, T in enumerate(q_lens):
        pick = synth.uniform_int(seed, 700 + b, per_seq, 0, T - 1).tolist() + [0, T - 1, 63, 64]
        rows += sorted({at + p for p in pick if p < T})
        at += T
    return np.array(rows, dtype=np.int64)


def test_small_stack_end_to_end_against_oracle_stack():
    base = synth.LayerShape(256, 8, 4, 4, 64, 8, 2, 128)
    q_lens, steps = [90, 41], 3
    st = Stack(base, 4, 31, q_lens, steps, wscale=2.0, keep_weights=range(4))
    x0 = synth.make_x(st.shapes[0], 31, sum(q_lens), "cuda")
    out, rec = st.forward(x0, [0, 0], decode=False, capture=range(4))
    assert out.shape == (sum(q_lens), 256)
    # teacher-forced, layer by layer
    for l in range(4):
        W = {k: v.cuda() for k, v in st.kept[l].items()}
        r = compare_with_oracle(st.shapes[l], W, rec[l]["x"], q_lens, [0, 0], rec[l]["cache"], st.kvs[l], rec[l]["out"],
                                rec[l]["aux"], stress=True)
    # free-running oracle stack (float64 all the way): report the drift, bound it loosely
    h = adapter.to_np(x0).astype(np.float64)
    for l in range(4):
        h = orc.foe_block(adapter.cfg_from_shape(st.shapes[l]), adapter.weights_to_numpy(st.kept[l]), h, q_lens)["out"]
    got = adapter.to_np(out).astype(np.float64)
    tok_err = np.abs(got - h).sum(-1) / np.abs(h).sum(-1)
    print("4-layer drift: median token rel err %.3e, max %.3e" % (np.median(tok_err), tok_err.max()))
    assert np.median(tok_err) < 2e-2
    # decode steps on top of the prefilled caches
    ctx = list(q_lens)
    for s in range(steps):
        xs = synth.make_x(st.shapes[0], 31, 2, "cuda", tid=synth.TID["x_step"] + s)
        o, rec = st.forward(xs, ctx, decode=True, capture=(0, 3))
        for l in (0, 3):
            W = {k: v.cuda() for k, v in st.kept[l].items()}
            compare_with_oracle(st.shapes[l], W, rec[l]["x"], [1, 1], ctx, rec[l]["cache"], st.kvs[l], rec[l]["out"],
                                rec[l]["aux"], stress=True)
        ctx = [c + 1 for c in ctx]
    st.close()


def _run_workload5(n_clusters, checked_layers, rows_per_seq, decode_steps, checked_steps):
    shape, info = synth.workload(5)
    if n_clusters == 1:            # the equal-size MoE baseline: one global router over the same 128 experts
        shape = dataclasses.replace(shape, n_clusters=1, experts_per_cluster=128, top_k_per_cluster=16)
    q_lens = info["q_lens"]
    L = info["layers"]
    st = Stack(shape, L, info["seed"], q_lens, decode_steps)
    x0 = synth.make_x(st.shapes[0], info["seed"], sum(q_lens), "cuda")
    out, rec = st.forward(x0, [0, 0], decode=False, capture=checked_layers)
    assert out.shape == (sum(q_lens), shape.hidden) and bool(torch.isfinite(out.float()).all())
    rows = _rows(q_lens, rows_per_seq, info["seed"])
    for l in checked_layers:
        W = synth.make_weights(st.shapes[l], info["seed"], "cuda", layer=l + 1)
        r = compare_with_oracle(st.shapes[l], W, rec[l]["x"], q_lens, [0, 0], rec[l]["cache"], st.kvs[l], rec[l]["out"],
                                rec[l]["aux"], rows=rows)
        print(f"workload 5 (H={n_clusters}) prefill layer {l + 1}: max {r['max_abs']:.2e} mean {r['rel_l1']:.2e} flips {r['flips']}")
        del W, rec[l]
    ctx = list(q_lens)
    for s in range(decode_steps):
        xs = synth.make_x(st.shapes[0], info["seed"], len(q_lens), "cuda", tid=synth.TID["x_step"] + s)
        cap = (0, L - 1) if s in checked_steps else ()
        o, rec = st.forward(xs, ctx, decode=True, capture=cap)
        for l in cap:
            W = synth.make_weights(st.shapes[l], info["seed"], "cuda", layer=l + 1)
            r = compare_with_oracle(st.shapes[l], W, rec[l]["x"], [1] * len(q_lens), ctx, rec[l]["cache"], st.kvs[l],
                                    rec[l]["out"], rec[l]["aux"])
            print(f"workload 5 (H={n_clusters}) decode step {s} layer {l + 1}: max {r['max_abs']:.2e} mean {r['rel_l1']:.2e}")
            del W
        ctx = [c + 1 for c in ctx]
    assert bool(torch.isfinite(o.float()).all())
    st.close()
    torch.cuda.empty_cache()


def test_workload5_foe_stack_prefill_and_128_decode_steps():
    _run_workload5(8, checked_layers=(0, 1, 15), rows_per_seq=10, decode_steps=128, checked_steps=(0, 127))


def test_workload5_one_cluster_moe_baseline_stack():
    _run_workload5(1, checked_layers=(0, 15), rows_per_seq=8, decode_steps=128, checked_steps=(127,))


def test_package_stack_helper_matches_layer_by_layer_calls():
    """paper_2605_06206_b200.stack.FoeStack (used by bench.py --stack) is plumbing over the same layer calls: its
    prefill and decode outputs equal those of hand-driven layers built from the same seeds, bit for bit."""
    from paper_2605_06206_b200.stack import FoeStack
    base = synth.LayerShape(256, 8, 4, 4, 64, 8, 2, 128)
    q_lens, L, extra = [150, 77], 3, 2
    st = FoeStack(base, L, 9, q_lens, extra)
    S = sum(q_lens)
    x = synth.make_x(st.shapes[0], 9, S, "cuda")
    out_p = st.forward(x, [0, 0], decode=False).clone()
    xs = synth.make_x(st.shapes[0], 9, len(q_lens), "cuda", tid=synth.TID["x_step"])
    out_d = st.forward(xs, q_lens, decode=True).clone()
    assert st.status() == 0
    st.close()
    # by hand
    layers, kvs = [], []
    for l in range(L):
        sh = dataclasses.replace(base, position=("first", "middle", "last")[l])
        W = synth.make_weights(sh, 9, "cuda", layer=l + 1)
        layers.append(binding.FoeLayer(sh, W, max_tokens=S, max_seqs=len(q_lens), max_context=max(q_lens) + extra))
        kvs.append(synth.make_paged_cache(base, 9, [0, 0], [q + extra for q in q_lens], "cuda", fill_random=False))
    h = x
    for layer, kv in zip(layers, kvs):
        kv.q_lens = torch.tensor(q_lens, dtype=torch.int32, device="cuda")
        h = layer.prefill(h, kv)
    assert torch.equal(h, out_p)
    h = xs
    for layer, kv in zip(layers, kvs):
        kv.context_lens = torch.tensor(q_lens, dtype=torch.int32, device="cuda")
        h = layer.decode(h, kv)
    assert torch.equal(h, out_d)
    for layer in layers:
        layer.close()
