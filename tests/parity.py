"""Shared machinery of the GPU parity tests: run the CUDA path through the C ABI, run the oracle on the
same seeded inputs, compare stage by stage with the tolerances the benchmark spec fixes.

Tolerances (bf16 weights and activations, fp32 accumulation on the GPU, float64 oracle):
  * routing: expert-id SETS equal for every (token, cluster) whose k-th / (k+1)-th oracle scores differ by
    at least 1e-5; gates equal to 1e-5 when matched by expert id   (both sides given the identical bf16 h);
  * dispatch maps: bit-exact against the oracle's permute() of the GPU's ids;
  * block output: max |err| <= 2e-2 * max |ref|  and  sum |err| / sum |ref| <= 5e-3.
The two output bounds are the task's, for the five workloads (weights N(0, 0.02^2)).  Stress cases that
scale the weights up make the attention and expert terms, each of which went through four to five bf16
roundings (unit roundoff 2^-8: folded gain, q/k/v, RoPE re-rounding, P, o / u, h_mid, y), dominate the
residual; for those the mean bound is 1.5e-2 (about five roundings in quadrature), and the same bound is used
for un-normalised intermediates (q, K/V pages, attention output, r_full, u) in every case.
Inside a full block the GPU's r_full carries bf16 noise far above 1e-5, so a few tokens legitimately pick
another expert.  The oracle is then evaluated with the GPU's ids for the experts stage, and every differing
(token, cluster) must be explainable: its oracle margin has to be below 2 * |u_gpu - u_ref|_2 * max_e |W_r[e]|_2
(how far input noise can move a score difference).
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from oracle import adapter
from oracle import foe_oracle as orc
from paper_2605_06206_b200 import binding, synth

MAX_ABS_TOL = 2e-2
MEAN_REL_TOL = 5e-3
STAGE_MAX_TOL = 3e-2      # intermediates and weight-scaled stress cases
STAGE_REL_TOL = 1.5e-2
TIE_MARGIN = 1e-5


def err_stats(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    err = np.abs(got - ref)
    return err.max() / max(np.abs(ref).max(), 1e-30), err.sum() / max(np.abs(ref).sum(), 1e-30)


def assert_close(got, ref, what, max_tol=MAX_ABS_TOL, rel_tol=MEAN_REL_TOL):
    mx, rel = err_stats(got, ref)
    assert mx <= max_tol and rel <= rel_tol, f"{what}: max_abs/max_ref={mx:.3e} (<= {max_tol}), rel_l1={rel:.3e} (<= {rel_tol})"
    return mx, rel


def scaled_weights(shape, seed, device, wscale=1.0, layer=0):
    W = synth.make_weights(shape, seed, device, layer=layer)
    if wscale != 1.0:
        for k in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down"):
            W[k] = (W[k].float() * wscale).to(torch.bfloat16)
        W["router_w"] = (W["router_w"] * wscale).to(torch.bfloat16).float()
    return W


def check_routing(shape, idx_gpu, w_gpu, logits_ref, idx_ref, w_ref):
    """Bit-exact routing check on identical inputs; returns the number of exempt (token, cluster) pairs."""
    cfg = adapter.cfg_from_shape(shape)
    margin = orc.topk_margin(cfg, logits_ref)
    exempt = margin < TIE_MARGIN
    gs, rs = np.sort(idx_gpu, -1), np.sort(idx_ref, -1)
    same = (gs == rs).all(-1)
    bad = ~same & ~exempt
    assert not bad.any(), f"{int(bad.sum())} non-exempt (token, cluster) pairs differ, first at {np.argwhere(bad)[:3].tolist()}"
    # gates matched by expert id
    og, orr = np.argsort(idx_gpu, -1), np.argsort(idx_ref, -1)
    wg = np.take_along_axis(w_gpu, og, -1)
    wr = np.take_along_axis(w_ref, orr, -1)
    dw = np.abs(wg - wr)[same]
    assert dw.size == 0 or dw.max() <= 1e-5, f"gate mismatch {dw.max():.3e}"
    np.testing.assert_allclose(w_gpu.sum(-1), 1.0, atol=1e-5)
    return int(exempt.sum())


def check_maps(shape, aux, idx_gpu):
    mp = orc.permute(idx_gpu, shape.n_experts)
    for k in ("counts", "offsets", "perm", "inv"):
        got = aux[k].cpu().numpy()
        assert np.array_equal(got, mp[k]), f"dispatch map {k} differs from the oracle's"
    return mp


def run_block_parity(shape, seed, q_lens: Sequence[int], ctx_lens: Sequence[int], decode=False, wscale=1.0,
                     router_bias: Optional[torch.Tensor] = None, rows: Optional[np.ndarray] = None,
                     shuffle_pages=True, weights=None, x=None, return_all=False) -> Dict:
    """One call through the C ABI against the oracle (all tokens, or the token subset `rows`)."""
    dev = "cuda"
    q_lens, ctx_lens = list(q_lens), list(ctx_lens)
    W = scaled_weights(shape, seed, dev, wscale) if weights is None else weights
    if router_bias is not None:
        W["router_b"] = router_bias.to(dev)
    S = sum(q_lens)
    x = synth.make_x(shape, seed, S, dev) if x is None else x
    kv = synth.make_paged_cache(shape, seed, ctx_lens, q_lens, dev, shuffle=shuffle_pages)
    cache = adapter.logical_cache(kv.k_pages, kv.v_pages, kv.block_table, ctx_lens, 64)
    layer = binding.FoeLayer(shape, W, max_tokens=max(S, 1), max_seqs=len(q_lens),
                             max_context=max(c + q for c, q in zip(ctx_lens, q_lens)))
    out = layer.decode(x, kv) if decode else layer.prefill(x, kv)
    assert layer.poll_status() == 0
    aux = layer.aux()
    launches = layer.last_launch_count()
    layer.close()
    res = compare_with_oracle(shape, W, x, q_lens, ctx_lens, cache, kv, out, aux, rows, stress=(wscale != 1.0))
    res["launches"] = launches
    if return_all:
        res.update(out=out, aux=aux, kv=kv, W=W, x=x)
    return res


def compare_with_oracle(shape, W, x, q_lens, ctx_lens, cache, kv, out, aux, rows=None, stress=False,
                        cluster_maps=None) -> Dict:
    """Stage-by-stage comparison of one finished GPU call (its output, intermediates `aux` and the cache `kv` it
    wrote) with the oracle run on the same inputs.  `cache` is the logical cache from before the call.
    `cluster_maps`: for a block that ran as one handle per cluster, the H per-cluster dispatch maps (each over the
    cluster's own E_c experts, ids local to the cluster) instead of one map over all experts in `aux`."""
    q_lens, ctx_lens = list(q_lens), list(ctx_lens)
    S = sum(q_lens)
    cfg = adapter.cfg_from_shape(shape)
    Wn = adapter.weights_to_numpy(W)
    xn = adapter.to_np(x)
    rsel = np.arange(S) if rows is None else np.asarray(rows)
    idx_gpu = aux["topk_idx"].cpu().numpy()
    ref = orc.foe_block(cfg, Wn, xn, q_lens, ctx_lens, cache, rows=rows)            # oracle's own routing
    ref_g = orc.moe_stage(cfg, Wn, ref["r_full"], idx_override=idx_gpu[rsel])      # experts with the GPU's ids

    # tier (i): everything up to the sync
    nq, nkv, dh = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    q_gpu = adapter.to_np(aux["q"])
    assert_close(q_gpu[rsel].reshape(len(rsel), nq, dh), ref["q"], "q after RoPE", STAGE_MAX_TOL, STAGE_REL_TOL)
    full = [c + q for c, q in zip(ctx_lens, q_lens)]
    newc = adapter.logical_cache(kv.k_pages, kv.v_pages, kv.block_table, full, 64)
    k_new = np.concatenate([newc[b][0][ctx_lens[b]:] for b in range(len(q_lens))])
    v_new = np.concatenate([newc[b][1][ctx_lens[b]:] for b in range(len(q_lens))])
    assert_close(k_new, ref["k_new"], "K written to the pages", STAGE_MAX_TOL, STAGE_REL_TOL)
    assert_close(v_new, ref["v_new"], "V written to the pages", STAGE_MAX_TOL, STAGE_REL_TOL)
    for b in range(len(q_lens)):                                                   # cached entries untouched
        if ctx_lens[b]:
            assert np.array_equal(newc[b][0][:ctx_lens[b]], cache[b][0]) and np.array_equal(newc[b][1][:ctx_lens[b]], cache[b][1])
    assert_close(adapter.to_np(aux["attn_o"])[rsel], ref["o"], "attention output", STAGE_MAX_TOL, STAGE_REL_TOL)
    # the attention stage by itself: the oracle's attend() on the GPU's own q and on the pages as the call left them
    # (both already bf16), so only the kernel's softmax and its two contractions are compared; the task's bounds
    qg = q_gpu[rsel].reshape(len(rsel), nq, dh).astype(np.float64)
    seq_of = np.repeat(np.arange(len(q_lens)), q_lens)
    o_iso = np.zeros((len(rsel), nq, dh))
    for b in range(len(q_lens)):
        sel = np.nonzero(seq_of[rsel] == b)[0]
        if len(sel):
            o_iso[sel] = orc.attend(qg[sel], ref["pos"][rsel[sel]], newc[b][0].astype(np.float64),
                                    newc[b][1].astype(np.float64), nq // nkv)
    assert_close(adapter.to_np(aux["attn_o"])[rsel], o_iso.reshape(len(rsel), -1), "attention on the GPU's q and pages")
    assert_close(adapter.to_np(aux["r_full"])[rsel], ref["r_full"], "r_full", STAGE_MAX_TOL, STAGE_REL_TOL)

    # tier (ii)/(iii): routing flips must be explained by the noise of the router input
    u_gpu = adapter.to_np(aux["u"])[rsel].astype(np.float64)
    same = (np.sort(idx_gpu[rsel], -1) == np.sort(ref["idx"], -1)).all(-1)          # [R, H]
    margin = orc.topk_margin(cfg, ref["logits"])
    r_gpu = adapter.to_np(aux["r_full"])[rsel].astype(np.float64)
    u_from_r = orc.rmsnorm(r_gpu, Wn["ffn_norm_g"], cfg.rms_eps)                    # GPU's fp32 u, before bf16 rounding
    tau = 2.0 * np.linalg.norm(u_from_r - ref["u"], axis=-1) * np.linalg.norm(Wn["router_w"].astype(np.float64), axis=-1).max()
    flips = ~same
    unexplained = flips & (margin >= tau[:, None] + TIE_MARGIN)
    assert not unexplained.any(), f"{int(unexplained.sum())} routing flips with margin above the noise bound"
    assert_close(u_gpu, ref["u"], "FFN-normed u", STAGE_MAX_TOL, STAGE_REL_TOL)

    H, kc = shape.n_clusters, shape.top_k_per_cluster
    Ec = shape.experts_per_cluster
    if cluster_maps is None:
        maps = check_maps(shape, aux, idx_gpu)
        assert int(maps["counts"].sum()) == S * H * kc
        for h in range(H):                                                         # every cluster gets S*k_c rows
            assert int(maps["counts"][h * Ec:(h + 1) * Ec].sum()) == S * kc
        counts = maps["counts"]
    else:
        per = []
        for h in range(H):
            mp = orc.permute(idx_gpu[:, h:h + 1] - h * Ec, Ec)
            for k in ("counts", "offsets", "perm", "inv"):
                assert np.array_equal(cluster_maps[h][k].cpu().numpy(), mp[k]), f"cluster {h}: dispatch map {k} differs"
            assert int(mp["counts"].sum()) == S * kc
            per.append(mp["counts"])
        counts = np.concatenate(per)

    got = adapter.to_np(out)
    got = got[:, rsel] if shape.grouped_output else got[rsel]
    # the experts stage by itself: the oracle fed the GPU's own fp32 r_full and ids, so that noise from before the sync
    # (which scaled weights amplify through the softmax) does not enter; the task's output bounds apply in every case
    iso = orc.moe_stage(cfg, Wn, r_gpu, idx_override=idx_gpu[rsel])
    assert_close(got, iso["out"], "experts stage on the GPU's r_full")
    if not stress:
        mx, rel = assert_close(got, ref_g["out"], "block output")
    else:
        mx, rel = assert_close(got, ref_g["out"], "block output (scaled weights)", STAGE_MAX_TOL, STAGE_REL_TOL)
    return dict(max_abs=mx, rel_l1=rel, flips=int(flips.sum()), counts=counts, ref=ref)


def check_every_row(shape, W, out, aux, kv, q_lens, ctx_lens, attn_seqs: Sequence[int], chunk: int = 4096) -> Dict:
    """Full-size parity over EVERY output row of one finished call, stage by stage, at the task's bounds.

    Experts stage: the oracle's moe_stage on the GPU's own fp32 r_full and expert ids, for all tokens (in chunks of
    tokens: the stage is per token, so chunking changes nothing), against the block output -- every row of every
    256-row tile of every expert's grouped GEMM enters the maximum.  Attention stage: the oracle's attend() on the
    GPU's q and on the pages as the call left them, for all rows of the sequences in `attn_seqs`, against the
    attention output -- every 128-row query block of those sequences."""
    q_lens, ctx_lens = list(q_lens), list(ctx_lens)
    S = sum(q_lens)
    cfg = adapter.cfg_from_shape(shape)
    Wn = adapter.weights_to_numpy(W)
    r_gpu = adapter.to_np(aux["r_full"])
    idx_gpu = aux["topk_idx"].cpu().numpy()
    got = adapter.to_np(out)
    max_err = max_ref = sum_err = sum_ref = 0.0
    worst_tok = -1
    for t0 in range(0, S, chunk):
        t1 = min(S, t0 + chunk)
        iso = orc.moe_stage(cfg, Wn, r_gpu[t0:t1].astype(np.float64), idx_override=idx_gpu[t0:t1])["out"]
        g = (got[:, t0:t1] if shape.grouped_output else got[t0:t1]).astype(np.float64)
        err = np.abs(g - iso)
        if err.max() > max_err:
            max_err = float(err.max())
            worst_tok = t0 + int(np.unravel_index(err.argmax(), err.shape)[-2])
        max_ref = max(max_ref, float(np.abs(iso).max()))
        sum_err += float(err.sum())
        sum_ref += float(np.abs(iso).sum())
    e_max, e_rel = max_err / max_ref, sum_err / sum_ref
    assert e_max <= MAX_ABS_TOL and e_rel <= MEAN_REL_TOL, \
        f"experts stage over all {S} tokens: max_abs/max_ref={e_max:.3e} at token {worst_tok}, rel_l1={e_rel:.3e}"

    nq, nkv, dh = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    starts = np.concatenate([[0], np.cumsum(q_lens)])
    full = [c + q for c, q in zip(ctx_lens, q_lens)]
    a_stats = []
    for b in attn_seqs:
        lo, hi = int(starts[b]), int(starts[b + 1])
        newc = adapter.logical_cache(kv.k_pages, kv.v_pages, kv.block_table[b:b + 1], [full[b]], 64)[0]
        qg = adapter.to_np(aux["q"][lo:hi]).reshape(hi - lo, nq, dh).astype(np.float64)
        pos = ctx_lens[b] + np.arange(hi - lo)
        o_iso = orc.attend(qg, pos, newc[0].astype(np.float64), newc[1].astype(np.float64), nq // nkv)
        a_stats.append(assert_close(adapter.to_np(aux["attn_o"][lo:hi]), o_iso.reshape(hi - lo, -1),
                                    f"attention, every row of sequence {b}"))
    return dict(experts_max=e_max, experts_rel=e_rel, attention=a_stats)
