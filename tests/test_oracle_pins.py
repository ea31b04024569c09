"""Pins for the CPU oracle: everything here checks oracle/foe_oracle.py against something
other than itself -- independently written torch code, library routines (SDPA, topk),
closed forms, invariants, brute force, and the closed forms printed in the paper."""
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import foe_oracle as orc
from paper_2605_06206_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def small_shape(H=4, position="middle", sync="mean", nq=8, nkv=4, Ec=6, kc=2):
    return synth.LayerShape(hidden=64, n_q_heads=nq, n_kv_heads=nkv, n_clusters=H, head_dim=16,
                            experts_per_cluster=Ec, top_k_per_cluster=kc, ffn_inter=32,
                            rope_theta=1.0e4, rms_eps=1.0e-6, position=position, sync=sync)


def to_cfg(s: synth.LayerShape) -> orc.FoeConfig:
    return orc.FoeConfig(s.hidden, s.n_q_heads, s.n_kv_heads, s.n_clusters, s.head_dim,
                         s.experts_per_cluster, s.top_k_per_cluster, s.ffn_inter, s.rope_theta,
                         s.rms_eps, s.position, s.sync)


def np_weights(s, seed=0, wscale=1.0):
    W = synth.make_weights(s, seed)
    out = {k: v.to(torch.float64).numpy() for k, v in W.items()}
    if wscale != 1.0:  # larger weights make attention/experts matter in tiny shapes
        for k in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "router_w"):
            out[k] = out[k] * wscale
    return out


def np_x(s, seed, S):
    return synth.make_x(s, seed, S).to(torch.float64).numpy()


# --------------------------------------------------------------------------------------
# independent pieces (torch, written separately from the oracle)
# --------------------------------------------------------------------------------------

def t_rmsnorm(x, g, eps):
    return x * torch.rsqrt((x * x).mean(-1, keepdim=True) + eps) * g


def t_rope_complex(t, pos, theta):
    """RoPE via complex multiplication on pairs (j, j + dh/2)."""
    dh = t.shape[-1]
    half = dh // 2
    z = torch.complex(t[..., :half], t[..., half:])
    freqs = theta ** (-torch.arange(0, half, dtype=torch.float64) * 2.0 / dh)
    ang = pos.to(torch.float64)[:, None] * freqs[None, :]
    rot = torch.polar(torch.ones_like(ang), ang)[:, None, :]
    z = z * rot
    return torch.cat([z.real, z.imag], dim=-1)


def t_gqa_attention(x, W, s, q_lens, first_pos=None):
    """Textbook pre-norm GQA attention with concatenated per-cluster weights; returns o @ W_O [S, d]."""
    x = torch.as_tensor(x)
    S = x.shape[0]
    wq = torch.cat([torch.as_tensor(W["wq"][h]) for h in range(s.n_clusters)], dim=1)
    wk = torch.cat([torch.as_tensor(W["wk"][h]) for h in range(s.n_clusters)], dim=1)
    wv = torch.cat([torch.as_tensor(W["wv"][h]) for h in range(s.n_clusters)], dim=1)
    n = t_rmsnorm(x, torch.as_tensor(W["attn_norm_g"]), s.rms_eps)
    q = (n @ wq).view(S, s.n_q_heads, s.head_dim)
    k = (n @ wk).view(S, s.n_kv_heads, s.head_dim)
    v = (n @ wv).view(S, s.n_kv_heads, s.head_dim)
    outs = []
    at = 0
    for b, T in enumerate(q_lens):
        p0 = 0 if first_pos is None else first_pos[b]
        pos = torch.arange(p0, p0 + T)
        qb = t_rope_complex(q[at:at + T], pos, s.rope_theta).transpose(0, 1)[None]
        kb = t_rope_complex(k[at:at + T], pos, s.rope_theta).transpose(0, 1)[None]
        vb = v[at:at + T].transpose(0, 1)[None]
        rep = s.n_q_heads // s.n_kv_heads
        kb = kb.repeat_interleave(rep, dim=1)
        vb = vb.repeat_interleave(rep, dim=1)
        ob = F.scaled_dot_product_attention(qb, kb, vb, is_causal=True)
        outs.append(ob[0].transpose(0, 1).reshape(T, -1))
        at += T
    o = torch.cat(outs, 0)
    return o @ torch.as_tensor(W["wo"])


def t_standard_moe_block(x, W, s, q_lens):
    """Left column of Table 2: a standard token-choice MoE block (global top-k)."""
    x = torch.as_tensor(x)
    r = x + t_gqa_attention(x, W, s, q_lens)
    u = t_rmsnorm(r, torch.as_tensor(W["ffn_norm_g"]), s.rms_eps)
    logits = (u @ torch.as_tensor(W["router_w"]).T + torch.as_tensor(W["router_b"])).to(torch.float32)
    k = s.top_k_per_cluster
    topv, topi = torch.topk(logits, k, dim=-1)
    gates = torch.softmax(topv.to(torch.float64), dim=-1)
    out = r.clone()
    for i in range(x.shape[0]):
        for j in range(k):
            e = int(topi[i, j])
            hmid = F.silu(u[i] @ torch.as_tensor(W["w_gate"][e])) * (u[i] @ torch.as_tensor(W["w_up"][e]))
            out[i] += gates[i, j] * (hmid @ torch.as_tensor(W["w_down"][e]))
    return out, topi, gates


# --------------------------------------------------------------------------------------
# pins
# --------------------------------------------------------------------------------------

@pytest.mark.parametrize("position", ["middle", "single", "first", "last"])
def test_one_cluster_is_a_standard_moe_block(position):
    s = small_shape(H=1, position=position, Ec=12, kc=3)
    W = np_weights(s, 1, wscale=8.0)
    q_lens = [9, 14]
    S = sum(q_lens)
    x = np_x(s, 1, S)
    res = orc.foe_block(to_cfg(s), W, x, q_lens)
    xin = x if not s.grouped_input else x[0]
    ref, topi, gates = t_standard_moe_block(xin, W, s, q_lens)
    out = res["out"] if not s.grouped_output else res["out"][0]
    assert np.array_equal(res["idx"][:, 0, :], topi.numpy())
    np.testing.assert_allclose(res["w"][:, 0, :], gates.numpy(), rtol=0, atol=1e-12)
    np.testing.assert_allclose(out, ref.numpy(), rtol=0, atol=1e-10)
    # sanity: attention and experts both matter at this weight scale
    assert np.abs(ref.numpy() - xin).max() > 1e-2


def test_brute_force_dense_experts():
    for position in ("middle", "last"):
        s = small_shape(H=4, position=position)
        cfg = to_cfg(s)
        W = np_weights(s, 2, wscale=8.0)
        S = 11
        rng = np.random.default_rng(0)
        r_full = rng.standard_normal((S, s.hidden))
        res = orc.moe_stage(cfg, W, r_full)
        u = torch.as_tensor(res["u"])
        E = s.n_experts
        dense = torch.stack([
            (F.silu(u @ torch.as_tensor(W["w_gate"][e])) * (u @ torch.as_tensor(W["w_up"][e])))
            @ torch.as_tensor(W["w_down"][e]) for e in range(E)], dim=1)          # [S, E, d]
        G = torch.zeros(S, E, dtype=torch.float64)
        for i in range(S):
            for h in range(s.n_clusters):
                for j in range(s.top_k_per_cluster):
                    G[i, res["idx"][i, h, j]] = res["w"][i, h, j]
        Ec = s.experts_per_cluster
        per_cluster = torch.stack([
            torch.as_tensor(r_full) + torch.einsum("se,sed->sd", G[:, h * Ec:(h + 1) * Ec],
                                                   dense[:, h * Ec:(h + 1) * Ec])
            for h in range(s.n_clusters)], dim=0)
        np.testing.assert_allclose(res["x_next"], per_cluster.numpy(), rtol=0, atol=1e-11)
        if position == "last":
            # last layer = one dense MoE with gates w / H
            one = torch.as_tensor(r_full) + torch.einsum("se,sed->sd", G / s.n_clusters, dense)
            np.testing.assert_allclose(res["out"], one.numpy(), rtol=0, atol=1e-11)
        else:
            np.testing.assert_allclose(res["out"], per_cluster.numpy(), rtol=0, atol=1e-11)


def test_gates_sum_to_one_and_three_formulations_agree():
    s = small_shape(H=4, Ec=8, kc=3)
    cfg = to_cfg(s)
    W = np_weights(s, 3, wscale=20.0)
    rng = np.random.default_rng(1)
    rt = orc.route(cfg, W, rng.standard_normal((50, s.hidden)))
    np.testing.assert_allclose(rt["w"].sum(-1), 1.0, rtol=0, atol=1e-12)
    assert (rt["w"] > 0).all()
    lg = torch.as_tensor(rt["logits"].astype(np.float64))
    Ec, kc = s.experts_per_cluster, s.top_k_per_cluster
    glob = torch.softmax(lg, dim=-1)                                  # global softmax, then slice
    for h in range(s.n_clusters):
        sl = slice(h * Ec, (h + 1) * Ec)
        v1, i1 = torch.topk(glob[:, sl], kc, dim=-1)
        w1 = v1 / v1.sum(-1, keepdim=True)
        v2, i2 = torch.topk(torch.softmax(lg[:, sl], dim=-1), kc, dim=-1)   # per-cluster softmax
        w2 = v2 / v2.sum(-1, keepdim=True)
        assert np.array_equal(i1.numpy() + h * Ec, rt["idx"][:, h])
        assert np.array_equal(i2.numpy() + h * Ec, rt["idx"][:, h])
        np.testing.assert_allclose(w1.numpy(), rt["w"][:, h], rtol=0, atol=1e-9)
        np.testing.assert_allclose(w2.numpy(), rt["w"][:, h], rtol=0, atol=1e-9)


def test_topk_matches_library_and_tie_rule():
    s = small_shape(H=3, nq=6, nkv=3, Ec=7, kc=3)
    cfg = to_cfg(s)
    rng = np.random.default_rng(2)
    logits = rng.standard_normal((200, s.n_experts)).astype(np.float32)
    idx, w = orc.topk_per_cluster(cfg, logits)
    for h in range(3):
        v, i = torch.topk(torch.as_tensor(logits[:, h * 7:(h + 1) * 7]), 3, dim=-1)
        assert np.array_equal(i.numpy() + h * 7, idx[:, h])
    # ties: lower index wins, list is ordered (descending value, ascending index)
    tie = np.zeros((1, s.n_experts), dtype=np.float32)
    tie[0, 2] = 1.0
    idx, w = orc.topk_per_cluster(cfg, tie)
    assert idx[0, 0].tolist() == [2, 0, 1]
    assert idx[0, 1].tolist() == [7, 8, 9]
    np.testing.assert_allclose(w[0, 1], 1.0 / 3.0, atol=1e-15)
    m = orc.topk_margin(cfg, tie)
    assert m[0, 0] == 0.0 and m[0, 1] == 0.0
    # bias shifts selection and gates alike
    Wb = dict(router_w=np.zeros((s.n_experts, s.hidden)), router_b=np.arange(s.n_experts, dtype=np.float64))
    lg = orc.router_logits(cfg, Wb, np.ones((1, s.hidden)))
    idx, w = orc.topk_per_cluster(cfg, lg)
    assert idx[0, 0].tolist() == [6, 5, 4]
    e = np.exp(np.array([0.0, -1.0, -2.0]))
    np.testing.assert_allclose(w[0, 0], e / e.sum(), atol=1e-12)


def test_topk_margin_on_hand_written_scores_and_by_brute_force():
    """The margin decides which (token, cluster) pairs the bit-exact routing check may skip, so it is pinned by
    itself: hand-written scores whose adjacent gaps all differ (an off-by-one in the position picks another gap),
    an unsorted row, a cluster with exactly k_c experts, and a definition that does not sort."""
    s = small_shape(H=2, nq=4, nkv=2, Ec=4, kc=2)
    cfg = to_cfg(s)
    # cluster 0: sorted gaps 2, 0.5, 1.5 -> k_c = 2 gives 3 - 2.5; cluster 1 is given unsorted: sorted 9, 4, 3, -1 -> 4 - 3
    logits = np.array([[5.0, 3.0, 2.5, 1.0, 3.0, -1.0, 9.0, 4.0]], dtype=np.float32)
    m = orc.topk_margin(cfg, logits)
    assert m.shape == (1, 2)
    assert m[0, 0] == 0.5 and m[0, 1] == 1.0
    # k_c = 1 and k_c = 3 on the same scores pick the other gaps
    assert orc.topk_margin(to_cfg(small_shape(H=2, nq=4, nkv=2, Ec=4, kc=1)), logits)[0].tolist() == [2.0, 5.0]
    assert orc.topk_margin(to_cfg(small_shape(H=2, nq=4, nkv=2, Ec=4, kc=3)), logits)[0].tolist() == [1.5, 4.0]
    # as many experts as selections: nothing can flip
    assert np.all(np.isinf(orc.topk_margin(to_cfg(small_shape(H=2, nq=4, nkv=2, Ec=4, kc=4)), logits)))
    # definition without sorting: the smallest selected score minus the largest score left out, with the selection
    # taken from topk_per_cluster
    s3 = small_shape(H=3, nq=6, nkv=3, Ec=7, kc=3)
    cfg3 = to_cfg(s3)
    rng = np.random.default_rng(5)
    lg = rng.standard_normal((300, s3.n_experts)).astype(np.float32)
    idx, _ = orc.topk_per_cluster(cfg3, lg)
    m3 = orc.topk_margin(cfg3, lg)
    for i in range(300):
        for h in range(3):
            chosen = set(idx[i, h].tolist())
            rest = [e for e in range(h * 7, (h + 1) * 7) if e not in chosen]
            want = float(min(lg[i, e] for e in chosen)) - float(max(lg[i, e] for e in rest))
            assert m3[i, h] == want and want >= 0.0


def test_dispatch_invariants():
    s = small_shape(H=4, Ec=8, kc=2)
    cfg = to_cfg(s)
    W = np_weights(s, 4, wscale=20.0)
    rng = np.random.default_rng(3)
    S = 97
    rt = orc.route(cfg, W, rng.standard_normal((S, s.hidden)))
    mp = orc.permute(rt["idx"], s.n_experts)
    E, Ec, kc, H = s.n_experts, s.experts_per_cluster, s.top_k_per_cluster, s.n_clusters
    R = S * H * kc
    # every cluster receives exactly S*k_c rows: the paper's load ratio of 1.0 across groups
    for h in range(H):
        assert mp["counts"][h * Ec:(h + 1) * Ec].sum() == S * kc
    assert mp["offsets"][0] == 0 and mp["offsets"][-1] == R
    assert (np.diff(mp["offsets"]) == mp["counts"]).all()
    assert sorted(mp["inv"].reshape(-1).tolist()) == list(range(R))          # bijection
    for i in range(S):
        for h in range(H):
            sl = mp["inv"][i, h]
            assert len(set(rt["idx"][i, h].tolist())) == kc                  # k_c distinct experts
            for j in range(kc):
                assert mp["perm"][sl[j]] == i
                e = rt["idx"][i, h, j]
                assert mp["offsets"][e] <= sl[j] < mp["offsets"][e + 1]
                assert h * Ec <= e < (h + 1) * Ec
    for e in range(E):                                                       # tokens ascend inside an expert
        seg = mp["perm"][mp["offsets"][e]:mp["offsets"][e + 1]]
        assert (np.diff(seg) > 0).all()
    # independent construction: stable sort of the flattened expert ids
    flat = rt["idx"].reshape(-1)
    order = np.argsort(flat, kind="stable")
    assert np.array_equal(mp["perm"], (order // (H * kc)).astype(np.int32))


def test_cluster_attention_sums_to_textbook_gqa_and_boundary_forms():
    s = small_shape(H=4)
    W = np_weights(s, 5, wscale=8.0)
    q_lens = [7, 12]
    S = sum(q_lens)
    x1 = np_x(small_shape(H=4, position="first"), 5, S)                  # [S, d]
    xrep = np.broadcast_to(x1, (4, S, s.hidden)).copy()
    gqa = t_gqa_attention(x1, W, s, q_lens).numpy()
    assert np.abs(gqa).max() > 1e-2
    mid = orc.attention_stage(to_cfg(s), W, xrep, q_lens)
    np.testing.assert_allclose(mid["a"].sum(0), gqa, rtol=0, atol=1e-11)
    np.testing.assert_allclose(mid["r_full"], x1 + gqa / 4.0, rtol=0, atol=1e-11)
    ssum = small_shape(H=4, sync="sum")
    msum = orc.attention_stage(to_cfg(ssum), W, xrep, q_lens)
    np.testing.assert_allclose(msum["r_full"], 4.0 * mid["r_full"], rtol=0, atol=1e-11)
    first = orc.attention_stage(to_cfg(small_shape(H=4, position="first")), W, x1, q_lens)
    np.testing.assert_allclose(first["r_full"], x1 + gqa, rtol=0, atol=1e-11)
    assert first["r"].shape == (S, s.hidden)
    # distinct streams: r[h] = x[h] + a[h] and r_full is their mean
    xd = np_x(s, 6, S)
    md = orc.attention_stage(to_cfg(s), W, xd, q_lens)
    np.testing.assert_allclose(md["r"], xd + md["a"], rtol=0, atol=0)
    np.testing.assert_allclose(md["r_full"], md["r"].mean(0), rtol=0, atol=1e-13)
    # each cluster's attention only sees its own stream
    xe = xd.copy()
    xe[2] += 1.0
    me = orc.attention_stage(to_cfg(s), W, xe, q_lens)
    for h in (0, 1, 3):
        assert np.array_equal(me["a"][h], md["a"][h])
    assert not np.array_equal(me["a"][2], md["a"][2])


def test_last_layer_is_mean_of_middle_output():
    s_mid, s_last = small_shape(H=4), small_shape(H=4, position="last")
    W = np_weights(s_mid, 7, wscale=8.0)
    q_lens = [10]
    x = np_x(s_mid, 7, 10)
    mid = orc.foe_block(to_cfg(s_mid), W, x, q_lens)
    last = orc.foe_block(to_cfg(s_last), W, x, q_lens)
    assert mid["out"].shape == (4, 10, s_mid.hidden) and last["out"].shape == (10, s_mid.hidden)
    np.testing.assert_allclose(last["out"], mid["out"].mean(0), rtol=0, atol=1e-13)
    # clusters differ only by their expert sums: x'[h] - r_full is the expert term
    assert not np.allclose(mid["out"][0], mid["out"][1])
    # "sum" changes the sync only; the last-layer mean stays a mean
    s_ls = small_shape(H=4, position="last", sync="sum")
    ls = orc.foe_block(to_cfg(s_ls), W, x, q_lens)
    np.testing.assert_allclose(ls["out"], ls["x_next"].mean(0), rtol=0, atol=1e-13)


def test_causality_and_batch_independence():
    s = small_shape(H=4)
    cfg = to_cfg(s)
    W = np_weights(s, 8, wscale=8.0)
    q_lens = [9, 6]
    x = np_x(s, 8, 15)
    base = orc.foe_block(cfg, W, x, q_lens)["out"]
    xp = x.copy()
    xp[:, 5, :] += 0.5                                  # perturb token 5 of sequence 0
    pert = orc.foe_block(cfg, W, xp, q_lens)["out"]
    assert np.array_equal(pert[:, :5], base[:, :5])     # earlier tokens bit-identical
    assert np.array_equal(pert[:, 9:], base[:, 9:])     # the other sequence too
    assert not np.array_equal(pert[:, 5:9], base[:, 5:9])
    alone = orc.foe_block(cfg, W, x[:, 9:], [6])["out"]
    np.testing.assert_allclose(alone, base[:, 9:], rtol=0, atol=1e-12)


def test_rope_is_a_rotation_and_shift_invariant():
    rng = np.random.default_rng(4)
    T, dh = 13, 16
    q = rng.standard_normal((T, 2, dh))
    k = rng.standard_normal((T, 1, dh))
    v = rng.standard_normal((T, 1, dh))
    pos = np.arange(T)
    r0 = orc.rope(q, pos, 1e4)
    np.testing.assert_allclose(np.linalg.norm(r0, axis=-1), np.linalg.norm(q, axis=-1), atol=1e-12)
    np.testing.assert_allclose(orc.rope(q, np.zeros(T, dtype=np.int64), 1e4), q, atol=0)
    ref = t_rope_complex(torch.as_tensor(q), torch.arange(T), 1e4).numpy()
    np.testing.assert_allclose(r0, ref, atol=1e-12)
    # explicit pair check for one element: (j, j+dh/2) rotated by p * theta^(-2j/dh)
    p, j = 7, 3
    ang = p * 1e4 ** (-2.0 * j / dh)
    np.testing.assert_allclose(r0[p, 1, j], q[p, 1, j] * math.cos(ang) - q[p, 1, j + 8] * math.sin(ang), atol=1e-13)
    np.testing.assert_allclose(r0[p, 1, j + 8], q[p, 1, j + 8] * math.cos(ang) + q[p, 1, j] * math.sin(ang), atol=1e-13)
    o0 = orc.attend(orc.rope(q, pos, 1e4), pos, orc.rope(k, pos, 1e4), v, 2)
    o1 = orc.attend(orc.rope(q, pos + 1000, 1e4), pos, orc.rope(k, pos + 1000, 1e4), v, 2)
    np.testing.assert_allclose(o0, o1, atol=1e-9)


def test_attend_matches_sdpa_with_cache_offset():
    rng = np.random.default_rng(5)
    Tk, Tq, dh = 21, 4, 16
    q = rng.standard_normal((Tq, 4, dh))
    K = rng.standard_normal((Tk, 2, dh))
    V = rng.standard_normal((Tk, 2, dh))
    qpos = np.arange(Tk - Tq, Tk)
    o = orc.attend(q, qpos, K, V, 2)
    mask = torch.as_tensor(np.arange(Tk)[None, :] <= qpos[:, None])
    ref = F.scaled_dot_product_attention(
        torch.as_tensor(q).transpose(0, 1)[None],
        torch.as_tensor(K).transpose(0, 1).repeat_interleave(2, 0)[None],
        torch.as_tensor(V).transpose(0, 1).repeat_interleave(2, 0)[None], attn_mask=mask)
    np.testing.assert_allclose(o, ref[0].transpose(0, 1).numpy(), atol=1e-12)
    # first position attends to itself only
    o1 = orc.attend(q[:1], np.array([0]), K, V, 2)
    np.testing.assert_allclose(o1[0, 3], V[0, 1], atol=1e-14)


def test_rmsnorm_scale_invariance_and_definition():
    rng = np.random.default_rng(6)
    x = rng.standard_normal((5, 64))
    g = 1.0 + 0.1 * rng.standard_normal(64)
    a = orc.rmsnorm(x, g, 0.0)
    b = orc.rmsnorm(37.5 * x, g, 0.0)
    np.testing.assert_allclose(a, b, rtol=1e-13)
    np.testing.assert_allclose((orc.rmsnorm(x, np.ones(64), 0.0) ** 2).mean(-1), 1.0, rtol=1e-13)
    ref = F.rms_norm(torch.as_tensor(x), (64,), torch.as_tensor(g), eps=1e-6).numpy()
    np.testing.assert_allclose(orc.rmsnorm(x, g, 1e-6), ref, rtol=1e-12)


def test_prefill_last_row_equals_prefill_plus_decode_step():
    s = small_shape(H=4)
    cfg = to_cfg(s)
    W = np_weights(s, 9, wscale=8.0)
    T = 12
    x = np_x(s, 9, T + 1)
    full = orc.foe_block(cfg, W, x, [T + 1])
    pre = orc.attention_stage(cfg, W, x[:, :T], [T])
    cache = [(pre["k_new"], pre["v_new"])]
    step = orc.foe_block(cfg, W, x[:, T:], [1], context_lens=[T], cache=cache)
    np.testing.assert_allclose(step["out"][:, 0], full["out"][:, T], rtol=0, atol=1e-11)
    np.testing.assert_allclose(step["k_new"][0], full["k_new"][T], rtol=0, atol=1e-12)
    # the row-subset form gives the same rows as the full computation
    sub = orc.foe_block(cfg, W, x, [T + 1], rows=np.array([0, 5, T]))
    np.testing.assert_allclose(sub["out"], full["out"][:, [0, 5, T]], rtol=0, atol=1e-12)


def test_idx_override_recomputes_gates_from_own_scores():
    s = small_shape(H=2, nq=4, nkv=2, Ec=4, kc=2)
    cfg = to_cfg(s)
    W = np_weights(s, 10, wscale=20.0)
    rng = np.random.default_rng(7)
    r = rng.standard_normal((6, s.hidden))
    base = orc.moe_stage(cfg, W, r)
    same = orc.moe_stage(cfg, W, r, idx_override=base["idx"])
    np.testing.assert_allclose(same["out"], base["out"], atol=1e-13)
    swapped = base["idx"][:, :, ::-1].copy()                    # same sets, other order
    sw = orc.moe_stage(cfg, W, r, idx_override=swapped)
    np.testing.assert_allclose(sw["out"], base["out"], atol=1e-12)


def _golden_rows():
    rows = []
    with open(os.path.join(GOLDEN, "comm_closed_forms.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, params, value, tol, _cite = [p.strip() for p in line.split("|")]
            kv = {k: float(v) for k, v in (p.split("=") for p in params.split())}
            rows.append((name, kv, float(value), float(tol)))
    return rows


def test_paper_closed_forms():
    rows = _golden_rows()
    assert len(rows) >= 6
    for name, p, value, tol in rows:
        if name == "single_node_ratio":
            vm, vf = orc.comm_volume_single_node(int(p["k"]), int(p["G"]), int(p["H"]))
            got = vm / vf
        elif name == "v_foe_single_node":
            got = orc.comm_volume_single_node(int(p["k"]), int(p["G"]), int(p["H"]))[1]
        elif name == "v_moe_single_node":
            got = orc.comm_volume_single_node(int(p["k"]), int(p["G"]), int(p["H"]))[0]
        elif name == "asymptote":
            got = orc.comm_time_ratio_asymptote(int(p["k"]), int(p["H"]), p["r"])
        elif name == "asymptote_within":
            full = orc.comm_time_ratio_multi_node(int(p["k"]), int(p["H"]), p["r"], int(p["N"]), int(p["Gn"]))
            asym = orc.comm_time_ratio_asymptote(int(p["k"]), int(p["H"]), p["r"])
            got = abs(asym - full) / asym
        else:
            raise AssertionError(name)
        assert abs(got - value) <= tol, (name, p, got, value)
    # the asymptote is the N -> infinity limit of the full formula
    big = orc.comm_time_ratio_multi_node(8, 8, 20.0, 100000, 8)
    assert abs(big - orc.comm_time_ratio_asymptote(8, 8, 20.0)) < 1e-3
