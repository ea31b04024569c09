"""CPU oracle for the forward pass of one Federation-of-Experts (FoE) transformer block.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the block
computes, written from the paper's definition of the layer (Table 2, the "Layer
boundaries" and "Routing" paragraphs of Section 3.1, and the notation of Table 1).
It is imported by the tests, by the smoke check and by the CPU-baseline leg of the
benchmark -- never by the product path, which shares no code with it.

Arithmetic: float64 throughout, on inputs that are bf16-valued numbers widened
exactly.  The one exception is the routing *decision*: router scores are rounded to
float32 before the top-k comparison and the gate softmax, because the CUDA router
works in float32 and an integer decision has to be taken in one precision on both
sides.  Library primitives used as steps: numpy matmul, argsort.

The paper leaves several details open (normalisation, RoPE form, tie rule, gate
normalisation, first-layer scaling, sum vs mean).  The readings taken here:
  * pre-norm RMSNorm with a gain before attention and before router+experts; the
    residuals carry un-normalised values;
  * RoPE on q and k with half-split pairs (j, j + d_h/2), angle p * theta^(-2j/d_h);
  * cluster h owns query heads h*g..(h+1)*g-1, KV heads h*c..(h+1)*c-1, the matching
    row block of W_O and experts h*E_c..(h+1)*E_c-1;
  * cross-cluster sync is the MEAN (Table 2, "Cross-group avg."); sync="sum" is offered
    because the abstract words it as a sum;
  * first layer: one shared attention, r = x + sum_h a_h, used in place of r_full;
  * last layer: appends the mean over clusters of x';
  * top-k inside each cluster's expert block, larger score first, equal scores -> lower
    index first; gates = softmax over the selected scores only;
  * dropless dispatch; expert slots ordered by global expert id, then token index.

Parity pins (tests/test_oracle_pins.py): H=1 equals an independently written MoE block;
dense brute force over all experts; torch SDPA / topk special cases; causality, RoPE
shift, RMSNorm scale invariances; sync/boundary closed forms; golden communication
closed forms from the paper.  No numeric example of the layer is printed in the paper,
so the readings listed above are "parity unpinned" with respect to the authors' code.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64


@dataclasses.dataclass
class FoeConfig:
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    n_clusters: int               # H
    head_dim: int
    experts_per_cluster: int      # E / H
    top_k_per_cluster: int        # k / H
    ffn_inter: int
    rope_theta: float = 1.0e4
    rms_eps: float = 1.0e-6
    position: str = "middle"      # middle | first | last | single (= first and last)
    sync: str = "mean"            # mean | sum

    @property
    def g(self) -> int:           # query heads per cluster
        return self.n_q_heads // self.n_clusters

    @property
    def c(self) -> int:           # KV heads per cluster
        return self.n_kv_heads // self.n_clusters

    @property
    def n_experts(self) -> int:
        return self.n_clusters * self.experts_per_cluster

    @property
    def is_first(self) -> bool:
        return self.position in ("first", "single")

    @property
    def is_last(self) -> bool:
        return self.position in ("last", "single")


def _f64(a) -> np.ndarray:
    return np.asarray(a, dtype=F64)


# ---------------------------------------------------------------------------
# elementary pieces
# ---------------------------------------------------------------------------

def rmsnorm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """x * rsqrt(mean(x^2) + eps) * gain over the last axis."""
    x = _f64(x)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * _f64(gain)


def rope(t: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding of t[T, heads, d_h] at integer positions pos[T]; pairs (j, j+d_h/2)."""
    t = _f64(t)
    dh = t.shape[-1]
    half = dh // 2
    j = np.arange(half, dtype=F64)
    inv_freq = theta ** (-2.0 * j / dh)
    ang = _f64(pos)[:, None] * inv_freq[None, :]          # [T, half]
    cos, sin = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    a, b = t[..., :half], t[..., half:]
    return np.concatenate([a * cos - b * sin, b * cos + a * sin], axis=-1)


def silu(z: np.ndarray) -> np.ndarray:
    return z / (1.0 + np.exp(-z))


def softmax_rows(s: np.ndarray) -> np.ndarray:
    m = np.max(s, axis=-1, keepdims=True)
    e = np.exp(s - m)
    return e / np.sum(e, axis=-1, keepdims=True)


# ---------------------------------------------------------------------------
# attention half of the block  (Table 2 rows "Attn. residual" and "Cross-group avg.")
# ---------------------------------------------------------------------------

def project_kv(cfg: FoeConfig, W: Dict[str, np.ndarray], x: np.ndarray, pos: np.ndarray
               ) -> Tuple[np.ndarray, np.ndarray]:
    """K (after RoPE) and V of every token for all KV heads: [S, n_kv, d_h] each.

    Cluster h projects its own stream x[h] (or the single shared x on a first layer)."""
    H, c, dh = cfg.n_clusters, cfg.c, cfg.head_dim
    S = x.shape[-2]
    k = np.empty((S, cfg.n_kv_heads, dh), dtype=F64)
    v = np.empty((S, cfg.n_kv_heads, dh), dtype=F64)
    for h in range(H):
        xin = x if cfg.is_first else x[h]
        n = rmsnorm(xin, W["attn_norm_g"], cfg.rms_eps)
        kh = (n @ _f64(W["wk"][h])).reshape(S, c, dh)
        vh = (n @ _f64(W["wv"][h])).reshape(S, c, dh)
        k[:, h * c:(h + 1) * c] = rope(kh, pos, cfg.rope_theta)
        v[:, h * c:(h + 1) * c] = vh
    return k, v


def project_q(cfg: FoeConfig, W: Dict[str, np.ndarray], x: np.ndarray, pos: np.ndarray,
              rows: np.ndarray) -> np.ndarray:
    """Q (after RoPE) of the tokens in ``rows`` for all query heads: [len(rows), n_q, d_h]."""
    H, g, dh = cfg.n_clusters, cfg.g, cfg.head_dim
    q = np.empty((len(rows), cfg.n_q_heads, dh), dtype=F64)
    for h in range(H):
        xin = (x if cfg.is_first else x[h])[rows]
        n = rmsnorm(xin, W["attn_norm_g"], cfg.rms_eps)
        qh = (n @ _f64(W["wq"][h])).reshape(len(rows), g, dh)
        q[:, h * g:(h + 1) * g] = rope(qh, pos[rows], cfg.rope_theta)
    return q


def attend(q: np.ndarray, qpos: np.ndarray, K: np.ndarray, V: np.ndarray, n_rep: int) -> np.ndarray:
    """Causal softmax(q k^T / sqrt(d_h)) v for one sequence.

    q[Tq, n_q, d_h] at absolute positions qpos[Tq]; K, V[Tk, n_kv, d_h] hold key positions
    0..Tk-1.  Query head a reads KV head a // n_rep.  Key j is visible to a query at position
    p iff j <= p.  Returns o[Tq, n_q, d_h]."""
    Tq, nq, dh = q.shape
    Tk = K.shape[0]
    o = np.empty_like(q)
    visible = np.arange(Tk)[None, :] <= np.asarray(qpos)[:, None]
    for a in range(nq):
        kv = a // n_rep
        s = (q[:, a, :] @ K[:, kv, :].T) / np.sqrt(F64(dh))
        s = np.where(visible, s, -np.inf)
        o[:, a, :] = softmax_rows(s) @ V[:, kv, :]
    return o


def attention_stage(cfg: FoeConfig, W: Dict[str, np.ndarray], x: np.ndarray,
                    q_lens: Sequence[int], context_lens: Optional[Sequence[int]] = None,
                    cache: Optional[List[Tuple[np.ndarray, np.ndarray]]] = None,
                    rows: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """Per-cluster attention residuals and their cross-cluster sync.

    x: [H, S, d] (middle/last) or [S, d] (first/single); the S tokens are the sequences' new
    tokens concatenated in sequence order, sequence b contributing q_lens[b] tokens at positions
    context_lens[b] ... ; cache[b] = (K, V) of the context_lens[b] tokens already cached
    ([ctx, n_kv, d_h], K stored after RoPE).  ``rows`` restricts the per-token outputs
    (q, o, a, r, r_full) to a subset of token indices; K and V are always produced for all S.

    Returns dict with pos[S], k_new, v_new [S, n_kv, d_h], q [R, n_q, d_h], o [R, n_q*d_h],
    a [H, R, d] (cluster h's o_h W_O^h), r ([H, R, d], or [R, d] on a first layer), r_full [R, d].
    """
    x = _f64(x)
    H, g, c, dh, d = cfg.n_clusters, cfg.g, cfg.c, cfg.head_dim, cfg.hidden
    S = x.shape[-2]
    q_lens = list(q_lens)
    assert sum(q_lens) == S
    context_lens = [0] * len(q_lens) if context_lens is None else list(context_lens)
    starts = np.concatenate([[0], np.cumsum(q_lens)]).astype(np.int64)
    pos = np.concatenate([ctx + np.arange(n) for ctx, n in zip(context_lens, q_lens)]).astype(np.int64)
    seq_of = np.concatenate([np.full(n, b) for b, n in enumerate(q_lens)]).astype(np.int64)
    rows = np.arange(S) if rows is None else np.asarray(rows, dtype=np.int64)

    k_new, v_new = project_kv(cfg, W, x, pos)
    q = project_q(cfg, W, x, pos, rows)

    n_rep = cfg.n_q_heads // cfg.n_kv_heads
    o = np.empty((len(rows), cfg.n_q_heads, dh), dtype=F64)
    for b in range(len(q_lens)):
        sel = np.nonzero(seq_of[rows] == b)[0]
        if len(sel) == 0:
            continue
        lo, hi = starts[b], starts[b + 1]
        if context_lens[b] > 0:
            Kc, Vc = cache[b]
            K = np.concatenate([_f64(Kc)[:context_lens[b]], k_new[lo:hi]], axis=0)
            V = np.concatenate([_f64(Vc)[:context_lens[b]], v_new[lo:hi]], axis=0)
        else:
            K, V = k_new[lo:hi], v_new[lo:hi]
        o[sel] = attend(q[sel], pos[rows[sel]], K, V, n_rep)

    wo = _f64(W["wo"])
    a = np.empty((H, len(rows), d), dtype=F64)
    for h in range(H):
        oh = o[:, h * g:(h + 1) * g, :].reshape(len(rows), g * dh)
        a[h] = oh @ wo[h * g * dh:(h + 1) * g * dh, :]

    if cfg.is_first:
        r = x[rows] + a.sum(axis=0)          # one shared attention, one residual
        r_full = r
    else:
        r = x[:, rows, :] + a                # r[h, i] = x[h, i] + Attn_h(x[h, :])[i]
        r_full = r.sum(axis=0)
        if cfg.sync == "mean":
            r_full = r_full / H
    return dict(pos=pos, k_new=k_new, v_new=v_new, q=q, o=o.reshape(len(rows), -1), a=a, r=r,
                r_full=r_full)


# ---------------------------------------------------------------------------
# routing  ("Routing" paragraph: one score vector, per-cluster top-k/H)
# ---------------------------------------------------------------------------

def router_logits(cfg: FoeConfig, W: Dict[str, np.ndarray], u: np.ndarray) -> np.ndarray:
    """g[i] = W_r u[i] + b, computed in float64 and rounded to float32 (the decision precision)."""
    l = _f64(u) @ _f64(W["router_w"]).T
    if W.get("router_b") is not None:
        l = l + _f64(W["router_b"])[None, :]
    return l.astype(np.float32)


def topk_per_cluster(cfg: FoeConfig, logits: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """idx[S, H, k_c] global expert ids (descending score, ties -> lower index) and gates w[S, H, k_c]
    = softmax over the selected scores of that cluster."""
    H, Ec, kc = cfg.n_clusters, cfg.experts_per_cluster, cfg.top_k_per_cluster
    S = logits.shape[0]
    idx = np.empty((S, H, kc), dtype=np.int32)
    w = np.empty((S, H, kc), dtype=F64)
    for h in range(H):
        blk = logits[:, h * Ec:(h + 1) * Ec]
        order = np.argsort(-blk, axis=1, kind="stable")[:, :kc]
        sel = np.take_along_axis(blk, order, axis=1).astype(F64)
        idx[:, h, :] = order + h * Ec
        w[:, h, :] = softmax_rows(sel)
    return idx, w


def topk_margin(cfg: FoeConfig, logits: np.ndarray) -> np.ndarray:
    """[S, H] gap between the k_c-th and (k_c+1)-th largest score inside each cluster (inf if E_c == k_c)."""
    H, Ec, kc = cfg.n_clusters, cfg.experts_per_cluster, cfg.top_k_per_cluster
    S = logits.shape[0]
    out = np.full((S, H), np.inf, dtype=F64)
    if Ec > kc:
        for h in range(H):
            srt = -np.sort(-logits[:, h * Ec:(h + 1) * Ec].astype(F64), axis=1)
            out[:, h] = srt[:, kc - 1] - srt[:, kc]
    return out


def route(cfg: FoeConfig, W: Dict[str, np.ndarray], r_full: np.ndarray) -> Dict[str, np.ndarray]:
    """FFN-norm, router scores, per-cluster top-k and gates for tokens r_full[S, d]."""
    u = rmsnorm(r_full, W["ffn_norm_g"], cfg.rms_eps)
    logits = router_logits(cfg, W, u)
    idx, w = topk_per_cluster(cfg, logits)
    return dict(u=u, logits=logits, idx=idx, w=w)


# ---------------------------------------------------------------------------
# dispatch maps (local form of the dispatch all-to-all)
# ---------------------------------------------------------------------------

def permute(idx: np.ndarray, n_experts: int) -> Dict[str, np.ndarray]:
    """counts[E], offsets[E+1] (exclusive scan), perm[R] (slot -> token), inv[S, H, k_c] (-> slot).

    Slots are grouped by global expert id; inside an expert, tokens ascend."""
    S, H, kc = idx.shape
    counts = np.zeros(n_experts, dtype=np.int32)
    for e in idx.reshape(-1):
        counts[e] += 1
    offsets = np.zeros(n_experts + 1, dtype=np.int32)
    offsets[1:] = np.cumsum(counts)
    fill = offsets[:-1].copy()
    perm = np.empty(S * H * kc, dtype=np.int32)
    inv = np.empty((S, H, kc), dtype=np.int32)
    for i in range(S):
        for h in range(H):
            for j in range(kc):
                e = idx[i, h, j]
                slot = fill[e]
                fill[e] += 1
                perm[slot] = i
                inv[i, h, j] = slot
    return dict(counts=counts, offsets=offsets, perm=perm, inv=inv)


# ---------------------------------------------------------------------------
# experts and combine  (Table 2 row "MoE update")
# ---------------------------------------------------------------------------

def experts(cfg: FoeConfig, W: Dict[str, np.ndarray], u: np.ndarray, maps: Dict[str, np.ndarray]
            ) -> np.ndarray:
    """y[slot] = W_d^e ( silu(W_g^e u_i) * (W_u^e u_i) ) for the (token i, expert e) of each slot."""
    R = maps["perm"].shape[0]
    y = np.zeros((R, cfg.hidden), dtype=F64)
    off = maps["offsets"]
    for e in range(cfg.n_experts):
        lo, hi = off[e], off[e + 1]
        if hi == lo:
            continue
        ue = _f64(u)[maps["perm"][lo:hi]]
        hmid = silu(ue @ _f64(W["w_gate"][e])) * (ue @ _f64(W["w_up"][e]))
        y[lo:hi] = hmid @ _f64(W["w_down"][e])
    return y


def combine(cfg: FoeConfig, r_full: np.ndarray, y: np.ndarray, w: np.ndarray, inv: np.ndarray
            ) -> Dict[str, np.ndarray]:
    """x'[h, i] = r_full[i] + sum_j w[i, h, j] y[inv[i, h, j]]; on a last layer also the mean over h."""
    S, H, kc = inv.shape
    xo = np.empty((H, S, cfg.hidden), dtype=F64)
    for h in range(H):
        acc = _f64(r_full).copy()
        for j in range(kc):
            acc += w[:, h, j][:, None] * y[inv[:, h, j]]
        xo[h] = acc
    out = xo.mean(axis=0) if cfg.is_last else xo
    return dict(x_next=xo, out=out)


def moe_stage(cfg: FoeConfig, W: Dict[str, np.ndarray], r_full: np.ndarray,
              idx_override: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """Everything after the sync for tokens r_full[S, d].  With ``idx_override`` the given expert
    ids are used in place of the top-k decision (gates recomputed from this side's scores)."""
    rt = route(cfg, W, r_full)
    if idx_override is not None:
        idx = np.asarray(idx_override, dtype=np.int32)
        sel = np.take_along_axis(rt["logits"], idx.reshape(idx.shape[0], -1).astype(np.int64), axis=1)
        rt["idx"] = idx
        rt["w"] = softmax_rows(sel.reshape(idx.shape).astype(F64))
    maps = permute(rt["idx"], cfg.n_experts)
    y = experts(cfg, W, rt["u"], maps)
    cb = combine(cfg, r_full, y, rt["w"], maps["inv"])
    out = dict(rt)
    out.update(maps)
    out.update(cb)
    out["y"] = y
    return out


def foe_block(cfg: FoeConfig, W: Dict[str, np.ndarray], x: np.ndarray, q_lens: Sequence[int],
              context_lens: Optional[Sequence[int]] = None,
              cache: Optional[List[Tuple[np.ndarray, np.ndarray]]] = None,
              rows: Optional[np.ndarray] = None,
              idx_override: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """Forward pass of one FoE block (prefill when q_lens > 1, decode when every q_len is 1).

    Output ``out`` is [H, R, d] (middle/first) or [R, d] (last/single) for the R tokens in ``rows``
    (all tokens when rows is None).  All intermediates are returned as well."""
    att = attention_stage(cfg, W, x, q_lens, context_lens, cache, rows)
    moe = moe_stage(cfg, W, att["r_full"], idx_override)
    res = dict(att)
    res.update(moe)
    return res


# ---------------------------------------------------------------------------
# analytic side results (Section 3.2) -- used only as pins for the closed forms
# ---------------------------------------------------------------------------

def comm_volume_single_node(k: int, G: int, H: int) -> Tuple[float, float]:
    """(V_moe, V_foe) per layer in units of S*d for one node with G <= H (Table 3)."""
    v_moe = 2.0 * k * (G - 1) / G
    v_foe = 2.0 * k * max(G - H, 0) / G + 2.0 * (min(G, H) - 1) / min(G, H)
    return v_moe, v_foe


def comm_time_ratio_multi_node(k: int, H: int, r: float, N: int, Gn: int) -> float:
    """T_moe / T_foe of Table 4 for N nodes of Gn GPUs."""
    G = Gn * N
    t_moe = 2.0 * k / N * (G - 1) / G * (1.0 + r * (N - 1))
    t_foe = 2.0 * k * (G - H) / G + 2.0 * (H - 1) / H * (1.0 + r * (N - 1)) / N
    return t_moe / t_foe


def comm_time_ratio_asymptote(k: int, H: int, r: float) -> float:
    return k * H * r / (k * H + r * (H - 1))
