"""Seeded synthetic inputs for the FoE block: weights, activations, KV caches, paging.

This module holds no arithmetic of the method itself.  It only produces numbers
(counter-based, so every element can be regenerated on demand on either device)
and lays logical KV caches out into physical pages.  Both the CUDA tests/bench and
the CPU checker draw their inputs from here so that they see identical values.

Value of element ``i`` of tensor ``tid`` under ``seed``:

    scale * Q[ top16( mix64(seed, tid, i) ) ]          rounded to bf16 (RNE)

``Q`` is a 65,536-entry table of standard-normal quantiles, so the values are
N(0, scale^2) to 16 bits of resolution.  Only 64-bit integer hashing and a table
lookup are involved, hence the result is bit-identical on CPU and GPU.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Tuple

import torch

# ----------------------------------------------------------------------------
# counter-based generator
# ----------------------------------------------------------------------------

_M1 = -0x40A7B892E31B1A47  # 0xBF58476D1CE4E5B9 as int64
_M2 = -0x6B2FB644ECCEEE15  # 0x94D049BB133111EB as int64
_GOLD = -0x61C8864680B583EB  # 0x9E3779B97F4A7C15 as int64
_MASK64 = (1 << 64) - 1

_QTABLE_CPU: Optional[torch.Tensor] = None
_QTABLE_DEV: Dict[str, torch.Tensor] = {}


def _qtable(device: torch.device) -> torch.Tensor:
    """65,536 standard-normal quantiles at the bin midpoints, fp32, built on the CPU."""
    global _QTABLE_CPU
    if _QTABLE_CPU is None:
        p = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
        _QTABLE_CPU = torch.special.ndtri(p).to(torch.float32)
    key = str(device)
    if key not in _QTABLE_DEV:
        _QTABLE_DEV[key] = _QTABLE_CPU.to(device)
    return _QTABLE_DEV[key]


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of an int64 tensor holding uint64 bit patterns."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def _to_i64(v: int) -> int:
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


def stream_key(seed: int, tid: int) -> int:
    """64-bit key of one (seed, tensor id) stream (python ints, uint64 arithmetic)."""
    z = (seed * 0xD1342543DE82EF95 + tid * 0xA0761D6478BD642F + 0x2545F4914F6CDD1D) & _MASK64
    z ^= z >> 29
    z = (z * 0xBF58476D1CE4E5B9) & _MASK64
    z ^= z >> 32
    return z


def hash16(seed: int, tid: int, idx: torch.Tensor) -> torch.Tensor:
    """Top 16 bits of mix64(seed, tid, idx) for an int64 index tensor."""
    z = idx * _GOLD + _to_i64(stream_key(seed, tid))
    z = (z ^ _lsr(z, 30)) * _M1
    z = (z ^ _lsr(z, 27)) * _M2
    z = z ^ _lsr(z, 31)
    return _lsr(z, 48)


def hash16_scalar(seed: int, tid: int, i: int) -> int:
    """Pure-python restatement of :func:`hash16` for one index (used by the tests)."""
    z = (i * 0x9E3779B97F4A7C15 + stream_key(seed, tid)) & _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    z ^= z >> 31
    return z >> 48


def normal_bf16(seed: int, tid: int, shape, scale: float = 1.0, offset: float = 0.0,
                device="cpu", start: int = 0, chunk: int = 1 << 25) -> torch.Tensor:
    """bf16 tensor of ``shape`` with element i = bf16(offset + scale * Q[hash16(seed, tid, start+i)])."""
    device = torch.device(device)
    n = int(math.prod(shape))
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    q = _qtable(device)
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        idx = torch.arange(start + lo, start + hi, dtype=torch.int64, device=device)
        v = q[hash16(seed, tid, idx)]
        if scale != 1.0:
            v = v * scale
        if offset != 0.0:
            v = v + offset
        out[lo:hi] = v.to(torch.bfloat16)
    return out.view(*shape)


def uniform_int(seed: int, tid: int, n: int, lo: int, hi: int) -> torch.Tensor:
    """n integers in [lo, hi] (inclusive) on the CPU, from the same hash."""
    idx = torch.arange(n, dtype=torch.int64)
    h = hash16(seed, tid, idx) * 65536 + hash16(seed, tid + 1, idx)
    return lo + (h % (hi - lo + 1))


def permutation(seed: int, tid: int, n: int) -> torch.Tensor:
    """A seeded permutation of range(n) on the CPU (sort of hashed keys, index as tie-break)."""
    idx = torch.arange(n, dtype=torch.int64)
    key = (hash16(seed, tid, idx) * 65536 + hash16(seed, tid + 1, idx)) * (1 << 24) + idx
    return torch.argsort(key)


# ----------------------------------------------------------------------------
# layer description (plain data; no method arithmetic)
# ----------------------------------------------------------------------------

@dataclasses.dataclass
class LayerShape:
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    n_clusters: int
    head_dim: int
    experts_per_cluster: int
    top_k_per_cluster: int
    ffn_inter: int
    rope_theta: float = 1.0e4
    rms_eps: float = 1.0e-6
    position: str = "middle"      # middle | first | last | single
    sync: str = "mean"            # mean | sum
    page_size: int = 64

    @property
    def q_per_cluster(self) -> int:
        return self.n_q_heads // self.n_clusters

    @property
    def kv_per_cluster(self) -> int:
        return self.n_kv_heads // self.n_clusters

    @property
    def n_experts(self) -> int:
        return self.n_clusters * self.experts_per_cluster

    @property
    def grouped_input(self) -> bool:
        return self.position in ("middle", "last")

    @property
    def grouped_output(self) -> bool:
        return self.position in ("middle", "first")


# tensor ids of the streams
TID = dict(attn_norm_g=1, wq=2, wk=3, wv=4, wo=5, ffn_norm_g=6, w_gate=7, w_up=8, w_down=9,
           router_w=10, router_b=11, x=20, k_cache=30, v_cache=31, ctx_lens=40, page_perm=42,
           bias_perm=44, x_step=100)


def make_weights(shape: LayerShape, seed: int, device="cpu", layer: int = 0) -> Dict[str, torch.Tensor]:
    """Weights of one FoE layer: projections/experts/router N(0, 0.02^2) bf16 values,
    norm gains 1 + 0.02 z.  Router weights are the bf16 values widened to fp32; the
    router bias is zero here (see :func:`zipf_router_bias`)."""
    s = shape
    H, d, dh = s.n_clusters, s.hidden, s.head_dim
    g, c, E, I = s.q_per_cluster, s.kv_per_cluster, s.n_experts, s.ffn_inter
    base = 1000 * layer

    def w(name, shp, scale=0.02, offset=0.0):
        return normal_bf16(seed, base + TID[name], shp, scale, offset, device)

    out = dict(
        attn_norm_g=w("attn_norm_g", (d,), 0.02, 1.0),
        wq=w("wq", (H, d, g * dh)),
        wk=w("wk", (H, d, c * dh)),
        wv=w("wv", (H, d, c * dh)),
        wo=w("wo", (s.n_q_heads * dh, d)),
        ffn_norm_g=w("ffn_norm_g", (d,), 0.02, 1.0),
        w_gate=w("w_gate", (E, d, I)),
        w_up=w("w_up", (E, d, I)),
        w_down=w("w_down", (E, I, d)),
        router_w=w("router_w", (E, d)).to(torch.float32),
        router_b=torch.zeros(E, dtype=torch.float32, device=device),
    )
    return out


def make_x(shape: LayerShape, seed: int, n_tokens: int, device="cpu", tid: Optional[int] = None) -> torch.Tensor:
    """Input hidden state, N(0,1) bf16: [H, S, d] when the layer takes grouped input, else [S, d]."""
    tid = TID["x"] if tid is None else tid
    shp = (shape.n_clusters, n_tokens, shape.hidden) if shape.grouped_input else (n_tokens, shape.hidden)
    return normal_bf16(seed, tid, shp, 1.0, 0.0, device)


def zipf_router_bias(shape: LayerShape, seed: int, sigma_logit: float, s_exp: float = 1.2,
                     dead_per_cluster: int = 0) -> torch.Tensor:
    """Router bias that skews per-cluster expert popularity towards Zipf(s_exp).

    b_e = beta * ln p_{pi(e)},  p_j ~ j^{-s_exp} over the experts of one cluster,  pi a seeded
    permutation per cluster,  beta = (sqrt(6)/pi) * sigma_logit  (matches a Gumbel of the
    logits' spread).  ``dead_per_cluster`` experts per cluster get bias -1e30 (never chosen)."""
    Ec, H = shape.experts_per_cluster, shape.n_clusters
    p = torch.arange(1, Ec + 1, dtype=torch.float64) ** (-s_exp)
    p = p / p.sum()
    beta = math.sqrt(6.0) / math.pi * sigma_logit
    b = torch.empty(H, Ec, dtype=torch.float64)
    for h in range(H):
        pi = permutation(seed, TID["bias_perm"] + 2 * h, Ec)
        b[h] = beta * torch.log(p[pi])
        if dead_per_cluster:
            b[h, pi[-dead_per_cluster:]] = -1.0e30
    return b.reshape(-1).to(torch.float32)


# ----------------------------------------------------------------------------
# paged KV cache
# ----------------------------------------------------------------------------

@dataclasses.dataclass
class PagedKV:
    k_pages: torch.Tensor        # [num_pages, n_kv, page, dh] bf16
    v_pages: torch.Tensor
    block_table: torch.Tensor    # [n_seqs, max_pages_per_seq] int32
    context_lens: torch.Tensor   # [n_seqs] int32, tokens cached before the call
    q_lens: torch.Tensor         # [n_seqs] int32, new tokens in the call

    @property
    def n_seqs(self) -> int:
        return int(self.block_table.shape[0])


def make_block_table(seed: int, total_lens: List[int], page_size: int, shuffle: bool = True
                     ) -> Tuple[torch.Tensor, int]:
    """Assign physical pages (a seeded permutation of the pool) to the logical pages of each sequence."""
    need = [(t + page_size - 1) // page_size for t in total_lens]
    num_pages = max(1, sum(need))
    max_pp = max(1, max(need))
    ids = permutation(seed, TID["page_perm"], num_pages) if shuffle else torch.arange(num_pages)
    bt = torch.zeros(len(total_lens), max_pp, dtype=torch.int32)
    at = 0
    for s, n in enumerate(need):
        bt[s, :n] = ids[at:at + n].to(torch.int32)
        at += n
    return bt, num_pages


def make_paged_cache(shape: LayerShape, seed: int, context_lens: List[int], q_lens: List[int],
                     device="cpu", fill_random: bool = True, shuffle: bool = True) -> PagedKV:
    """Paged cache sized for context+new tokens of every sequence.

    With ``fill_random`` every page slot is filled with N(0,1) bf16 values (page-major streams), so
    the first ``context_lens[s]`` logical positions of sequence s hold random "already rotated" K and
    V; the rest is overwritten by the call."""
    ps, nkv, dh = shape.page_size, shape.n_kv_heads, shape.head_dim
    total = [c + q for c, q in zip(context_lens, q_lens)]
    bt, num_pages = make_block_table(seed, total, ps, shuffle)
    shp = (num_pages, nkv, ps, dh)
    if fill_random and any(c > 0 for c in context_lens):
        kp = normal_bf16(seed, TID["k_cache"], shp, 1.0, 0.0, device)
        vp = normal_bf16(seed, TID["v_cache"], shp, 1.0, 0.0, device)
    else:
        kp = torch.zeros(shp, dtype=torch.bfloat16, device=device)
        vp = torch.zeros(shp, dtype=torch.bfloat16, device=device)
    return PagedKV(kp, vp, bt.to(device), torch.tensor(context_lens, dtype=torch.int32, device=device),
                   torch.tensor(q_lens, dtype=torch.int32, device=device))


def gather_logical_cache(kv: PagedKV, seq: int, length: int, page_size: int
                         ) -> Tuple[torch.Tensor, torch.Tensor]:
    """Logical [length, n_kv, dh] K and V of one sequence read back through the block table (CPU copies)."""
    npg = (length + page_size - 1) // page_size
    ids = kv.block_table[seq, :npg].long().cpu()
    k = kv.k_pages[ids.to(kv.k_pages.device)].cpu()   # [npg, n_kv, page, dh]
    v = kv.v_pages[ids.to(kv.v_pages.device)].cpu()
    k = k.permute(0, 2, 1, 3).reshape(npg * page_size, k.shape[1], k.shape[3])[:length]
    v = v.permute(0, 2, 1, 3).reshape(npg * page_size, v.shape[1], v.shape[3])[:length]
    return k, v


# ----------------------------------------------------------------------------
# the five workloads
# ----------------------------------------------------------------------------

def workload(n: int) -> Tuple[LayerShape, dict]:
    """Layer shape and call shape of workload n (1..5).  Returns (shape, info) where info has
    seed, mode ('prefill' | 'decode'), q_lens and context_lens."""
    if n == 1:
        s = LayerShape(256, 8, 4, 4, 64, 8, 2, 128, 1.0e4)
        return s, dict(seed=0, mode="prefill", q_lens=[128], context_lens=[0])
    if n == 2:
        s = LayerShape(2048, 16, 4, 4, 128, 16, 2, 1024, 1.0e4)
        return s, dict(seed=2, mode="prefill", q_lens=[4096] * 4, context_lens=[0] * 4)
    if n == 3:
        s = LayerShape(2048, 16, 4, 4, 128, 16, 2, 1024, 1.0e4)
        ctx = uniform_int(3, TID["ctx_lens"], 64, 4096, 16384).tolist()
        return s, dict(seed=3, mode="decode", q_lens=[1] * 64, context_lens=ctx)
    if n == 4:
        s = LayerShape(2048, 16, 8, 8, 128, 32, 4, 768, 1.0e4)
        return s, dict(seed=4, mode="prefill", q_lens=[2048] * 8, context_lens=[0] * 8, zipf=1.2)
    if n == 5:
        s = LayerShape(4096, 32, 8, 8, 128, 16, 2, 1408, 1.0e4)
        return s, dict(seed=5, mode="stack", q_lens=[16384] * 2, context_lens=[0] * 2, layers=16,
                       decode_steps=128)
    raise ValueError(f"no workload {n}")
