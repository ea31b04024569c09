"""Glue between torch tensors (as the seeded input generator produces them) and the numpy oracle.

TEST INFRASTRUCTURE ONLY, like the rest of this directory.  Holds no arithmetic of the method.
"""
from __future__ import annotations

from typing import Dict, List, Sequence, Tuple

import numpy as np
import torch

from . import foe_oracle as orc


def cfg_from_shape(s) -> orc.FoeConfig:
    """FoeConfig from any object with the layer-shape attributes (duck typed)."""
    return orc.FoeConfig(s.hidden, s.n_q_heads, s.n_kv_heads, s.n_clusters, s.head_dim, s.experts_per_cluster,
                         s.top_k_per_cluster, s.ffn_inter, s.rope_theta, s.rms_eps, s.position, s.sync)


def to_np(t: torch.Tensor) -> np.ndarray:
    """Exact widening: bf16/fp32 torch tensor (any device) -> float32 numpy (values preserved)."""
    return t.detach().to("cpu", torch.float32).numpy()


def weights_to_numpy(W: Dict[str, torch.Tensor]) -> Dict[str, np.ndarray]:
    return {k: (None if v is None else to_np(v)) for k, v in W.items()}


def logical_cache(k_pages: torch.Tensor, v_pages: torch.Tensor, block_table: torch.Tensor,
                  context_lens: Sequence[int], page_size: int) -> List[Tuple[np.ndarray, np.ndarray]]:
    """Per-sequence logical (K, V) [ctx, n_kv, dh] read back through the block table."""
    out = []
    bt = block_table.cpu().long()
    for b, ctx in enumerate(context_lens):
        npg = (ctx + page_size - 1) // page_size
        if npg == 0:
            nkv, dh = k_pages.shape[1], k_pages.shape[3]
            out.append((np.zeros((0, nkv, dh), np.float32), np.zeros((0, nkv, dh), np.float32)))
            continue
        ids = bt[b, :npg].to(k_pages.device)
        k = k_pages[ids].permute(0, 2, 1, 3).reshape(npg * page_size, k_pages.shape[1], k_pages.shape[3])[:ctx]
        v = v_pages[ids].permute(0, 2, 1, 3).reshape(npg * page_size, v_pages.shape[1], v_pages.shape[3])[:ctx]
        out.append((to_np(k), to_np(v)))
    return out
