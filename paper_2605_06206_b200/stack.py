"""A stack of FoE layers (first, middle..., last) on one GPU: the layers share one workspace and each has its own
paged KV cache.  Plumbing only: every layer call goes through the C ABI binding."""
from __future__ import annotations

import dataclasses
from typing import List, Sequence

import torch

from . import binding, synth


class FoeStack:
    def __init__(self, base_shape: synth.LayerShape, n_layers: int, seed: int, q_lens: Sequence[int], extra_tokens: int,
                 device: str = "cuda"):
        self.n_layers, self.seed, self.device = n_layers, seed, device
        self.q_lens = list(q_lens)
        self.n_seqs = len(self.q_lens)
        S = sum(self.q_lens)
        self.max_context = max(self.q_lens) + extra_tokens
        self.layers: List[binding.FoeLayer] = []
        self.shapes: List[synth.LayerShape] = []
        for l in range(n_layers):
            pos = "single" if n_layers == 1 else ("first" if l == 0 else ("last" if l == n_layers - 1 else "middle"))
            sh = dataclasses.replace(base_shape, position=pos)
            W = synth.make_weights(sh, seed, device, layer=l + 1)
            self.layers.append(binding.FoeLayer(sh, W, max_tokens=S, max_seqs=self.n_seqs, max_context=self.max_context,
                                                share_workspace_with=self.layers[0] if self.layers else None))
            self.shapes.append(sh)
            del W
        torch.cuda.empty_cache()
        total = [q + extra_tokens for q in self.q_lens]
        self.kvs = [synth.make_paged_cache(base_shape, seed, [0] * self.n_seqs, total, device, fill_random=False)
                    for _ in range(n_layers)]
        ql = torch.tensor(self.q_lens, dtype=torch.int32, device=device)
        for kv in self.kvs:
            kv.q_lens = ql

    def forward(self, x: torch.Tensor, context_lens: Sequence[int], decode: bool) -> torch.Tensor:
        ctx = torch.tensor(list(context_lens), dtype=torch.int32, device=self.device)
        h = x
        for layer, kv in zip(self.layers, self.kvs):
            kv.context_lens = ctx
            h = layer.decode(h, kv) if decode else layer.prefill(h, kv)
        return h

    def status(self) -> int:
        return self.layers[0].poll_status()

    def close(self) -> None:
        for layer in self.layers:
            layer.close()
        self.layers = []
