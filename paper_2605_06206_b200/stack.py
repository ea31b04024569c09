"""A stack of FoE layers (first, middle..., last) on one GPU: the layers share one workspace and each has its own
paged KV cache.  Plumbing only: a forward pass of the whole stack is ONE call into the C ABI (foe_stack_forward), the
context lengths live on the device and are advanced there (foe_context_advance), so a decode step crosses from Python
into the library twice whatever the number of layers, and can be replayed from a CUDA graph."""
from __future__ import annotations

import ctypes
import dataclasses
from typing import List, Optional, Sequence

import torch

from . import binding, synth


class FoeStack:
    def __init__(self, base_shape: synth.LayerShape, n_layers: int, seed: int, q_lens: Sequence[int], extra_tokens: int,
                 device: str = "cuda"):
        self.n_layers, self.seed, self.device = n_layers, seed, device
        self.q_lens = list(q_lens)
        self.n_seqs = len(self.q_lens)
        S = sum(self.q_lens)
        self.max_tokens = S
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
        # one device array of context lengths for all layers; it only changes through set_context / advance
        self.ctx = torch.zeros(self.n_seqs, dtype=torch.int32, device=device)
        for kv in self.kvs:
            kv.q_lens = ql
            kv.context_lens = self.ctx
        self.lib = binding.load_library()
        self._handles = (ctypes.c_void_p * n_layers)(*[l.handle.value for l in self.layers])
        H, d = base_shape.n_clusters, base_shape.hidden
        self._work = [torch.empty((H, S, d), dtype=torch.bfloat16, device=device) for _ in range(min(2, n_layers - 1))]
        self._kv_arrays = {}

    # ---- marshalling
    def _kv_array(self, decode: bool):
        """The per-layer cache descriptions as one ctypes array (built once per call kind: pointers do not change)."""
        if decode not in self._kv_arrays:
            n_tok = self.n_seqs if decode else sum(self.q_lens)
            mq = 1 if decode else max(self.q_lens)
            arr = (binding.FoeKvCache * self.n_layers)()
            for i, (layer, kv) in enumerate(zip(self.layers, self.kvs)):
                arr[i] = layer._kv(kv, n_tok, mq, decode)
            self._kv_arrays[decode] = arr
        return self._kv_arrays[decode]

    def set_context(self, context_lens: Sequence[int]) -> None:
        self.ctx.copy_(torch.tensor(list(context_lens), dtype=torch.int32), non_blocking=False)

    def advance(self, by: int = 1, stream=None) -> None:
        binding._check(self.lib.foe_context_advance(self.ctx.data_ptr(), self.n_seqs, by, binding._stream_ptr(stream)),
                       "foe_context_advance")

    def run(self, x: torch.Tensor, decode: bool, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """All layers on the context lengths currently on the device (foe_stack_forward)."""
        assert x.is_cuda and x.is_contiguous() and x.dtype == torch.bfloat16
        n_tok = self.n_seqs if decode else sum(self.q_lens)
        if out is None:
            out = self.layers[-1]._out_like(n_tok)
        w0 = self._work[0].data_ptr() if len(self._work) > 0 else None
        w1 = self._work[1].data_ptr() if len(self._work) > 1 else None
        binding._check(self.lib.foe_stack_forward(self._handles, self.n_layers, x.data_ptr(), self._kv_array(decode),
                                                  out.data_ptr(), w0, w1, 1 if decode else 0, binding._stream_ptr(stream)),
                       "foe_stack_forward")
        return out

    def forward(self, x: torch.Tensor, context_lens: Sequence[int], decode: bool) -> torch.Tensor:
        """One pass with the given context lengths (a host list, copied to the device first)."""
        self.set_context(context_lens)
        return self.run(x, decode)

    def status(self) -> int:
        return self.layers[0].poll_status()

    def close(self) -> None:
        for layer in self.layers:
            layer.close()
        self.layers = []
