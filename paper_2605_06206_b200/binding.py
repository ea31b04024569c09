"""Thin ctypes binding over the C ABI in include/foe.h.

Argument marshalling only: every step of the block runs inside libfoe.so.  torch is used for
device memory and streams.  There is no fallback: if the library is missing or no CUDA device is
present the calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfoe.so")

FOE_OK = 0
POSITIONS = {"middle": 0, "first": 1, "last": 2, "single": 3}
SYNCS = {"mean": 0, "sum": 1}

EXPORTS = ["foe_layer_create", "foe_layer_destroy", "foe_prefill", "foe_decode", "foe_route", "foe_get_aux",
           "foe_poll_status", "foe_last_launch_count", "foe_status_string", "foe_set_profiling", "foe_num_stages",
           "foe_stage_name", "foe_get_stage_ms", "foe_route_noalloc", "foe_layer_create_shared",
           "foe_route_partial_capacity", "foe_route_partial_floats", "foe_stack_forward", "foe_context_advance"]


class FoeConfig(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("hidden", "n_q_heads", "n_kv_heads", "n_clusters", "head_dim", "experts_per_cluster",
                 "top_k_per_cluster", "ffn_inter", "page_size", "max_tokens", "max_seqs", "max_context")] + \
               [("rope_theta", ctypes.c_float), ("rms_eps", ctypes.c_float),
                ("position", ctypes.c_int), ("sync", ctypes.c_int)]


class FoeWeights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("attn_norm_g", "wq", "wk", "wv", "wo", "ffn_norm_g", "w_gate", "w_up", "w_down", "router_w",
                 "router_b")]


class FoeKvCache(ctypes.Structure):
    _fields_ = [("k_pages", ctypes.c_void_p), ("v_pages", ctypes.c_void_p), ("block_table", ctypes.c_void_p),
                ("context_lens", ctypes.c_void_p), ("q_lens", ctypes.c_void_p), ("n_seqs", ctypes.c_int),
                ("max_pages_per_seq", ctypes.c_int), ("num_pages", ctypes.c_int), ("n_tokens", ctypes.c_int),
                ("max_q_len", ctypes.c_int)]


class FoeAux(ctypes.Structure):
    _fields_ = [("n_tokens", ctypes.c_int)] + [(n, ctypes.c_void_p) for n in
                                               ("r_full", "u", "logits", "topk_idx", "topk_w", "counts", "offsets",
                                                "perm", "inv", "q", "attn_o")]


_lib = None


def load_library() -> ctypes.CDLL:
    """Load libfoe.so (built by paper_2605_06206_b200.build) and declare the prototypes."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2605_06206_b200.build` "
                           "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci = ctypes.c_void_p, ctypes.c_int
    lib.foe_layer_create.argtypes = [ctypes.POINTER(FoeConfig), ctypes.POINTER(FoeWeights), ctypes.POINTER(vp)]
    lib.foe_layer_create.restype = ci
    lib.foe_layer_create_shared.argtypes = [ctypes.POINTER(FoeConfig), ctypes.POINTER(FoeWeights), vp, ctypes.POINTER(vp)]
    lib.foe_layer_create_shared.restype = ci
    lib.foe_layer_destroy.argtypes = [vp]
    lib.foe_layer_destroy.restype = ci
    for name in ("foe_prefill", "foe_decode"):
        fn = getattr(lib, name)
        fn.argtypes = [vp, vp, ctypes.POINTER(FoeKvCache), vp, vp]
        fn.restype = ci
    lib.foe_route.argtypes = [vp, vp, ci, vp, vp, vp]
    lib.foe_route.restype = ci
    lib.foe_get_aux.argtypes = [vp, ctypes.POINTER(FoeAux)]
    lib.foe_get_aux.restype = ci
    lib.foe_poll_status.argtypes = [vp, ctypes.POINTER(ci)]
    lib.foe_poll_status.restype = ci
    lib.foe_last_launch_count.argtypes = [vp]
    lib.foe_last_launch_count.restype = ci
    lib.foe_status_string.argtypes = [ci]
    lib.foe_status_string.restype = ctypes.c_char_p
    lib.foe_set_profiling.argtypes = [vp, ci]
    lib.foe_set_profiling.restype = ci
    lib.foe_num_stages.argtypes = []
    lib.foe_num_stages.restype = ci
    lib.foe_stage_name.argtypes = [ci]
    lib.foe_stage_name.restype = ctypes.c_char_p
    lib.foe_get_stage_ms.argtypes = [vp, ctypes.POINTER(ctypes.c_float), ci]
    lib.foe_get_stage_ms.restype = ci
    lib.foe_route_noalloc.argtypes = [ci, ci, ci, ci, ctypes.c_float, vp, vp, vp, vp, ci, vp, vp, vp]
    lib.foe_route_noalloc.restype = ci
    lib.foe_route_partial_capacity.argtypes = [ci, ci, ci]
    lib.foe_route_partial_capacity.restype = ctypes.c_size_t
    lib.foe_route_partial_floats.argtypes = [ci, ci, ci, ci, ctypes.c_size_t]
    lib.foe_route_partial_floats.restype = ctypes.c_size_t
    lib.foe_stack_forward.argtypes = [ctypes.POINTER(vp), ci, vp, ctypes.POINTER(FoeKvCache), vp, vp, vp, ci, vp]
    lib.foe_stack_forward.restype = ci
    lib.foe_context_advance.argtypes = [vp, ci, ci, vp]
    lib.foe_context_advance.restype = ci
    _lib = lib
    return lib


class FoeError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = load_library().foe_status_string(code).decode()
        super().__init__(f"{where}: {msg} ({code})")


def _check(code: int, where: str) -> None:
    if code != FOE_OK:
        raise FoeError(code, where)


class _DevView:
    """Exposes a raw device pointer to torch through the CUDA array interface."""

    def __init__(self, ptr: int, shape, typestr: str):
        self.__cuda_array_interface__ = dict(shape=tuple(shape), typestr=typestr, data=(int(ptr), False), version=2)


def _view(ptr, shape, dtype: torch.dtype) -> torch.Tensor:
    if any(s == 0 for s in shape):
        return torch.empty(shape, dtype=dtype, device="cuda")
    ts = {torch.float32: "<f4", torch.int32: "<i4", torch.bfloat16: "<i2"}[dtype]
    t = torch.as_tensor(_DevView(ptr, shape, ts), device="cuda")
    return t.view(torch.bfloat16) if dtype == torch.bfloat16 else t


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream_ptr(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


class FoeLayer:
    """One FoE block on the current CUDA device (foe_layer_create / foe_prefill / foe_decode / foe_route)."""

    def __init__(self, shape, weights: Dict[str, torch.Tensor], max_tokens: int, max_seqs: int, max_context: int,
                 share_workspace_with: Optional["FoeLayer"] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("FoeLayer needs a CUDA device: the block has no CPU path")
        self.lib = load_library()
        self.shape = shape
        cfg = FoeConfig(shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.n_clusters, shape.head_dim,
                        shape.experts_per_cluster, shape.top_k_per_cluster, shape.ffn_inter, shape.page_size,
                        max_tokens, max_seqs, max_context, shape.rope_theta, shape.rms_eps,
                        POSITIONS[shape.position], SYNCS[shape.sync])
        w = FoeWeights()
        for name, _ in FoeWeights._fields_:
            t = weights.get(name)
            if t is not None:
                want = torch.float32 if name.startswith("router") else torch.bfloat16
                assert t.is_cuda and t.is_contiguous() and t.dtype == want, name
            setattr(w, name, _ptr(t))
        h = ctypes.c_void_p()
        torch.cuda.synchronize()
        donor = share_workspace_with.handle if share_workspace_with is not None else None
        _check(self.lib.foe_layer_create_shared(ctypes.byref(cfg), ctypes.byref(w), donor, ctypes.byref(h)),
               "foe_layer_create")
        self.handle = h
        self.max_tokens, self.max_seqs, self.max_context = max_tokens, max_seqs, max_context

    def close(self) -> None:
        if getattr(self, "handle", None):
            self.lib.foe_layer_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- marshalling helpers
    def _kv(self, kv, n_tokens: int, max_q_len: int, decode: bool) -> FoeKvCache:
        for t in (kv.k_pages, kv.v_pages, kv.block_table, kv.context_lens):
            assert t.is_cuda and t.is_contiguous()
        assert kv.block_table.dtype == torch.int32 and kv.context_lens.dtype == torch.int32
        q = None if decode else kv.q_lens
        if q is not None:
            assert q.is_cuda and q.dtype == torch.int32
        return FoeKvCache(kv.k_pages.data_ptr(), kv.v_pages.data_ptr(), kv.block_table.data_ptr(),
                          kv.context_lens.data_ptr(), _ptr(q), kv.block_table.shape[0], kv.block_table.shape[1],
                          kv.k_pages.shape[0], n_tokens, max_q_len)

    def _out_like(self, n_tokens: int) -> torch.Tensor:
        s = self.shape
        shp = (s.n_clusters, n_tokens, s.hidden) if s.grouped_output else (n_tokens, s.hidden)
        return torch.empty(shp, dtype=torch.bfloat16, device="cuda")

    # ---- the four calls
    def prefill(self, x: torch.Tensor, kv, n_tokens: Optional[int] = None, max_q_len: Optional[int] = None,
                out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """foe_prefill.  n_tokens / max_q_len default to what x and kv.q_lens say (a host read of q_lens)."""
        assert x.is_cuda and x.is_contiguous() and x.dtype == torch.bfloat16
        if n_tokens is None:
            n_tokens = x.shape[-2]
        if max_q_len is None:
            max_q_len = int(kv.q_lens.max().item()) if n_tokens else 0
        out = self._out_like(n_tokens) if out is None else out
        c = self._kv(kv, n_tokens, max_q_len, False)
        _check(self.lib.foe_prefill(self.handle, x.data_ptr(), ctypes.byref(c), out.data_ptr(), _stream_ptr(stream)),
               "foe_prefill")
        return out

    def decode(self, x_step: torch.Tensor, kv, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        assert x_step.is_cuda and x_step.is_contiguous() and x_step.dtype == torch.bfloat16
        n = kv.block_table.shape[0]
        out = self._out_like(n) if out is None else out
        c = self._kv(kv, n, 1, True)
        _check(self.lib.foe_decode(self.handle, x_step.data_ptr(), ctypes.byref(c), out.data_ptr(), _stream_ptr(stream)),
               "foe_decode")
        return out

    def route(self, h: torch.Tensor, stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
        assert h.is_cuda and h.is_contiguous() and h.dtype == torch.bfloat16
        n = h.shape[0]
        s = self.shape
        idx = torch.empty((n, s.n_clusters, s.top_k_per_cluster), dtype=torch.int32, device="cuda")
        w = torch.empty((n, s.n_clusters, s.top_k_per_cluster), dtype=torch.float32, device="cuda")
        _check(self.lib.foe_route(self.handle, h.data_ptr(), n, idx.data_ptr(), w.data_ptr(), _stream_ptr(stream)),
               "foe_route")
        return idx, w

    # ---- introspection
    def aux(self) -> Dict[str, torch.Tensor]:
        """Copies of the last call's intermediates (see foe_aux)."""
        a = FoeAux()
        _check(self.lib.foe_get_aux(self.handle, ctypes.byref(a)), "foe_get_aux")
        torch.cuda.synchronize()
        s = self.shape
        S, H, kc, E, d = a.n_tokens, s.n_clusters, s.top_k_per_cluster, s.n_experts, s.hidden
        spec = dict(r_full=((S, d), torch.float32), u=((S, d), torch.bfloat16), logits=((S, E), torch.float32),
                    topk_idx=((S, H, kc), torch.int32), topk_w=((S, H, kc), torch.float32),
                    counts=((E,), torch.int32), offsets=((E + 1,), torch.int32), perm=((S * H * kc,), torch.int32),
                    inv=((S, H, kc), torch.int32), q=((S, s.n_q_heads, 128 if s.head_dim == 96 else s.head_dim), torch.bfloat16),
                    attn_o=((S, s.n_q_heads * s.head_dim), torch.bfloat16))
        out = {k: _view(getattr(a, k), shp, dt).clone() for k, (shp, dt) in spec.items()}
        # q is kept with its heads padded to the attention kernels' tile width (head_dim 96 -> 128)
        out["q"] = out["q"][:, :, :s.head_dim].reshape(S, s.n_q_heads * s.head_dim).contiguous()
        return out

    def poll_status(self) -> int:
        v = ctypes.c_int(0)
        _check(self.lib.foe_poll_status(self.handle, ctypes.byref(v)), "foe_poll_status")
        return v.value

    def last_launch_count(self) -> int:
        return self.lib.foe_last_launch_count(self.handle)

    def set_profiling(self, on) -> None:
        """False / 0: off; True / 1: the last call; n > 1: the n most recent calls (stage_ms returns their mean)."""
        _check(self.lib.foe_set_profiling(self.handle, int(on)), "foe_set_profiling")

    def stage_ms(self) -> Dict[str, float]:
        n = self.lib.foe_num_stages()
        buf = (ctypes.c_float * n)()
        _check(self.lib.foe_get_stage_ms(self.handle, buf, n), "foe_get_stage_ms")
        return {self.lib.foe_stage_name(i).decode(): float(buf[i]) for i in range(n)}


def route_noalloc(shape, ffn_norm_g: torch.Tensor, router_w: torch.Tensor, router_b: Optional[torch.Tensor],
                  h: torch.Tensor, idx: torch.Tensor, w: torch.Tensor, stream=None) -> None:
    """foe_route_noalloc: routing for callers that must not allocate device memory.  The caller supplies the
    outputs idx / w ([n, H, k_c] int32 / fp32); the library works on its built-in scratch area and this
    wrapper creates no tensors either.  Calls on one device must not overlap (they share the scratch)."""
    lib = load_library()
    assert h.is_cuda and h.is_contiguous() and h.dtype == torch.bfloat16
    assert idx.is_cuda and idx.dtype == torch.int32 and idx.is_contiguous()
    assert w.is_cuda and w.dtype == torch.float32 and w.is_contiguous()
    assert ffn_norm_g.dtype == torch.bfloat16 and router_w.dtype == torch.float32
    _check(lib.foe_route_noalloc(shape.hidden, shape.n_clusters, shape.experts_per_cluster, shape.top_k_per_cluster,
                                 shape.rms_eps, ffn_norm_g.data_ptr(), router_w.data_ptr(), _ptr(router_b),
                                 h.data_ptr(), h.shape[0], idx.data_ptr(), w.data_ptr(), _stream_ptr(stream)),
           "foe_route_noalloc")
