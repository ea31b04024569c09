"""One cluster per GPU: binding of include/foe_shard.h and the host plumbing around it.

Argument marshalling and bookkeeping only; the exchange itself (partials pushed into peer memory from the
O-projection's epilogue, owner-side reduction, all-gather, bounded waits) runs inside libfoe.so.

Two ways to form a group of H ranks:
  * `LocalGroup`: all H ranks on the current device, each with its own exchange buffer, layer handle and KV cache.
    Kernels of different ranks never run concurrently here, so every phase is issued for all ranks before the
    next phase starts and no device-side wait ever spins.  This is how the sharded path is checked on one GPU.
  * `connect`: one process per GPU under torch.distributed.  Every rank allocates its buffer, the 64-byte CUDA IPC
    handles travel through `all_gather`, and each rank maps the others' buffers.  A rank then simply calls
    attend, reduce, ffn back to back.
"""
from __future__ import annotations

import ctypes
import dataclasses
from typing import Callable, Dict, List, Optional, Sequence

import torch

from . import binding
from .binding import FoeKvCache, _check, _stream_ptr

SHARD_EXPORTS = ["foe_shard_buffer_bytes", "foe_shard_buffer_alloc", "foe_shard_buffer_free", "foe_shard_buffer_export",
                 "foe_shard_buffer_import", "foe_shard_buffer_close", "foe_shard_create", "foe_shard_destroy",
                 "foe_shard_attend", "foe_shard_push", "foe_shard_reduce", "foe_shard_ffn", "foe_shard_gather",
                 "foe_shard_poll_status"]

HANDLE_BYTES = 64


class FoeShardConfig(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("rank", "n_ranks", "hidden", "max_tokens", "wait_limit_ms")]


_declared = False


def load_library() -> ctypes.CDLL:
    """libfoe.so with the prototypes of foe_shard.h declared."""
    global _declared
    lib = binding.load_library()
    if _declared:
        return lib
    vp, ci = ctypes.c_void_p, ctypes.c_int
    cfgp = ctypes.POINTER(FoeShardConfig)
    lib.foe_shard_buffer_bytes.argtypes = [cfgp]
    lib.foe_shard_buffer_bytes.restype = ctypes.c_size_t
    lib.foe_shard_buffer_alloc.argtypes = [cfgp, ctypes.POINTER(vp)]
    lib.foe_shard_buffer_free.argtypes = [vp]
    lib.foe_shard_buffer_export.argtypes = [vp, ctypes.c_char_p]
    lib.foe_shard_buffer_import.argtypes = [ctypes.c_char_p, ctypes.POINTER(vp)]
    lib.foe_shard_buffer_close.argtypes = [vp]
    lib.foe_shard_create.argtypes = [cfgp, ctypes.POINTER(vp), ctypes.POINTER(vp)]
    lib.foe_shard_destroy.argtypes = [vp]
    lib.foe_shard_attend.argtypes = [vp, vp, vp, ctypes.POINTER(FoeKvCache), ci, vp]
    lib.foe_shard_push.argtypes = [vp, vp, ci, ctypes.c_float, vp]
    lib.foe_shard_reduce.argtypes = [vp, vp]
    lib.foe_shard_ffn.argtypes = [vp, vp, vp, vp]
    lib.foe_shard_gather.argtypes = [vp, vp, vp]
    lib.foe_shard_poll_status.argtypes = [vp, ctypes.POINTER(ci)]
    for name in SHARD_EXPORTS:
        if name != "foe_shard_buffer_bytes":
            getattr(lib, name).restype = ci
    _declared = True
    return lib


# ------------------------------------------------------------------ what one rank holds

def cluster_shape(shape, h: int):
    """Layer description of cluster h alone (the handle rank h creates): one cluster with the cluster's heads
    and experts.  Position and sync keep their meaning.  The cluster's own query width (query heads per cluster x
    head width) must be a multiple of 128, as for any layer handle."""
    assert 0 <= h < shape.n_clusters
    if (shape.q_per_cluster * shape.head_dim) % 128:
        raise ValueError("one cluster per rank needs a per-cluster query width that is a multiple of 128")
    return dataclasses.replace(shape, n_clusters=1, n_q_heads=shape.q_per_cluster, n_kv_heads=shape.kv_per_cluster)


def cluster_weights(shape, weights: Dict[str, torch.Tensor], h: int) -> Dict[str, torch.Tensor]:
    """Views of the weights rank h needs (no copies: every slice is contiguous in the full tensors)."""
    Ec, gd = shape.experts_per_cluster, shape.q_per_cluster * shape.head_dim
    e0, e1 = h * Ec, (h + 1) * Ec
    out = dict(attn_norm_g=weights["attn_norm_g"], ffn_norm_g=weights["ffn_norm_g"],
               wq=weights["wq"][h:h + 1], wk=weights["wk"][h:h + 1], wv=weights["wv"][h:h + 1],
               wo=weights["wo"][h * gd:(h + 1) * gd],
               w_gate=weights["w_gate"][e0:e1], w_up=weights["w_up"][e0:e1], w_down=weights["w_down"][e0:e1],
               router_w=weights["router_w"][e0:e1])
    if weights.get("router_b") is not None:
        out["router_b"] = weights["router_b"][e0:e1]
    return out


def exchange_config(shape, rank: int, max_tokens: int, wait_limit_ms: int = 0) -> FoeShardConfig:
    return FoeShardConfig(rank, shape.n_clusters, shape.hidden, max_tokens, wait_limit_ms)


class ExchangeBuffer:
    """One rank's exchange buffer (foe_shard_buffer_alloc / _free), or a peer's buffer mapped through CUDA IPC."""

    def __init__(self, cfg: FoeShardConfig, imported_from: Optional[bytes] = None):
        self.lib = load_library()
        p = ctypes.c_void_p()
        self.imported = imported_from is not None
        if self.imported:
            assert len(imported_from) == HANDLE_BYTES
            _check(self.lib.foe_shard_buffer_import(imported_from, ctypes.byref(p)), "foe_shard_buffer_import")
        else:
            _check(self.lib.foe_shard_buffer_alloc(ctypes.byref(cfg), ctypes.byref(p)), "foe_shard_buffer_alloc")
        self.ptr = p.value
        self.bytes = self.lib.foe_shard_buffer_bytes(ctypes.byref(cfg))

    def export(self) -> bytes:
        buf = ctypes.create_string_buffer(HANDLE_BYTES)
        _check(self.lib.foe_shard_buffer_export(self.ptr, buf), "foe_shard_buffer_export")
        return buf.raw

    def close(self) -> None:
        if getattr(self, "ptr", None):
            (self.lib.foe_shard_buffer_close if self.imported else self.lib.foe_shard_buffer_free)(self.ptr)
            self.ptr = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Exchange:
    """One rank's end of the group's exchange (foe_shard_create ... foe_shard_poll_status)."""

    def __init__(self, cfg: FoeShardConfig, buffer_ptrs: Sequence[int]):
        self.lib = load_library()
        assert len(buffer_ptrs) == cfg.n_ranks
        self.cfg = cfg
        table = (ctypes.c_void_p * cfg.n_ranks)(*buffer_ptrs)
        h = ctypes.c_void_p()
        _check(self.lib.foe_shard_create(ctypes.byref(cfg), table, ctypes.byref(h)), "foe_shard_create")
        self.handle = h

    def push(self, src: torch.Tensor, scale: float = 1.0, stream=None) -> None:
        assert src.is_cuda and src.is_contiguous() and src.dtype == torch.bfloat16 and src.shape[-1] == self.cfg.hidden
        _check(self.lib.foe_shard_push(self.handle, src.data_ptr(), src.shape[0], scale, _stream_ptr(stream)),
               "foe_shard_push")
        self._n = src.shape[0]

    def reduce(self, stream=None) -> None:
        _check(self.lib.foe_shard_reduce(self.handle, _stream_ptr(stream)), "foe_shard_reduce")

    def gather(self, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        if out is None:
            out = torch.empty((self._n, self.cfg.hidden), dtype=torch.bfloat16, device="cuda")
        _check(self.lib.foe_shard_gather(self.handle, out.data_ptr(), _stream_ptr(stream)), "foe_shard_gather")
        return out

    def poll_status(self) -> int:
        v = ctypes.c_int(0)
        _check(self.lib.foe_shard_poll_status(self.handle, ctypes.byref(v)), "foe_shard_poll_status")
        return v.value

    def close(self) -> None:
        if getattr(self, "handle", None):
            self.lib.foe_shard_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class ShardedLayer:
    """Rank h's part of one FoE block: the layer handle of cluster h plus the rank's end of the exchange."""

    def __init__(self, shape, weights_h: Dict[str, torch.Tensor], h: int, exchange: Exchange, max_tokens: int,
                 max_seqs: int, max_context: int, share_workspace_with: Optional["ShardedLayer"] = None):
        self.full_shape, self.h, self.exchange = shape, h, exchange
        self.layer = binding.FoeLayer(cluster_shape(shape, h), weights_h, max_tokens, max_seqs, max_context,
                                      share_workspace_with.layer if share_workspace_with is not None else None)
        self.lib = load_library()
        self._n = 0

    def attend(self, x: torch.Tensor, kv, decode: bool = False, stream=None) -> None:
        """foe_shard_attend: x is x[h] ([S, hidden]); kv is this cluster's own cache."""
        assert x.is_cuda and x.is_contiguous() and x.dtype == torch.bfloat16 and x.dim() == 2
        n = kv.block_table.shape[0] if decode else x.shape[0]
        mq = 1 if decode else (int(kv.q_lens.max().item()) if n else 0)
        c = self.layer._kv(kv, n, mq, decode)
        _check(self.lib.foe_shard_attend(self.layer.handle, self.exchange.handle, x.data_ptr(), ctypes.byref(c),
                                         1 if decode else 0, _stream_ptr(stream)), "foe_shard_attend")
        self._n = n

    def reduce(self, stream=None) -> None:
        self.exchange.reduce(stream)

    def ffn(self, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """foe_shard_ffn: returns x'[h] ([S, hidden])."""
        if out is None:
            out = torch.empty((self._n, self.full_shape.hidden), dtype=torch.bfloat16, device="cuda")
        _check(self.lib.foe_shard_ffn(self.layer.handle, self.exchange.handle, out.data_ptr(), _stream_ptr(stream)),
               "foe_shard_ffn")
        return out

    def forward(self, x: torch.Tensor, kv, decode: bool = False, stream=None) -> torch.Tensor:
        """All three steps back to back: the call of a rank that has its GPU to itself."""
        self.attend(x, kv, decode, stream)
        self.reduce(stream)
        return self.ffn(stream=stream)

    def close(self) -> None:
        self.layer.close()


# ------------------------------------------------------------------ forming a group

def gather_handles(my_handle: bytes, my_cfg: Sequence[int], rank: int, world: int,
                   all_gather: Callable[[torch.Tensor], List[torch.Tensor]]) -> List[bytes]:
    """Every rank's 64-byte handle, in rank order.  `all_gather(t)` returns the list of every rank's `t` (uint8).
    The ranks also compare their exchange descriptions (n_ranks, hidden, max_tokens): a group whose members
    disagree would compute different buffer layouts, so that is an error on every rank."""
    assert len(my_handle) == HANDLE_BYTES
    desc = ",".join(str(int(v)) for v in my_cfg).encode()
    assert len(desc) <= 60
    msg = torch.zeros(HANDLE_BYTES + 64, dtype=torch.uint8)
    msg[:HANDLE_BYTES] = torch.frombuffer(bytearray(my_handle), dtype=torch.uint8)
    msg[HANDLE_BYTES] = rank
    msg[HANDLE_BYTES + 1] = len(desc)
    msg[HANDLE_BYTES + 2:HANDLE_BYTES + 2 + len(desc)] = torch.frombuffer(bytearray(desc), dtype=torch.uint8)
    parts = all_gather(msg)
    if len(parts) != world:
        raise RuntimeError(f"expected {world} handles, got {len(parts)}")
    out: List[Optional[bytes]] = [None] * world
    for p in parts:
        p = p.cpu()
        r = int(p[HANDLE_BYTES])
        n = int(p[HANDLE_BYTES + 1])
        their = bytes(p[HANDLE_BYTES + 2:HANDLE_BYTES + 2 + n].tolist())
        if their != desc:
            raise RuntimeError(f"rank {r} describes the exchange as ({their.decode()}), this rank as ({desc.decode()})")
        if not (0 <= r < world) or out[r] is not None:
            raise RuntimeError(f"bad or duplicate rank {r} among the gathered handles")
        out[r] = bytes(p[:HANDLE_BYTES].tolist())
    return out  # type: ignore[return-value]


def connect(shape, max_tokens: int, wait_limit_ms: int = 0,
            make_buffer: Callable[..., object] = ExchangeBuffer, make_exchange: Callable[..., object] = Exchange):
    """One process per GPU (torch.distributed initialised, world size = n_clusters): allocate this rank's buffer,
    swap IPC handles, map the peers' buffers, create the exchange.  Returns (exchange, buffers); keep `buffers`
    alive as long as the exchange.  `make_buffer` / `make_exchange` exist so that the plumbing can be exercised
    without a device."""
    import torch.distributed as dist
    rank, world = dist.get_rank(), dist.get_world_size()
    if world != shape.n_clusters:
        raise RuntimeError(f"{world} ranks for {shape.n_clusters} clusters: the group has one rank per cluster")
    cfg = exchange_config(shape, rank, max_tokens, wait_limit_ms)
    mine = make_buffer(cfg)

    def all_gather(t: torch.Tensor) -> List[torch.Tensor]:
        dev = torch.device("cuda", torch.cuda.current_device()) if dist.get_backend() == "nccl" else torch.device("cpu")
        t = t.to(dev)
        parts = [torch.empty_like(t) for _ in range(world)]
        dist.all_gather(parts, t)
        return parts

    handles = gather_handles(mine.export(), (cfg.n_ranks, cfg.hidden, cfg.max_tokens), rank, world, all_gather)
    buffers = [mine if r == rank else make_buffer(cfg, imported_from=handles[r]) for r in range(world)]
    ex = make_exchange(cfg, [b.ptr for b in buffers])
    dist.barrier()          # nobody pushes before every rank has mapped every buffer
    return ex, buffers


class LocalGroup:
    """All H ranks of a group on the current device: H exchange buffers, H exchanges and, per block, H layer
    handles.  Phases are issued rank by rank -- every attend, then every reduce, then every ffn -- on one stream."""

    def __init__(self, shape, max_tokens: int, wait_limit_ms: int = 0):
        self.shape, self.H = shape, shape.n_clusters
        cfgs = [exchange_config(shape, h, max_tokens, wait_limit_ms) for h in range(self.H)]
        self.buffers = [ExchangeBuffer(c) for c in cfgs]
        ptrs = [b.ptr for b in self.buffers]
        self.exchanges = [Exchange(c, ptrs) for c in cfgs]

    def make_layer(self, shape, weights: Dict[str, torch.Tensor], max_tokens: int, max_seqs: int, max_context: int
                   ) -> List[ShardedLayer]:
        return [ShardedLayer(shape, cluster_weights(shape, weights, h), h, self.exchanges[h], max_tokens, max_seqs,
                             max_context) for h in range(self.H)]

    def forward(self, layers: List[ShardedLayer], x: torch.Tensor, kvs, decode: bool = False) -> torch.Tensor:
        """x: [H, S, hidden] (or [S, hidden] on a first layer); kvs: the H per-cluster caches.  Returns
        [H, S, hidden], or the [S, hidden] mean over clusters on a last layer."""
        shape = layers[0].full_shape
        for h, l in enumerate(layers):
            l.attend(x if not shape.grouped_input else x[h], kvs[h], decode)
        for l in layers:
            l.reduce()
        outs = [l.ffn() for l in layers]
        if shape.grouped_output:
            return torch.stack(outs)
        return self.allreduce(outs, 1.0 / self.H)[0]

    def allreduce(self, tensors: List[torch.Tensor], scale: float = 1.0) -> List[torch.Tensor]:
        """sum_h scale * tensors[h] on every rank (push, reduce, gather as three phases over all ranks)."""
        for ex, t in zip(self.exchanges, tensors):
            ex.push(t, scale)
        for ex in self.exchanges:
            ex.reduce()
        return [ex.gather() for ex in self.exchanges]

    def poll_status(self) -> int:
        bad = [s for s in (ex.poll_status() for ex in self.exchanges) if s != 0]
        return bad[0] if bad else 0

    def close(self) -> None:
        for ex in self.exchanges:
            ex.close()
        for b in self.buffers:
            b.close()


def split_cache(shape, kv, h: int):
    """Cluster h's own cache cut out of a cache over all KV heads (copies: pages hold the heads interleaved)."""
    c = shape.kv_per_cluster
    return dataclasses.replace(kv, k_pages=kv.k_pages[:, h * c:(h + 1) * c].contiguous(),
                               v_pages=kv.v_pages[:, h * c:(h + 1) * c].contiguous())
