"""One PROCESS per rank with real CUDA IPC handles (foe_shard_buffer_export / _import), both ranks on the one device
there is.  Kernels of different processes must not wait on one another on a shared device, so the ranks move in
lock step: after every phase each rank drains its stream and joins a host barrier, and every device-side wait finds
its counters already at their targets (the waits are bounded anyway).  The results must equal, bit for bit, what the
same group computes inside one process."""
import os
import socket

import pytest
import torch
import torch.multiprocessing as mp

from paper_2605_06206_b200 import shard, synth

pytestmark = pytest.mark.gpu

SEED, Q_LENS, CTX = 31, [130, 75], [0, 64]
DEC_CTX = [5, 64, 127, 300, 1]


def the_shape():
    return synth.LayerShape(256, 4, 2, 2, 64, 8, 2, 128)


def allreduce_inputs(shape, rank):
    g = torch.Generator(device="cuda").manual_seed(100 + rank)
    return [torch.randn(n, shape.hidden, device="cuda", generator=g).to(torch.bfloat16) for n in (77, 205, 1, 205)]


def rank_main(rank: int, world: int, port: int, tmp: str) -> None:
    import torch.distributed as dist
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    torch.cuda.set_device(0)
    shape = the_shape()
    S = sum(Q_LENS)

    def in_step():
        torch.cuda.synchronize()
        dist.barrier()

    ex, buffers = shard.connect(shape, max_tokens=S, wait_limit_ms=200)
    W = synth.make_weights(shape, SEED, "cuda")
    layer = shard.ShardedLayer(shape, shard.cluster_weights(shape, W, rank), rank, ex, S, len(DEC_CTX), 512)
    res = {}
    for name, q_lens, ctx, decode in [("prefill", Q_LENS, CTX, False), ("decode", [1] * len(DEC_CTX), DEC_CTX, True)]:
        x = synth.make_x(shape, SEED, sum(q_lens), "cuda")[rank].contiguous()
        kv = shard.split_cache(shape, synth.make_paged_cache(shape, SEED, ctx, q_lens, "cuda"), rank)
        layer.attend(x, kv, decode)
        in_step()
        layer.reduce()
        in_step()
        res[name] = layer.ffn().cpu()
        in_step()
    res["allreduce"] = []
    for t in allreduce_inputs(shape, rank):
        ex.push(t, 0.5)
        in_step()
        ex.reduce()
        in_step()
        res["allreduce"].append(ex.gather().cpu())
        in_step()
    res["status"] = (ex.poll_status(), layer.layer.poll_status())
    torch.save(res, os.path.join(tmp, f"rank{rank}.pt"))
    layer.close()
    ex.close()
    for r, b in enumerate(buffers):            # mappings of the peers' buffers go before their owners free them
        if r != rank:
            b.close()
    in_step()
    buffers[rank].close()
    dist.destroy_process_group()


def test_two_processes_with_ipc_handles_match_the_one_process_group(tmp_path):
    world = 2
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    procs = [ctx.Process(target=rank_main, args=(r, world, port, str(tmp_path))) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=240)
    hung = [p for p in procs if p.is_alive()]
    for p in hung:
        p.kill()
    assert not hung and all(p.exitcode == 0 for p in procs), [p.exitcode for p in procs]
    got = [torch.load(tmp_path / f"rank{r}.pt") for r in range(world)]
    assert all(g["status"] == (0, 0) for g in got)

    shape = the_shape()
    S = sum(Q_LENS)
    group = shard.LocalGroup(shape, max_tokens=S)
    W = synth.make_weights(shape, SEED, "cuda")
    layers = group.make_layer(shape, W, S, len(DEC_CTX), 512)
    for name, q_lens, cl, decode in [("prefill", Q_LENS, CTX, False), ("decode", [1] * len(DEC_CTX), DEC_CTX, True)]:
        x = synth.make_x(shape, SEED, sum(q_lens), "cuda")
        kv = synth.make_paged_cache(shape, SEED, cl, q_lens, "cuda")
        want = group.forward(layers, x, [shard.split_cache(shape, kv, h) for h in range(world)], decode)
        for r in range(world):
            assert torch.equal(got[r][name], want[r].cpu()), f"{name}, rank {r}"
    ins = [allreduce_inputs(shape, r) for r in range(world)]
    for i in range(len(ins[0])):
        want = group.allreduce([ins[r][i] for r in range(world)], 0.5)
        for r in range(world):
            assert torch.equal(got[r]["allreduce"][i], want[r].cpu()), f"all-reduce {i}, rank {r}"
    assert group.poll_status() == 0
    for l in layers:
        l.close()
    group.close()
