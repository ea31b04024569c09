"""Opt-in soak: the seeded generators of the fuzz tests (and three wider ones) with OTHER seeds than the committed
cases, on one device (the one-cluster-per-rank generator runs its ranks one after the other there).  Skipped unless FOE_SOAK=<draws per generator> is set; FOE_SOAK_BASE moves the seed range.

    FOE_SOAK=300 FOE_SOAK_BASE=70000 python -m pytest tests/test_gpu_soak.py -m gpu -q

Every draw is reproducible from (generator, seed), which a failure prints.  The committed second fuzz series and the
fixed head-width-96 decode cases come from a run of this file."""
import os
import random

import pytest

from paper_2605_06206_b200 import synth

from parity import run_block_parity
from test_gpu_shard import run_group
import test_gpu_fuzz as fuzz

pytestmark = [pytest.mark.gpu, pytest.mark.timeout(3600)]

DRAWS = int(os.environ.get("FOE_SOAK", "0"))
BASE = int(os.environ.get("FOE_SOAK_BASE", "100000"))
needs_soak = pytest.mark.skipif(DRAWS <= 0, reason="set FOE_SOAK=<draws> to run")


def _run(kind, make):
    for seed in range(BASE, BASE + DRAWS):
        rng = random.Random(seed)
        shape, q_lens, ctx_lens, decode = make(rng)
        try:
            run_block_parity(shape, seed, q_lens, ctx_lens, decode=decode)
        except Exception as e:
            raise AssertionError(f"{kind} draw {seed}: {shape} decode={decode} q_lens={q_lens} ctx={ctx_lens}") from e


@needs_soak
def test_soak_fuzz_generator_other_seeds():
    def make(rng):
        shape = fuzz.draw_shape(rng)
        decode = rng.random() < 0.5
        q, c = fuzz.draw_batch(rng, decode)
        return shape, q, c, decode
    _run("shape-and-batch", make)


@needs_soak
def test_soak_mixed_batches_of_many_sequences():
    def make(rng):
        shape = fuzz.draw_shape(rng)
        ns = rng.choice([1, 2, 7, 16, 17, 33, 60])
        if rng.random() < 0.5:       # mostly decode tokens plus a few prompt chunks
            q = [rng.choice([1, 1, 1, 1, 2, 17, 64, 65, 130]) for _ in range(ns)]
        else:
            q = [rng.choice([1, 5, 63, 64, 65, 257, 300, 600]) for _ in range(min(ns, 12))]
        c = [rng.choice([0, 0, 1, 63, 64, 200, 1000, 2500]) for _ in q]
        return shape, q, c, False
    _run("mixed-batch", make)


@needs_soak
def test_soak_decode_steps_of_many_sequences():
    def make(rng):
        shape = fuzz.draw_shape(rng)
        ns = rng.choice([65, 150, 256, 257, 300, 600])
        hi = rng.choice([300, 2000, 6000])
        c = [rng.choice([0, 63, 64, rng.randint(0, hi)]) for _ in range(ns)]
        return shape, [1] * ns, c, True
    _run("large-decode", make)


@needs_soak
def test_soak_wide_groups_and_odd_cluster_counts():
    def make(rng):
        while True:
            H = rng.choice([1, 2, 6, 7]); g = rng.choice([8, 16]); dh = rng.choice([64, 96, 128])
            if (H * g * dh) % 128 == 0 and H * g * dh <= 8192:
                break
        Ec = rng.choice([2, 4, 8])
        shape = synth.LayerShape(128 * rng.choice([2, 4, 7]), H * g, H, H, dh, Ec, rng.randint(1, min(Ec, 2)), 128,
                                 position=rng.choice(["middle", "first", "last"]) if H > 1 else "single")
        decode = rng.random() < 0.5
        if decode:
            ns = rng.choice([3, 70, 150])
            return shape, [1] * ns, [rng.choice([0, 63, 64, 200, 700]) for _ in range(ns)], True
        q = [rng.choice([1, 65, 257, 600]) for _ in range(rng.randint(1, 3))]
        return shape, q, [rng.choice([0, 64, 191]) for _ in q], False
    _run("wide-groups", make)


@needs_soak
def test_soak_wide_expert_sets_with_skewed_routing():
    for seed in range(BASE, BASE + DRAWS):
        rng = random.Random(seed)
        H = rng.choice([1, 2, 4, 8])
        Ec = rng.choice([32, 64, 128, 24, 100])
        k = min(rng.choice([1, 2, 4, 8, 16]), Ec)
        hidden = 128 * rng.choice([2, 4, 8])
        shape = synth.LayerShape(hidden, 2 * H, H, H, rng.choice([64, 128]), Ec, k, 128 * rng.choice([1, 2]),
                                 position=rng.choice(["middle", "first", "last"]) if H > 1 else "single")
        bias = synth.zipf_router_bias(shape, seed, 1.0, 1.2, dead_per_cluster=rng.choice([0, 5])) if seed % 2 else None
        decode = rng.random() < 0.5
        if decode:
            n = rng.choice([3, 64, 200, 256, 257])
            q_lens, ctx_lens = [1] * n, [rng.choice([0, 63, 64, 300]) for _ in range(n)]
        else:
            q_lens = [rng.choice([20, 257, 700, 1500]) for _ in range(rng.randint(1, 2))]
            ctx_lens = [rng.choice([0, 64, 100]) for _ in q_lens]
        try:
            run_block_parity(shape, seed, q_lens, ctx_lens, decode=decode, wscale=4.0 if hidden <= 512 else 2.0,
                             router_bias=bias)
        except Exception as e:
            raise AssertionError(f"wide-experts draw {seed}: {shape} decode={decode} q_lens={q_lens}") from e


@needs_soak
def test_soak_one_cluster_per_rank():
    for seed in range(BASE, BASE + DRAWS):
        rng = random.Random(seed)
        while True:
            shape = fuzz.draw_shape(rng)
            if (shape.n_clusters > 1 and shape.hidden % (32 * shape.n_clusters) == 0
                    and (shape.q_per_cluster * shape.head_dim) % 128 == 0):
                break
        decode = rng.random() < 0.5
        q_lens, ctx_lens = fuzz.draw_batch(rng, decode)
        try:
            run_group(shape, seed, q_lens, ctx_lens, decode=decode)
        except Exception as e:
            raise AssertionError(f"group draw {seed}: {shape} decode={decode} q_lens={q_lens} ctx={ctx_lens}") from e
