"""Seeded random layer shapes and batches against the oracle: every draw is reproducible from its case number.
The draws cover what the fixed cases do not pair up: head widths with group sizes, cluster counts with expert counts,
token counts on both sides of the sizes at which the library changes kernels, cached context with ragged chunks."""
import random

import pytest

from paper_2605_06206_b200 import synth

from parity import run_block_parity
from test_gpu_shard import run_group

pytestmark = pytest.mark.gpu


def draw_shape(rng: random.Random) -> synth.LayerShape:
    while True:
        H = rng.choice([1, 2, 3, 4, 5, 8])
        dh = rng.choice([64, 96, 128])
        c = rng.choice([1, 2])                      # KV heads per cluster
        group = rng.choice([1, 2, 4])               # query heads per KV head
        n_kv, n_q = H * c, H * c * group
        if (n_q * dh) % 128 or n_q * dh > 2048:
            continue
        hidden = 128 * rng.choice([1, 2, 3, 4, 8])
        Ec = rng.choice([1, 2, 4, 8, 16])
        k = rng.randint(1, min(Ec, 4))
        inter = 128 * rng.choice([1, 2, 3])
        position = rng.choice(["middle", "middle", "first", "last", "single"] if H > 1 else ["middle", "single"])
        sync = rng.choice(["mean", "sum"])
        return synth.LayerShape(hidden, n_q, n_kv, H, dh, Ec, k, inter, position=position, sync=sync)


def draw_batch(rng: random.Random, decode: bool):
    if decode:
        n = rng.choice([1, 2, 7, 64, 65, 150])
        return [1] * n, [rng.choice([0, 1, 63, 64, 65, 127, 200, 513]) for _ in range(n)]
    n = rng.randint(1, 4)
    q = [rng.choice([1, 5, 63, 64, 65, 130, 257, 300]) for _ in range(n)]
    ctx = [rng.choice([0, 0, 64, 130, 191]) for _ in range(n)]
    return q, ctx


@pytest.mark.parametrize("case", range(64))
def test_random_shape_and_batch(case):
    rng = random.Random(7000 + case)
    shape = draw_shape(rng)
    decode = rng.random() < 0.4
    q_lens, ctx_lens = draw_batch(rng, decode)
    run_block_parity(shape, 7000 + case, q_lens, ctx_lens, decode=decode)


@pytest.mark.timeout(300)
@pytest.mark.parametrize("case", range(20100, 20148))
def test_random_shape_and_batch_second_series(case):
    """A second series of draws with decode steps as likely as prefill calls.  Draw 20122 (head width 96, five
    clusters, 150 sequences) is the one that found the weight-streaming QKV kernel waiting forever in a CTA's second
    task: a full-mask shuffle sat behind a row test that the lanes of a ragged last chunk fail."""
    rng = random.Random(case)
    shape = draw_shape(rng)
    decode = rng.random() < 0.5
    q_lens, ctx_lens = draw_batch(rng, decode)
    run_block_parity(shape, case, q_lens, ctx_lens, decode=decode)


@pytest.mark.parametrize("case", range(16))
def test_random_shape_and_batch_one_cluster_per_rank(case):
    rng = random.Random(9000 + case)
    while True:
        shape = draw_shape(rng)
        if (shape.n_clusters > 1 and shape.hidden % (32 * shape.n_clusters) == 0
                and (shape.q_per_cluster * shape.head_dim) % 128 == 0):
            break
    decode = rng.random() < 0.4
    q_lens, ctx_lens = draw_batch(rng, decode)
    run_group(shape, 9000 + case, q_lens, ctx_lens, decode=decode)


@pytest.mark.parametrize("case", range(16))
def test_random_wide_expert_sets_with_skewed_routing(case):
    """Many experts per cluster (up to the 128 the library takes), wider top-k, a popularity-skewed router bias with
    dead experts on every other case, scaled weights so that the routing logits spread."""
    rng = random.Random(11000 + case)
    H = rng.choice([1, 2, 4, 8])
    Ec = rng.choice([32, 64, 128])
    k = rng.choice([1, 2, 4, 8])
    hidden = 128 * rng.choice([2, 4, 8])
    shape = synth.LayerShape(hidden, 2 * H, H, H, rng.choice([64, 128]), Ec, k, 128 * rng.choice([1, 2]),
                             position=rng.choice(["middle", "first", "last"]) if H > 1 else "single")
    bias = synth.zipf_router_bias(shape, 11000 + case, 1.0, 1.2, dead_per_cluster=rng.choice([0, 5])) if case % 2 else None
    decode = rng.random() < 0.4
    if decode:
        n = rng.choice([3, 64, 200])
        q_lens, ctx_lens = [1] * n, [rng.choice([0, 63, 64, 300]) for _ in range(n)]
    else:
        q_lens = [rng.choice([20, 257, 700, 1500]) for _ in range(rng.randint(1, 2))]
        ctx_lens = [rng.choice([0, 64, 100]) for _ in q_lens]
    # wider layers take a smaller factor: attention logits grow with the square of the factor and with the width,
    # and past a point the softmax turns bf16 noise in q and k into errors beyond the stress bounds
    run_block_parity(shape, 11000 + case, q_lens, ctx_lens, decode=decode, wscale=4.0 if hidden <= 512 else 2.0,
                     router_bias=bias)
