"""Request-level harness on the GPU: continuous batching over a small FoE stack.  What a request computes must not
depend on which other requests share its batches or on how its prompt was chunked."""
import pytest
import torch

from paper_2605_06206_b200 import serving as sv
from paper_2605_06206_b200 import synth

pytestmark = pytest.mark.gpu


def _runner():
    shape = synth.LayerShape(256, 8, 4, 4, 64, 8, 2, 128)
    return sv.FoeStackRunner(shape, n_layers=3, seed=9, num_pages=64, max_batch_tokens=512, max_seqs=8, max_context=640)


def test_batched_serving_matches_each_request_served_alone():
    runner = _runner()
    reqs = sv.synthetic_trace(7, rate=4000.0, seed=3, prompt_range=(40, 500), output_range=(2, 7))
    pool = sv.PagePool(64)
    runner.collect = {}
    eng = sv.Engine(sv.Scheduler(pool, max_batch_tokens=512, max_seqs=8, chunk=128), runner.forward)
    done = eng.run(reqs)
    assert len(done) == 7 and pool.free == 64
    assert max(eng.batch_tokens) <= 512 and max(eng.batch_tokens) > 128          # batches really were shared
    together = {rid: torch.cat(rows, 0).float() for rid, rows in runner.collect.items()}
    rep = sv.latency_report(reqs)
    assert rep["ttft_ms"]["n"] == 7 and rep["ttft_ms"]["mean"] > 0 and rep["e2e_ms"]["p99"] >= rep["e2e_ms"]["p50"]
    # the same requests, one at a time, prompts in 64-token chunks: other batches, other tile positions
    for r in reqs:
        alone = sv.Request(r.rid, 0.0, r.prompt_len, r.output_len)
        runner.collect = {}
        sv.Engine(sv.Scheduler(sv.PagePool(64), 512, 8, 64), runner.forward).run([alone])
        mine = torch.cat(runner.collect[r.rid], 0).float()
        ref = together[r.rid]
        assert mine.shape == ref.shape == (r.prompt_len + r.output_len - 1, 256)
        err = (mine - ref).abs().max().item() / ref.abs().max().item()
        assert err <= 1e-2, f"request {r.rid}: batching changed its output by {err:.2e}"
    runner.close()
