"""Host logic of the request-level harness (page pool, continuous-batching scheduler, latency bookkeeping) with a
stand-in for the device call: no GPU needed."""
import math

import pytest

from paper_2605_06206_b200 import serving as sv


def fake_forward(cost_per_token=1e-5, fixed=1e-4, log=None):
    def f(items):
        if log is not None:
            log.append([(it.req.rid, it.context, it.q_len) for it in items])
        return fixed + cost_per_token * sum(it.q_len for it in items)
    return f


def test_page_pool_hands_out_and_takes_back():
    pool = sv.PagePool(10)
    a = pool.take(4)
    b = pool.take(6)
    assert sorted(a + b) == list(range(10)) and pool.free == 0
    with pytest.raises(MemoryError):
        pool.take(1)
    pool.give(a)
    assert pool.free == 4 and sorted(pool.take(4)) == sorted(a)
    assert sv.pages_for(0) == 0 and sv.pages_for(1) == 1 and sv.pages_for(64) == 1 and sv.pages_for(65) == 2


def test_every_request_finishes_budgets_hold_and_no_page_leaks():
    reqs = sv.synthetic_trace(40, rate=200.0, seed=5, prompt_range=(100, 3000), output_range=(4, 40))
    pool = sv.PagePool(400)
    log = []
    sched = sv.Scheduler(pool, max_batch_tokens=2048, max_seqs=16, chunk=512)
    eng = sv.Engine(sched, fake_forward(log=log))
    done = eng.run(reqs)
    assert len(done) == len(reqs) and pool.free == 400 and not sched.running and not sched.waiting
    for batch in log:
        assert 0 < sum(q for _, _, q in batch) <= 2048 and len(batch) <= 16
        assert len({rid for rid, _, _ in batch}) == len(batch)          # a request appears once per iteration
    # per request: contexts are contiguous from 0 and cover prompt + output - 1 positions (the last generated token
    # is never fed back); chunks respect the chunk size; decode phases are single tokens
    by = {}
    for batch in log:
        for rid, ctx, q in batch:
            by.setdefault(rid, []).append((ctx, q))
    for r in reqs:
        at = 0
        for ctx, q in by[r.rid]:
            assert ctx == at and q <= 512
            if ctx >= r.prompt_len:
                assert q == 1
            at += q
        assert at == r.prompt_len + r.output_len - 1
        assert r.generated == r.output_len and len(r.token_times) == r.output_len
        assert r.finished == r.token_times[-1] and r.token_times[0] >= r.arrival
        assert all(b > a for a, b in zip(r.token_times, r.token_times[1:]))


def test_admission_is_first_come_first_served_and_waits_for_pages():
    # the pool holds one request at a time: the second may only start after the first has finished
    reqs = [sv.Request(0, 0.0, 640, 3), sv.Request(1, 0.0, 640, 3)]
    pool = sv.PagePool(sv.pages_for(643))
    log = []
    eng = sv.Engine(sv.Scheduler(pool, 4096, 8, 1024), fake_forward(log=log))
    done = eng.run(reqs)
    assert [r.rid for r in done] == [0, 1]
    first_of_1 = next(i for i, b in enumerate(log) if any(rid == 1 for rid, _, _ in b))
    last_of_0 = max(i for i, b in enumerate(log) if any(rid == 0 for rid, _, _ in b))
    assert first_of_1 > last_of_0
    with pytest.raises(MemoryError):                                     # a request larger than the whole pool
        sv.Engine(sv.Scheduler(sv.PagePool(2), 4096, 8, 1024), fake_forward()).run([sv.Request(0, 0.0, 1000, 5)])


def test_clock_idles_until_an_arrival_and_latencies_add_up():
    reqs = [sv.Request(0, 1.0, 128, 2), sv.Request(1, 5.0, 64, 1)]
    eng = sv.Engine(sv.Scheduler(sv.PagePool(16), 1024, 4, 256), fake_forward(cost_per_token=0.0, fixed=0.25))
    eng.run(reqs)
    r0, r1 = reqs
    assert r0.token_times == [1.25, 1.5] and r0.finished == 1.5          # prefill iteration, one decode iteration
    assert r1.token_times == [5.25]
    rep = sv.latency_report(reqs)
    assert rep["ttft_ms"]["mean"] == pytest.approx(250.0) and rep["tbt_ms"]["n"] == 1
    assert rep["tbt_ms"]["mean"] == pytest.approx(250.0) and rep["e2e_ms"]["p50"] == pytest.approx(375.0)


def test_percentile_and_poisson_trace():
    assert sv.percentile([1, 2, 3, 4], 50) == 2.5 and sv.percentile([5], 99) == 5 and math.isnan(sv.percentile([], 50))
    reqs = sv.synthetic_trace(2000, rate=10.0, seed=1)
    gaps = [b.arrival - a.arrival for a, b in zip(reqs, reqs[1:])]
    assert abs(sum(gaps) / len(gaps) - 0.1) < 0.01                        # mean inter-arrival 1 / rate
    assert all(1024 <= r.prompt_len <= 16384 and 32 <= r.output_len <= 256 for r in reqs)
    again = sv.synthetic_trace(2000, rate=10.0, seed=1)
    assert [(r.arrival, r.prompt_len, r.output_len) for r in reqs] == [(r.arrival, r.prompt_len, r.output_len) for r in again]
