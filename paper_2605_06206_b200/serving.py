"""Request-level harness on top of the block calls: continuous batching over a stack of FoE layers.

The paper evaluates its engine per request (Section 5: time to first token, time between tokens and end-to-end
latency, mean / p50 / p99, requests arriving as a Poisson process).  This module is the single-GPU counterpart for
the kernels of this package: a page pool, a scheduler that mixes prompt chunks of waiting requests with the decode
tokens of running ones into one batch per iteration (the serving mode of the paper's engine: chunked prefill and
paged attention), and the latency bookkeeping.  It holds no arithmetic of the method: every iteration is one
`foe_prefill` call per layer on a mixed batch.

Time is the device's: each iteration advances a simulated clock by its measured duration (CUDA events), and
requests become visible to the scheduler when the clock passes their arrival time.  The model is "vocabulary-free":
the hidden state fed for a token is a seeded synthetic row, so nothing depends on sampled tokens.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Callable, Dict, List, Optional, Sequence, Tuple

PAGE = 64


# ------------------------------------------------------------------------------------------------ page pool
class PagePool:
    """Free-list allocator of physical KV pages (ids 0..num_pages-1), shared by all layers of a stack."""

    def __init__(self, num_pages: int):
        self.num_pages = num_pages
        self._free = list(range(num_pages - 1, -1, -1))      # pop() hands out ascending ids

    @property
    def free(self) -> int:
        return len(self._free)

    def take(self, n: int) -> List[int]:
        if n > len(self._free):
            raise MemoryError(f"page pool exhausted: {n} wanted, {len(self._free)} free")
        return [self._free.pop() for _ in range(n)]

    def give(self, pages: Sequence[int]) -> None:
        self._free.extend(reversed(list(pages)))


def pages_for(tokens: int) -> int:
    return (tokens + PAGE - 1) // PAGE


# ------------------------------------------------------------------------------------------------ requests
@dataclasses.dataclass
class Request:
    rid: int
    arrival: float                  # seconds on the simulated clock
    prompt_len: int
    output_len: int                 # tokens generated after the prompt (>= 1)
    # filled in by the engine
    pages: List[int] = dataclasses.field(default_factory=list)
    cached: int = 0                 # tokens of this request whose K/V are in the cache
    generated: int = 0
    token_times: List[float] = dataclasses.field(default_factory=list)   # clock at which each output token appeared
    finished: Optional[float] = None

    @property
    def total_len(self) -> int:
        return self.prompt_len + self.output_len

    @property
    def prefilling(self) -> bool:
        return self.cached < self.prompt_len


def poisson_requests(n: int, rate: float, prompt_lens: Sequence[int], output_lens: Sequence[int], u01: Sequence[float]
                     ) -> List[Request]:
    """n requests with exponential inter-arrival times of mean 1/rate (u01: n uniform numbers in (0, 1))."""
    t, out = 0.0, []
    for i in range(n):
        t += -math.log(max(1e-12, 1.0 - u01[i])) / rate
        out.append(Request(i, t, int(prompt_lens[i]), max(1, int(output_lens[i]))))
    return out


# ------------------------------------------------------------------------------------------------ scheduler
@dataclasses.dataclass
class BatchItem:
    req: Request
    q_len: int                      # new tokens of this request in the iteration
    context: int                    # tokens already cached before the iteration


class Scheduler:
    """Continuous batching with chunked prefill.

    Every iteration first gives each running request in its decode phase one token, then fills what is left of the
    token budget with prompt chunks: requests that are already part-way through their prompt first, then waiting
    requests in arrival order, as long as the page pool can hold a request's whole prompt + output (pages are
    reserved at admission, so a running request can never be starved of pages)."""

    def __init__(self, pool: PagePool, max_batch_tokens: int, max_seqs: int, chunk: int):
        assert chunk % PAGE == 0 and chunk > 0
        self.pool, self.max_batch_tokens, self.max_seqs, self.chunk = pool, max_batch_tokens, max_seqs, chunk
        self.waiting: List[Request] = []
        self.running: List[Request] = []

    def add(self, req: Request) -> None:
        self.waiting.append(req)

    def next_batch(self) -> List[BatchItem]:
        items: List[BatchItem] = []
        budget = self.max_batch_tokens
        for r in self.running:                                  # decode tokens
            if not r.prefilling and budget > 0 and len(items) < self.max_seqs:
                items.append(BatchItem(r, 1, r.cached))
                budget -= 1
        for r in self.running:                                  # prompts in progress
            if r.prefilling and budget > 0 and len(items) < self.max_seqs:
                q = min(self.chunk, r.prompt_len - r.cached, budget)
                items.append(BatchItem(r, q, r.cached))
                budget -= q
        while self.waiting and budget > 0 and len(items) < self.max_seqs:      # admissions, first come first served
            r = self.waiting[0]
            need = pages_for(r.total_len)
            if need > self.pool.free:
                break
            self.waiting.pop(0)
            r.pages = self.pool.take(need)
            self.running.append(r)
            q = min(self.chunk, r.prompt_len, budget)
            items.append(BatchItem(r, q, 0))
            budget -= q
        return items

    def commit(self, items: Sequence[BatchItem], now: float) -> List[Request]:
        """Book the iteration that just finished at clock `now`; returns the requests that completed."""
        done = []
        for it in items:
            r = it.req
            was_prefilling = r.prefilling
            r.cached += it.q_len
            if was_prefilling and not r.prefilling:
                r.generated = 1                                 # the last prompt position yields the first token
                r.token_times.append(now)
            elif not was_prefilling:
                r.generated += 1
                r.token_times.append(now)
            if r.generated >= r.output_len:
                r.finished = now
                done.append(r)
        for r in done:
            self.running.remove(r)
            self.pool.give(r.pages)
            r.pages = []
        return done


# ------------------------------------------------------------------------------------------------ metrics
def percentile(xs: Sequence[float], p: float) -> float:
    if not xs:
        return float("nan")
    s = sorted(xs)
    k = (len(s) - 1) * p / 100.0
    lo, hi = int(math.floor(k)), int(math.ceil(k))
    return s[lo] + (s[hi] - s[lo]) * (k - lo)


def latency_report(reqs: Sequence[Request]) -> Dict[str, Dict[str, float]]:
    """TTFT, TBT and end-to-end latency in milliseconds: mean, p50, p99 (the format of the paper's latency tables)."""
    ttft = [1e3 * (r.token_times[0] - r.arrival) for r in reqs if r.token_times]
    e2e = [1e3 * (r.finished - r.arrival) for r in reqs if r.finished is not None]
    tbt = [1e3 * (b - a) for r in reqs for a, b in zip(r.token_times, r.token_times[1:])]
    out = {}
    for name, xs in (("ttft_ms", ttft), ("tbt_ms", tbt), ("e2e_ms", e2e)):
        out[name] = dict(mean=sum(xs) / len(xs) if xs else float("nan"), p50=percentile(xs, 50), p99=percentile(xs, 99),
                         n=len(xs))
    return out


# ------------------------------------------------------------------------------------------------ engine
class Engine:
    """Drives a forward function with the scheduler's batches.

    forward(items) runs one iteration on the device and returns its duration in seconds; it is the only part that
    touches the GPU (see FoeStackRunner).  Anything callable with that contract can stand in for it, which is how the
    host logic is tested without a GPU."""

    def __init__(self, scheduler: Scheduler, forward: Callable[[Sequence[BatchItem]], float]):
        self.sched, self.forward = scheduler, forward
        self.clock = 0.0
        self.iterations = 0
        self.batch_tokens: List[int] = []

    def run(self, requests: Sequence[Request], max_iterations: int = 1 << 30) -> List[Request]:
        pending = sorted(requests, key=lambda r: r.arrival)
        at, finished = 0, []
        while (at < len(pending) or self.sched.waiting or self.sched.running) and self.iterations < max_iterations:
            while at < len(pending) and pending[at].arrival <= self.clock:
                self.sched.add(pending[at])
                at += 1
            items = self.sched.next_batch()
            if not items:
                if at < len(pending):                       # idle until the next arrival
                    self.clock = max(self.clock, pending[at].arrival)
                    continue
                if self.sched.waiting:
                    raise MemoryError("a waiting request does not fit the page pool even when it is empty")
                break
            self.clock += self.forward(items)
            self.iterations += 1
            self.batch_tokens.append(sum(i.q_len for i in items))
            finished += self.sched.commit(items, self.clock)
        return finished


class FoeStackRunner:
    """forward() for Engine on a stack of FoE layers (first, middle..., last) with per-layer page pools.

    One batch = one foe_prefill per layer (foe_decode when every sequence contributes a single token): sequences in scheduler order, their new tokens concatenated; the
    block table row of a sequence lists the pages reserved for the request."""

    def __init__(self, base_shape, n_layers: int, seed: int, num_pages: int, max_batch_tokens: int, max_seqs: int,
                 max_context: int, device: str = "cuda"):
        import torch
        from . import binding, synth
        self.torch, self.synth = torch, synth
        self.shape, self.seed, self.device = base_shape, seed, device
        self.max_pages_per_seq = pages_for(max_context)
        self.layers = []
        for l in range(n_layers):
            pos = "single" if n_layers == 1 else ("first" if l == 0 else ("last" if l == n_layers - 1 else "middle"))
            sh = dataclasses.replace(base_shape, position=pos)
            W = synth.make_weights(sh, seed, device, layer=l + 1)
            self.layers.append(binding.FoeLayer(sh, W, max_tokens=max_batch_tokens, max_seqs=max_seqs,
                                                max_context=max_context,
                                                share_workspace_with=self.layers[0] if self.layers else None))
            del W
        torch.cuda.empty_cache()
        nkv, dh = base_shape.n_kv_heads, base_shape.head_dim
        self.k = [torch.zeros((num_pages, nkv, PAGE, dh), dtype=torch.bfloat16, device=device) for _ in range(n_layers)]
        self.v = [torch.zeros((num_pages, nkv, PAGE, dh), dtype=torch.bfloat16, device=device) for _ in range(n_layers)]
        self.step = 0
        self.collect: Optional[Dict[int, list]] = None      # set to {} to keep every request's output rows (tests)

    def inputs(self, items: Sequence[BatchItem]):
        """Seeded hidden rows for the batch: row (request, position) is always the same, whatever batch it is in."""
        torch, synth = self.torch, self.synth
        d = self.shape.hidden
        rows = [synth.normal_bf16(self.seed + 7919 * (it.req.rid + 1), 31, (it.q_len, d), 1.0, 0.0, self.device,
                                  start=it.context * d) for it in items]
        return torch.cat(rows, 0).contiguous()

    def forward(self, items: Sequence[BatchItem]) -> float:
        torch, synth = self.torch, self.synth
        n = len(items)
        bt = torch.zeros((n, self.max_pages_per_seq), dtype=torch.int32)
        for s, it in enumerate(items):
            bt[s, :len(it.req.pages)] = torch.tensor(it.req.pages, dtype=torch.int32)
        ctx = torch.tensor([it.context for it in items], dtype=torch.int32)
        ql = torch.tensor([it.q_len for it in items], dtype=torch.int32)
        bt, ctx, ql = bt.to(self.device), ctx.to(self.device), ql.to(self.device)
        x = self.inputs(items)
        S, mq = int(x.shape[0]), max(it.q_len for it in items)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        h = x
        for l, layer in enumerate(self.layers):
            kv = synth.PagedKV(self.k[l], self.v[l], bt, ctx, ql)
            # an iteration of decode tokens only takes the decode entry point (split-KV attention, weight streaming)
            h = layer.decode(h, kv) if mq == 1 else layer.prefill(h, kv, n_tokens=S, max_q_len=mq)
        e1.record()
        torch.cuda.synchronize()
        status = self.layers[0].poll_status()
        if status != 0:
            raise RuntimeError(f"device status {status}")
        if self.collect is not None:
            at = 0
            for it in items:
                self.collect.setdefault(it.req.rid, []).append(h[at:at + it.q_len].cpu())
                at += it.q_len
        self.step += 1
        return e0.elapsed_time(e1) * 1e-3

    def close(self):
        for layer in self.layers:
            layer.close()


def synthetic_trace(n: int, rate: float, seed: int, prompt_range: Tuple[int, int] = (1024, 16384),
                    output_range: Tuple[int, int] = (32, 256)) -> List[Request]:
    """Long-prompt request mix standing in for the paper's long-context suite: prompt lengths log-uniform in
    prompt_range, output lengths uniform in output_range, Poisson arrivals.  Seeded with the package's counter hash."""
    from . import synth
    u = [(int(synth.hash16_scalar(seed, 41, i)) + 0.5) / 65536.0 for i in range(3 * n)]
    lo, hi = prompt_range
    prompts = [int(round(math.exp(math.log(lo) + u[i] * (math.log(hi) - math.log(lo))))) for i in range(n)]
    outs = [output_range[0] + int(u[n + i] * (output_range[1] - output_range[0] + 1)) for i in range(n)]
    return poisson_requests(n, rate, prompts, outs, u[2 * n:])
