#!/usr/bin/env python
"""Benchmark of the FoE block forward pass on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload prefill|decode] [--impl ours|reference]

A step is one pass of the whole block (every stage: norms, projections, attention, sync, routing,
dispatch maps, experts, combine) over one batch of seeded synthetic input.  The default workload is the
single-block prefill (hidden 2048, 16q/4kv heads, 4 clusters x 16 experts, top-2 per cluster, 4 x 4096
tokens); the decode workload (64 sequences, contexts 4096..16384, paged KV) is measured in the same run and
reported under "decode".  With N > 1 (torchrun) every rank runs an independent replica of the workload:
the path has no sharding and no collective, so the aggregate is N x tokens / max-over-ranks time.

Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2605_06206_b200 import replicas, synth  # noqa: E402


def profile_traffic(profile_file: str, kernel: str):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of `kernel` (a substring of its section title) from a
    committed ncu summary under profiles/: the figure is read from the file the JSON line names, never retyped.
    Returns (bytes or None, source string)."""
    path = os.path.join(ROOT, "profiles", profile_file)
    src = f"dram read+write bytes per launch of {kernel}, profiles/{profile_file}"
    try:
        text = open(path).read()
    except OSError:
        return None, src + " (file missing)"
    scale = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    for sec in text.split("\n## ")[1:]:
        title, _, body = sec.partition("\n")
        if kernel not in title:
            continue
        tot, seen = 0.0, 0
        for line in body.splitlines():
            cells = [c.strip() for c in line.strip().strip("|").split("|")]
            if len(cells) >= 3 and cells[0] in ("dram__bytes_read.sum", "dram__bytes_write.sum") and cells[2] in scale:
                tot += float(cells[1].replace(",", "")) * scale[cells[2]]
                seen += 1
        if seen == 2:
            return tot, src
    return None, src + " (kernel not found)"


# ----------------------------------------------------------------------------------------------
def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            m = json.load(f)
        return dict(hbm_gbs=float(m["hbm_gbs"]), bf16_tflops=float(m["bf16_tflops"]),
                    bf16_tflops_sustained=float(m.get("bf16_tflops_sustained", m["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    samples=len(sm), reasons=sorted(reasons))


# ----------------------------------------------------------------------------------------------
def build_workload(kind: str, device, seed_offset: int = 0):
    """Layer + inputs of the prefill (workload 2) or decode (workload 3) benchmark on `device`."""
    from paper_2605_06206_b200 import binding
    n = 2 if kind == "prefill" else 3
    shape, info = synth.workload(n)
    seed = info["seed"] + 1000 * seed_offset
    W = synth.make_weights(shape, seed, device)
    q_lens, ctx = info["q_lens"], info["context_lens"]
    S = sum(q_lens)
    x = synth.make_x(shape, seed, S, device)
    kv = synth.make_paged_cache(shape, seed, ctx, q_lens, device)
    layer = binding.FoeLayer(shape, W, max_tokens=S if kind == "prefill" else 1, max_seqs=len(q_lens),
                             max_context=max(c + q for c, q in zip(ctx, q_lens)))
    del W
    torch.cuda.empty_cache()
    return dict(kind=kind, shape=shape, info=info, layer=layer, x=x, kv=kv, S=S, n=n)


def step_fn(wl):
    layer, x, kv, S = wl["layer"], wl["x"], wl["kv"], wl["S"]
    out = torch.empty_like(x) if wl["shape"].grouped_output == wl["shape"].grouped_input else None
    mq = max(wl["info"]["q_lens"])
    if wl["kind"] == "prefill":
        return (lambda: layer.prefill(x, kv, n_tokens=S, max_q_len=mq, out=out)), out
    return (lambda: layer.decode(x, kv, out=out)), out


def timed_loop(fn, steps, warmup, dist_on):
    """W untimed steps, then exactly K steps between CUDA events, bracketed by a barrier and a device
    synchronisation on both sides; returns this rank's milliseconds for the K steps."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    replicas.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    replicas.barrier()
    return ms


def sustained_profile(layer, fn, ms_per_step, seconds=1.2, ring=64):
    """Runs the step back to back for about `seconds` of device time (no host synchronisation in between) and, without
    a pause, `ring` more steps with the library's stage events on.  Returns (ms per step over the long run, mean
    per-stage ms of the profiled steps, number of steps of the long run): the stage times are taken where the GPU has
    settled to the clocks it sustains.  (The stage events themselves cost a few microseconds per step and keep
    neighbouring kernels from overlapping, so the stage times of a step of many short kernels add up to a little more
    than the step.)"""
    n = max(8, int(seconds * 1e3 / max(ms_per_step, 1e-3)) + 1)
    if seconds <= 0:                   # profiler runs: no long run, a handful of profiled steps
        n, ring = 1, min(ring, 4)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(n):
        fn()
    e1.record()
    layer.set_profiling(ring)
    for _ in range(ring):
        fn()
    torch.cuda.synchronize()
    stages = layer.stage_ms()
    layer.set_profiling(0)
    return e0.elapsed_time(e1) / n, stages, n


def library_gemm_same_shape(R, K, N, seconds=0.6):
    """Context for the tensor roofline, not part of the path: the vendor library's bf16 GEMM (torch.matmul) on ONE dense
    problem with the row count, reduction length and output width of an expert GEMM launch ([R, K] x [K, N]), run
    back to back for `seconds` so that it meets the same power cap.  The measured peak in MEASURED_PEAKS.json is an
    8192^3 problem, whose reduction is four to eight times longer per output element than an expert GEMM's."""
    a = torch.randn(R, K, device="cuda", dtype=torch.bfloat16)
    b = torch.randn(K, N, device="cuda", dtype=torch.bfloat16)
    c = torch.empty(R, N, device="cuda", dtype=torch.bfloat16)
    for _ in range(3):
        torch.matmul(a, b, out=c)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    torch.matmul(a, b, out=c)
    e1.record()
    torch.cuda.synchronize()
    n = max(4, int(seconds * 1e3 / max(e0.elapsed_time(e1), 1e-3)))
    for _ in range(n // 2):                       # settle to the sustained clock, then time the second half
        torch.matmul(a, b, out=c)
    e0.record()
    for _ in range(n - n // 2):
        torch.matmul(a, b, out=c)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / (n - n // 2)
    del a, b, c
    return dict(tflops=2.0 * R * K * N / (ms * 1e-3) / 1e12, ms=ms, shape=[R, K, N], seconds=seconds,
                note="torch.matmul (vendor library) on one dense problem of the launch's size, sustained; context only")


def expert_row_histogram(counts):
    """Rows per expert of the last call: how ragged the grouped GEMMs' tiles were."""
    c = counts.double()
    tiles = int(((counts + 255) // 256).sum())
    return dict(max=int(c.max()), mean=float(c.mean()), min=int(c.min()), empty=int((counts == 0).sum()),
                experts=int(counts.numel()), tiles_of_256_rows=tiles, rows_in_tiles=tiles * 256)


def algorithmic_work(wl):
    """Flops / bytes the method itself must do for this call, from the actual routing of the last call."""
    s, info, S = wl["shape"], wl["info"], wl["S"]
    aux = wl["layer"].aux()
    counts = aux["counts"].cpu()
    touched = int((counts > 0).sum())
    R = int(counts.sum())
    d, I, dh = s.hidden, s.ffn_inter, s.head_dim
    nq, nkv = s.n_q_heads, s.n_kv_heads
    w = dict(rows=R, touched_experts=touched)
    w["gemm1_flops"] = 2.0 * R * d * 2 * I
    w["gemm2_flops"] = 2.0 * R * I * d
    w["qkv_flops"] = 2.0 * S * d * (nq + 2 * nkv) * dh
    w["oproj_flops"] = 2.0 * S * nq * dh * d
    w["router_flops"] = 2.0 * S * d * s.n_experts
    if wl["kind"] == "prefill":
        w["attn_flops"] = sum(2.0 * (c + q) * q * dh * nq * 2 * 0.5 if c == 0 else 4.0 * q * (c + q / 2.0) * dh * nq
                              for c, q in zip(info["context_lens"], info["q_lens"]))
    else:
        w["attn_flops"] = sum(4.0 * (c + 1) * dh * nq for c in info["context_lens"])
    w["total_flops"] = sum(v for k, v in w.items() if k.endswith("_flops"))
    # decode bytes: valid KV tokens, touched experts only, attention + router weights, activations in/out
    kv_bytes = sum((c + 1) for c in info["context_lens"]) * nkv * dh * 2 * 2 if wl["kind"] == "decode" else 0
    w["kv_bytes"] = kv_bytes
    w["gemm1_weight_bytes"] = touched * 2 * I * d * 2
    w["gemm2_weight_bytes"] = touched * I * d * 2
    w["attn_weight_bytes"] = ((nq + 2 * nkv) * dh * d + nq * dh * d) * 2
    w["router_bytes"] = s.n_experts * d * 4
    H = s.n_clusters
    w["act_bytes"] = (H * S * d * 2) * 2
    w["total_bytes"] = (kv_bytes + w["gemm1_weight_bytes"] + w["gemm2_weight_bytes"] + w["attn_weight_bytes"] +
                        w["router_bytes"] + w["act_bytes"])
    return w


def e2e_loop(wl, steps, warmup):
    """Same call with HOST buffers: every step copies its input from pinned host memory to the device, runs the
    block through the C ABI and copies the result back to pinned host memory.  The three legs run on three
    streams with two sets of device buffers, so the copy of step i+1 and the read-back of step i-1 overlap the
    compute of step i (the layer's workspace keeps the compute legs in order)."""
    layer, kv, S = wl["layer"], wl["kv"], wl["S"]
    x_host = wl["x"].cpu().pin_memory()
    mq = max(wl["info"]["q_lens"])
    probe = layer.prefill(wl["x"], kv, n_tokens=S, max_q_len=mq) if wl["kind"] == "prefill" else layer.decode(wl["x"], kv)
    x_dev = [torch.empty_like(wl["x"]) for _ in range(2)]
    out_dev = [torch.empty_like(probe) for _ in range(2)]
    out_host = [torch.empty(probe.shape, dtype=probe.dtype).pin_memory() for _ in range(2)]
    s_in, s_comp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_comp = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]
    torch.cuda.synchronize()

    def one(i):
        b = i & 1
        with torch.cuda.stream(s_in):
            s_in.wait_event(ev_comp[b])                     # the compute that last read x_dev[b] is done
            x_dev[b].copy_(x_host, non_blocking=True)
            ev_in[b].record(s_in)
        with torch.cuda.stream(s_comp):
            s_comp.wait_event(ev_in[b])
            s_comp.wait_event(ev_out[b])                    # the read-back that last used out_dev[b] is done
            if wl["kind"] == "prefill":
                layer.prefill(x_dev[b], kv, n_tokens=S, max_q_len=mq, out=out_dev[b], stream=s_comp)
            else:
                layer.decode(x_dev[b], kv, out=out_dev[b], stream=s_comp)
            ev_comp[b].record(s_comp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_comp[b])
            out_host[b].copy_(out_dev[b], non_blocking=True)
            ev_out[b].record(s_out)

    for i in range(warmup):
        one(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(s_comp)
    for i in range(steps):
        one(i)
    s_comp.wait_event(ev_out[(steps - 1) & 1])
    if steps > 1:
        s_comp.wait_event(ev_out[steps & 1])
    e1.record(s_comp)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    return ms, x_host.numel() * 2, out_host[0].numel() * 2


# ----------------------------------------------------------------------------------------------
def oracle_sample(kind: str, n_tokens: int, seed: int = 0, n_seqs: int = 1):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload.  Returns (seconds, tokens,
    threads, description)."""
    import numpy as np
    from oracle import adapter, foe_oracle as orc
    n = 2 if kind == "prefill" else 3
    shape, info = synth.workload(n)
    W = adapter.weights_to_numpy(synth.make_weights(shape, info["seed"]))
    cfg = adapter.cfg_from_shape(shape)
    threads = os.cpu_count() or 1
    if kind == "prefill":
        x = adapter.to_np(synth.make_x(shape, info["seed"] + seed, n_tokens * n_seqs))
        t0 = time.perf_counter()
        orc.foe_block(cfg, W, x, [n_tokens] * n_seqs)
        dt = time.perf_counter() - t0
        return dt, n_tokens * n_seqs, threads, f"{n_seqs} sequence(s) of {n_tokens} tokens, full block, workload-2 layer"
    n_seqs = n_tokens
    ctx = info["context_lens"][:n_seqs]
    kv = synth.make_paged_cache(shape, info["seed"], ctx, [1] * n_seqs)
    cache = adapter.logical_cache(kv.k_pages, kv.v_pages, kv.block_table, ctx, 64)
    x = adapter.to_np(synth.make_x(shape, info["seed"] + seed, n_seqs))
    t0 = time.perf_counter()
    orc.foe_block(cfg, W, x, [1] * n_seqs, ctx, cache)
    dt = time.perf_counter() - t0
    return dt, n_seqs, threads, f"{n_seqs} of the 64 sequences, one decode step, workload-3 layer and contexts"


def run_reference(args, rank):
    """The reference arm: the CPU oracle on host cores, bounded sample per step."""
    if rank != 0:
        return
    kind = args.workload
    n_tok = 256 if kind == "prefill" else 8
    for _ in range(args.warmup):
        oracle_sample(kind, n_tok)
    tot_s, tot_tok, thr, desc = 0.0, 0, 1, ""
    for i in range(args.steps):
        dt, ntk, thr, desc = oracle_sample(kind, n_tok, seed=i)
        tot_s += dt
        tot_tok += ntk
    val = tot_tok / tot_s
    unit = "tokens/s"
    line = dict(impl="reference", metric=f"foe_block_{kind}_tokens_per_s", value=val, unit=unit, n_gpus=args.gpus,
                steps=args.steps, warmup=args.warmup, ms_per_step=1e3 * tot_s / args.steps, higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload=f"workload {2 if kind == 'prefill' else 3} ({kind}), bounded sample: {desc}"),
                cpu_baseline=dict(value=val, unit=unit, cores=thr, kind="oracle", sample=desc),
                e2e=dict(value=val, unit=unit, h2d_bytes_per_step=0, d2h_bytes_per_step=0), gpu_launches=0)
    print(json.dumps(line))


def roofline_of(kind, work, stages, step_ms, peaks, wl_n):
    """The roofline object of the dominant kernel: achieved = algorithmic flops (bytes) of one launch / its mean
    duration inside the seconds-long run; peak = the measured sustained GEMM rate (copy bandwidth)."""
    if kind == "prefill":
        t = stages["expert_gemm1_swiglu"] * 1e-3
        ach = work["gemm1_flops"] / t / 1e12
        peak = peaks["bf16_tflops_sustained"]
        extra = {}
        if wl_n == 2:
            traffic, tsrc = profile_traffic("ncu_full_prefill_kernels_workload2.md", "gemm_tcgen05_kernel<1, 1>")
        else:     # the full workload-4 batch is too large to capture; the committed capture is of half the batch
            half, tsrc = profile_traffic("ncu_expert_gemms_workload4_half_batch.md", "gemm_tcgen05_kernel<1, 1>")
            traffic, extra = None, dict(traffic_half_batch=half)
            tsrc += " (4 of the 8 sequences: weights do not grow with the batch, activations do; not scaled)"
        return dict(**extra, bound="tensor", kernel="gemm_tcgen05_kernel<SwiGLU, gather> (expert GEMM 1, CTA pairs)", achieved=ach,
                    peak=peak, unit="TFLOP/s", frac=ach / peak, traffic=traffic, traffic_source=tsrc,
                    peak_source=f"{peaks['source']} sustained bf16 (kernel timed deep inside a seconds-long run of steps)",
                    frac_of_burst=ach / peaks["bf16_tflops"], frac_of_nominal_2250=ach / 2250.0,
                    gemm2_tflops=work["gemm2_flops"] / (stages["expert_gemm2"] * 1e-3) / 1e12,
                    attention_tflops=work["attn_flops"] / (stages["attention"] * 1e-3) / 1e12,
                    whole_step_tflops=work["total_flops"] / (step_ms * 1e-3) / 1e12,
                    whole_step_frac=work["total_flops"] / (step_ms * 1e-3) / 1e12 / peak)
    t = stages["attention"] * 1e-3
    ach = work["kv_bytes"] / t / 1e9
    peak = peaks["hbm_gbs"]
    g1 = work["gemm1_weight_bytes"] / (stages["expert_gemm1_swiglu"] * 1e-3) / 1e9
    g2 = work["gemm2_weight_bytes"] / (stages["expert_gemm2"] * 1e-3) / 1e9
    traffic, tsrc = profile_traffic("ncu_full_decode_kernels_workload3.md", "attn_decode_kernel")
    return dict(bound="hbm", kernel="attn_decode_kernel (paged split-KV attention)", achieved=ach,
                peak=peak, unit="GB/s", frac=ach / peak, traffic=traffic, traffic_source=tsrc,
                algorithmic_bytes=work["kv_bytes"],
                peak_source=f"{peaks['source']} copy bandwidth", frac_of_nominal_8000=ach / 8000.0,
                gemm1_gbs=g1, gemm2_gbs=g2,
                whole_step_gbs=work["total_bytes"] / (step_ms * 1e-3) / 1e9,
                whole_step_frac=work["total_bytes"] / (step_ms * 1e-3) / 1e9 / peak)


# ----------------------------------------------------------------------------------------------
def measure(kind, args, dist_on, rank, world, peaks, with_cpu):
    dev = torch.device("cuda", torch.cuda.current_device())
    wl = build_workload(kind, dev, seed_offset=rank)
    fn, _ = step_fn(wl)
    fn()
    torch.cuda.synchronize()
    st = wl["layer"].poll_status()
    if st != 0:
        raise RuntimeError(f"device status {st} after the first {kind} step")
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    ms_local = timed_loop(fn, args.steps, args.warmup, dist_on)
    tokens_per_s, ms = replicas.job_throughput(wl["S"], args.steps, ms_local, device="cuda")
    launches = wl["layer"].last_launch_count()
    # The contract's K steps are a short region (tens of milliseconds): the stage times and the roofline come from a
    # second, seconds-long run of the same steps back to back, which is where the sustained GEMM peak is the right
    # denominator; the clock sampler stays on through both.
    sus_ms, stages, sus_steps = sustained_profile(wl["layer"], fn, ms / 1.0, seconds=args.sustain_seconds)
    clocks = sampler.stop()
    work = algorithmic_work(wl)
    S = wl["S"]
    mhz = clocks.get("sm_mhz") or 0.0
    res = dict(ms_per_step=ms, tokens_per_s=tokens_per_s, launches_per_step=launches, stages_ms=stages,
               stage_sm_mcycles={k: v * mhz * 1e-3 for k, v in stages.items()},     # time x median SM clock, in 10^6 cycles
               sustained=dict(ms_per_step=sus_ms, tokens_per_s=world * S / (sus_ms * 1e-3), steps=sus_steps,
                              seconds=sus_ms * sus_steps * 1e-3,
                              note="the same step back to back for about a second; stages_ms are the mean of the 64 steps that follow it without a pause"),
               clocks=clocks, tokens_per_step=S, expert_rows=expert_row_histogram(wl["layer"].aux()["counts"].cpu()))
    res["roofline"] = roofline_of(kind, work, stages, sus_ms, peaks, wl["n"])
    if kind == "prefill" and rank == 0:
        sh = wl["shape"]
        res["roofline"]["library_gemm_same_shape"] = dict(
            gemm1=library_gemm_same_shape(work["rows"], sh.hidden, 2 * sh.ffn_inter),
            gemm2=library_gemm_same_shape(work["rows"], sh.ffn_inter, sh.hidden))
    res["work"] = {k: v for k, v in work.items()}
    e_ms, h2d, d2h = e2e_loop(wl, max(4, min(args.steps, 10)), 3)
    res["e2e"] = dict(value=world * S / (e_ms * 1e-3), unit="tokens/s", ms_per_step=e_ms, h2d_bytes_per_step=h2d,
                      d2h_bytes_per_step=d2h)
    wl["layer"].close()
    del wl
    torch.cuda.empty_cache()
    if with_cpu:
        dt, ntk, thr, desc = oracle_sample(kind, 4096 if kind == "prefill" else 64, n_seqs=2)   # about 10 s of host work
        res["cpu_baseline"] = dict(value=ntk / dt, unit="tokens/s", cores=thr, kind="oracle", sample=desc,
                                   seconds=dt)
    return res


def measure_skew(args, peaks, clock_index, n_seqs=None):
    """Workload 4, the routing stress: 8 clusters x 32 experts top-4, inter 768, 8 x 2048 tokens, router bias that makes
    per-cluster expert popularity Zipf(1.2), two experts per cluster guaranteed empty.  Same measurement as the headline
    (K steps, then a seconds-long run for the stage times), no end-to-end leg."""
    from paper_2605_06206_b200 import binding
    shape, info = synth.workload(4)
    dev = "cuda"
    seed, q_lens, ctx = info["seed"], info["q_lens"], info["context_lens"]
    if n_seqs:                                              # a reduced batch of the same sequences (profiler captures)
        q_lens, ctx = q_lens[:n_seqs], ctx[:n_seqs]
    S = sum(q_lens)
    W = synth.make_weights(shape, seed, dev)
    layer = binding.FoeLayer(shape, W, max_tokens=S, max_seqs=len(q_lens), max_context=max(q_lens))
    # the bias scale follows the spread of the unbiased scores, measured with the library on a sample
    layer.route(synth.normal_bf16(seed, 79, (2048, shape.hidden), 1.0, 0.0, dev))
    sigma = float(layer.aux()["logits"].std())
    layer.close()
    W["router_b"] = synth.zipf_router_bias(shape, seed, sigma, info["zipf"], dead_per_cluster=2).to(dev)
    layer = binding.FoeLayer(shape, W, max_tokens=S, max_seqs=len(q_lens), max_context=max(q_lens))
    del W
    torch.cuda.empty_cache()
    x = synth.make_x(shape, seed, S, dev)
    kv = synth.make_paged_cache(shape, seed, ctx, q_lens, dev)
    out = torch.empty_like(x)
    mq = max(q_lens)
    fn = lambda: layer.prefill(x, kv, n_tokens=S, max_q_len=mq, out=out)
    wl = dict(kind="prefill", shape=shape, info=info, layer=layer, x=x, kv=kv, S=S, n=4)
    fn()
    torch.cuda.synchronize()
    if layer.poll_status() != 0:
        raise RuntimeError("device status after the first workload-4 step")
    sampler = ClockSampler(clock_index)
    sampler.start()
    steps = max(5, min(args.steps, 20))
    ms = timed_loop(fn, steps, 3, False) / steps
    sus_ms, stages, sus_steps = sustained_profile(layer, fn, ms, seconds=args.sustain_seconds)
    clocks = sampler.stop()
    work = algorithmic_work(wl)
    mhz = clocks.get("sm_mhz") or 0.0
    hist = expert_row_histogram(layer.aux()["counts"].cpu())
    res = dict(workload=f"workload 4: hidden 2048, 16q/8kv heads, 8 clusters x 32 experts top-4, inter 768, {len(q_lens)} x 2048 tokens, "
                        "Zipf(1.2) router bias, 2 dead experts per cluster",
               ms_per_step=ms, tokens_per_s=S / (ms * 1e-3), steps=steps, stages_ms=stages,
               stage_sm_mcycles={k: v * mhz * 1e-3 for k, v in stages.items()},
               sustained=dict(ms_per_step=sus_ms, tokens_per_s=S / (sus_ms * 1e-3), steps=sus_steps),
               clocks=clocks, expert_rows=hist, roofline=roofline_of("prefill", work, stages, sus_ms, peaks, 4),
               launches_per_step=layer.last_launch_count(),
               work=dict(rows=work["rows"], gemm1_flops=work["gemm1_flops"], gemm2_flops=work["gemm2_flops"],
                         total_flops=work["total_flops"]))
    # what the ragged tiles cost: flops of the rows the 256-row tiles actually hold against the useful ones
    res["roofline"]["tile_fill"] = work["rows"] / max(1, hist["rows_in_tiles"])
    layer.close()
    del wl, layer, x, kv, out
    torch.cuda.empty_cache()
    return res


def stack_decode_bytes(st, shape, xs, ctx0):
    """Algorithmic bytes of one decode step of the stack: per layer the weights of the experts the step touches (read
    from the dispatch counts of a layer-by-layer pass, untimed), valid K/V entries, attention and router weights."""
    d, I, dh, nq, nkv = shape.hidden, shape.ffn_inter, shape.head_dim, shape.n_q_heads, shape.n_kv_heads
    touched = []
    st.set_context(ctx0)
    h = xs
    for layer, kv in zip(st.layers, st.kvs):
        h = layer.decode(h, kv)
        touched.append(int((layer.aux()["counts"] > 0).sum()))
    kv_bytes = sum(c + 1 for c in ctx0) * nkv * dh * 2 * 2
    attn_w = ((nq + 2 * nkv) * dh * d + nq * dh * d) * 2
    per_layer = [t * 3 * d * I * 2 + kv_bytes + attn_w + shape.n_experts * d * 4 for t in touched]
    return sum(per_layer), touched


def measure_stack(args, peaks, clock_index, one_cluster=False):
    """Workload 5 as FoE: 16 layers (hidden 4096, 32q/8kv heads, 8 clusters x 16 experts top-2, inter 1408; 72 GB of
    weights), prefill of 2 x 16,384 tokens, then 128 decode steps on the caches it wrote.  A decode step is one
    foe_stack_forward + foe_context_advance; it is timed issued directly and replayed from a CUDA graph.
    one_cluster: the equal-size MoE baseline on the same kernels (1 cluster x 128 experts, top-16)."""
    import dataclasses
    from paper_2605_06206_b200.stack import FoeStack
    shape, info = synth.workload(5)
    if one_cluster:
        shape = dataclasses.replace(shape, n_clusters=1, experts_per_cluster=128, top_k_per_cluster=16)
    q_lens, L, steps = info["q_lens"], info["layers"], info.get("decode_steps", 128)
    st = FoeStack(shape, L, info["seed"], q_lens, steps + 8)
    S, B = sum(q_lens), len(q_lens)
    x0 = synth.make_x(st.shapes[0], info["seed"], S, "cuda")
    out_p = st.forward(x0, [0] * B, decode=False)                        # warm-up (also writes the caches)
    torch.cuda.synchronize()
    sampler = ClockSampler(clock_index)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = 3
    e0.record()
    for _ in range(reps):
        st.run(x0, decode=False, out=out_p)
    e1.record()
    torch.cuda.synchronize()
    prefill_ms = e0.elapsed_time(e1) / reps
    clocks_prefill = sampler.stop()
    d, I, dh, nq, nkv, H = shape.hidden, shape.ffn_inter, shape.head_dim, shape.n_q_heads, shape.n_kv_heads, shape.n_clusters
    R = S * H * shape.top_k_per_cluster
    flops_layer = (R * 3 * d * I * 2.0 + 2.0 * S * d * (nq + 2 * nkv) * dh + sum(2.0 * q * q * dh * nq for q in q_lens) +
                   2.0 * S * nq * dh * d + 2.0 * S * d * shape.n_experts)
    xs = [synth.make_x(st.shapes[0], info["seed"], B, "cuda", tid=synth.TID["x_step"] + s) for s in range(steps)]
    step_bytes, touched = stack_decode_bytes(st, shape, xs[0], list(q_lens))
    out_d = torch.empty_like(xs[0])

    def timed_steps(step_fn):
        st.set_context(q_lens)
        for s in range(3):                                               # warm-up steps (contexts restored below)
            step_fn(s)
        st.set_context(q_lens)
        torch.cuda.synchronize()
        e0.record()
        for s in range(steps):
            step_fn(s)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps

    def direct(s):
        st.run(xs[s], decode=True, out=out_d)
        st.advance(1)

    sampler = ClockSampler(clock_index)
    sampler.start()
    direct_ms = timed_steps(direct)
    # the same step captured once (all layers + the advance) and replayed; its input is copied into a fixed buffer
    x_in = torch.empty_like(xs[0])
    g = torch.cuda.CUDAGraph()
    st.set_context(q_lens)
    torch.cuda.synchronize()
    with torch.cuda.graph(g):
        st.run(x_in, decode=True, out=out_d)
        st.advance(1)

    def replay(s):
        x_in.copy_(xs[s], non_blocking=True)
        g.replay()

    graph_ms = timed_steps(replay)
    clocks_decode = sampler.stop()
    status = st.status()
    st.close()
    del st, x0, xs
    torch.cuda.empty_cache()
    if status != 0:
        raise RuntimeError(f"device status {status} in the stack run")
    best = min(direct_ms, graph_ms)
    gbs = step_bytes / (best * 1e-3) / 1e9
    pf = L * flops_layer / (prefill_ms * 1e-3) / 1e12
    return dict(workload="workload 5: 16-layer stack, hidden 4096, 32q/8kv heads, "
                         + ("1 cluster x 128 experts top-16 (the equal-size MoE baseline)" if one_cluster else "8 clusters x 16 experts top-2")
                         + ", inter 1408; prefill 2 x 16384 tokens, then 128 decode steps of 2 tokens",
                prefill_ms=prefill_ms, prefill_tokens_per_s=S / (prefill_ms * 1e-3), prefill_tflops=pf,
                prefill_frac_of_sustained=pf / peaks["bf16_tflops_sustained"], prefill_frac_of_burst=pf / peaks["bf16_tflops"],
                decode_ms_per_step=best, decode_ms_per_step_direct=direct_ms, decode_ms_per_step_graph=graph_ms,
                decode_tokens_per_s=B / (best * 1e-3), decode_steps=steps,
                decode_bytes_per_step=step_bytes, touched_experts_per_layer_mean=sum(touched) / len(touched),
                decode_gbs=gbs, decode_frac_of_hbm=gbs / peaks["hbm_gbs"], peak_source=f"{peaks['source']} copy bandwidth",
                bytes_note="touched experts (from one step's dispatch counts), valid K/V entries, attention and router weights, per layer",
                clocks_prefill=clocks_prefill, clocks_decode=clocks_decode)


def run_sweep(args):
    """Latency of one block at the paper's 7B (or 1B) layer shape for the token-batch sizes of its forward-latency table
    (1 ... 24,576 tokens, as sequences of at most 2,048 tokens), on one GPU.  Context for that table's shape only:
    the paper's numbers are whole 16-layer models on 8 H100s."""
    from paper_2605_06206_b200 import binding
    if args.sweep_shape == "1b":
        shape = synth.LayerShape(768, 8, 8, 8, 96, 8, 1, 384, rope_theta=5.0e5)
        desc = "paper 1B layer shape (hidden 768, 8q/8kv heads of 96, 8 groups x 8 experts top-1, inter 384)"
    else:
        shape = synth.LayerShape(2048, 16, 8, 8, 128, 8, 1, 1024, rope_theta=5.0e5)
        desc = "paper 7B layer shape (hidden 2048, 16q/8kv, 8 groups x 8 experts top-1, inter 1024)"
    W = synth.make_weights(shape, 7, "cuda")
    sizes = [1, 64, 128, 256, 512, 1024, 2048, 4096, 8192, 12288, 16384, 24576]
    layer = binding.FoeLayer(shape, W, max_tokens=max(sizes), max_seqs=16, max_context=2048)
    rows = []
    for S in sizes:
        q_lens = [2048] * (S // 2048) + ([S % 2048] if S % 2048 else [])
        x = synth.make_x(shape, 7, S, "cuda")
        kv = synth.make_paged_cache(shape, 7, [0] * len(q_lens), q_lens, "cuda", fill_random=False)
        out = torch.empty_like(x)
        fn = lambda: layer.prefill(x, kv, n_tokens=S, max_q_len=max(q_lens), out=out)
        ms = timed_loop(fn, args.steps, args.warmup, False) / args.steps
        rows.append(dict(tokens=S, ms_per_block=ms, tokens_per_s=S / (ms * 1e-3)))
    layer.close()
    print(json.dumps(dict(metric="foe_block_latency_sweep", unit="ms", data="synthetic", dtype="bf16",
                          config=dict(workload=desc + ", prefill of S tokens in sequences of <= 2048"),
                          steps=args.steps, warmup=args.warmup, sweep=rows)))


def run_serve(args):
    """Request-level run: Poisson arrivals of long-prompt requests served with continuous batching (chunked prefill
    mixed with decode tokens) by a 4-layer stack of the workload-2 layer; TTFT / TBT / end-to-end latency as mean,
    p50, p99 (the format of the paper's latency tables; its numbers are whole models on 8 GPUs, context only)."""
    from paper_2605_06206_b200 import serving as sv
    shape, _ = synth.workload(2)
    n_layers, max_batch_tokens, max_seqs, chunk, max_context = 4, 8192, 64, 2048, 16384 + 256
    n_req, rate = args.requests, args.rate
    reqs = sv.synthetic_trace(n_req, rate=rate, seed=11)
    num_pages = 4096                                        # 262,144 tokens of KV per layer
    runner = sv.FoeStackRunner(shape, n_layers, seed=2, num_pages=num_pages, max_batch_tokens=max_batch_tokens,
                               max_seqs=max_seqs, max_context=max_context)
    # Warm-up: every kernel family the run can launch (large and small prefill chunks, mixed batches, decode steps of
    # several sizes) once, so that no one-time cost of a first launch (module loading, kernel attributes) lands inside
    # an iteration whose device time is charged to the requests waiting on it.  The collector is off during the run for
    # the same reason: an iteration's time is taken between two events and includes any pause of the launching thread.
    import gc
    for seed, n, pr, orr in ((12, 3, (512, 4096), (2, 4)), (13, 12, (64, 9000), (2, 12))):
        warm = sv.synthetic_trace(n, rate=1e6, seed=seed, prompt_range=pr, output_range=orr)
        sv.Engine(sv.Scheduler(sv.PagePool(num_pages), max_batch_tokens, max_seqs, chunk), runner.forward).run(warm)
    eng = sv.Engine(sv.Scheduler(sv.PagePool(num_pages), max_batch_tokens, max_seqs, chunk), runner.forward)
    gc.collect()
    gc.disable()
    try:
        done = eng.run(reqs)
    finally:
        gc.enable()
    runner.close()
    rep = sv.latency_report(done)
    toks = sum(r.prompt_len + r.output_len - 1 for r in done)
    print(json.dumps(dict(metric="foe_stack_request_latency", unit="ms", data="synthetic", dtype="bf16",
                          config=dict(workload=f"{n_layers}-layer stack of the workload-2 layer; {n_req} requests, Poisson "
                                               f"{rate} req/s, prompts log-uniform 1024..16384, outputs 32..256; continuous "
                                               f"batching, <= {max_batch_tokens} tokens and {max_seqs} sequences per iteration, "
                                               f"prompt chunks of {chunk}"),
                          requests=len(done), iterations=eng.iterations, busy_seconds=eng.clock,
                          tokens_per_s=toks / eng.clock, mean_batch_tokens=sum(eng.batch_tokens) / max(1, len(eng.batch_tokens)),
                          **rep)))


def run_stack(args):
    """The 16-layer stack (workload 5) once as FoE and once as the equal-size one-cluster MoE (128 experts, top-16) on
    the same kernels: prefill of 2 x 16,384 tokens, then 128 decode steps on the caches it wrote."""
    peaks = measured_peaks()
    dev = torch.cuda.current_device()
    rows = [measure_stack(args, peaks, dev, one_cluster=False), measure_stack(args, peaks, dev, one_cluster=True)]
    print(json.dumps(dict(metric="foe_stack_tokens_per_s", unit="tokens/s", data="synthetic", dtype="bf16",
                          config=dict(workload="workload 5, FoE and its one-cluster MoE twin"), stacks=rows)))


def run_shard(args):
    """One cluster per rank, all ranks on this one device: what each rank's own kernels cost.  Ranks on one device run
    one after the other, so a rank's time is the sum of its three phases (attention + push, owner-side reduce +
    all-gather, wait + routing + experts + combine), taken with CUDA events around each; the exchange moves through
    local memory here, so the NVLink time is NOT in these numbers -- its bytes are reported beside them."""
    from paper_2605_06206_b200 import shard
    rows = []
    for kind in ("prefill", "decode"):
        n = 2 if kind == "prefill" else 3
        shape, info = synth.workload(n)
        H, d = shape.n_clusters, shape.hidden
        seed, q_lens, ctx = info["seed"], info["q_lens"], info["context_lens"]
        S = sum(q_lens)
        decode = kind == "decode"
        W = synth.make_weights(shape, seed, "cuda")
        x = synth.make_x(shape, seed, S, "cuda")
        kv = synth.make_paged_cache(shape, seed, ctx, q_lens, "cuda")
        kvs = [shard.split_cache(shape, kv, h) for h in range(H)]
        max_ctx = max(c + q for c, q in zip(ctx, q_lens))
        one = build_workload(kind, "cuda")
        fn, _ = step_fn(one)
        one_ms = timed_loop(fn, args.steps, args.warmup, False) / args.steps
        one["layer"].close()
        del one, kv
        group = shard.LocalGroup(shape, max_tokens=S)
        layers = group.make_layer(shape, W, S, len(q_lens), max_ctx)
        del W
        torch.cuda.empty_cache()
        outs = [torch.empty(S, d, dtype=torch.bfloat16, device="cuda") for _ in range(H)]
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(6)] for _ in range(H)]
        acc = [[0.0, 0.0, 0.0] for _ in range(H)]
        for it in range(args.warmup + args.steps):
            torch.cuda._sleep(20_000_000)      # ~10 ms of device spin: the host queues the whole step behind it, so the
                                               # events see kernel time, not launch gaps
            for h, l in enumerate(layers):
                ev[h][0].record(); l.attend(x[h], kvs[h], decode); ev[h][1].record()
            for h, l in enumerate(layers):
                ev[h][2].record(); l.reduce(); ev[h][3].record()
            for h, l in enumerate(layers):
                ev[h][4].record(); l.ffn(out=outs[h]); ev[h][5].record()
            torch.cuda.synchronize()
            if it >= args.warmup:
                for h in range(H):
                    for p in range(3):
                        acc[h][p] += ev[h][2 * p].elapsed_time(ev[h][2 * p + 1])
        assert group.poll_status() == 0 and all(l.layer.poll_status() == 0 for l in layers)
        per = [[v / args.steps for v in a] for a in acc]
        rank_ms = [sum(a) for a in per]
        # per rank and layer: reduce-scatter sends (H-1)/H of its [S][d] bf16 partial, all-gather sends its d/H columns
        # to H-1 peers: 2 * S * d * 2 * (H-1)/H bytes out (and as many in).  Conventional expert parallelism over the
        # same H GPUs moves every token to its k experts and back: 2 * S * k * d * 2 * (H-1)/H bytes (Section 3.2).
        k = H * shape.top_k_per_cluster
        sync_bytes = 2 * S * d * 2 * (H - 1) / H
        ep_bytes = 2 * S * k * d * 2 * (H - 1) / H
        rows.append(dict(workload=f"workload {n} ({kind})", n_ranks=H, tokens=S, one_device_ms=one_ms,
                         rank_ms_max=max(rank_ms), rank_ms_mean=sum(rank_ms) / H,
                         phases_ms_mean=dict(attend_push=sum(a[0] for a in per) / H, reduce_allgather=sum(a[1] for a in per) / H,
                                             wait_route_experts_combine=sum(a[2] for a in per) / H),
                         launches_per_rank=layers[0].layer.last_launch_count() + 1,
                         sync_bytes_out_per_rank=sync_bytes, sync_ms_at_770_GBs=sync_bytes / 770e9 * 1e3,
                         expert_parallel_alltoall_bytes_out_per_rank=ep_bytes, bytes_ratio=ep_bytes / sync_bytes))
        for l in layers:
            l.close()
        group.close()
        del layers, group, kvs, outs
        torch.cuda.empty_cache()
    print(json.dumps(dict(metric="foe_rank_ms_per_layer", unit="ms", data="synthetic", dtype="bf16",
                          config=dict(workload="one cluster per rank, all ranks emulated on one device; exchange through local "
                                               "memory (NVLink time not included: see sync_ms_at_770_GBs)",
                                      steps=args.steps, warmup=args.warmup),
                          groups=rows)))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", choices=["prefill", "decode"], default="prefill")
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-secondary", action="store_true", help="skip the other workload's measurement")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip timing the CPU oracle (profiler runs)")
    ap.add_argument("--no-extra", action="store_true", help="skip the skewed-routing (workload 4) and 16-layer stack (workload 5) keys")
    ap.add_argument("--only", choices=["skew", "stack"], help="run just that measurement and print its object (profiler captures)")
    ap.add_argument("--skew-seqs", type=int, default=0, help="--only skew: use the first N of the 8 sequences")
    ap.add_argument("--sustain-seconds", type=float, default=1.2,
                    help="length of the back-to-back run the stage times are taken from (0: just 72 steps)")
    ap.add_argument("--sweep", action="store_true", help="token-batch latency sweep at the paper's 7B layer shape")
    ap.add_argument("--sweep-shape", choices=["7b", "1b"], default="7b")
    ap.add_argument("--stack", action="store_true", help="16-layer stack (workload 5): FoE and the one-cluster MoE twin")
    ap.add_argument("--shard", action="store_true", help="one cluster per rank, all ranks emulated on this device: per-rank kernel time")
    ap.add_argument("--serve", action="store_true", help="request-level latency run (continuous batching on a 4-layer stack)")
    ap.add_argument("--requests", type=int, default=48)
    ap.add_argument("--rate", type=float, default=20.0, help="--serve: Poisson arrival rate, requests per second")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (the block has no CPU path)")
    torch.cuda.set_device(local)
    if args.sweep:
        run_sweep(args)
        return
    if args.serve:
        run_serve(args)
        return
    if args.stack:
        run_stack(args)
        return
    if args.shard:
        run_shard(args)
        return
    peaks = measured_peaks()
    if args.only:
        res = measure_skew(args, peaks, local, args.skew_seqs or None) if args.only == "skew" else measure_stack(args, peaks, local)
        print(json.dumps(res))
        return
    dist_on = replicas.init("nccl", torch.device("cuda", local))

    main_kind = args.workload
    other = "decode" if main_kind == "prefill" else "prefill"
    m = measure(main_kind, args, dist_on, rank, world, peaks, with_cpu=(rank == 0 and world == 1 and not args.no_cpu_baseline))
    o = None if args.no_secondary else measure(other, args, dist_on, rank, world, peaks,
                                               with_cpu=(rank == 0 and world == 1 and not args.no_cpu_baseline))
    extra = {}
    if rank == 0 and world == 1 and not args.no_extra and not args.no_secondary:
        extra["skew"] = measure_skew(args, peaks, local)
        extra["stack"] = measure_stack(args, peaks, local)
    if rank == 0:
        wl_n = 2 if main_kind == "prefill" else 3
        line = dict(metric=f"foe_block_{main_kind}_tokens_per_s", value=m["tokens_per_s"], unit="tokens/s",
                    n_gpus=world, steps=args.steps, warmup=args.warmup, ms_per_step=m["ms_per_step"],
                    higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16", data="synthetic",
                    config=dict(workload=f"workload {wl_n}: single FoE block {main_kind}, hidden 2048, 16q/4kv heads, "
                                         f"4 clusters x 16 experts top-2, inter 1024, "
                                         + ("4 x 4096 tokens causal" if main_kind == "prefill" else
                                            "64 sequences x 1 token, paged KV (page 64), contexts U[4096,16384]"),
                                tokens_per_step=m["tokens_per_step"], replicas=world,
                                l2="inputs larger than L2: weights 0.8 GB + activations/KV >= 0.5 GB per step"),
                    clocks=m["clocks"], roofline=m["roofline"], e2e=m["e2e"],
                    gpu_launches=m["launches_per_step"] * args.steps, stages_ms=m["stages_ms"],
                    stage_sm_mcycles=m["stage_sm_mcycles"], sustained=m["sustained"], expert_rows=m["expert_rows"])
        line.update(extra)
        if "cpu_baseline" in m:
            line["cpu_baseline"] = m["cpu_baseline"]
        if o is not None:
            line[other] = dict(tokens_per_s=o["tokens_per_s"], ms_per_step=o["ms_per_step"], roofline=o["roofline"],
                               e2e=o["e2e"], stages_ms=o["stages_ms"], clocks=o["clocks"], sustained=o["sustained"],
                               stage_sm_mcycles=o["stage_sm_mcycles"], expert_rows=o["expert_rows"],
                               gpu_launches=o["launches_per_step"] * args.steps,
                               cpu_baseline=o.get("cpu_baseline"))
        print(json.dumps(line))
    replicas.shutdown()


if __name__ == "__main__":
    main()
