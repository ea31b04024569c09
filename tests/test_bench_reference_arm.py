"""The benchmark's reference arm (`bench.py --impl reference`) needs no GPU: it times the CPU oracle on a bounded sample
of the benchmark workload and prints the same one-line record as the CUDA arm."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line_without_a_gpu():
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                       env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True, timeout=600, cwd=ROOT)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "foe_block_prefill_tokens_per_s" and d["unit"] == "tokens/s"
    assert d["value"] > 0 and d["higher_is_better"] is True and d["dtype"] == "f64" and d["vs_baseline"] is None
    assert d["steps"] == 1 and d["n_gpus"] == 1 and "workload" in d["config"]
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] == d["value"] and cb["sample"]
    assert d["e2e"] == dict(value=d["value"], unit="tokens/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0)


def test_other_ranks_of_the_reference_arm_exit_without_work():
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True, timeout=120, cwd=ROOT)
    assert p.returncode == 0, p.stderr[-2000:]
    assert not [l for l in p.stdout.strip().splitlines() if l.startswith("{")]


def test_roofline_traffic_is_read_from_the_committed_profiles():
    """The `traffic` figure of the bench line is parsed out of the ncu summary the line names, not kept in the source:
    the committed summaries must hold the two kernels' DRAM byte rows, and the figures must be near the algorithmic
    bytes they are compared with (1.0-1.5 x: a smaller or far larger value means the wrong section was read)."""
    import importlib.util
    spec = importlib.util.spec_from_file_location("bench_mod", os.path.join(ROOT, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    t, src = bench.profile_traffic("ncu_full_prefill_kernels_workload2.md", "gemm_tcgen05_kernel<1, 1>")
    assert t is not None and "profiles/ncu_full_prefill_kernels_workload2.md" in src
    assert 0.872e9 <= t <= 1.5 * 0.872e9               # weights 537 MB + output 268 MB + distinct activations 67 MB
    t, src = bench.profile_traffic("ncu_full_decode_kernels_workload3.md", "attn_decode_kernel")
    assert t is not None and 1.34e9 <= t <= 1.1 * 1.344e9
    t, src = bench.profile_traffic("ncu_full_decode_kernels_workload3.md", "no_such_kernel")
    assert t is None and "not found" in src
    t, src = bench.profile_traffic("no_such_file.md", "x")
    assert t is None and "missing" in src
