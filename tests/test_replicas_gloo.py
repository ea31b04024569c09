"""The benchmark's N > 1 plumbing (barrier, max-over-ranks time, whole-job throughput) on two CPU processes
over the gloo backend."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent("""
    import sys, json
    sys.path.insert(0, %r)
    from paper_2605_06206_b200 import replicas
    rank, size, local = replicas.world()
    assert replicas.init("gloo")
    replicas.barrier()
    local_ms = 10.0 if rank == 0 else 25.0            # rank 1 is the slow replica
    tput, ms_step = replicas.job_throughput(units_per_rank_step=1000, steps=5, ms_total_local=local_ms)
    mx = replicas.max_over_ranks(float(rank))
    replicas.barrier()
    print(json.dumps(dict(rank=rank, size=size, tput=tput, ms_step=ms_step, mx=mx)))
    replicas.shutdown()
""") % ROOT


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_two_replicas_agree_on_job_time_and_throughput():
    import json
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", LOCAL_RANK=str(r), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        o, e = p.communicate(timeout=120)
        assert p.returncode == 0, e
        outs.append(json.loads(o.strip().splitlines()[-1]))
    for o in outs:
        assert o["size"] == 2
        assert abs(o["ms_step"] - 5.0) < 1e-9                      # max(10, 25) ms over 5 steps
        assert abs(o["tput"] - 2 * 1000 * 5 / 25e-3) < 1e-6        # both replicas' units over the slowest time
        assert o["mx"] == 1.0


def test_single_process_is_a_no_op():
    from paper_2605_06206_b200 import replicas
    env_backup = {k: os.environ.pop(k, None) for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    try:
        assert replicas.world() == (0, 1, 0)
        assert replicas.init("gloo") is False
        replicas.barrier()
        assert replicas.max_over_ranks(3.5) == 3.5
        tput, ms = replicas.job_throughput(100, 4, 8.0)
        assert abs(tput - 100 * 4 / 8e-3) < 1e-9 and ms == 2.0
    finally:
        for k, v in env_backup.items():
            if v is not None:
                os.environ[k] = v
