"""The N > 1 bookkeeping (independent replicas: barrier, slowest-rank time, whole-job throughput, one printed line)
exercised with two CPU processes over gloo."""

import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, sys.argv[1])
from paper_2506_01206_b200 import replicas
rank, world = replicas.init("gloo")
assert world == 2
replicas.barrier(world)
ms = replicas.max_over_ranks(10.0 + 5.0 * rank, world)          # rank 1 is the slow one
seed = replicas.replica_seed(7, rank)
value = replicas.whole_job_throughput(1000.0, ms, world)
replicas.barrier(world)
if rank == 0:
    print(json.dumps({"ms": ms, "value": value, "seed": seed, "world": world}))
else:
    assert seed == 8
replicas.finish(world)
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_replicas_over_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e
    lines = [l for l in outs[0][0].splitlines() if l.startswith("{")]
    assert len(lines) == 1 and not outs[1][0].strip(), "exactly one rank prints exactly one line"
    j = json.loads(lines[0])
    assert j["ms"] == 15.0, "the job lasts as long as its slowest replica"
    assert abs(j["value"] - 2 * 1000.0 / 15e-3) < 1e-6, "throughput counts the work of all replicas"
    assert j["seed"] == 7 and j["world"] == 2


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    from paper_2506_01206_b200 import replicas
    assert replicas.max_over_ranks(3.5, 1) == 3.5
    assert replicas.whole_job_throughput(10.0, 2.0, 1) == 5000.0
    replicas.barrier(1)


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and not r.stdout.strip(), "ranks other than 0 leave the reference arm without work or output"
