"""bench.py on more than one rank is N independent replicas: the only traffic between ranks is the
rendezvous, the barriers around the timed region and the max of the per-rank times.  That host logic
is run here on CPU with two gloo ranks; the reference arm must print from rank 0 only."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, os.environ["REPO_ROOT"])
import bench
rank, world, local = bench.dist_setup(backend="gloo")
bench.barrier_sync(world, device="cpu")
ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, device="cpu")     # rank 1 is the slow one
bench.barrier_sync(world, device="cpu")
value = bench.job_throughput(1000.0, 4, ms, world)
print(json.dumps({"rank": rank, "world": world, "ms": ms, "value": value}), flush=True)
"""


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def run_ranks(code_or_args, world=2, use_file=False):
    port = free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), REPO_ROOT=ROOT)
        cmd = [sys.executable] + (code_or_args if use_file else ["-c", code_or_args])
        procs.append(subprocess.Popen(cmd, env=env, cwd=ROOT, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=300)
        assert p.returncode == 0, err[-2000:]
        outs.append(out)
    return outs


def test_two_gloo_ranks_take_the_slowest_time():
    outs = run_ranks(WORKER)
    recs = [json.loads(o.strip().splitlines()[-1]) for o in outs]
    assert sorted(r["rank"] for r in recs) == [0, 1] and all(r["world"] == 2 for r in recs)
    for r in recs:
        assert r["ms"] == 15.0                                   # max over ranks, on every rank
        assert r["value"] == 2 * 1000.0 * 4 / 15.0e-3            # whole-job units / slowest time


def test_reference_arm_prints_from_rank_zero_only():
    outs = run_ranks(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                      "--workload", "c1"], use_file=True)
    lines = [[l for l in o.splitlines() if l.startswith("{")] for o in outs]
    assert len(lines[0]) == 1 and lines[1] == []
    rec = json.loads(lines[0][0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["cpu_baseline"]["kind"] == "oracle"
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["value"] > 0
