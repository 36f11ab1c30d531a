"""The N > 1 path on CPU: two gloo ranks exchange only timing (max) and unit counts (sum)."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, %r)
from paper_2603_03592_b200 import replicas
rank, world, local = replicas.init_from_env(backend="gloo")
assert world == 2 and rank == local
replicas.barrier()
ms = replicas.max_over_ranks(10.0 + 5.0 * rank)           # rank 1 is the slow one
units = replicas.sum_over_ranks(100.0 * (rank + 1))
thr = replicas.aggregate_throughput(100.0 * (rank + 1), 10.0 + 5.0 * rank)
mine = replicas.boundaries_of_rank(8, rank, world)
replicas.shutdown()
print(json.dumps({"rank": rank, "ms": ms, "units": units, "thr": thr, "mine": mine}))
""" % ROOT


def test_two_gloo_ranks_reduce_time_and_units(tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err
        outs.append(__import__("json").loads(out.strip().splitlines()[-1]))
    for o in outs:
        assert o["ms"] == 15.0 and o["units"] == 300.0
        assert o["thr"] == 300.0 / 15e-3
    assert sorted(outs[0]["mine"] + outs[1]["mine"]) == list(range(8))
    assert not set(outs[0]["mine"]) & set(outs[1]["mine"])


def test_single_process_needs_no_process_group():
    from paper_2603_03592_b200 import replicas
    assert replicas.max_over_ranks(3.5) == 3.5 and replicas.sum_over_ranks(2.0) == 2.0
    replicas.barrier()
    assert replicas.boundaries_of_rank(5, 0, 1) == [0, 1, 2, 3, 4]


def test_reference_arm_runs_on_cpu_and_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--steps", "1", "--warmup", "0", "--workload", "cfg1"],
                         capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    rec = __import__("json").loads(lines[0])
    assert rec["impl"] == "reference" and rec["unit"] == "GB/s" and rec["value"] > 0
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["e2e"]["h2d_bytes_per_step"] == 0
