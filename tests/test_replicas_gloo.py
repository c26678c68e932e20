"""World-size-2 test (gloo, CPU) of the benchmark's multi-process plumbing: replicas only, the
barrier, max-over-ranks time and summed units; and the reference arm's rank rule."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, os.environ["KMIP_ROOT"])
from paper_2604_03815_b200 import dist as kdist
rank, local_rank, world = kdist.init(backend="gloo")
kdist.barrier()
secs = 2.0 if rank == 0 else 3.0          # rank 1 is the slow replica
value, tmax = kdist.aggregate_throughput(100.0 * (rank + 1), secs)
mx = kdist.max_over_ranks(float(rank))
kdist.barrier()
print(json.dumps({"rank": rank, "world": world, "value": value, "tmax": tmax, "mx": mx}))
kdist.shutdown()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_replicas_aggregate_over_gloo():
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), KMIP_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        o, e = p.communicate(timeout=120)
        assert p.returncode == 0, e
        outs.append(json.loads(o.strip().splitlines()[-1]))
    for o in outs:
        assert o["world"] == 2
        assert o["tmax"] == 3.0                 # slowest rank decides
        assert abs(o["value"] - 300.0 / 3.0) < 1e-12   # units of all ranks / max time
        assert o["mx"] == 1.0


def test_single_process_needs_no_process_group():
    from paper_2604_03815_b200 import dist as kdist
    env = {k: os.environ.pop(k, None) for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE")}
    try:
        assert kdist.env_world() == (0, 0, 1)
        assert kdist.aggregate_throughput(10.0, 2.0) == (5.0, 2.0)
    finally:
        for k, v in env.items():
            if v is not None:
                os.environ[k] = v


def test_reference_arm_runs_on_rank0_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
