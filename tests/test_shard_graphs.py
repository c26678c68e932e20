"""Sharding a batch by whole graphs (paper_2604_03815_b200.dist.partition_graphs / shard_of): a query only sees the
nodes of its own graph, so each rank can run its own contiguous run of graphs and the pieces are exactly the slices
of the unsharded result.  The partition arithmetic on CPU, a world-size-2 gloo run in which each rank evaluates its
shard with the oracle and the gathered pieces are compared with the oracle on the whole batch, and (GPU) the same
through the library, the shards run one after the other on one device."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

from paper_2604_03815_b200 import dist as kdist
from paper_2604_03815_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _check_partition(offs, world):
    parts = kdist.partition_graphs(offs, world)
    G = len(offs) - 1
    assert len(parts) == world and parts[0][0] == 0
    for (a, b), (c, d) in zip(parts, parts[1:]):
        assert a <= b == c <= d                       # contiguous, in order
    assert parts[-1][1] == G or all(p == (G, G) for p in parts if p[0] == G)
    assert max(b for _, b in parts) == G
    cost = [(offs[g + 1] - offs[g]) ** 2 for g in range(G)]
    worst = max(sum(cost[a:b]) for a, b in parts)
    return parts, cost, worst


def test_partition_is_contiguous_complete_and_optimal_on_small_cases():
    rng = np.random.default_rng(3)
    for _ in range(200):
        G = int(rng.integers(0, 9))
        world = int(rng.integers(1, 6))
        sizes = rng.integers(0, 50, size=G)
        offs = [0] + np.cumsum(sizes).tolist()
        parts, cost, worst = _check_partition(offs, world)
        # brute force over all contiguous splits into at most `world` runs
        best = None
        def rec(start, left, cur_max):
            nonlocal best
            if left == 1 or start == G:
                m = max(cur_max, sum(cost[start:]))
                best = m if best is None else min(best, m)
                return
            for end in range(start, G + 1):
                rec(end, left - 1, max(cur_max, sum(cost[start:end])))
        rec(0, world, 0)
        assert worst == best


def test_partition_of_the_hub_batch_and_degenerate_inputs():
    offs = [0, 200_000, 400_000, 600_000, 800_000]          # config 5: one graph per rank at four ranks
    assert kdist.partition_graphs(offs, 4) == [(0, 1), (1, 2), (2, 3), (3, 4)]
    assert kdist.partition_graphs(offs, 2) == [(0, 2), (2, 4)]
    assert kdist.partition_graphs(offs, 8)[4:] == [(4, 4)] * 4   # more ranks than graphs: the rest stay empty
    assert kdist.shard_of(offs, 4, 2) == (400_000, 600_000, [0, 200_000], 2)
    assert kdist.partition_graphs([0], 3) == [(0, 0)] * 3
    with pytest.raises(ValueError):
        kdist.partition_graphs([0, 5, 3], 2)


WORKER = r"""
import json, os, sys
import numpy as np
sys.path.insert(0, os.environ["KMIP_ROOT"])
import torch.distributed as dist
from paper_2604_03815_b200 import dist as kdist, workloads as wl
from oracle import kmip_oracle as ko
rank, local_rank, world = kdist.init(backend="gloo")
w = wl.iid_workload("s", 77, [40, 0, 300, 7, 129, 64, 1, 250], 2, 16, 5, wl.MODE_BF16_TC)
lo, hi, offs, g0 = kdist.shard_of(w.graph_offsets, world, rank)
mine = ko.forward(w.Q[lo:hi], w.K[lo:hi], w.V[lo:hi], np.asarray(offs, dtype=np.int32), w.k)
idx = np.where(mine["idx"] >= 0, mine["idx"] + lo, -1)          # back to node numbers of the whole batch
dQ, dK, dV = ko.backward(w.Q[lo:hi], w.K[lo:hi], w.V[lo:hi], w.dOut[lo:hi], mine["idx"])
pieces = [None] * world
dist.all_gather_object(pieces, {"lo": lo, "hi": hi, "out": mine["out"], "idx": idx, "dK": dK})
ok = True
if rank == 0:
    full = ko.forward(w.Q, w.K, w.V, w.graph_offsets, w.k)
    fQ, fK, fV = ko.backward(w.Q, w.K, w.V, w.dOut, full["idx"])
    pieces.sort(key=lambda p: p["lo"])
    assert pieces[0]["lo"] == 0 and pieces[-1]["hi"] == w.N and all(a["hi"] == b["lo"] for a, b in zip(pieces, pieces[1:]))
    ok = (np.array_equal(np.concatenate([p["out"] for p in pieces]), full["out"])
          and np.array_equal(np.concatenate([p["idx"] for p in pieces]), full["idx"])
          and np.array_equal(np.concatenate([p["dK"] for p in pieces]), fK))
kdist.barrier()
print(json.dumps({"rank": rank, "ok": bool(ok), "nodes": hi - lo}))
kdist.shutdown()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_ranks_by_graphs_reproduce_the_whole_batch_over_gloo():
    from oracle import kmip_oracle as ko
    ko.build()
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), KMIP_ROOT=ROOT, OMP_NUM_THREADS="2")
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        o, e = p.communicate(timeout=300)
        assert p.returncode == 0, e
        outs.append(json.loads(o.strip().splitlines()[-1]))
    assert all(o["ok"] for o in outs)
    assert sum(o["nodes"] for o in outs) == 40 + 300 + 7 + 129 + 64 + 1 + 250 and min(o["nodes"] for o in outs) > 0


@pytest.mark.gpu
def test_shards_through_the_library_equal_the_unsharded_call():
    import torch
    from paper_2604_03815_b200 import binding as kb
    w = wl.iid_workload("s", 78, [3000, 129, 0, 5000, 1, 2000, 383, 64], 2, 32, 16, wl.MODE_BF16_TC)
    dt = kb.storage_dtype(w.mode)
    Q, K, V, dO = (torch.from_numpy(getattr(w, n)).to("cuda", dt) for n in ("Q", "K", "V", "dOut"))
    full = kb.forward(Q, K, V, torch.from_numpy(w.graph_offsets).cuda(), w.k, w.mode)
    fb = kb.backward(Q, K, V, torch.from_numpy(w.graph_offsets).cuda(), w.k, w.mode, full, dO)
    world = 3
    covered = 0
    for rank in range(world):
        lo, hi, offs, _ = kdist.shard_of(w.graph_offsets, world, rank)
        if hi == lo:
            continue
        o = torch.tensor(offs, dtype=torch.int32, device="cuda")
        part = kb.forward(Q[lo:hi].contiguous(), K[lo:hi].contiguous(), V[lo:hi].contiguous(), o, w.k, w.mode)
        idx = torch.where(part.topk_idx >= 0, part.topk_idx + lo, part.topk_idx)
        assert torch.equal(idx, full.topk_idx[lo:hi])
        assert torch.equal(part.topk_score, full.topk_score[lo:hi])
        assert torch.equal(part.out, full.out[lo:hi])
        pb = kb.backward(Q[lo:hi].contiguous(), K[lo:hi].contiguous(), V[lo:hi].contiguous(), o, w.k, w.mode, part,
                         dO[lo:hi].contiguous())
        assert torch.equal(pb.dQ, fb.dQ[lo:hi]) and torch.equal(pb.dK, fb.dK[lo:hi]) and torch.equal(pb.dV, fb.dV[lo:hi])
        covered += hi - lo
    assert covered == w.N
