"""Multi-process plumbing: one process per GPU.

The k-MIP hot path has no exchange step between graphs (a query only sees the nodes of its own graph, Eq. 1 with
the batching of graphs by offsets), so it shards without a data-path collective in two ways:
  * replicas (the benchmark's default): N processes run N independent copies of the workload;
  * whole graphs per rank (`partition_graphs`, `shard_of`): the graphs of one batch are split into contiguous
    runs, one per rank, balanced by the number of scores (sum of n_g^2); each rank calls the library on its own
    slice of Q, K, V with its own offsets, and the results are the corresponding slices of the unsharded result
    (indices shifted by the slice's first node).  Nothing crosses the link.
A single graph larger than one GPU's share would need its query rows split and K, V gathered into every rank's own
memory first; the library's calls take one node count for queries and keys, so that variant is not built.
torch.distributed is used only for the barrier around the timed region and to take the maximum time / the sum of
processed units over ranks.  Works with NCCL (GPU) and gloo (CPU tests).
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world():
    """(rank, local_rank, world_size) from the launcher's environment (1 process if absent)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str | None = None) -> tuple[int, int, int]:
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        if backend is None:
            backend = "nccl" if torch.cuda.is_available() else "gloo"
        if backend == "nccl":
            torch.cuda.set_device(local_rank)
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def _device():
    if dist.is_initialized() and dist.get_backend() == "nccl":
        return torch.device("cuda", torch.cuda.current_device())
    return torch.device("cpu")


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(x: float) -> float:
    if not dist.is_initialized():
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=_device())
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(x: float) -> float:
    if not dist.is_initialized():
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=_device())
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def aggregate_throughput(units_this_rank: float, seconds_this_rank: float) -> tuple[float, float]:
    """Whole-job throughput of independent replicas: units of all ranks / slowest rank's time.
    Returns (units per second, max seconds)."""
    t = max_over_ranks(seconds_this_rank)
    u = sum_over_ranks(units_this_rank)
    return (u / t if t > 0 else 0.0), t


def partition_graphs(graph_offsets, world: int) -> list[tuple[int, int]]:
    """Contiguous runs of graphs, one per rank: [(first graph, one past the last graph)] * world.

    The cost of a graph is n_g^2 (its scores; the forward sweep dominates a step).  The split minimises the largest
    cost of a rank over all contiguous splits (binary search on that bound with a greedy feasibility test), so it is
    deterministic and the same on every rank.  Ranks beyond the number of non-empty runs get an empty range."""
    offs = [int(x) for x in graph_offsets]
    G = len(offs) - 1
    if world < 1 or G < 0 or any(b < a for a, b in zip(offs, offs[1:])):
        raise ValueError("partition_graphs: offsets must be non-decreasing and world >= 1")
    cost = [(offs[g + 1] - offs[g]) ** 2 for g in range(G)]

    def runs_needed(bound):
        runs, acc = 1, 0
        for c in cost:
            if c > bound:
                return world + 1
            if acc + c > bound:
                runs, acc = runs + 1, c
            else:
                acc += c
        return runs

    lo, hi = (max(cost) if cost else 0), sum(cost)
    while lo < hi:
        mid = (lo + hi) // 2
        if runs_needed(mid) <= world:
            hi = mid
        else:
            lo = mid + 1
    parts, g, acc, start = [], 0, 0, 0
    for g in range(G):
        if acc + cost[g] > lo and g > start:
            parts.append((start, g))
            start, acc = g, 0
        acc += cost[g]
    parts.append((start, G))
    parts += [(G, G)] * (world - len(parts))
    return parts[:world]


def shard_of(graph_offsets, world: int, rank: int):
    """This rank's slice of a batch split by whole graphs: (first node, one past the last node, local offsets as a
    list starting at 0, first graph).  Slice Q, K, V, dOut [first:last]; add `first node` to the indices that come
    back to name nodes of the whole batch."""
    g_lo, g_hi = partition_graphs(graph_offsets, world)[rank]
    offs = [int(x) for x in graph_offsets]
    n_lo, n_hi = offs[g_lo], offs[g_hi]
    return n_lo, n_hi, [o - n_lo for o in offs[g_lo:g_hi + 1]], g_lo


def shutdown() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
