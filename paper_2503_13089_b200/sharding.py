"""Multi-GPU scheduling: whole matrices per rank, nothing exchanged.

The paper notes that the clustering of different weight matrices is independent, so the path
shards at matrix granularity with no data-path collective.  Rank r of a benchmark run clusters
its own copy of the workload's matrices, drawn from seeds shifted by the rank (weak scaling);
a model-compression job hands out its list of matrices round-robin by size.
"""
from __future__ import annotations

from dataclasses import replace
from typing import List, Sequence, Tuple

from .workloads import MatrixSpec, Workload


def matrices_for_rank(w: Workload, rank: int) -> Tuple[MatrixSpec, ...]:
    """The matrices rank `rank` clusters in a benchmark step (rank 0: the workload as defined)."""
    if rank == 0:
        return w.matrices
    return tuple(replace(m, data_seed=m.data_seed + 1000 * rank, init_seed=m.init_seed + 1000 * rank)
                 for m in w.matrices)


def assign_matrices(sizes: Sequence[int], world: int) -> List[List[int]]:
    """Longest-processing-time-first split of matrix indices over `world` ranks (cost = size)."""
    order = sorted(range(len(sizes)), key=lambda i: (-sizes[i], i))
    loads = [0] * world
    out: List[List[int]] = [[] for _ in range(world)]
    for i in order:
        r = min(range(world), key=lambda k: (loads[k], k))
        out[r].append(i)
        loads[r] += sizes[i]
    return [sorted(v) for v in out]


def max_over_ranks(value: float, group=None) -> float:
    """Max of a host scalar over the ranks of an initialised process group (any backend)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64)
    if dist.get_backend(group) == "nccl":
        t = t.cuda()
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())
