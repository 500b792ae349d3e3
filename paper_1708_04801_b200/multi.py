"""Multi-GPU layout of the path: nodes are independent until the single aggregation of Algorithm 1,
so they are partitioned over the ranks; every rank combines its own nodes with their global Eq. 6
weights and one all-reduce (sum) of d floats finishes v. No rank reads another rank's memory."""
from __future__ import annotations

from typing import List, Sequence

import numpy as np

from . import binding


def partition_nodes(n_steps: Sequence[int], world_size: int) -> List[np.ndarray]:
    """Longest-processing-time assignment of nodes to ranks by step count. Returns, per rank, the
    sorted global node ids it owns. Deterministic; every node appears exactly once."""
    n = np.asarray(n_steps, dtype=np.int64)
    order = sorted(range(len(n)), key=lambda j: (-int(n[j]), j))
    load = [0] * world_size
    owned: List[List[int]] = [[] for _ in range(world_size)]
    for j in order:
        r = min(range(world_size), key=lambda q: (load[q], q))
        owned[r].append(j)
        load[r] += int(n[j])
    return [np.array(sorted(o), dtype=np.int64) for o in owned]


def local_weights(n_steps_global, owned: np.ndarray, eta0: float, sched: int, lam: float, r: float = 0.0) -> np.ndarray:
    """Eq. 6 / Eq. 8 weights computed over ALL nodes (so that the delays refer to the globally fastest
    node and the weights sum to one over the cluster), restricted to this rank's nodes."""
    w, _, _ = binding.weights(n_steps_global, eta0, sched, lam, r)
    return w[np.asarray(owned, dtype=np.int64)]


def allreduce_sum(partial_v, group=None):
    """Sum of the ranks' partial combinations, in place (the aggregation's single exchange)."""
    import torch.distributed as dist

    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(partial_v, op=dist.ReduceOp.SUM, group=group)
    return partial_v
