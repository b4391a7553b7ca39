"""Host-side sharding of the batch generator across GPUs.

The path shards by instance: every rank owns whole candidate pools and its own Assistant
(the paper trains one Assistant per GPU on that GPU's data chunk, Sec. "Machine Translation"), so there is no
data-path collective.  Instance ids stay global (id_base per pool), so the keep/skip decisions
do not depend on how many ranks share the data.  The only cross-rank exchange is the reduction
of the timing numbers for reporting.
"""
from __future__ import annotations

from dataclasses import dataclass


@dataclass
class ShardPlan:
    pool_ids: list      # global ids of the pools this rank owns
    id_bases: list      # instance id of row 0 of each owned pool


def plan(rank: int, world: int, pools_per_rank: int, pool_rows: int) -> ShardPlan:
    if not (0 <= rank < world) or pools_per_rank < 1 or pool_rows < 0:
        raise ValueError("bad shard request")
    ids = [rank * pools_per_rank + j for j in range(pools_per_rank)]
    return ShardPlan(pool_ids=ids, id_bases=[pid * pool_rows for pid in ids])


def aggregate(dist, device, elapsed_ms: float, units: int) -> dict:
    """Whole-job numbers: slowest rank's time, all ranks' units.  dist=None means a single process."""
    if dist is None:
        return {"ms": float(elapsed_ms), "units": int(units)}
    import torch

    t = torch.tensor([float(elapsed_ms)], dtype=torch.float64, device=device)
    u = torch.tensor([float(units)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return {"ms": float(t.item()), "units": int(u.item())}
