"""The N>1 host logic on CPU: two gloo ranks shard the pools, keep global instance ids, and
reduce timing as max-over-ranks / sum-of-units.  Also checks on the oracle that a pool screened
as two shards with the right id_base gives the decisions of the whole pool."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import aa_oracle as O
from paper_1905_03381_b200 import sharding


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    plan = sharding.plan(rank, world, 3, 1000)
    ms = 10.0 + 5.0 * rank            # rank 1 is the slow one
    agg = sharding.aggregate(dist, torch.device("cpu"), ms, 3 * 1000 * (rank + 1))
    out.put((rank, plan.pool_ids, plan.id_bases, agg))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_plan_and_aggregation():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, pools0, bases0, agg0), (r1, pools1, bases1, agg1) = got
    assert pools0 == [0, 1, 2] and pools1 == [3, 4, 5]
    assert bases0 == [0, 1000, 2000] and bases1 == [3000, 4000, 5000]
    assert agg0 == agg1 == {"ms": 15.0, "units": 9000}    # slowest rank's time, everybody's units


def test_single_process_aggregate_and_bad_requests():
    assert sharding.aggregate(None, None, 2.5, 7) == {"ms": 2.5, "units": 7}
    for bad in ((2, 2, 1, 10), (0, 1, 0, 10), (-1, 1, 1, 10)):
        try:
            sharding.plan(*bad)
        except ValueError:
            continue
        raise AssertionError(bad)


def test_sharded_screening_equals_whole_pool_screening():
    rng = np.random.default_rng(0)
    n, d = 2000, 12
    x = rng.standard_normal((n, d)).astype(np.float32)
    w = (rng.standard_normal(d) * 0.5).astype(np.float32)
    whole = O.screen_linear_dense(x, w, 0.1, 0.1, seed=5, step=2, id_base=0)
    half = n // 2
    a = O.screen_linear_dense(x[:half], w, 0.1, 0.1, seed=5, step=2, id_base=0)
    b = O.screen_linear_dense(x[half:], w, 0.1, 0.1, seed=5, step=2, id_base=half)
    assert np.array_equal(np.concatenate([a["keep"], b["keep"]]), whole["keep"])
    assert np.array_equal(np.concatenate([a["B"], b["B"] + half]), whole["B"])
