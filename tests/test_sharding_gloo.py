"""World-size-2 check (gloo, CPU) of the replica sharding used by multi-GPU runs."""
import os

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import fcsim_oracle as orc
from paper_2604_11001_b200 import sharding
from paper_2604_11001_b200 import workloads as wl


def _group_totals(cfg, counters):
    s = orc.summarize(cfg, counters, None, cfg.T_max)
    return torch.tensor([[g[n] for n in orc.COUNTER_NAMES] for g in s], dtype=torch.int64)


def _worker(rank, world, port, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = wl.config2(replicas=3, T=600)
    mine = sharding.shard_for_rank(cfg, rank)
    out = orc.run(mine, trace=False, complog=False)
    total = sharding.combine_group_totals(_group_totals(mine, out["counters"]), dist)
    if rank == 0:
        ret["total"] = total.numpy().copy()
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_equal_one_simulation_with_twice_the_replicas():
    world = 2
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(world, 29517, ret), nprocs=world, join=True)
    cfg = wl.config2(replicas=3, T=600)
    assert sharding.id_span(cfg) == 3
    # the union of the shards: every group twice, second copy with ids shifted by the span
    both = cfg.with_(groups=tuple(g for r in range(world) for g in sharding.shard_for_rank(cfg, r).groups))
    out = orc.run(both, trace=False, complog=False)
    t = _group_totals(both, out["counters"]).numpy()
    expect = t[:2].copy()
    other = t[2:]
    for f in range(t.shape[1]):
        if f in sharding.MAX_FIELDS:
            expect[:, f] = np.maximum(expect[:, f], other[:, f])
        elif f in sharding.OR_FIELDS:
            expect[:, f] |= other[:, f]
        else:
            expect[:, f] += other[:, f]
    assert (ret["total"] == expect).all()
    # shards really are different replicas
    a = orc.run(sharding.shard_for_rank(cfg, 0), trace=False, complog=False)["counters"]
    b = orc.run(sharding.shard_for_rank(cfg, 1), trace=False, complog=False)["counters"]
    assert (a[:, orc.CIDX["sum_U"]] != b[:, orc.CIDX["sum_U"]]).all()
