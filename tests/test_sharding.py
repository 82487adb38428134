"""Element sharding across ranks: pure host logic plus a world_size-2 gloo run in which
each rank applies the (CPU oracle) operator to its shard and the gathered result equals
the single-process result -- the multi-GPU path has no data-path collective, so this is
all there is to it."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2604_19906_b200 import sharding


def test_shard_range_partitions_exactly():
    for E in (0, 1, 7, 64, 131072, 131075):
        for world in (1, 2, 3, 8):
            ranges = [sharding.shard_range(E, r, world) for r in range(world)]
            assert ranges[0][0] == 0 and ranges[-1][1] == E
            assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
            sizes = [b - a for a, b in ranges]
            assert max(sizes) - min(sizes) <= 1
    assert sharding.weak_range(100, 3, 8) == (300, 400)
    with pytest.raises(ValueError):
        sharding.shard_range(10, 2, 2)


def _worker(rank, world, port, E, n, ret):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2604_19906_b200 import inputs
    wl = inputs.Workload(0, "inv_helmholtz", (n, n, n), (n, n, n), E)
    e0, e1 = sharding.shard_range(E, rank, world)
    host = inputs.host_case(wl, e0, e1)
    v = torch.from_numpy(oracle.inv_helmholtz(host["S"], host["D"], host["u"], threads=1))
    parts = [None] * world
    dist.all_gather_object(parts, v)                      # caller-side gather, not on the data path
    t = torch.tensor([float(e1 - e0)])
    dist.all_reduce(t, op=dist.ReduceOp.MAX)              # the bench's max-over-ranks pattern
    if rank == 0:
        ret["v"] = torch.cat(parts).numpy()
        ret["max"] = float(t.item())
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("E", [10, 11])
def test_two_ranks_reproduce_the_single_process_result(E):
    import oracle
    from paper_2604_19906_b200 import inputs
    n, world = 4, 2
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    ret = ctx.Manager().dict()
    procs = [ctx.Process(target=_worker, args=(r, world, port, E, n, ret)) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    wl = inputs.Workload(0, "inv_helmholtz", (n, n, n), (n, n, n), E)
    host = inputs.host_case(wl)
    want = oracle.inv_helmholtz(host["S"], host["D"], host["u"])
    assert np.array_equal(ret["v"], want)
    assert ret["max"] == float((E + 1) // 2)
