"""The N > 1 path on CPU: two gloo ranks own disjoint layer units and agree on the slowest time."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2601_21896_b200 import sharding


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close(); return p


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    units = sharding.units_for_rank(7, rank, world)
    slowest = sharding.max_over_ranks(10.0 + rank)
    total = sharding.sum_over_ranks(len(units))
    q.put((rank, units, slowest, total))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_share_units_without_overlap():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    out = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    units = [u for (_, us, _, _) in out for u in us]
    assert sorted(units) == list(range(7))                     # every unit exactly once
    assert all(s == 11.0 for (_, _, s, _) in out)               # max over ranks
    assert all(t == 7.0 for (_, _, _, t) in out)


def test_single_process_is_identity():
    assert sharding.units_for_rank(5, 0, 1) == [0, 1, 2, 3, 4]
    assert sharding.max_over_ranks(3.5) == 3.5
