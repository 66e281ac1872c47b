"""Host logic of the multi-rank path, on CPU ranks (gloo, world_size 2): the whole-matrix
partition is a partition, is balanced, is identical on every rank, and the step time of a job is
the maximum over its ranks."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_16341_b200 import sharding, workloads as wl


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = wl.workload("cfg4", layers=4)
    shapes = [(s.m, s.n, s.r) for s in w.matrices]
    parts = sharding.partition_matrices(shapes, world)
    # every rank must see the same partition: gather and compare
    gathered = [None] * world
    dist.all_gather_object(gathered, parts)
    same = all(g == parts for g in gathered)
    # the slowest rank defines the step time
    t = sharding.max_over_ranks(10.0 + rank, dist)
    out.put((rank, same, parts[rank], t))
    dist.barrier()
    dist.destroy_process_group()


def test_partition_and_timing_on_two_gloo_ranks():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    w = wl.workload("cfg4", layers=4)
    n = len(w.matrices)
    assert all(r[1] for r in res)
    mine = [r[2] for r in res]
    assert sorted(mine[0] + mine[1]) == list(range(n))          # a partition: no loss, no overlap
    assert all(r[3] == 11.0 for r in res)                       # max over ranks, on every rank
    cost = [sum(sharding.step_cost(w.matrices[i].m, w.matrices[i].n, w.matrices[i].r) for i in part) for part in mine]
    assert abs(cost[0] - cost[1]) <= 0.05 * max(cost)


def test_partition_single_rank_and_more_ranks_than_matrices():
    shapes = [(256, 512, 16), (128, 128, 16), (512, 512, 32)]
    assert sharding.partition_matrices(shapes, 1) == [[0, 1, 2]]
    parts = sharding.partition_matrices(shapes, 5)
    assert sorted(i for p in parts for i in p) == [0, 1, 2]
    assert sum(1 for p in parts if not p) == 2
    assert sharding.max_over_ranks(3.5) == 3.5
