"""Host logic of the multi-rank paths, on CPU ranks (gloo): the whole-matrix partition is a
partition, is balanced (world sizes 2, 4, 8 on both grouped workloads), is identical on every
rank, and the step time of a job is the maximum over its ranks; and the algebra of the
column-sharded step (sum of shard products, local right factors, one reduced r x r Gram matrix)
gives the oracle's step of the whole matrix when two ranks hold half of the columns each."""
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


def test_partition_balance_for_the_strong_scaling_runs():
    # the split `bench.py --scaling strong` uses, for every world size it may be asked for
    for cfg in ("cfg3", "cfg4"):
        w = wl.workload(cfg)
        shapes = [(s.m, s.n, s.r) for s in w.matrices]
        for world in (2, 4, 8):
            parts = sharding.partition_matrices(shapes, world)
            assert sorted(i for p in parts for i in p) == list(range(len(shapes)))
            cost = [sum(sharding.step_cost(*shapes[i]) for i in p) for p in parts]
            assert (max(cost) - min(cost)) <= 0.05 * max(cost), (cfg, world, cost)


def test_shard_columns_cover_and_balance():
    for n, world in ((4096, 8), (14336, 8), (1024, 3), (640, 4), (200, 2)):
        rg = sharding.shard_columns(n, world)
        assert len(rg) == world and rg[0][0] == 0 and rg[-1][1] == n
        assert all(a[1] == b[0] for a, b in zip(rg, rg[1:]))
        widths = [e - b for b, e in rg]
        assert all(wd % 128 == 0 for wd in widths[:-1]) and max(widths) - min(widths) <= 128 + (n % 128)


def _shard_worker(rank, world, port, out):
    import numpy as np
    from oracle import orthdion_oracle as orc
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    m, n, r, eta, mu = 96, 256, 8, 0.01, 0.95
    g = np.random.default_rng(3)                       # the same full matrices on every rank
    X, M, G = 0.02 * g.standard_normal((m, n)), 0.3 * g.standard_normal((m, n)), g.standard_normal((m, n))
    Q0, _ = orc.thin_qr_pos(g.standard_normal((n, r)))
    c0, c1 = sharding.shard_columns(n, world, multiple=8)[rank]
    B_j, Q_j = (M + G)[:, c0:c1], Q0[c0:c1]

    def allreduce(a):
        t = torch.from_numpy(np.ascontiguousarray(a))
        dist.all_reduce(t)
        return t.numpy()

    Y = allreduce(B_j @ Q_j)                           # B Q_prev = sum_j B_j Q_j
    P, _ = orc.thin_qr_pos(Y)                          # the same on every rank
    R_j = B_j.T @ P                                    # rows c0..c1 of R = B^T P
    gram = allreduce(R_j.T @ R_j)                      # R^T R = sum_j R_j^T R_j
    L = np.linalg.cholesky(gram)                       # R = Q L^T with diag(L) > 0: the thin QR of R
    Qn_j = np.linalg.solve(L, R_j.T).T
    Mn_j = B_j - (1.0 - mu) * (P @ R_j.T)
    Xn_j = X[:, c0:c1] - eta * (P @ Qn_j.T)
    ref = orc.step(X, M, G, Q0, eta=eta, mu=mu)
    err = max(np.abs(P - ref["P"]).max(), np.abs(Qn_j - ref["Q"][c0:c1]).max(),
              np.abs(Mn_j - ref["M"][:, c0:c1]).max(), np.abs(Xn_j - ref["X"][:, c0:c1]).max())
    out.put((rank, float(err), int(Y.size + gram.size), int(m * n)))
    dist.barrier()
    dist.destroy_process_group()


def test_column_shard_algebra_matches_the_oracle_on_two_gloo_ranks():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_shard_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, err, exchanged, elements in res:
        assert err <= 1e-10, (rank, err)
        assert exchanged < elements / 8                 # (m + r) r numbers cross the ranks, not m n
