"""Splitting a model's weight matrices over ranks.

The optimizer steps of two matrices are independent (nothing in Algorithm 1 couples them), so the
grouped step shards over whole matrices with no exchange on the data path: every rank steps its
own matrices.  The assignment balances the cost model of one step,
8 m n r + 6 (m + n) r^2 flops per matrix, with the longest-processing-time rule.

One matrix can also be split by columns over the ranks (the paper's FSDP setting, Section 2,
"FSDP communication"): `shard_columns` gives the column ranges and `sharded_step` drives the
library's local phases with one all-reduce of a small buffer between two of them.
"""
from __future__ import annotations


def step_cost(m: int, n: int, r: int) -> float:
    """Logical flops of one Orth-Dion step of an m x n matrix at rank r (four m*n*r contractions,
    two CholeskyQR2)."""
    return 8.0 * m * n * r + 6.0 * (m + n) * r * r


def partition_matrices(shapes, world_size: int):
    """shapes: sequence of (m, n, r).  Returns `world_size` lists of matrix indices: heaviest
    matrix first, each to the currently lightest rank (ties: lowest rank), so the result is the
    same on every rank."""
    if world_size < 1:
        raise ValueError("world_size must be >= 1")
    order = sorted(range(len(shapes)), key=lambda i: (-step_cost(*shapes[i]), i))
    load = [0.0] * world_size
    parts = [[] for _ in range(world_size)]
    for i in order:
        k = min(range(world_size), key=lambda j: (load[j], j))
        parts[k].append(i)
        load[k] += step_cost(*shapes[i])
    for p in parts:
        p.sort()
    return parts


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """The largest `value` over all ranks of the default process group (the time of a multi-rank
    step is the time of its slowest rank).  With no process group: the value itself."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def shard_columns(n: int, world_size: int, multiple: int = 128):
    """Column ranges [(begin, end), ...] of an m x n matrix over `world_size` ranks: contiguous,
    covering, as even as possible in units of `multiple` columns (the last range takes the
    remainder; ranges may be empty when there are more ranks than units)."""
    if world_size < 1 or n < 1 or multiple < 1:
        raise ValueError("bad arguments")
    units = -(-n // multiple)
    base, extra = divmod(units, world_size)
    out, begin = [], 0
    for k in range(world_size):
        take = (base + (1 if k < extra else 0)) * multiple
        end = min(n, begin + take)
        out.append((begin, end))
        begin = end
    return out


def sharded_step(od, h, orth: bool, X, M, G, Q, workspace, dist=None, stream=None):
    """One optimizer step of this rank's column shard (X, M, G: m x n_j; Q: n_j x r; `h` a plan
    created with (m, n_j, r)): the local phases of the library with the sums over the ranks in
    between (all-reduce over the default process group; none when `dist` is None or has one rank).
    `od` is the binding module."""
    phases = 4 if orth else 3
    multi = dist is not None and dist.is_initialized() and dist.get_world_size() > 1
    for phase in range(phases):
        od.orthdion_shard_phase(h, phase, X, M, G, Q, workspace, stream)
        if phase < phases - 1 and multi:
            dist.all_reduce(od.orthdion_shard_reduce_buffer(h, phase, workspace))
