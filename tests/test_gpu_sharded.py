"""Column-sharded step on one GPU: the k shards of one matrix are stepped phase by phase through the
C ABI, each with its own workspace, and the buffers the phases leave for the cross-rank sums are
summed over the shards here (on real ranks that sum is an all-reduce).  The result, put back
together, must be the float64 oracle's step of the whole matrix.  Not run on more than one GPU.
"""
import numpy as np
import pytest
import torch

from oracle import orthdion_oracle as orc
from paper_2605_16341_b200 import binding as od
from paper_2605_16341_b200 import sharding

from parity_util import TOL_ORTHO, TOL_STEP, f64, poisoned_workspace, rel
from test_gpu_parity import make_problem

pytestmark = pytest.mark.gpu
BF16 = torch.bfloat16


@pytest.mark.parametrize("shape,k", [((768, 1024, 128), 2), ((768, 1024, 128), 4), ((640, 1152, 256), 3)])
@pytest.mark.parametrize("mode", [od.MODE_ORTH, od.MODE_COLNORM])
def test_sharded_step_matches_the_oracle_on_the_whole_matrix(shape, k, mode):
    m, n, r = shape
    spec, X, M, G, Q = make_problem(m, n, r, BF16, BF16, seed=m + n + k)
    ranges = sharding.shard_columns(n, k)
    assert ranges[0][0] == 0 and ranges[-1][1] == n
    orth = mode == od.MODE_ORTH
    shards = []
    for (c0, c1) in ranges:
        h = od.orthdion_create(m, c1 - c0, r, 0.95, 0.01, 0.0, mode)
        ws = poisoned_workspace(od.orthdion_workspace_bytes(h))
        shards.append(dict(h=h, ws=ws, X=X[:, c0:c1].contiguous().cuda(), M=M[:, c0:c1].contiguous().cuda(),
                           G=G[:, c0:c1].contiguous().cuda(), Q=Q[c0:c1].contiguous().cuda()))
    phases = 4 if orth else 3
    for phase in range(phases):
        for s in shards:
            od.orthdion_shard_phase(s["h"], phase, s["X"], s["M"], s["G"], s["Q"], s["ws"])
        torch.cuda.synchronize()
        if phase < phases - 1:
            bufs = [od.orthdion_shard_reduce_buffer(s["h"], phase, s["ws"]) for s in shards]
            total = torch.stack(bufs).sum(0)                 # stands in for the all-reduce
            for b in bufs:
                b.copy_(total)
    torch.cuda.synchronize()
    for s in shards:
        assert od.orthdion_last_status([s["h"]], s["ws"])[0] & ~od.STATUS_SHIFTED_RIGHT == 0
    ref = orc.step(f64(X), f64(M), f64(G), f64(Q), eta=0.01, mu=0.95,
                   mode=orc.ORTH if orth else orc.COLNORM)
    Pd = [od.orthdion_get_factors([s["h"]], 0, s["ws"], (m, s["X"].shape[1], r))[0] for s in shards]
    for P in Pd[1:]:
        assert torch.equal(P, Pd[0])                          # the left factor is the same on every rank
    Pn = f64(Pd[0])
    Qn = np.concatenate([f64(s["Q"]) for s in shards], axis=0)
    Mn = np.concatenate([f64(s["M"]) for s in shards], axis=1)
    assert rel(Pn, ref["P"]) <= TOL_STEP and rel(Qn, ref["Q"]) <= TOL_STEP and rel(Mn, ref["M"]) <= TOL_STEP
    assert rel(-0.01 * (Pn @ Qn.T), ref["X"] - f64(X)) <= TOL_STEP
    assert np.abs(Pn.T @ Pn - np.eye(r)).max() <= TOL_ORTHO
    if orth:
        assert np.abs(Qn.T @ Qn - np.eye(r)).max() <= TOL_ORTHO
    # stored bf16 weights: within one bf16 step of the oracle's, plus the single-pass product bound
    Xn = np.concatenate([f64(s["X"]) for s in shards], axis=1)
    slack = 0.01 * (np.abs(Pn) @ np.abs(Qn).T) * 2.0 ** -8
    assert (np.abs(Xn - ref["X"]) - slack <= np.maximum(np.abs(ref["X"]), 2.0 ** -120) * 2.0 ** -7).all()
    for s in shards:
        od.orthdion_destroy(s["h"])


def test_one_shard_without_reduction_is_the_plain_step():
    spec, X, M, G, Q = make_problem(512, 640, 64, BF16, BF16, seed=5)
    h = od.orthdion_create(512, 640, 64, 0.95, 0.01, 0.0, od.MODE_ORTH)
    ws = poisoned_workspace(od.orthdion_workspace_bytes(h))
    a = [t.cuda() for t in (X, M, Q)]
    b = [t.cuda() for t in (X, M, Q)]
    Gd = G.cuda()
    od.orthdion_step(h, a[0], a[1], Gd, a[2], ws)
    torch.cuda.synchronize()
    ws2 = poisoned_workspace(od.orthdion_workspace_bytes(h))
    sharding.sharded_step(od, h, True, b[0], b[1], Gd, b[2], ws2)
    torch.cuda.synchronize()
    assert rel(f64(b[1]), f64(a[1])) <= TOL_STEP and rel(f64(b[2]), f64(a[2])) <= TOL_STEP
    od.orthdion_destroy(h)
