"""Repeatability of the grouped step on the GPU: the same seeded model stepped twice from the same
state, over several chained steps with alternating gradients, must give bit-identical X, M and Q.

Nothing in the path accumulates with atomics or in a run-dependent order, so any difference
between the two runs means that some kernel read an operand tile, an accumulator or a workspace
region before its producer had finished with it (a missing wait between the roles of the
tensor-core kernels, between the two CTAs of a pair, or between launches).  Both runs start from
workspaces filled with 0x7f bytes.  Orthonormality of every Q is checked on the way.
"""
import pytest
import torch

from paper_2605_16341_b200 import binding as od
from paper_2605_16341_b200 import workloads as wl

from parity_util import TOL_ORTHO, poisoned_workspace

pytestmark = pytest.mark.gpu


def _run(w, steps, mode):
    dev = torch.device("cuda", 0)
    hs, Xs, Ms, Qs, Gs, plans = [], [], [], [], [[], []], {}
    for i, spec in enumerate(w.matrices):
        key = (spec.m, spec.n, spec.r)
        if key not in plans:
            h = od.orthdion_create(spec.m, spec.n, spec.r, w.mu, w.eta, w.wd, mode)
            od.orthdion_set_dtypes(h, spec.x_dtype, spec.g_dtype)
            plans[key] = h
        hs.append(plans[key])
        X, M, Q = wl.initial_state(spec, 11, i, device=dev)
        basis = wl.grad_basis(w, spec, 11, i, device=dev)
        Xs.append(X); Ms.append(M); Qs.append(Q)
        for k in range(2):
            Gs[k].append(wl.gradient(w, spec, 11, i, k, basis, device=dev))
    ws = poisoned_workspace(od.orthdion_workspace_bytes_grouped(hs))
    tables = [od.PointerTable(hs, Xs, Ms, Gs[k], Qs) for k in range(2)]
    for s in range(steps):
        od.orthdion_step_grouped(tables[s % 2], ws)
    torch.cuda.synchronize()
    status = od.orthdion_last_status(hs, ws)
    for h in plans.values():
        od.orthdion_destroy(h)
    return Xs, Ms, Qs, status


@pytest.mark.parametrize("name,layers", [("cfg3", 2), ("cfg4", 1)])
@pytest.mark.parametrize("mode", [od.MODE_ORTH, od.MODE_COLNORM])
def test_two_runs_are_bit_identical(name, layers, mode):
    w = wl.workload(name, layers=layers)
    a = _run(w, 6, mode)
    b = _run(w, 6, mode)
    assert set(a[3]) == {0} and set(b[3]) == {0}
    for i in range(len(a[0])):
        for t, what in enumerate(("X", "M", "Q")):
            assert torch.equal(a[t][i], b[t][i]), f"{what} of matrix {i} differs between two identical runs"
    if mode == od.MODE_ORTH:
        for Q in a[2]:
            g = Q.double().T @ Q.double()
            g -= torch.eye(g.shape[0], dtype=torch.float64, device=g.device)
            assert float(g.abs().max()) <= TOL_ORTHO
