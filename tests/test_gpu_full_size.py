"""Full-size cases in the launch configuration the benchmark times (grouped step, tensor engine,
default passes): one layer of the 8B-shape and of the 1.1B-shape workload (all shape classes at
r = 512) and the ends of the rank sweep on the 11008 x 4096 matrix (r = 32 and r = 1024).

Every shape class of a layer is compared with the float64 oracle in full: P, R, Q, M and dX of
its first matrix, by relative Frobenius norm and by largest element.  Every matrix of the layer
is also checked on what holds at any size, in float64 from the device's own factors:
orthonormality of P and Q, the error-feedback identity M' = a B - b P R^T and the weight update
on sampled entries, and R = B^T P on sampled entries.
"""
import numpy as np
import pytest
import torch

from oracle import orthdion_oracle as orc
from paper_2605_16341_b200 import binding as od
from paper_2605_16341_b200 import workloads as wl

from parity_util import TOL_MAXABS, TOL_ORTHO, TOL_STEP, f64, poisoned_workspace, rel, rel_max

pytestmark = pytest.mark.gpu


def _gram_dev(A):
    """max |A^T A - I| in float64 on the device."""
    a = A.double()
    g = a.T @ a
    g -= torch.eye(g.shape[0], dtype=torch.float64, device=g.device)
    return float(g.abs().max())


def _sampled_checks(spec, X0, M0, G, Xd, Md, Qd, P, R, eta, mu, mode, rng, samples=2048):
    m, n = spec.m, spec.n
    ii = torch.from_numpy(rng.integers(0, m, samples)).cuda()
    jj = torch.from_numpy(rng.integers(0, n, samples)).cuda()
    Pd, Rd, Qn = P.double(), R.double(), Qd.double()
    b = M0[ii, jj].double() + G[ii, jj].double()
    prt = (Pd[ii] * Rd[jj]).sum(1)
    m_expect = b - (1.0 - mu) * prt
    scale_b = float(b.abs().max())
    assert float((Md[ii, jj].double() - m_expect).abs().max()) <= 1e-4 * scale_b
    pqt = (Pd[ii] * Qn[jj]).sum(1)
    x_expect = X0[ii, jj].double() - eta * pqt
    x_got = Xd[ii, jj].double()
    # stored bf16 weights: half a bf16 spacing (at most |x| 2^-8) for the round-to-nearest-even store,
    # plus the bound of the single fp16 pass that feeds it (each operand rounded to 11 bits)
    half_ulp = torch.clamp(x_expect.abs(), min=2.0 ** -126) * 2.0 ** -8
    slack = eta * (Pd[ii].abs() * Qn[jj].abs()).sum(1) * 2.0 ** -10
    assert float(((x_got - x_expect).abs() - slack - half_ulp * (1 + 1e-3)).max()) <= 0.0
    # R = B^T P on sampled (column of B, factor column) pairs
    cols = torch.from_numpy(rng.integers(0, n, 16)).cuda()
    Bc = (M0[:, cols].double() + G[:, cols].double())                  # m x 16
    r_expect = Bc.T @ Pd                                               # 16 x r
    assert float((Rd[cols] - r_expect).norm() / r_expect.norm()) <= TOL_STEP


@pytest.mark.parametrize("cfg,mode", [("cfg4", od.MODE_ORTH), ("cfg4", od.MODE_COLNORM), ("cfg3", od.MODE_ORTH)])
def test_one_layer_of_the_grouped_workloads(cfg, mode):
    w = wl.workload(cfg, layers=1)
    dev = torch.device("cuda")
    plan = {}
    hs, X0s, M0s, Gs, Xs, Ms, Qs, Q0s = [], [], [], [], [], [], [], []
    for i, spec in enumerate(w.matrices):
        key = (spec.m, spec.n, spec.r)
        if key not in plan:
            plan[key] = od.orthdion_create(spec.m, spec.n, spec.r, w.mu, w.eta, w.wd, mode)
        hs.append(plan[key])
        X, M, Q = wl.initial_state(spec, 0, i, device=dev)
        # a non-trivial residual so that the buffer is not just the gradient
        M = 0.02 * torch.randn(spec.m, spec.n, device=dev, generator=torch.Generator(device=dev).manual_seed(50 + i))
        basis = wl.grad_basis(w, spec, 0, i, device=dev)
        G = wl.gradient(w, spec, 0, i, 0, basis, device=dev)
        X0s.append(X.clone()); M0s.append(M.clone()); Q0s.append(Q.clone()); Gs.append(G)
        Xs.append(X); Ms.append(M); Qs.append(Q)
    ws = poisoned_workspace(od.orthdion_workspace_bytes_grouped(hs))
    table = od.PointerTable(hs, Xs, Ms, Gs, Qs)
    od.orthdion_step_grouped(table, ws)
    torch.cuda.synchronize()
    assert od.orthdion_last_status(hs, ws) == [0] * len(hs)
    rng = np.random.default_rng(0)
    seen = set()
    for i, spec in enumerate(w.matrices):
        P, R = od.orthdion_get_factors(hs, i, ws, (spec.m, spec.n, spec.r))
        assert _gram_dev(P) <= TOL_ORTHO
        if mode == od.MODE_ORTH:
            assert _gram_dev(Qs[i]) <= TOL_ORTHO
        else:
            assert float((Qs[i].double().norm(dim=0) - 1).abs().max()) <= TOL_ORTHO
        _sampled_checks(spec, X0s[i], M0s[i], Gs[i], Xs[i], Ms[i], Qs[i], P, R, w.eta, w.mu, mode, rng)
        # full oracle parity on the first matrix of every shape class (cfg4: 4096 x 4096,
        # 1024 x 4096, 14336 x 4096, 4096 x 14336; cfg3: 2048 x 2048, 5632 x 2048, 2048 x 5632)
        if (spec.m, spec.n) not in seen:
            seen.add((spec.m, spec.n))
            ref = orc.step(f64(X0s[i]), f64(M0s[i]), f64(Gs[i]), f64(Q0s[i]), eta=w.eta, mu=w.mu, wd=w.wd,
                           mode=orc.ORTH if mode == od.MODE_ORTH else orc.COLNORM)
            assert ref["status"] == orc.STATUS_OK
            dx_gpu = -w.eta * (f64(P) @ f64(Qs[i]).T)
            dx_ref = ref["X"] - f64(X0s[i])
            got = dict(dx=dx_gpu, M=f64(Ms[i]), P=f64(P), R=f64(R), Q=f64(Qs[i]))
            want = dict(dx=dx_ref, M=ref["M"], P=ref["P"], R=ref["R"], Q=ref["Q"])
            errs = {k: rel(got[k], want[k]) for k in got}
            emax = {k: rel_max(got[k], want[k]) for k in got}
            print(f"{cfg} mode {mode} {spec.m}x{spec.n}: frobenius {errs} largest element {emax}")
            assert max(errs.values()) <= TOL_STEP, (spec.name, errs)
            assert max(emax.values()) <= TOL_MAXABS, (spec.name, emax)
            del ref, got, want, dx_gpu, dx_ref
    assert len(seen) == len({(s.m, s.n) for s in w.matrices})
    for h in plan.values():
        od.orthdion_destroy(h)


@pytest.mark.parametrize("r", [32, 1024])
@pytest.mark.parametrize("mode", [od.MODE_ORTH, od.MODE_COLNORM])
def test_rank_sweep_ends_on_the_mlp_matrix(r, mode):
    w = wl.workload("cfg2", r=r)
    spec = w.matrices[0]
    dev = torch.device("cuda")
    X, M, Q = wl.initial_state(spec, 0, 0, device=dev)
    M = 0.05 * torch.randn(spec.m, spec.n, device=dev, generator=torch.Generator(device=dev).manual_seed(7))
    basis = wl.grad_basis(w, spec, 0, 0, device=dev)
    G = wl.gradient(w, spec, 0, 0, 0, basis, device=dev)
    X0, M0, Q0 = X.clone(), M.clone(), Q.clone()
    h = od.orthdion_create(spec.m, spec.n, spec.r, w.mu, w.eta, w.wd, mode)
    ws = poisoned_workspace(od.orthdion_workspace_bytes(h))
    od.orthdion_step(h, X, M, G, Q, ws)
    torch.cuda.synchronize()
    assert od.orthdion_last_status([h], ws) == [0]
    P, R = od.orthdion_get_factors([h], 0, ws, (spec.m, spec.n, spec.r))
    assert _gram_dev(P) <= TOL_ORTHO
    if mode == od.MODE_ORTH:
        assert _gram_dev(Q) <= TOL_ORTHO
        # the update direction P Q^T has r unit singular values (Lemma 4.1): Q^T Q = I with P^T P = I
    else:
        # Dion's column normalisation: unit columns, but nu = sigma_1(Q) may exceed 1 (Prop. 3.1)
        assert float((Q.double().norm(dim=0) - 1).abs().max()) <= TOL_ORTHO
        nu = float(torch.linalg.matrix_norm(Q.double(), ord=2))
        assert 1.0 - 1e-6 <= nu <= np.sqrt(r) + 1e-6
    _sampled_checks(spec, X0, M0, G, X, M, Q, P, R, w.eta, w.mu, mode, np.random.default_rng(1))
    if r == 32:
        ref = orc.step(f64(X0), f64(M0), f64(G), f64(Q0), eta=w.eta, mu=w.mu, wd=w.wd,
                       mode=orc.ORTH if mode == od.MODE_ORTH else orc.COLNORM)
        dx_gpu = -w.eta * (f64(P) @ f64(Q).T)
        assert rel(dx_gpu, ref["X"] - f64(X0)) <= TOL_STEP
        assert rel(f64(M), ref["M"]) <= TOL_STEP
    od.orthdion_destroy(h)
