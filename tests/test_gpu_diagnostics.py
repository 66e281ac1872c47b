"""On-device diagnostics against the float64 oracle's own step (not against the GPU's factors):
nu = ||Q||_op (Proposition 3.1), the effective-rank estimate from the column norms of R,
<B, P Q^T> (Lemma 4.2: tr T_2 for Orth-Dion, the sum of the column norms for Dion), ||R||_F,
||M'||_F, ||G||_F and the derived ||B||_F.

Tolerances: 1e-4 relative for everything that is a plain sum; 1e-3 relative for nu, which comes
from a Lanczos iteration on Q^T Q that stops after at most 96 products.
"""
import math

import numpy as np
import pytest
import torch

from oracle import orthdion_oracle as orc
from paper_2605_16341_b200 import binding as od
from paper_2605_16341_b200 import workloads as wl

from parity_util import GpuMatrix, f64, oracle_mode, poisoned_workspace

pytestmark = pytest.mark.gpu

F32, BF16 = torch.float32, torch.bfloat16
TOL_SUM = 1e-4
TOL_NU = 1e-3


def low_rank_problem(m, n, r, xdt, gdt, seed, k=12, noise=0.05):
    """Gradient and momentum with a decaying spectrum, so that the column norms of R are far from
    uniform and ColNorm(R) is far from orthonormal (nu > 1)."""
    spec = wl.MatrixSpec("t", m, n, r, xdt, gdt)
    g = torch.Generator().manual_seed(seed)
    U = wl.random_orthonormal(m, k, g)
    V = wl.random_orthonormal(n, k, g)
    s = torch.tensor([8.0 / (i + 1) for i in range(k)])
    G = ((U * s) @ V.T + noise * torch.randn(m, n, generator=g)).to(gdt)
    M = 0.5 * ((U * s.flip(0)) @ V.T) + 0.3 * noise * torch.randn(m, n, generator=g)
    X = (0.02 * torch.randn(m, n, generator=g)).to(xdt)
    Q = wl.random_orthonormal(n, r, g)
    return spec, X, M, G, Q


def oracle_diagnostics(ref, G, mode):
    out = dict(nu=orc.nu(ref["Q"]), erank=orc.effective_rank_estimate(ref["R"]),
               tr_t2=float(np.sum(ref["B"] * ref["D"])), norm_r=float(np.linalg.norm(ref["R"])),
               norm_m=float(np.linalg.norm(ref["M"])), norm_g=float(np.linalg.norm(f64(G))),
               norm_b=float(np.linalg.norm(ref["B"])))
    # Lemma 4.2 / its Dion counterpart, on the oracle itself
    if mode == od.MODE_ORTH:
        assert abs(out["tr_t2"] - np.trace(ref["T2"])) <= 1e-9 * abs(out["tr_t2"])
    else:
        assert abs(out["tr_t2"] - np.sum(ref["colnorms"])) <= 1e-9 * abs(out["tr_t2"])
    return out


def compare(d, want, mask):
    assert abs(d["nu"] - want["nu"]) <= TOL_NU * want["nu"], (d, want)
    names = ["erank", "tr_t2", "norm_r"] + (["norm_m", "norm_g", "norm_b"] if mask == 3 else [])
    for k in names:
        assert abs(d[k] - want[k]) <= TOL_SUM * abs(want[k]), (k, d, want)
    if mask != 3:
        assert d["norm_m"] == 0.0 and d["norm_g"] == 0.0 and d["norm_b"] == 0.0
    assert 1 <= d["iterations"] <= 96


CASES = [
    # m, n, r, x dtype, g dtype, engine
    (200, 328, 24, F32, F32, od.ENGINE_SIMT),
    (300, 77, 5, F32, BF16, od.ENGINE_SIMT),
    (256, 512, 16, F32, F32, od.ENGINE_TENSOR),
    (384, 640, 64, BF16, BF16, od.ENGINE_TENSOR),
    (1000, 264, 128, BF16, BF16, od.ENGINE_TENSOR),
    (640, 1160, 272, BF16, BF16, od.ENGINE_TENSOR),
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: f"{c[0]}x{c[1]}r{c[2]}e{c[5]}")
@pytest.mark.parametrize("mode", [od.MODE_ORTH, od.MODE_COLNORM], ids=["orth", "colnorm"])
@pytest.mark.parametrize("mask", [1, 3])
def test_diagnostics_match_oracle(case, mode, mask):
    m, n, r, xdt, gdt, engine = case
    spec, X, M, G, Q = low_rank_problem(m, n, r, xdt, gdt, seed=m + n + r)
    gm = GpuMatrix(spec, X, M, Q, mu=0.95, eta=0.01, mode=mode, engine=engine)
    od.orthdion_set_diagnostics(gm.h, mask)
    gm.step(G)
    assert gm.status() & ~(od.STATUS_SHIFTED_LEFT | od.STATUS_SHIFTED_RIGHT) == 0
    d = od.orthdion_last_diagnostics([gm.h], gm.ws)[0]
    ref = orc.step(f64(X), f64(M), f64(G), f64(Q), eta=0.01, mu=0.95, mode=oracle_mode(mode))
    want = oracle_diagnostics(ref, G, mode)
    compare(d, want, mask)
    if mode == od.MODE_ORTH:
        assert abs(d["nu"] - 1.0) <= 1e-5           # Proposition 3.1, Orth-Dion end
    else:
        assert 1.0 - 1e-5 <= d["nu"] <= math.sqrt(r) * (1 + 1e-5)
        assert want["nu"] > 1.05                      # the case is not a trivial one
    assert 1.0 <= d["erank"] <= r * (1 + 1e-6)
    gm.close()


def test_diagnostics_paper_error_feedback_form():
    """(a, b) = (beta, beta): ||B||_F is recovered from ||M'||_F and ||R||_F."""
    spec, X, M, G, Q = low_rank_problem(384, 640, 64, BF16, BF16, seed=5)
    gm = GpuMatrix(spec, X, M, Q, mu=0.95, eta=0.01, mode=od.MODE_ORTH, engine=od.ENGINE_TENSOR, ef=(0.9, 0.9))
    od.orthdion_set_diagnostics(gm.h, 3)
    gm.step(G)
    d = od.orthdion_last_diagnostics([gm.h], gm.ws)[0]
    ref = orc.step(f64(X), f64(M), f64(G), f64(Q), eta=0.01, ef=(0.9, 0.9), mode=orc.ORTH)
    compare(d, oracle_diagnostics(ref, G, od.MODE_ORTH), 3)
    gm.close()


def test_diagnostics_do_not_change_the_step_and_index_by_matrix():
    """Grouped call with mixed masks: state after the step is bit-identical with diagnostics on
    and off, every record sits at its matrix's position, a plan without diagnostics reports zeros."""
    shapes = [(256, 512, 16), (384, 640, 64), (256, 512, 16), (200, 328, 48)]
    masks = [3, 0, 1, 3]
    probs = [low_rank_problem(m, n, r, BF16, BF16, seed=10 + i) for i, (m, n, r) in enumerate(shapes)]
    results = {}
    for with_diag in (False, True):
        hs, Xs, Ms, Gs, Qs = [], [], [], [], []
        for (spec, X, M, G, Q), mask in zip(probs, masks):
            h = od.orthdion_create(spec.m, spec.n, spec.r, 0.95, 0.01, 0.0, od.MODE_COLNORM)
            od.orthdion_set_dtypes(h, spec.x_dtype, spec.g_dtype)
            if with_diag:
                od.orthdion_set_diagnostics(h, mask)
            hs.append(h)
            Xs.append(X.cuda().clone()); Ms.append(M.cuda().clone())
            Gs.append(G.cuda().clone()); Qs.append(Q.cuda().clone())
        ws = poisoned_workspace(od.orthdion_workspace_bytes_grouped(hs))
        od.orthdion_step_grouped(od.PointerTable(hs, Xs, Ms, Gs, Qs), ws)
        torch.cuda.synchronize()
        assert all(s == 0 for s in od.orthdion_last_status(hs, ws))
        results[with_diag] = (Xs, Ms, Qs, od.orthdion_last_diagnostics(hs, ws))
        for h in hs:
            od.orthdion_destroy(h)
    for a, b in zip(results[False][:3], results[True][:3]):
        for ta, tb in zip(a, b):
            assert torch.equal(ta, tb)
    assert all(all(v == 0.0 for v in d.values()) for d in results[False][3])
    diags = results[True][3]
    assert all(v == 0.0 for v in diags[1].values())
    for i in (0, 2, 3):
        spec, X, M, G, Q = probs[i]
        ref = orc.step(f64(X), f64(M), f64(G), f64(Q), eta=0.01, mu=0.95, mode=orc.COLNORM)
        compare(diags[i], oracle_diagnostics(ref, G, od.MODE_COLNORM), masks[i])


def test_diagnostics_of_a_failed_step_are_nan():
    spec = wl.MatrixSpec("t", 256, 512, 16, BF16, BF16)
    g = torch.Generator().manual_seed(1)
    X = (0.02 * torch.randn(256, 512, generator=g)).to(BF16)
    Z = torch.zeros(256, 512)
    gm = GpuMatrix(spec, X, Z, wl.random_orthonormal(512, 16, g), mu=0.95, eta=0.01)
    od.orthdion_set_diagnostics(gm.h, 3)
    gm.step(Z.to(BF16))
    assert gm.status() & (od.STATUS_RANK_DEFICIENT | od.STATUS_NONFINITE)
    d = od.orthdion_last_diagnostics([gm.h], gm.ws)[0]
    assert all(math.isnan(v) for v in d.values())
    gm.close()


def test_set_diagnostics_rejects_bad_masks():
    h = od.orthdion_create(256, 512, 16, 0.95, 0.01, 0.0, od.MODE_ORTH)
    for bad in (-1, 4, 7):
        with pytest.raises(od.OrthDionError):
            od.orthdion_set_diagnostics(h, bad)
    od.orthdion_destroy(h)


@pytest.mark.parametrize("mode", [od.MODE_ORTH, od.MODE_COLNORM], ids=["orth", "colnorm"])
def test_diagnostics_at_full_size_in_the_grouped_launch(mode):
    """One layer of the 8B workload (r = 512, n up to 14336) in the benchmark's launch
    configuration.  Every matrix: against float64 library routines applied to the device's own
    state (matrix 2-norm of Q, column norms of R, Frobenius norms).  The 1024 x 4096 matrix also
    against the oracle's own step."""
    w = wl.workload("cfg4", layers=1)
    dev = torch.device("cuda")
    plan, hs, M0s, Gs, Xs, Ms, Qs, Q0s, X0s = {}, [], [], [], [], [], [], [], []
    for i, spec in enumerate(w.matrices):
        key = (spec.m, spec.n, spec.r)
        if key not in plan:
            plan[key] = od.orthdion_create(spec.m, spec.n, spec.r, w.mu, w.eta, w.wd, mode)
            od.orthdion_set_diagnostics(plan[key], 3)
        hs.append(plan[key])
        X, M, Q = wl.initial_state(spec, 0, i, device=dev)
        M = 0.02 * torch.randn(spec.m, spec.n, device=dev, generator=torch.Generator(device=dev).manual_seed(50 + i))
        G = wl.gradient(w, spec, 0, i, 0, wl.grad_basis(w, spec, 0, i, device=dev), device=dev)
        X0s.append(X.clone()); M0s.append(M.clone()); Q0s.append(Q.clone()); Gs.append(G)
        Xs.append(X); Ms.append(M); Qs.append(Q)
    ws = poisoned_workspace(od.orthdion_workspace_bytes_grouped(hs))
    od.orthdion_step_grouped(od.PointerTable(hs, Xs, Ms, Gs, Qs), ws)
    torch.cuda.synchronize()
    assert od.orthdion_last_status(hs, ws) == [0] * len(hs)
    diags = od.orthdion_last_diagnostics(hs, ws)
    by_oracle = 0
    for i, spec in enumerate(w.matrices):
        d = diags[i]
        P, R = od.orthdion_get_factors(hs, i, ws, (spec.m, spec.n, spec.r))
        Rd, Qd = R.double(), Qs[i].double()
        s = Rd.norm(dim=0)
        p = s / s.sum()
        want = dict(nu=float(torch.linalg.matrix_norm(Qd, ord=2)),
                    erank=float(torch.exp(-(p * torch.log(p)).sum())),
                    tr_t2=float((Rd * Qd).sum()), norm_r=float(Rd.norm()),
                    norm_m=float(Ms[i].double().norm()), norm_g=float(Gs[i].double().norm()),
                    norm_b=float((M0s[i].double() + Gs[i].double()).norm()))
        compare(d, want, 3)
        if mode == od.MODE_ORTH:
            assert abs(d["nu"] - 1.0) <= 1e-5
        if spec.name == "l0.k":
            ref = orc.step(f64(X0s[i]), f64(M0s[i]), f64(Gs[i]), f64(Q0s[i]), eta=w.eta, mu=w.mu, wd=w.wd,
                           mode=oracle_mode(mode))
            compare(d, oracle_diagnostics(ref, Gs[i], mode), 3)
            by_oracle += 1
    assert by_oracle == 1
    for h in plan.values():
        od.orthdion_destroy(h)
