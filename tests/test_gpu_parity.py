"""GPU-vs-oracle parity of the optimizer step, through the C-ABI, element by element.

Tolerances: one step from identical state  ||dX_gpu - dX_or||_F / ||dX_or||_F <= 1e-4,
<= 1e-3 after 10 chained steps (GPU carries its own fp32 M, Q; the oracle float64), and
max |Q^T Q - I| <= 1e-5.
"""
import numpy as np
import pytest
import torch

from oracle import orthdion_oracle as orc
from paper_2605_16341_b200 import binding as od
from paper_2605_16341_b200 import workloads as wl

from parity_util import (TOL_CHAIN, TOL_ORTHO, TOL_STEP, GpuMatrix, bf16_steps_apart, check_bf16_rounding,
                         delta_x_from_factors, f64, oracle_mode, poisoned_workspace, rel, single_pass_slack)

pytestmark = pytest.mark.gpu

ENGINES = [od.ENGINE_SIMT, od.ENGINE_TENSOR]
ENGINE_IDS = ["simt", "tensor"]
MODES = [od.MODE_ORTH, od.MODE_COLNORM]
F32, BF16 = torch.float32, torch.bfloat16


def make_problem(m, n, r, xdt, gdt, seed, m_scale=0.3):
    spec = wl.MatrixSpec("t", m, n, r, xdt, gdt)
    g = torch.Generator().manual_seed(seed)
    X = (0.02 * torch.randn(m, n, generator=g)).to(xdt)
    M = m_scale * torch.randn(m, n, generator=g)
    G = torch.randn(m, n, generator=g).to(gdt)
    Q = wl.random_orthonormal(n, r, g)
    return spec, X, M, G, Q


def one_step_compare(spec, X, M, G, Q, *, mode, engine, mu=0.95, eta=0.01, wd=0.0, ef=None, scale=None,
                     tol=TOL_STEP, passes=None):
    gm = GpuMatrix(spec, X, M, Q, mu=mu, eta=eta, wd=wd, mode=mode, engine=engine, ef=ef, scale=scale,
                   passes=passes)
    gm.step(G)
    assert gm.status() & ~(od.STATUS_SHIFTED_LEFT | od.STATUS_SHIFTED_RIGHT) == 0
    kw = dict(ef=ef) if ef is not None else dict(mu=mu)
    ref = orc.step(f64(X), f64(M), f64(G), f64(Q), eta=eta, wd=wd, scale=1.0 if scale is None else scale,
                   mode=oracle_mode(mode), **kw)
    P, R = gm.factors()
    sc = 1.0 if scale is None else scale
    dx_ref = ref["X"] - f64(X)
    if spec.x_dtype == F32:
        dx_gpu = f64(gm.X) - f64(X)
    else:
        dx_gpu = delta_x_from_factors(P, gm.Q, X, eta, wd, sc)
        assert check_bf16_rounding(gm.X, X, P, gm.Q, eta, wd, sc) <= 1.0 + 1e-6
    errs = dict(dx=rel(dx_gpu, dx_ref), M=rel(f64(gm.M), ref["M"]), Q=rel(f64(gm.Q), ref["Q"]),
                P=rel(f64(P), ref["P"]), R=rel(f64(R), ref["R"]))
    assert errs["dx"] <= tol, errs
    assert errs["M"] <= tol, errs
    assert errs["P"] <= tol and errs["R"] <= tol and errs["Q"] <= tol, errs
    Pn = f64(P)
    assert np.abs(Pn.T @ Pn - np.eye(spec.r)).max() <= TOL_ORTHO
    Qn = f64(gm.Q)
    if mode == od.MODE_ORTH:
        assert np.abs(Qn.T @ Qn - np.eye(spec.r)).max() <= TOL_ORTHO
    else:
        assert np.abs(np.linalg.norm(Qn, axis=0) - 1.0).max() <= TOL_ORTHO
    gm.close()
    return errs


# ------------------------------------------------------------------ cfg0: 10 chained steps
@pytest.mark.parametrize("engine", ENGINES, ids=ENGINE_IDS)
def test_cfg0_chained_both_modes(engine):
    w = wl.workload("cfg0")
    spec = w.matrices[0]
    m_traj = {}
    for mode in MODES:
        X, M, Q = wl.initial_state(spec, 0, 0)
        gm = GpuMatrix(spec, X, M, Q, mu=w.mu, eta=w.eta, wd=w.wd, mode=mode, engine=engine)
        Xo, Mo, Qo = f64(X), f64(M), f64(Q)
        m_traj[mode] = []
        for t in range(10):
            G = wl.gradient(w, spec, 0, 0, t, None)
            x_before_gpu = f64(gm.X)
            gm.step(G)
            assert gm.status() == 0
            ref = orc.step(Xo, Mo, f64(G), Qo, eta=w.eta, mu=w.mu, wd=w.wd, mode=oracle_mode(mode))
            dx_gpu = f64(gm.X) - x_before_gpu
            dx_ref = ref["X"] - Xo
            tol = TOL_STEP if t == 0 else TOL_CHAIN
            assert rel(dx_gpu, dx_ref) <= tol, (mode, t, rel(dx_gpu, dx_ref))
            assert rel(f64(gm.M), ref["M"]) <= tol
            assert rel(f64(gm.X), ref["X"]) <= 1e-5
            Qn = f64(gm.Q)
            if mode == od.MODE_ORTH:
                assert np.abs(Qn.T @ Qn - np.eye(spec.r)).max() <= TOL_ORTHO
            Xo, Mo, Qo = ref["X"], ref["M"], ref["Q"]
            m_traj[mode].append(f64(gm.M))
        gm.close()
    # Lemma 4.3 on the device: the residual trajectory does not depend on the mode
    for a, b in zip(m_traj[od.MODE_ORTH], m_traj[od.MODE_COLNORM]):
        assert rel(a, b) <= 1e-4


# ------------------------------------------------------------------ one step, several shapes
SHAPES_ANY = [(200, 328, 24), (129, 520, 8), (64, 64, 64), (520, 136, 40), (96, 1000, 1), (300, 77, 5)]
SHAPES_TENSOR = [(256, 512, 16), (384, 640, 64), (200, 328, 48), (1000, 264, 128), (136, 2056, 32),
                 (640, 384, 272), (64, 64, 64), (96, 1000, 16), (48, 136, 16), (16, 16, 16),
                 # ranks that are multiples of 256 run as CTA pairs: odd and even numbers of 128-row
                 # tiles on either side, a ragged last tile, two 512-column tiles (r = 1024)
                 (384, 640, 256), (1000, 1032, 256), (1152, 768, 512), (1300, 1024, 1024)]


@pytest.mark.parametrize("shape", SHAPES_ANY)
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("dt", [(F32, F32), (BF16, BF16)])
def test_one_step_simt_shapes(shape, mode, dt):
    m, n, r = shape
    spec, X, M, G, Q = make_problem(m, n, r, dt[0], dt[1], seed=m * 7 + n)
    one_step_compare(spec, X, M, G, Q, mode=mode, engine=od.ENGINE_SIMT)


@pytest.mark.parametrize("shape", SHAPES_TENSOR)
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("dt", [(F32, F32), (BF16, BF16), (F32, BF16), (BF16, F32)])
def test_one_step_tensor_shapes(shape, mode, dt):
    m, n, r = shape
    spec, X, M, G, Q = make_problem(m, n, r, dt[0], dt[1], seed=m * 7 + n)
    one_step_compare(spec, X, M, G, Q, mode=mode, engine=od.ENGINE_TENSOR)


@pytest.mark.parametrize("shape", [(384, 640, 64), (1000, 264, 128), (136, 2056, 32), (640, 384, 272)])
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("m_scale", [0.3, 3e-4, 300.0])
def test_one_step_fused_pass_in_fp16(shape, mode, m_scale):
    # the error-feedback and weight-update products as one fp16 pass (R scaled by a power of two):
    # same tolerances, also when the buffer is far from unit scale
    m, n, r = shape
    spec, X, M, G, Q = make_problem(m, n, r, BF16, BF16, seed=m * 3 + n, m_scale=m_scale)
    G = (G.float() * (m_scale / 0.3)).to(BF16)
    one_step_compare(spec, X, M, G, Q, mode=mode, engine=od.ENGINE_TENSOR, passes={2: 1, 3: 1})


@pytest.mark.parametrize("engine", ENGINES, ids=ENGINE_IDS)
def test_paper_error_feedback_form_and_decay(engine):
    spec, X, M, G, Q = make_problem(256, 384, 32, F32, F32, seed=3)
    beta = 0.7
    gm = GpuMatrix(spec, X, M, Q, mu=0.95, eta=0.01, mode=od.MODE_ORTH, engine=engine, ef=(beta, beta))
    gm.step(G)
    ref = orc.step(f64(X), f64(M), f64(G), f64(Q), eta=0.01, ef=(beta, beta))
    P, _ = gm.factors()
    # R_{t+1} = beta (I - U U^T) M_t is orthogonal to the left factor (up to fp32 cancellation)
    assert np.abs(f64(P).T @ f64(gm.M)).max() <= 2e-3 * np.abs(ref["B"]).max() * np.sqrt(spec.m)
    assert rel(f64(gm.M), ref["M"]) <= TOL_STEP
    gm.close()
    one_step_compare(spec, X, M, G, Q, mode=od.MODE_ORTH, engine=engine, wd=0.1, scale=0.5, eta=0.02)


# ------------------------------------------------------------------ the paper's own shape classes
@pytest.mark.parametrize("shape", [(768, 768, 192), (768, 2048, 192), (2048, 768, 192)])
@pytest.mark.parametrize("mode", MODES)
def test_shape_classes_of_the_320m_model(shape, mode):
    # hidden width 768, MLP width 2048, rank fraction 0.25 of the smaller side, the paper's
    # error-feedback form (beta, beta) and its learning rate and weight decay
    m, n, r = shape
    spec, X, M, G, Q = make_problem(m, n, r, BF16, BF16, seed=m + 3 * n)
    one_step_compare(spec, X, M, G, Q, mode=mode, engine=od.ENGINE_TENSOR, ef=(0.95, 0.95), eta=0.012, wd=0.1)


# ------------------------------------------------------------------ degenerate inputs
@pytest.mark.parametrize("engine", ENGINES, ids=ENGINE_IDS)
def test_zero_buffer_is_flagged_and_state_untouched(engine):
    spec, X, M, G, Q = make_problem(256, 256, 16, BF16, BF16, seed=5)
    M.zero_(); G.zero_()
    gm = GpuMatrix(spec, X, M, Q, mu=0.95, eta=0.01, engine=engine)
    gm.step(G)
    assert gm.status() & od.STATUS_RANK_DEFICIENT
    assert torch.equal(gm.X.cpu(), X) and torch.equal(gm.Q.cpu(), Q) and torch.equal(gm.M.cpu(), M)
    ref = orc.step(f64(X), f64(M), f64(G), f64(Q), eta=0.01, mu=0.95)
    assert ref["status"] == orc.STATUS_RANK_DEFICIENT
    gm.close()


@pytest.mark.parametrize("engine", ENGINES, ids=ENGINE_IDS)
def test_nonfinite_gradient_is_flagged_and_state_untouched(engine):
    spec, X, M, G, Q = make_problem(256, 256, 16, F32, F32, seed=6)
    G[3, 5] = float("nan")
    gm = GpuMatrix(spec, X, M, Q, mu=0.95, eta=0.01, engine=engine)
    gm.step(G)
    assert gm.status() & (od.STATUS_NONFINITE | od.STATUS_RANK_DEFICIENT)
    assert torch.equal(gm.X.cpu(), X) and torch.equal(gm.Q.cpu(), Q) and torch.equal(gm.M.cpu(), M)
    gm.close()


@pytest.mark.parametrize("engine", ENGINES, ids=ENGINE_IDS)
def test_ill_conditioned_projection_takes_shifted_path(engine):
    # B Q_prev with a condition number near 1e6: CholeskyQR2 alone would break down
    m, n, r = 512, 384, 32
    g = torch.Generator().manual_seed(7)
    spec = wl.MatrixSpec("t", m, n, r, F32, F32)
    U = wl.random_orthonormal(m, r, g)
    Q = wl.random_orthonormal(n, r, g)
    s = torch.logspace(0, -6, r)
    G = ((U * s[None, :]) @ Q.T).contiguous()
    X = torch.zeros(m, n)
    M = torch.zeros(m, n)
    gm = GpuMatrix(spec, X, M, Q, mu=0.95, eta=0.01, engine=engine)
    gm.step(G)
    st = gm.status()
    assert st & od.STATUS_SHIFTED_LEFT and not (st & od.STATUS_RANK_DEFICIENT)
    P, _ = gm.factors()
    Pn = f64(P)
    assert np.isfinite(Pn).all()
    assert np.abs(Pn.T @ Pn - np.eye(r)).max() <= TOL_ORTHO
    # the well-conditioned leading directions agree with the oracle
    ref = orc.step(f64(X), f64(M), f64(G), f64(Q), eta=0.01, mu=0.95)
    assert np.abs(Pn[:, :8] - ref["P"][:, :8]).max() <= 1e-3
    gm.close()


# ------------------------------------------------------------------ grouped == single, resume
@pytest.mark.parametrize("engine", ENGINES, ids=ENGINE_IDS)
def test_grouped_matches_single_and_is_deterministic(engine):
    shapes = [(256, 384, 32), (384, 256, 32), (256, 384, 32), (128, 128, 16), (384, 256, 32), (256, 384, 32)]
    specs, st, Gs = [], [], []
    for i, (m, n, r) in enumerate(shapes):
        spec, X, M, G, Q = make_problem(m, n, r, BF16, BF16, seed=100 + i)
        specs.append(spec); st.append((X, M, Q)); Gs.append(G)
    hs = []
    for spec in specs:
        h = od.orthdion_create(spec.m, spec.n, spec.r, 0.95, 0.01, 0.0, od.MODE_ORTH)
        od.orthdion_set_engine(h, engine)
        hs.append(h)
    dev = [tuple(t.cuda() for t in s) for s in st]
    Gd = [g.cuda() for g in Gs]
    ws = poisoned_workspace(od.orthdion_workspace_bytes_grouped(hs))
    table = od.PointerTable(hs, [d[0] for d in dev], [d[1] for d in dev], Gd, [d[2] for d in dev])
    for _ in range(2):
        od.orthdion_step_grouped(table, ws)
    torch.cuda.synchronize()
    assert od.orthdion_last_status(hs, ws) == [0] * len(hs)
    for i, spec in enumerate(specs):
        gm = GpuMatrix(spec, *st[i], mu=0.95, eta=0.01, engine=engine)
        for _ in range(2):
            gm.step(Gs[i])
        assert torch.equal(gm.X, dev[i][0]) and torch.equal(gm.M, dev[i][1]) and torch.equal(gm.Q, dev[i][2])
        P, R = od.orthdion_get_factors(hs, i, ws, (spec.m, spec.n, spec.r))
        P1, R1 = gm.factors()
        assert torch.equal(P, P1) and torch.equal(R, R1)
        gm.close()
    for h in hs:
        od.orthdion_destroy(h)


def test_internal_streams_change_no_bit():
    """A grouped call runs its launch batches on 1 to 8 internal streams: two steps of five classes
    (twelve matrices) leave the same bits whatever the number of streams."""
    shapes = [(256, 384, 32)] * 3 + [(384, 256, 64)] * 2 + [(520, 392, 48)] * 3 + [(128, 1024, 16)] * 2 + \
             [(640, 384, 256)] * 2
    probs = [make_problem(m, n, r, BF16, BF16, seed=300 + i) for i, (m, n, r) in enumerate(shapes)]
    hs = []
    for spec, *_ in probs:
        h = od.orthdion_create(spec.m, spec.n, spec.r, 0.95, 0.01, 0.0, od.MODE_ORTH)
        od.orthdion_set_dtypes(h, BF16, BF16)
        hs.append(h)
    outs = []
    try:
        for lanes in (1, 2, 4, 8):
            od.orthdion_set_concurrency(lanes)
            Xs = [p[1].cuda() for p in probs]; Ms = [p[2].cuda() for p in probs]
            Gd = [p[3].cuda() for p in probs]; Qs = [p[4].cuda() for p in probs]
            ws = poisoned_workspace(od.orthdion_workspace_bytes_grouped(hs))
            table = od.PointerTable(hs, Xs, Ms, Gd, Qs)
            for _ in range(2):
                od.orthdion_step_grouped(table, ws)
            torch.cuda.synchronize()
            assert od.orthdion_last_status(hs, ws) == [0] * len(hs)
            outs.append((Xs, Ms, Qs))
    finally:
        od.orthdion_set_concurrency(4)
    for other in outs[1:]:
        for k in range(3):
            for a, b in zip(outs[0][k], other[k]):
                assert torch.equal(a, b)
    with pytest.raises(Exception):
        od.orthdion_set_concurrency(0)
    with pytest.raises(Exception):
        od.orthdion_set_concurrency(9)
    for h in hs:
        od.orthdion_destroy(h)


# (the last case also has more matrices of one plan than a launch batch holds: two batches)
@pytest.mark.parametrize("shape,count", [((128, 192, 64), 150), ((128, 192, 64), 40), ((512, 640, 512), 150),
                                         ((512, 640, 512), 40), ((64, 64, 16), 300)])
def test_factor_kernel_forms_agree_bit_for_bit(shape, count):
    """The r x r factor kernel runs one CTA per matrix when a call holds more matrices than the
    device has room for clusters, and shares a matrix among the 2, 4, 8 or (from rank 512) 16 CTAs
    of a cluster when it holds fewer.  Every form does the same arithmetic in the same order: a
    matrix stepped inside a call of 150 (one CTA each) or 40 (clusters of two) gets the bits it
    gets when stepped alone (the largest cluster)."""
    m, n, r = shape
    specs, st, Gs = [], [], []
    for i in range(count):
        spec, X, M, G, Q = make_problem(m, n, r, BF16, BF16, seed=7000 + i)
        specs.append(spec); st.append((X, M, Q)); Gs.append(G)
    h = od.orthdion_create(m, n, r, 0.95, 0.01, 0.0, od.MODE_ORTH)
    od.orthdion_set_dtypes(h, BF16, BF16)
    hs = [h] * count
    dev = [tuple(t.cuda() for t in s) for s in st]
    Gd = [g.cuda() for g in Gs]
    ws = poisoned_workspace(od.orthdion_workspace_bytes_grouped(hs))
    table = od.PointerTable(hs, [d[0] for d in dev], [d[1] for d in dev], Gd, [d[2] for d in dev])
    od.orthdion_step_grouped(table, ws)
    torch.cuda.synchronize()
    flags = od.orthdion_last_status(hs, ws)
    assert all(f & ~(od.STATUS_SHIFTED_LEFT | od.STATUS_SHIFTED_RIGHT) == 0 for f in flags)
    for i in (0, count // 2, count - 1):
        gm = GpuMatrix(specs[i], *st[i], mu=0.95, eta=0.01, engine=od.ENGINE_TENSOR)
        gm.step(Gs[i])
        assert gm.status() == flags[i]
        assert torch.equal(gm.X, dev[i][0]) and torch.equal(gm.M, dev[i][1]) and torch.equal(gm.Q, dev[i][2])
        P, R = od.orthdion_get_factors(hs, i, ws, (m, n, r))
        P1, R1 = gm.factors()
        assert torch.equal(P, P1) and torch.equal(R, R1)
        gm.close()
    od.orthdion_destroy(h)


@pytest.mark.parametrize("engine", ENGINES, ids=ENGINE_IDS)
def test_state_is_only_m_and_q(engine):
    # 4 steps in one go == 2 steps, state copied out and back, 2 more steps (bitwise)
    spec, X, M, G, Q = make_problem(256, 384, 32, BF16, BF16, seed=11)
    g = torch.Generator().manual_seed(12)
    Gs = [torch.randn(256, 384, generator=g).to(BF16) for _ in range(4)]
    a = GpuMatrix(spec, X, M, Q, mu=0.95, eta=0.01, engine=engine)
    for t in range(4):
        a.step(Gs[t])
    b = GpuMatrix(spec, X, M, Q, mu=0.95, eta=0.01, engine=engine)
    for t in range(2):
        b.step(Gs[t])
    c = GpuMatrix(spec, b.X.cpu(), b.M.cpu(), b.Q.cpu(), mu=0.95, eta=0.01, engine=engine)
    for t in range(2, 4):
        c.step(Gs[t])
    assert torch.equal(a.X, c.X) and torch.equal(a.M, c.M) and torch.equal(a.Q, c.Q)
    for x in (a, b, c):
        x.close()


# ------------------------------------------------------------------ chained steps with bf16 storage
def chain_compare(w, specs, ids, steps, mode, passes=None, seed=0):
    """`steps` chained steps of the matrices `ids` of workload `w`, as one grouped call per step.
    The device carries its own state (bf16 X, fp32 M and Q); the oracle carries its own (float64
    M and Q, and X rounded to bf16 after every step, which is what storing it means).  Per step
    and matrix: dX formed in float64 from the device's fp32 factors against the oracle's, M, the
    orthonormality of P and Q, the stored weights against the oracle's rounded ones."""
    dev = torch.device("cuda")
    hs, Xs, Ms, Qs, bases, state = [], [], [], [], [], []
    for i in ids:
        spec = specs[i]
        h = od.orthdion_create(spec.m, spec.n, spec.r, w.mu, w.eta, w.wd, mode)
        od.orthdion_set_dtypes(h, spec.x_dtype, spec.g_dtype)
        for k, v in (passes or {}).items():
            od.orthdion_set_passes(h, k, v)
        hs.append(h)
        X, M, Q = wl.initial_state(spec, seed, i)
        bases.append(wl.grad_basis(w, spec, seed, i))
        state.append([f64(X), f64(M), f64(Q)])
        Xs.append(X.to(dev)); Ms.append(M.to(dev)); Qs.append(Q.to(dev))
    ws = poisoned_workspace(od.orthdion_workspace_bytes_grouped(hs))
    worst = dict(dx=0.0, M=0.0, ulps=0.0, differ=0.0)
    for t in range(steps):
        Gs = [wl.gradient(w, specs[i], seed, i, t, bases[k]) for k, i in enumerate(ids)]
        Gd = [g.to(dev) for g in Gs]
        Xb = [x.clone() for x in Xs]
        od.orthdion_step_grouped(od.PointerTable(hs, Xs, Ms, Gd, Qs), ws)
        torch.cuda.synchronize()
        # (a QR may take its third pass: the spike makes B Q_prev less well conditioned as the
        # warm start aligns with it; that is a flag, not a failure)
        assert all(f & ~(od.STATUS_SHIFTED_LEFT | od.STATUS_SHIFTED_RIGHT) == 0 for f in od.orthdion_last_status(hs, ws))
        tol = TOL_STEP if t == 0 else TOL_CHAIN
        for k, i in enumerate(ids):
            spec = specs[i]
            Xo, Mo, Qo = state[k]
            ref = orc.step(Xo, Mo, f64(Gs[k]), Qo, eta=w.eta, mu=w.mu, wd=w.wd, mode=oracle_mode(mode))
            assert ref["status"] == orc.STATUS_OK
            P, R = od.orthdion_get_factors(hs, k, ws, (spec.m, spec.n, spec.r))
            dx_gpu = delta_x_from_factors(P, Qs[k], Xb[k], w.eta, w.wd, 1.0)
            e_dx, e_m = rel(dx_gpu, ref["X"] - Xo), rel(f64(Ms[k]), ref["M"])
            assert e_dx <= tol and e_m <= tol, (spec.name, t, e_dx, e_m)
            Pn, Qn = f64(P), f64(Qs[k])
            assert np.abs(Pn.T @ Pn - np.eye(spec.r)).max() <= TOL_ORTHO
            if mode == od.MODE_ORTH:
                assert np.abs(Qn.T @ Qn - np.eye(spec.r)).max() <= TOL_ORTHO
            assert check_bf16_rounding(Xs[k], Xb[k], P, Qs[k], w.eta, w.wd, 1.0) <= 1.0 + 1e-6
            # stored weights: the oracle's X', rounded to bf16 like the device's, on the entries
            # whose value before the step was the same on both sides
            x_ref = orc.round_to_bf16(ref["X"])
            ulps, differ = bf16_steps_apart(Xs[k], x_ref, Xb[k], Xo, single_pass_slack(P, Qs[k], w.eta))
            assert ulps <= 1.0 and differ <= 0.02, (spec.name, t, ulps, differ)
            state[k] = [x_ref.astype(np.float64), ref["M"], ref["Q"]]
            worst = dict(dx=max(worst["dx"], e_dx), M=max(worst["M"], e_m), ulps=max(worst["ulps"], ulps),
                         differ=max(worst["differ"], differ))
    print(f"{w.name} mode {mode} passes {passes} {steps} chained steps: worst {worst}")
    for h in hs:
        od.orthdion_destroy(h)
    return worst


# cfg1: 4096 x 4096, r = 256, bf16 X and G.  Ten steps with the default passes (the fused pass as
# one fp16 pass), three with the error-feedback product from split terms.
@pytest.mark.parametrize("mode,fused,steps", [(od.MODE_ORTH, "default", 10), (od.MODE_COLNORM, "default", 10),
                                              (od.MODE_ORTH, "bf16x3", 3), (od.MODE_COLNORM, "bf16x3", 3)])
def test_cfg1_chained_steps(mode, fused, steps):
    w = wl.workload("cfg1")
    chain_compare(w, w.matrices, [0], steps, mode, passes=None if fused == "default" else {2: 3, 3: 1})


# One matrix of every shape class of the 1.1B-shape model (2048 x 2048, 5632 x 2048, 2048 x 5632,
# r = 512), stepped together for ten steps with the default passes.
def test_cfg3_ten_chained_steps_of_one_matrix_per_shape_class():
    w = wl.workload("cfg3", layers=1)
    ids = [i for i, s in enumerate(w.matrices) if s.name in ("l0.q", "l0.gate", "l0.down")]
    assert len(ids) == 3
    chain_compare(w, w.matrices, ids, 10, od.MODE_ORTH)


# The accuracy of the single-pass fused products before any storage rounding: fp32 weights (so
# that X' itself can be compared) stepped with the passes a bf16 weight matrix gets by default.
@pytest.mark.parametrize("mode", MODES)
def test_single_pass_update_accuracy_on_fp32_weights(mode):
    spec, X, M, G, Q = make_problem(1000, 1032, 256, F32, BF16, seed=77)
    gm = GpuMatrix(spec, X, M, Q, mu=0.95, eta=0.01, mode=mode, passes={2: 1, 3: 1})
    gm.step(G)
    assert gm.status() == 0
    ref = orc.step(f64(X), f64(M), f64(G), f64(Q), eta=0.01, mu=0.95, mode=oracle_mode(mode))
    P, _ = gm.factors()
    dx_applied = f64(gm.X) - f64(X)                       # what the fused pass really subtracted
    dx_factors = delta_x_from_factors(P, gm.Q, X, 0.01, 0.0, 1.0)
    dx_ref = ref["X"] - f64(X)
    e_applied, e_factors = rel(dx_applied, dx_ref), rel(dx_factors, dx_ref)
    print(f"single-pass update, mode {mode}: applied dX rel err {e_applied:.3e}, from fp32 factors {e_factors:.3e}")
    # the factors meet the step tolerance; the applied update carries the rounding of one
    # 11-bit-operand pass on top (2^-11 per operand: a few 1e-4), and the fp32 storage of X
    assert e_factors <= TOL_STEP
    assert e_applied <= 1e-3
    gm.close()


# ------------------------------------------------------------------ ranks above 1024
# The paper's wide-model study runs 16384-wide blocks at rank fraction 0.25 (r = 4096).  These
# reduced cases take the same path: several 512-column sweeps of the two products with the
# buffer, Gram matrices of more than four tile rows, and an r x r factor kernel whose lists of
# tile products exceed one table (r > 1152) and whose row sums span two column blocks.
@pytest.mark.parametrize("shape,mode", [((2048, 1792, 1536), od.MODE_ORTH), ((1408, 1536, 1280), od.MODE_ORTH),
                                        ((1408, 1536, 1280), od.MODE_COLNORM)])
def test_one_step_rank_above_1024(shape, mode):
    m, n, r = shape
    spec, X, M, G, Q = make_problem(m, n, r, BF16, BF16, seed=m + n + r)
    one_step_compare(spec, X, M, G, Q, mode=mode, engine=od.ENGINE_TENSOR)


def test_one_step_at_the_largest_rank():
    """r = 4096 (the paper's 16384-wide blocks at rank fraction 0.25) on a 6144 x 8192 matrix.  The
    float64 oracle's QR would take minutes here; the results are held to what defines them, formed
    in float64 on the device: P and Q orthonormal, R = B^T P, col(P) = col(B Q_prev), Q R-factor
    upper triangular with positive diagonal, M' = a B - b P R^T."""
    m, n, r = 6144, 8192, 4096
    g = torch.Generator(device="cuda").manual_seed(5)
    X = (0.02 * torch.randn(m, n, generator=g, device="cuda")).to(BF16)
    M = 0.3 * torch.randn(m, n, generator=g, device="cuda")
    G = torch.randn(m, n, generator=g, device="cuda").to(BF16)
    Q0 = torch.linalg.qr(torch.randn(n, r, generator=g, device="cuda", dtype=torch.float64))[0].float().contiguous()
    h = od.orthdion_create(m, n, r, 0.95, 0.01, 0.0, od.MODE_ORTH)
    ws = poisoned_workspace(od.orthdion_workspace_bytes(h))
    Xd, Md, Qd = X.clone(), M.clone(), Q0.clone()
    od.orthdion_step(h, Xd, Md, G, Qd, ws)
    torch.cuda.synchronize()
    st = od.orthdion_last_status([h], ws)[0]
    assert st & ~(od.STATUS_SHIFTED_LEFT | od.STATUS_SHIFTED_RIGHT) == 0
    P, R = od.orthdion_get_factors([h], 0, ws, (m, n, r))
    B = M.double() + G.double()
    P64, R64, Q64 = P.double(), R.double(), Qd.double()
    eye = torch.eye(r, device="cuda", dtype=torch.float64)
    assert (P64.T @ P64 - eye).abs().max().item() <= TOL_ORTHO
    assert (Q64.T @ Q64 - eye).abs().max().item() <= TOL_ORTHO
    Rref = B.T @ P64
    assert ((R64 - Rref).norm() / Rref.norm()).item() <= TOL_STEP
    Y = B @ Q0.double()
    assert ((Y - P64 @ (P64.T @ Y)).norm() / Y.norm()).item() <= TOL_STEP          # col(Y) inside col(P)
    T = Q64.T @ R64                                                                    # R = Q T
    assert ((R64 - Q64 @ T).norm() / R64.norm()).item() <= TOL_STEP
    assert (torch.tril(T, -1).norm() / T.norm()).item() <= TOL_STEP and (torch.diagonal(T) > 0).all()
    Mref = B - 0.05 * (P64 @ R64.T)
    assert ((Md.double() - Mref).norm() / Mref.norm()).item() <= TOL_STEP
    dX = -0.01 * (P64 @ Q64.T)
    got = Xd.double() - X.double()
    # stored bf16 weights: within one bf16 step of the exact update (plus the single-pass bound)
    ulp = X.double().abs().clamp_min(2.0 ** -126) * 2.0 ** -7
    slack = 0.01 * 2.0 ** -8 * (P64.abs() @ Q64.abs().T)
    assert (((got - dX).abs() - slack) / ulp).max().item() <= 1.0 + 1e-6
    od.orthdion_destroy(h)


def test_rank_limits():
    # 4096 is the largest rank; beyond 1024 only the tensor engine (r % 16 == 0) and no diagnostics
    h = od.orthdion_create(8192, 4096, 4096, 0.95, 0.01, 0.0, od.MODE_ORTH)
    assert od.orthdion_workspace_bytes(h) > 0
    with pytest.raises(od.OrthDionError):
        od.orthdion_set_engine(h, od.ENGINE_SIMT)
    with pytest.raises(od.OrthDionError):
        od.orthdion_set_diagnostics(h, 1)
    od.orthdion_destroy(h)
    for bad in ((8192, 8192, 4112), (4096, 4096, 1030)):
        with pytest.raises(od.OrthDionError):
            od.orthdion_create(*bad, 0.95, 0.01, 0.0, od.MODE_ORTH)


def test_tensor_engine_rejects_unsupported_rank():
    h = od.orthdion_create(128, 128, 5, 0.95, 0.01, 0.0, od.MODE_ORTH)
    with pytest.raises(od.OrthDionError):
        od.orthdion_set_engine(h, od.ENGINE_TENSOR)
    od.orthdion_destroy(h)
