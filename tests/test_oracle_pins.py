"""Pins for the float64 oracle: what the paper and plain mathematics fix about one step.

Each test names the passage it rests on.  None of these retypes the oracle's own formula:
they check it against LAPACK factorisations, brute-force SVDs, closed-form special cases
and identities stated in the paper.
"""
import os

import numpy as np
import pytest

from oracle import orthdion_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")
TOL = 1e-11


def rng(seed):
    return np.random.default_rng(seed)


def rand_orth(g, n, r):
    q, t = np.linalg.qr(g.standard_normal((n, r)))
    return q * np.sign(np.diag(t))[None, :]


def problem(seed, m=24, n=40, r=6):
    g = rng(seed)
    X = 0.02 * g.standard_normal((m, n))
    M = 0.3 * g.standard_normal((m, n))
    G = g.standard_normal((m, n))
    Qp = rand_orth(g, n, r)
    return X, M, G, Qp


# ------------------------------------------------------------------ thin QR (orth)
@pytest.mark.parametrize("shape", [(7, 1), (9, 9), (40, 6), (200, 33), (64, 64)])
def test_thin_qr_matches_lapack_and_is_unique(shape):
    g = rng(shape[0] * 100 + shape[1])
    Y = g.standard_normal(shape)
    F, T = orc.thin_qr_pos(Y)
    r = shape[1]
    assert np.allclose(F.T @ F, np.eye(r), atol=TOL)
    assert np.allclose(F @ T, Y, atol=TOL)
    assert np.all(np.diag(T) > 0) and np.allclose(T, np.triu(T))
    # LAPACK QR with the sign fixed
    q, t = np.linalg.qr(Y)
    d = np.sign(np.diag(t))
    assert np.allclose(F, q * d[None, :], atol=1e-10)
    assert np.allclose(T, t * d[:, None], atol=1e-10)
    # uniqueness: the Cholesky factor of the Gram matrix is the same triangle
    L = np.linalg.cholesky(Y.T @ Y)
    assert np.allclose(T, L.T, atol=1e-9 * np.linalg.norm(Y) ** 1)


def test_thin_qr_gram_schmidt_bruteforce_tiny():
    # classical Gram-Schmidt written out for a 4 x 3 matrix with small integers
    Y = np.array([[2.0, -1.0, 0.0], [1.0, 3.0, 1.0], [0.0, 1.0, -2.0], [2.0, 0.0, 1.0]])
    cols = []
    T_expected = np.zeros((3, 3))
    for j in range(3):
        v = Y[:, j].copy()
        for i, q in enumerate(cols):
            T_expected[i, j] = q @ Y[:, j]
            v -= T_expected[i, j] * q
        T_expected[j, j] = np.linalg.norm(v)
        cols.append(v / T_expected[j, j])
    F, T = orc.thin_qr_pos(Y)
    assert np.allclose(F, np.stack(cols, axis=1), atol=1e-13)
    assert np.allclose(T, T_expected, atol=1e-13)
    # first column: closed form  (2,1,0,2)/3
    assert np.allclose(F[:, 0], np.array([2, 1, 0, 2]) / 3.0, atol=1e-15)


def test_thin_qr_negative_leading_entries_still_positive_diag():
    Y = -np.abs(rng(5).standard_normal((12, 4)))
    F, T = orc.thin_qr_pos(Y)
    assert np.all(np.diag(T) > 0)
    assert np.allclose(F @ T, Y, atol=TOL)


# ------------------------------------------------------------------ ColNorm (Prop. 3.1)
def test_colnorm_unit_columns_and_nu_range():
    g = rng(11)
    R = g.standard_normal((30, 8)) * np.logspace(-2, 2, 8)[None, :]
    Q, norms = orc.col_norm(R)
    assert np.allclose(np.diag(Q.T @ Q), 1.0, atol=1e-14)
    assert np.allclose(norms, np.linalg.norm(R, axis=0))
    v = orc.nu(Q)
    assert 1.0 - 1e-12 <= v <= np.sqrt(8) + 1e-12


def test_colnorm_nu_extremes():
    # orthogonal columns -> nu = 1 ; colinear columns -> nu = sqrt(r)   (Prop. 3.1 and Section 4)
    g = rng(12)
    r = 9
    Qo = rand_orth(g, 25, r) * np.linspace(0.5, 7, r)[None, :]
    assert abs(orc.nu(orc.col_norm(Qo)[0]) - 1.0) < 1e-12
    w = g.standard_normal(25)
    Rc = np.outer(w, np.linspace(1.0, 3.0, r))
    assert abs(orc.nu(orc.col_norm(Rc)[0]) - np.sqrt(r)) < 1e-12


# ------------------------------------------------------------------ Lemma 4.1 and Frobenius norm
@pytest.mark.parametrize("mode", [orc.ORTH, orc.COLNORM])
def test_update_direction_norms(mode):
    X, M, G, Qp = problem(1)
    out = orc.step(X, M, G, Qp, eta=0.01, mu=0.95, mode=mode)
    r = Qp.shape[1]
    D = out["P"] @ out["Q"].T
    assert np.allclose(out["P"].T @ out["P"], np.eye(r), atol=TOL)
    # ||P Q^T||_F = sqrt(r) in both modes (Section 3, geometric interpretation)
    assert abs(np.linalg.norm(D) - np.sqrt(r)) < 1e-11
    s = np.linalg.svd(D, compute_uv=False)
    if mode == orc.ORTH:
        # Lemma 4.1: r unit singular values, the rest zero; dual norm 1
        assert np.allclose(s[:r], 1.0, atol=1e-11) and np.all(s[r:] < 1e-11)
        assert np.allclose(out["Q"].T @ out["Q"], np.eye(r), atol=TOL)
        assert abs(orc.dual_norm(D, r) - 1.0) < 1e-11
    else:
        # Prop. 3.1: nu = ||Q||_op = dual norm of D, in [1, sqrt(r)], > 1 for generic R
        v = orc.nu(out["Q"])
        assert abs(s[0] - v) < 1e-11
        assert abs(orc.dual_norm(D, r) - v) < 1e-11
        assert 1.0 + 1e-6 < v <= np.sqrt(r)


# ------------------------------------------------------------------ error feedback (Alg. 1, error-feedback step)
def test_error_feedback_identities():
    X, M, G, Qp = problem(2)
    mu = 0.95
    out = orc.step(X, M, G, Qp, eta=0.01, mu=mu)
    B, P, R = M + G, out["P"], out["R"]
    # momentum form: B = M' + (1-mu) P R^T
    assert np.allclose(out["M"] + (1 - mu) * P @ R.T, B, atol=TOL)
    # P R^T is the projection of B on col(P)
    assert np.allclose(P @ R.T, P @ (P.T @ B), atol=TOL)
    # paper form  R_{t+1} = beta (I - U U^T) M_t :  P^T M' = 0 and M' = beta (B - P P^T B)
    beta = 0.7
    out2 = orc.step(X, M, G, Qp, eta=0.01, ef=(beta, beta))
    assert np.abs(P.T @ out2["M"]).max() < 1e-11
    proj = np.eye(B.shape[0]) - P @ P.T
    assert np.allclose(out2["M"], beta * proj @ B, atol=TOL)
    # the factors do not depend on the EF coefficients
    assert np.allclose(out2["Q"], out["Q"], atol=0) and np.allclose(out2["X"], out["X"], atol=0)


def test_weight_update_line():
    X, M, G, Qp = problem(3)
    eta = 0.013
    out = orc.step(X, M, G, Qp, eta=eta, mu=0.9)
    assert np.allclose(out["X"], X - eta * out["P"] @ out["Q"].T, atol=1e-15)
    # decoupled decay / scale: algebraic identity only (no equation in the paper: unpinned)
    out2 = orc.step(X, M, G, Qp, eta=eta, mu=0.9, wd=0.1, scale=0.5)
    assert np.allclose(out2["X"] - (1 - eta * 0.1) * X, -eta * 0.5 * out["P"] @ out["Q"].T, atol=1e-15)


# ------------------------------------------------------------------ closed-form special cases
def test_exact_rank_r_buffer_is_reconstructed():
    g = rng(4)
    m, n, r = 20, 30, 5
    U, V = rand_orth(g, m, r), rand_orth(g, n, r)
    S = np.diag(np.linspace(3.0, 1.0, r))
    B = U @ S @ V.T
    G = g.standard_normal((m, n))
    M = B - G
    # Q_prev spans the row space of B but is not V itself
    Qp = rand_orth(g, r, r)
    Qp = V @ Qp
    mu = 0.95
    out = orc.step(np.zeros((m, n)), M, G, Qp, eta=0.1, mu=mu)
    assert np.allclose(out["P"] @ out["R"].T, B, atol=1e-10)
    assert np.allclose(out["M"], mu * B, atol=1e-10)
    out_b = orc.step(np.zeros((m, n)), M, G, Qp, eta=0.1, ef=(1.0, 1.0))
    assert np.abs(out_b["M"]).max() < 1e-10


def test_aligned_case_gives_polar_factor_and_modes_agree():
    # B = U S V^T and Q_prev = V  =>  P = U, T1 = T2 = S, Q = V, P Q^T = rank-r polar factor
    g = rng(5)
    m, n, r = 18, 26, 4
    U, V = rand_orth(g, m, r), rand_orth(g, n, r)
    s = np.array([5.0, 3.0, 2.0, 0.5])
    tail_u, tail_v = rand_orth(g, m, m)[:, :2], rand_orth(g, n, n)[:, :2]
    # add an orthogonal tail below sigma_r so that the truncated SVD is U, V
    tail_u -= U @ (U.T @ tail_u); tail_u = np.linalg.qr(tail_u)[0]
    tail_v -= V @ (V.T @ tail_v); tail_v = np.linalg.qr(tail_v)[0]
    B = U @ np.diag(s) @ V.T + tail_u @ np.diag([0.1, 0.05]) @ tail_v.T
    out = orc.step(np.zeros((m, n)), np.zeros((m, n)), B, V, eta=1.0, mu=0.95)
    assert np.allclose(out["P"], U, atol=1e-11)
    assert np.allclose(out["T1"], np.diag(s), atol=1e-11)
    assert np.allclose(out["T2"], np.diag(s), atol=1e-11)
    assert np.allclose(out["Q"], V, atol=1e-11)
    assert np.allclose(out["P"] @ out["Q"].T, orc.rank_r_polar(B, r), atol=1e-10)
    assert abs(orc.defect(B, out["P"], out["Q"], r)) < 1e-10
    out_c = orc.step(np.zeros((m, n)), np.zeros((m, n)), B, V, eta=1.0, mu=0.95, mode=orc.COLNORM)
    assert np.allclose(out_c["Q"], out["Q"], atol=1e-11)
    assert np.allclose(out_c["X"], out["X"], atol=1e-11)


def test_rank_one_modes_coincide():
    X, M, G, Qp = problem(6, r=1)
    a = orc.step(X, M, G, Qp, eta=0.01, mu=0.95, mode=orc.ORTH)
    b = orc.step(X, M, G, Qp, eta=0.01, mu=0.95, mode=orc.COLNORM)
    assert np.allclose(a["Q"], b["Q"], atol=1e-13) and np.allclose(a["X"], b["X"], atol=1e-13)
    # and for a rank-1 buffer the update is u1 v1^T
    g = rng(7)
    u, v = g.standard_normal(10), g.standard_normal(14)
    B = 2.5 * np.outer(u, v)
    q0 = g.standard_normal((14, 1)); q0 /= np.linalg.norm(q0)
    out = orc.step(np.zeros((10, 14)), np.zeros((10, 14)), B, q0, eta=1.0, mu=0.9)
    sgn = np.sign(v @ q0[:, 0])
    # P = sgn*u/|u|, Q = sgn*v/|v| (positive diagonal), product independent of sgn
    assert np.allclose(out["P"] @ out["Q"].T, np.outer(u, v) / (np.linalg.norm(u) * np.linalg.norm(v)), atol=1e-12)
    assert np.allclose(out["P"][:, 0], sgn * u / np.linalg.norm(u), atol=1e-12)


# ------------------------------------------------------------------ Lemma 4.2 (defect) with brute-force SVD
@pytest.mark.parametrize("seed", range(5))
def test_defect_nonnegative_and_inner_product_is_trace(seed):
    X, M, G, Qp = problem(20 + seed, m=9, n=7, r=3)
    out = orc.step(X, M, G, Qp, eta=0.01, mu=0.95)
    B = M + G
    ip = float(np.sum(B * (out["P"] @ out["Q"].T)))
    assert abs(ip - np.trace(out["T2"])) < 1e-11          # <B, P Q^T> = tr(T2) > 0
    assert ip > 0
    sv = np.sqrt(np.clip(np.linalg.eigvalsh(B.T @ B)[::-1], 0, None))   # SVD by eigenvalues
    assert sv[:3].sum() - ip >= -1e-11                    # Lemma 4.2
    assert abs(orc.defect(B, out["P"], out["Q"], 3) - (sv[:3].sum() - ip)) < 1e-10


# ------------------------------------------------------------------ Lemma 4.3 (same tracking)
def test_same_tracking_across_modes_chained():
    g = rng(30)
    m, n, r = 32, 48, 6
    X = 0.02 * g.standard_normal((m, n))
    Qp = rand_orth(g, n, r)
    st = {orc.ORTH: (X, np.zeros((m, n)), Qp), orc.COLNORM: (X, np.zeros((m, n)), Qp)}
    for t in range(10):
        G = g.standard_normal((m, n))
        res = {}
        for mode in st:
            Xc, Mc, Qc = st[mode]
            res[mode] = orc.step(Xc, Mc, G, Qc, eta=0.01, mu=0.95, mode=mode)
            st[mode] = (res[mode]["X"], res[mode]["M"], res[mode]["Q"])
        qo, qc = res[orc.ORTH]["Q"], res[orc.COLNORM]["Q"]
        # equal column spaces: equal projectors
        proj_c = qc @ np.linalg.solve(qc.T @ qc, qc.T)
        assert np.allclose(qo @ qo.T, proj_c, atol=1e-9)
        # hence the whole residual trajectory is the same
        assert np.allclose(res[orc.ORTH]["M"], res[orc.COLNORM]["M"], atol=1e-9)
    assert not np.allclose(st[orc.ORTH][0], st[orc.COLNORM][0], atol=1e-6)   # the weights do differ


def test_sign_invariance_of_warm_start():
    X, M, G, Qp = problem(8)
    d = np.array([1, -1, 1, -1, -1, 1.0])
    a = orc.step(X, M, G, Qp, eta=0.01, mu=0.95)
    b = orc.step(X, M, G, Qp * d[None, :], eta=0.01, mu=0.95)
    assert np.allclose(a["X"], b["X"], atol=1e-12) and np.allclose(a["M"], b["M"], atol=1e-12)


def test_residual_operator_norm_bound():
    # ||M'||_op <= sigma_{r+1}(B) + eps_t sigma_1(B) for beta = 1 (appendix, self-consistent bound)
    for seed in range(4):
        X, M, G, Qp = problem(40 + seed, m=12, n=15, r=4)
        out = orc.step(X, M, G, Qp, eta=0.01, ef=(1.0, 1.0))
        B = M + G
        U, s, _ = np.linalg.svd(B)
        P = out["P"]
        eps = np.linalg.norm(P @ P.T - U[:, :4] @ U[:, :4].T, 2)
        assert np.linalg.norm(out["M"], 2) <= s[4] + eps * s[0] + 1e-10


def test_transposed_operand_would_be_caught():
    # Y = B Q_prev (not B^T ...): for a non-square problem P must be m x r and satisfy
    # col(P) = col(B Q_prev); R = B^T P must be n x r.
    X, M, G, Qp = problem(9, m=10, n=17, r=3)
    out = orc.step(X, M, G, Qp, eta=0.01, mu=0.95)
    B = M + G
    assert out["P"].shape == (10, 3) and out["R"].shape == (17, 3)
    Y = B @ Qp
    assert np.linalg.matrix_rank(np.concatenate([Y, out["P"]], axis=1), tol=1e-9) == 3
    assert np.allclose(out["R"], B.T @ out["P"], atol=TOL)


def test_rank_deficient_is_flagged_and_state_untouched():
    m, n, r = 8, 12, 3
    Qp = rand_orth(rng(10), n, r)
    X = np.ones((m, n))
    out = orc.step(X, np.zeros((m, n)), np.zeros((m, n)), Qp, eta=0.1, mu=0.95)
    assert out["status"] == orc.STATUS_RANK_DEFICIENT
    assert np.array_equal(out["X"], X) and np.array_equal(out["Q"], Qp)


# ------------------------------------------------------------------ numbers printed in the paper
def _golden(name):
    vals = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split("=")
                vals[k.strip()] = float(v)
    return vals


def test_printed_values():
    gold = _golden("paper_printed_values.txt")
    A = np.eye(3)
    assert abs(orc.dual_norm(A, 2) - gold["dual_norm_I3_r2"]) < 1e-12
    assert abs(orc.dual_norm_body_formula(A, 2) ** 2 - gold["body_formula_I3_r2_squared"]) < 1e-12
    # attained by B = I/2 with Ky Fan 2-norm 1
    Bm = 0.5 * np.eye(3)
    assert abs(orc.ky_fan(Bm, 2) - 1.0) < 1e-12 and abs(np.sum(A * Bm) - gold["dual_norm_I3_r2"]) < 1e-12
    # coupling ratio (1 + sqrt(r)) / 2 at r = 256, with nu = sqrt(r) attained by colinear columns
    r = 256
    Rc = np.outer(np.arange(1.0, 301.0), np.ones(r))
    v = orc.nu(orc.col_norm(Rc)[0])
    assert abs((1 + v) / 2 - gold["coupling_ratio_r256"]) < 1e-9
    assert abs(v * v - gold["smoothness_ratio_r256"]) < 1e-6


def test_round_to_bf16_matches_torch():
    import torch
    g = rng(50)
    x = np.concatenate([g.standard_normal(4000) * 10.0 ** g.integers(-6, 3, 4000),
                        np.array([1.0, 1.00390625, 1.001953125, 1.005859375, 0.0, -3.0])])
    ours = orc.round_to_bf16(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).float().numpy()   # fp64 -> bf16, RN-even
    assert np.array_equal(ours, ref)


def test_effective_rank_estimate_extremes():
    assert abs(orc.effective_rank_estimate(np.eye(6)) - 6.0) < 1e-12       # flat spectrum
    R = np.zeros((5, 4)); R[:, 0] = 1.0; R[:, 1:] = 1e-300
    assert abs(orc.effective_rank_estimate(R) - 1.0) < 1e-9                  # one dominant column


# ------------------------------------------------------------------ rank selection (Ada-Orth-Dion)
def test_rank_policy_worked_examples():
    # alpha = 1: no memory; gamma = 1: the target is the estimate itself, rounded up to an integer
    assert orc.rank_policy(40.0, 64, 123.0, 8, 512, 1.0, 1.0) == (40.0, 40)
    assert orc.rank_policy(40.2, 64, 0.0, 8, 512, 1.0, 1.0) == (40.2, 40)        # ceil 41 -> nearest multiple 40
    assert orc.rank_policy(43.5, 64, 0.0, 8, 512, 1.0, 1.0)[1] == 48             # ceil 44: tie goes up
    assert orc.rank_policy(44.5, 64, 0.0, 8, 512, 1.0, 1.0)[1] == 48             # ceil 45 -> 48
    # EMA by hand: 0.25 * 100 + 0.75 * 60 = 70; gamma 1.5 -> 105 -> 104
    ema, r = orc.rank_policy(100.0, 64, 60.0, 8, 512, 0.25, 1.5)
    assert ema == 70.0 and r == 104
    # clipping at both ends, with bounds that are multiples of 16
    assert orc.rank_policy(3.0, 64, 3.0, 16, 256, 0.5, 1.1, multiple=16)[1] == 16
    assert orc.rank_policy(900.0, 64, 900.0, 16, 256, 0.5, 1.1, multiple=16)[1] == 256
    # alpha = 0 keeps the old average whatever the new estimate says
    assert orc.rank_policy(500.0, 64, 32.0, 8, 512, 0.0, 1.0) == (32.0, 32)
    with pytest.raises(ValueError):
        orc.rank_policy(10.0, 64, 10.0, 12, 512, 0.5, 1.1)                        # bound not a multiple of 8


def test_rank_policy_is_monotone_and_stays_in_bounds():
    g = np.random.default_rng(3)
    for _ in range(200):
        e, prev = g.uniform(1, 600, 2)
        alpha, gamma = g.uniform(0, 1), g.uniform(0.8, 1.6)
        ema, r = orc.rank_policy(e, 64, prev, 16, 512, alpha, gamma)
        assert min(e, prev) - 1e-9 <= ema <= max(e, prev) + 1e-9
        assert 16 <= r <= 512 and r % 8 == 0
        assert abs(r - min(max(np.ceil(gamma * ema), 16), 512)) <= 4              # nearest multiple of 8
        assert orc.rank_policy(e + 50, 64, prev, 16, 512, alpha, gamma)[1] >= r    # monotone in the estimate


def test_effective_rank_estimate_of_k_equal_columns_is_k():
    R = np.zeros((7, 10))
    R[:, :4] = np.random.default_rng(0).standard_normal((7, 4))
    R[:, :4] /= np.linalg.norm(R[:, :4], axis=0)
    assert abs(orc.effective_rank_estimate(3.0 * R) - 4.0) < 1e-12                # scale-free, counts equal columns
    R[:, 1] *= 2.0                                                                # p = (1/5, 2/5, 1/5, 1/5)
    want = np.exp(-(3 * 0.2 * np.log(0.2) + 0.4 * np.log(0.4)))
    assert abs(orc.effective_rank_estimate(R) - want) < 1e-12


def test_resize_factor_truncates_and_pads():
    Q = np.arange(12.0).reshape(4, 3)
    assert np.array_equal(orc.resize_factor(Q, 2), Q[:, :2])
    assert np.array_equal(orc.resize_factor(Q, 3), Q)
    pad = -np.ones((4, 2))
    out = orc.resize_factor(Q, 5, pad)
    assert out.shape == (4, 5) and np.array_equal(out[:, :3], Q) and np.array_equal(out[:, 3:], pad)
    with pytest.raises(ValueError):
        orc.resize_factor(Q, 5, np.ones((4, 1)))
