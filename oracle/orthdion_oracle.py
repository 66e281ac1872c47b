"""Float64 CPU oracle for one Orth-Dion / Stripped-Dion optimizer step.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what the
optimizer step computes, written from the paper.  It shares no code with the CUDA
path and must never be imported by the product library; only the test-suite, the
smoke check and the benchmark's CPU-baseline leg may call it.

Notation.  The paper (Algorithm 1) writes the buffer as M_t = G_t + R_t, the factors
as U_t, W_t, V_t.  This code uses the letters of the library's C interface:

    library      paper (Algorithm 1)
    G            G_t        gradient                         m x n
    M            R_t        error-feedback residual (state)  m x n
    B = M + G    M_t        buffer                           m x n
    Qp, Q        V_{t-1}, V_t   right factor (state)         n x r
    P            U_t        left factor                      m x r
    R            W_t        un-normalised right factor       n x r

Everything is float64; callers widen stored bf16/fp32 values exactly before calling.
numpy's matmul is used as a library primitive for the matrix products; the thin QR is
a Householder factorisation written out below.

Parity pins: every function here is pinned by tests/test_oracle_pins.py against
identities the paper states (Lemma 4.1, Prop. 3.1, Lemma 4.2, Lemma 4.3, the
error-feedback step of Algorithm 1), closed forms, LAPACK QR / SVD, and the worked
numbers the paper prints.  The weight-decay and scale factors of `step` have no
equation in the paper: for wd != 0 or scale != 1 the parity is UNPINNED beyond the
algebraic identity X' - (1 - eta*wd) X = -eta*scale*P Q^T.
"""
from __future__ import annotations

import numpy as np

ORTH = 0      # Algorithm 1, normalisation step, Orth-Dion branch: QR of the right factor
COLNORM = 1   # Algorithm 1, normalisation step, Dion branch: unit-length columns

STATUS_OK = 0
STATUS_RANK_DEFICIENT = 1   # a triangular factor has a (relatively) vanishing pivot
STATUS_ZERO_COLUMN = 2      # COLNORM met a zero column of R

RANK_TOL = 1e-12


# ----------------------------------------------------------------------------------
# orth(.) : thin QR with positive diagonal  (Section 2, "orth(W_t) (QR)"; Alg. 1, left-factor and normalisation steps)
# ----------------------------------------------------------------------------------
def thin_qr_pos(Y: np.ndarray):
    """Thin QR factorisation Y = F T by Householder reflections, diag(T) > 0.

    Y is k x r with k >= r.  Returns (F, T): F k x r with orthonormal columns, T r x r
    upper triangular.  For full column rank this factorisation is unique, which is the
    meaning given to the paper's `orth(.)`.  (The paper only says "QR"; the positive
    diagonal is the convention that makes the result unique.)
    """
    Y = np.array(Y, dtype=np.float64, copy=True)
    k, r = Y.shape
    if k < r:
        raise ValueError("thin_qr_pos needs rows >= columns")
    A = Y                       # overwritten by the triangular factor
    V = np.zeros((k, r))        # Householder vectors, column j lives in rows j..k-1
    tau = np.zeros(r)
    for j in range(r):
        x = A[j:, j]
        normx = np.sqrt(np.dot(x, x))
        if normx == 0.0:
            tau[j] = 0.0
            continue
        # reflect x onto -sign(x0) * |x| e_1 (the cancellation-free choice)
        alpha = -normx if x[0] >= 0.0 else normx
        v = x.copy()
        v[0] -= alpha
        vnorm2 = np.dot(v, v)
        tau[j] = 2.0 / vnorm2
        V[j:, j] = v
        # apply H = I - tau v v^T to the trailing columns
        w = tau[j] * (v @ A[j:, j:])
        A[j:, j:] -= np.outer(v, w)
    T = np.triu(A[:r, :])
    # accumulate F = H_0 H_1 ... H_{r-1} [I_r; 0]
    F = np.zeros((k, r))
    F[:r, :r] = np.eye(r)
    for j in range(r - 1, -1, -1):
        if tau[j] == 0.0:
            continue
        v = V[j:, j]
        w = tau[j] * (v @ F[j:, :])
        F[j:, :] -= np.outer(v, w)
    # flip signs so that diag(T) > 0:  Y = (F D)(D T), D = diag(+-1)
    d = np.where(np.diag(T) < 0.0, -1.0, 1.0)
    F *= d[None, :]
    T *= d[:, None]
    return F, T


def col_norm(R: np.ndarray):
    """ColNorm(W): every column scaled to unit Euclidean length (Section 3; Alg. 1, normalisation step, Dion).

    Returns (Q, norms).  A zero column stays zero (its norm is reported as 0)."""
    R = np.asarray(R, dtype=np.float64)
    norms = np.sqrt(np.sum(R * R, axis=0))
    safe = np.where(norms > 0.0, norms, 1.0)
    return R / safe[None, :], norms


# ----------------------------------------------------------------------------------
# One optimizer step (Algorithm 1; appendix algorithms "Stripped Dion" / "Orth-Dion")
# ----------------------------------------------------------------------------------
def step(X, M, G, Qp, *, eta, mode=ORTH, mu=None, ef=None, wd=0.0, scale=1.0):
    """One step.  Returns a dict with X, M, Q (the new state) and P, R, T1, T2, B, status.

    Error feedback: M' = a*B - b*P R^T.
      * `mu` given  ->  (a, b) = (1, 1 - mu)        the momentum form M <- B - (1-mu) P R^T
      * `ef=(a,b)`  ->  explicit; the paper's error-feedback step, R_{t+1} = beta (M_t - U_t U_t^T M_t),
                        is ef=(beta, beta).
    Weight update: X' = (1 - eta*wd) X - eta*scale * P Q^T   (Alg. 1, update step, has wd=0, scale=1).
    If a triangular factor is numerically singular the state is returned unchanged and
    status = STATUS_RANK_DEFICIENT (the paper assumes full rank)."""
    if (mu is None) == (ef is None):
        raise ValueError("give exactly one of mu, ef")
    a, b = (1.0, 1.0 - float(mu)) if ef is None else (float(ef[0]), float(ef[1]))
    X = np.asarray(X, dtype=np.float64)
    M = np.asarray(M, dtype=np.float64)
    G = np.asarray(G, dtype=np.float64)
    Qp = np.asarray(Qp, dtype=np.float64)

    B = M + G                                   # Alg. 1, buffer step
    Y = B @ Qp
    P, T1 = thin_qr_pos(Y)                      # Alg. 1, left-factor step
    status = STATUS_OK
    if _deficient(T1):
        status = STATUS_RANK_DEFICIENT
    R = B.T @ P                                 # Alg. 1, right-factor step (un-normalised)
    T2 = None
    colnorms = None
    if status == STATUS_OK:
        if mode == ORTH:
            Q, T2 = thin_qr_pos(R)              # Alg. 1, normalisation step: Orth-Dion
            if _deficient(T2):
                status = STATUS_RANK_DEFICIENT
        elif mode == COLNORM:
            Q, colnorms = col_norm(R)           # Alg. 1, normalisation step: Dion
            if np.any(colnorms == 0.0):
                status = STATUS_ZERO_COLUMN
        else:
            raise ValueError("mode")
    if status == STATUS_RANK_DEFICIENT:
        return dict(X=X.copy(), M=M.copy(), Q=Qp.copy(), P=P, R=R, T1=T1, T2=T2, B=B,
                    Y=Y, colnorms=colnorms, status=status)
    D = P @ Q.T                                 # Alg. 1, update step: direction
    Xn = (1.0 - eta * wd) * X - (eta * scale) * D   # Alg. 1, update step
    Mn = a * B - b * (P @ R.T)                  # Alg. 1, error-feedback step (P R^T = P P^T B)
    return dict(X=Xn, M=Mn, Q=Q, P=P, R=R, T1=T1, T2=T2, B=B, Y=Y, D=D,
                colnorms=colnorms, status=status)


def _deficient(T):
    d = np.abs(np.diag(T))
    return bool(d.min() <= RANK_TOL * d.max())


# ----------------------------------------------------------------------------------
# Norms and per-iteration quantities (appendix "Norms and Key Quantities")
# ----------------------------------------------------------------------------------
def singular_values(A):
    return np.linalg.svd(np.asarray(A, dtype=np.float64), compute_uv=False)


def ky_fan(A, r):
    """Ky Fan r-norm: sum of the r largest singular values."""
    return float(np.sum(singular_values(A)[:r]))


def dual_norm(A, r):
    """Dual of the Ky Fan r-norm, appendix form: max{sigma_1, nuclear/r}."""
    s = singular_values(A)
    return float(max(s[0], np.sum(s) / r))


def dual_norm_body_formula(A, r):
    """The body-text formula max{sigma_1, frobenius/sqrt(r)}, which the appendix footnote
    corrects; kept only so the printed counter-example can be reproduced."""
    s = singular_values(A)
    return float(max(s[0], np.sqrt(np.sum(s * s)) / np.sqrt(r)))


def nu(Q):
    """nu_t = ||Q||_op, the dual-norm factor of P Q^T when P has orthonormal columns
    (Proposition 3.1)."""
    return float(singular_values(Q)[0])


def defect(B, P, Q, r):
    """Oracle defect delta_t = ||B||_{KF,r} - <B, P Q^T>  (Eq. 1)."""
    return ky_fan(B, r) - float(np.sum(B * (P @ Q.T)))


def rank_r_polar(A, r):
    """Rank-r polar factor U_r V_r^T from the truncated SVD (Section 2)."""
    U, s, Vt = np.linalg.svd(np.asarray(A, dtype=np.float64), full_matrices=False)
    return U[:, :r] @ Vt[:r, :]


def effective_rank_estimate(R):
    """exp(-sum p log p) with p_i proportional to the column norms of R (Section 6)."""
    s = np.sqrt(np.sum(np.asarray(R, dtype=np.float64) ** 2, axis=0))
    p = s / np.sum(s)
    p = p[p > 0]
    return float(np.exp(-np.sum(p * np.log(p))))


# ----------------------------------------------------------------------------------
# Ada-Orth-Dion rank selection (appendix algorithm "Ada-Orth-Dion Rank Selection")
# ----------------------------------------------------------------------------------
def rank_policy(e_t, r_t, ema_prev, r_min, r_max, alpha, gamma, multiple=8):
    """One application of the rank-selection rule.  Returns (ema_t, r_next).

        ema_t    = alpha * e_t + (1 - alpha) * ema_prev
        r_target = ceil(gamma * ema_t)
        r_next   = clip(r_target, r_min, r_max), rounded to a multiple of `multiple`

    Readings where the paper is silent: "rounded" is to the nearest multiple, a tie going up;
    r_min and r_max are multiples of `multiple` themselves, so rounding cannot leave the bounds;
    all arithmetic in float64.  r_t is carried only because the rule is stated with it (the
    resize happens when r_next != r_t)."""
    if r_min % multiple or r_max % multiple or r_min < multiple or r_max < r_min:
        raise ValueError("bounds must be positive multiples of `multiple`")
    ema_t = float(alpha) * float(e_t) + (1.0 - float(alpha)) * float(ema_prev)
    r_target = int(np.ceil(float(gamma) * ema_t))
    clipped = min(max(r_target, r_min), r_max)
    r_next = int(np.floor(clipped / multiple + 0.5)) * multiple
    return ema_t, r_next


def resize_factor(Q, r_new, pad=None):
    """Resize the warm-start factor to r_new columns: keep the leading columns (truncate), or
    append the given columns (pad).  The paper only says "truncate or pad"; the reading taken is
    that the new columns are supplied by the caller (any columns that keep B Q of full rank will
    do for the power iteration; the tests draw them N(0, 1/n))."""
    Q = np.asarray(Q, dtype=np.float64)
    n, r = Q.shape
    if r_new <= r:
        return Q[:, :r_new].copy()
    pad = np.asarray(pad, dtype=np.float64)
    if pad.shape != (n, r_new - r):
        raise ValueError("pad must be n x (r_new - r)")
    return np.concatenate([Q, pad], axis=1)


# ----------------------------------------------------------------------------------
# Storage rounding (bf16 round-to-nearest-even), for comparing stored weights
# ----------------------------------------------------------------------------------
def round_to_bf16(x):
    """Round float64/float32 values to the nearest bfloat16 (ties to even); returns float32.

    Done on the float32 bit pattern after a correctly-rounded float64->float32 conversion
    would double-round, so the rounding is carried out on the float64 value directly."""
    x = np.asarray(x, dtype=np.float64)
    out = np.empty(x.shape, dtype=np.float32)
    flat = x.ravel()
    m, e = np.frexp(flat)                 # x = m * 2^e, 0.5 <= |m| < 1
    # bf16 keeps 8 significant bits: quantum = 2^(e-8); subnormal range not needed here
    q = np.ldexp(1.0, e - 8)
    y = np.round(flat / q) * q            # np.round is ties-to-even
    y = np.where(flat == 0.0, 0.0, y)
    out.ravel()[:] = y.astype(np.float32)
    return out
