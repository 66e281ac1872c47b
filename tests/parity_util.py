"""Helpers for the GPU-vs-oracle parity tests: run the CUDA library and the float64 oracle on the
same seeded tensors and compare the quantities the tolerances are stated on."""
from __future__ import annotations

import numpy as np
import torch

from oracle import orthdion_oracle as orc
from paper_2605_16341_b200 import binding as od
from paper_2605_16341_b200 import workloads as wl

TOL_STEP = 1e-4       # ||dX_gpu - dX_or||_F / ||dX_or||_F after one step from identical state
TOL_CHAIN = 1e-3      # the same after 10 chained steps
TOL_ORTHO = 1e-5      # max |Q^T Q - I|
# Largest element-wise error, relative to the largest element of the reference.  An error of
# relative Frobenius size e spread evenly over N entries has its largest entry near
# sqrt(2 ln N) ~ 6 times the error's root mean square, and the reference's largest entry is
# about as many of its own root mean squares away, so a result inside TOL_STEP has a largest
# error of about TOL_STEP of the largest reference entry (twice that is allowed); a localised fault (one wrong tile, one
# dropped depth block) exceeds this while barely moving the Frobenius norm.
TOL_MAXABS = 2e-4


def poisoned_workspace(nbytes: int) -> torch.Tensor:
    """A workspace whose every byte is 0x7f (floats of 3.4e38, bf16/fp16 values far out of range):
    the step must not depend on what the workspace held before, and anything it reads without
    having written it first shows up as a wrong result instead of passing on zeroed memory."""
    ws = od.alloc_workspace(nbytes)
    ws.fill_(0x7F)
    return ws


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().double().cpu().numpy()


def rel(a, b):
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def rel_max(a, b):
    """Largest element-wise difference over the largest reference element."""
    return float(np.abs(a - b).max() / max(np.abs(b).max(), 1e-300))


def bf16_steps_apart(x_dev, x_ref32, x_before, x_ref_before, slack):
    """Stored bf16 weights after a step against reference values that are already rounded to bf16.

    bf16 accumulation of updates that are smaller than the spacing is chaotic: an entry whose
    exact new value sits on a rounding boundary may go either way (about one entry in a thousand
    per step), and from then on the two copies can sit in different binades, where the same later
    updates round away in one and are applied in the other.  So the two trajectories are compared
    where that has not happened yet: on the entries whose value BEFORE the step was identical on
    both sides, the values after the step may differ by one bf16 step (measured at the larger of the
    old and the new magnitude) beyond `slack`, the per-entry bound on the error of the single-pass
    product that feeds the update.  Returns (largest such distance in bf16 steps, fraction of all
    entries that differ after the step)."""
    a = x_dev.detach().float().cpu().numpy().astype(np.float64)
    b = np.asarray(x_ref32, dtype=np.float64)
    a0 = x_before.detach().float().cpu().numpy().astype(np.float64)
    b0 = np.asarray(x_ref_before, dtype=np.float64)
    mag = np.maximum(np.maximum(np.abs(a), np.abs(b)), np.abs(a0))
    _, e = np.frexp(np.maximum(mag, 2.0 ** -120))          # mag = f * 2^e, 0.5 <= f < 1
    step = np.ldexp(1.0, e - 8)                            # bf16 keeps 8 significant bits
    d = np.abs(a - b)
    dist = np.where(a0 == b0, np.maximum(d - slack, 0.0) / step, 0.0)
    return float(dist.max()), float(np.count_nonzero(d) / d.size)


def single_pass_slack(P, Q, eta, scale=1.0, bits=8):
    """Per-entry bound on the error of eta*scale*(P Q^T) when the product is one tensor-core pass
    with operands rounded to `bits` significant bits: 2^-bits * sum_k |p_ik q_jk|."""
    return eta * scale * (np.abs(f64(P)) @ np.abs(f64(Q)).T) * 2.0 ** -bits


class GpuMatrix:
    """One matrix on the GPU with its plan and workspace."""

    def __init__(self, spec, X, M, Q, *, mu, eta, wd=0.0, mode=od.MODE_ORTH, engine=None, ef=None,
                 scale=None, passes=None):
        self.spec = spec
        self.h = od.orthdion_create(spec.m, spec.n, spec.r, mu, eta, wd, mode)
        od.orthdion_set_dtypes(self.h, spec.x_dtype, spec.g_dtype)
        if engine is not None:
            od.orthdion_set_engine(self.h, engine)
        if ef is not None:
            od.orthdion_set_ef(self.h, *ef)
        if scale is not None:
            od.orthdion_set_scale(self.h, scale)
        for k, v in (passes or {}).items():
            od.orthdion_set_passes(self.h, k, v)
        self.X, self.M, self.Q = X.cuda().contiguous(), M.cuda().contiguous(), Q.cuda().contiguous()
        self.ws = poisoned_workspace(od.orthdion_workspace_bytes(self.h))
        self.eta, self.wd, self.scale = eta, wd, 1.0 if scale is None else scale

    def step(self, G):
        self.G = G.cuda().contiguous()
        od.orthdion_step(self.h, self.X, self.M, self.G, self.Q, self.ws)
        torch.cuda.synchronize()

    def factors(self):
        return od.orthdion_get_factors([self.h], 0, self.ws, (self.spec.m, self.spec.n, self.spec.r))

    def status(self):
        return od.orthdion_last_status([self.h], self.ws)[0]

    def close(self):
        od.orthdion_destroy(self.h)


def delta_x_from_factors(P, Q, X_before, eta, wd, scale):
    """dX formed in float64 from the GPU's fp32 factors (what the weight update applies before
    the storage rounding of X)."""
    return -eta * scale * (f64(P) @ f64(Q).T) - eta * wd * f64(X_before)


def check_bf16_rounding(X_after, X_before, P, Q, eta, wd, scale, sample=4096, seed=0):
    """Stored bf16 weights against the float64 value of c*X - d*(P Q^T) formed from the GPU's own
    fp32 factors, on sampled entries.  Returns the largest excess over the allowed deviation in
    bf16 ulps: one ulp for the storage rounding plus the bound 2^-8 * d * sum_k |p_ik q_jk| on the
    single-pass bf16 product that feeds a bf16 weight matrix (each operand rounded to 8 bits)."""
    g = np.random.default_rng(seed)
    m, n = X_after.shape
    ii, jj = g.integers(0, m, sample), g.integers(0, n, sample)
    Pn, Qn = f64(P), f64(Q)
    d = np.einsum("ik,ik->i", Pn[ii], Qn[jj])
    dabs = np.einsum("ik,ik->i", np.abs(Pn[ii]), np.abs(Qn[jj]))
    xb = f64(X_before)[ii, jj]
    exact = (1.0 - eta * wd) * xb - eta * scale * d
    got = f64(X_after)[ii, jj]
    ulp = np.maximum(np.abs(exact), 2.0 ** -126) * 2.0 ** -7
    slack = eta * scale * dabs * 2.0 ** -8
    return float(np.max((np.abs(got - exact) - slack) / ulp))


def oracle_mode(mode):
    return orc.ORTH if mode == od.MODE_ORTH else orc.COLNORM
