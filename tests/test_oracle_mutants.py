"""The pins must be sharp: a plausible mistake planted in (a copy of) the oracle has to be
caught by the battery below.  Mistakes are planted in the oracle's source text, on the CPU."""
import inspect
import types

import numpy as np
import pytest

from oracle import orthdion_oracle as orc


def rand_orth(g, n, r):
    q, t = np.linalg.qr(g.standard_normal((n, r)))
    return q * np.sign(np.diag(t))[None, :]


def battery(mod):
    """Closed-form / identity checks that use only the module's public functions.
    Raises AssertionError (or any exception) when the module is wrong."""
    g = np.random.default_rng(123)
    m, n, r = 14, 22, 4
    U, V = rand_orth(g, m, r), rand_orth(g, n, r)
    s = np.array([4.0, 3.0, 2.0, 1.0])
    Blow = U @ np.diag(s) @ V.T
    G = g.standard_normal((m, n))
    M = Blow - G
    X0 = g.standard_normal((m, n))
    mu, eta = 0.9, 0.5
    # (1) aligned case: everything is known in closed form
    out = mod.step(X0, M, G, V, eta=eta, mu=mu, mode=mod.ORTH)
    assert np.allclose(out["P"], U, atol=1e-10)
    assert np.allclose(out["Q"], V, atol=1e-10)
    assert np.allclose(out["T1"], np.diag(s), atol=1e-10) and np.allclose(out["T2"], np.diag(s), atol=1e-10)
    assert np.allclose(out["X"], X0 - eta * U @ V.T, atol=1e-10)
    assert np.allclose(out["M"], mu * Blow, atol=1e-10)
    outp = mod.step(X0, M, G, V, eta=eta, ef=(0.6, 0.6), mode=mod.ORTH)
    assert np.abs(outp["M"]).max() < 1e-10
    # (2) generic buffer: projection identities and LAPACK factors
    M2 = g.standard_normal((m, n))
    Qp = rand_orth(g, n, r)
    for mode in (mod.ORTH, mod.COLNORM):
        o = mod.step(X0, M2, G, Qp, eta=eta, mu=mu, mode=mode)
        B = M2 + G
        q, t = np.linalg.qr(B @ Qp)
        q = q * np.sign(np.diag(t))[None, :]
        assert np.allclose(o["P"], q, atol=1e-10)
        assert np.allclose(o["P"] @ o["R"].T, q @ q.T @ B, atol=1e-10)
        assert np.allclose(B - o["M"], (1 - mu) * q @ q.T @ B, atol=1e-10)
        if mode == mod.ORTH:
            q2, t2 = np.linalg.qr(B.T @ q)
            q2 = q2 * np.sign(np.diag(t2))[None, :]
            assert np.allclose(o["Q"], q2, atol=1e-10)
            assert np.allclose((X0 - o["X"]) / eta, q @ q2.T, atol=1e-10)
        else:
            W = B.T @ q
            assert np.allclose(np.linalg.norm(o["Q"], axis=0), 1.0, atol=1e-12)
            assert np.allclose(o["Q"] * np.linalg.norm(W, axis=0)[None, :], W, atol=1e-10)
    # (3) decay / scale algebra
    o3 = mod.step(X0, M2, G, Qp, eta=eta, mu=mu, wd=0.2, scale=3.0)
    o1 = mod.step(X0, M2, G, Qp, eta=eta, mu=mu)
    assert np.allclose(o3["X"], (1 - eta * 0.2) * X0 + 3.0 * (o1["X"] - X0), atol=1e-10)


def test_battery_passes_on_the_oracle():
    battery(orc)


MUTATIONS = [
    ("B = M + G      ", "B = M - G      "),
    ("Y = B @ Qp", "Y = M @ Qp"),
    ("R = B.T @ P ", "R = G.T @ P "),
    ("Mn = a * B - b * (P @ R.T)", "Mn = a * B + b * (P @ R.T)"),
    ("Mn = a * B - b * (P @ R.T)", "Mn = a * M - b * (P @ R.T)"),
    ("Mn = a * B - b * (P @ R.T)", "Mn = a * B - b * (P @ R.T).T @ np.eye(B.shape[0], B.shape[1])"),
    ("(1.0, 1.0 - float(mu))", "(1.0, float(mu))"),
    ("Xn = (1.0 - eta * wd) * X - (eta * scale) * D", "Xn = (1.0 - eta * wd) * X + (eta * scale) * D"),
    ("Xn = (1.0 - eta * wd) * X - (eta * scale) * D", "Xn = (1.0 - eta * wd) * (X - (eta * scale) * D)"),
    ("Xn = (1.0 - eta * wd) * X - (eta * scale) * D", "Xn = (1.0 - wd) * X - (eta * scale) * D"),
    ("D = P @ Q.T ", "D = P @ R.T "),
    ("Q, T2 = thin_qr_pos(R) ", "Q, T2 = thin_qr_pos(R * np.arange(1, R.shape[1] + 1)[None, ::-1] @ np.eye(R.shape[1])[::-1]) "),
    ("d = np.where(np.diag(T) < 0.0, -1.0, 1.0)", "d = np.ones(r)"),
    ("tau[j] = 2.0 / vnorm2", "tau[j] = 1.0 / vnorm2"),
    ("norms = np.sqrt(np.sum(R * R, axis=0))", "norms = np.sum(np.abs(R), axis=0)"),
    ("norms = np.sqrt(np.sum(R * R, axis=0))", "norms = np.sqrt(np.sum(R * R, axis=1))[: R.shape[1]]"),
]


@pytest.mark.parametrize("idx", range(len(MUTATIONS)))
def test_planted_mistake_is_caught(idx):
    old, new = MUTATIONS[idx]
    src = inspect.getsource(orc)
    assert src.count(old) == 1, f"mutation anchor not unique: {old!r}"
    mutant = types.ModuleType("oracle_mutant")
    exec(compile(src.replace(old, new), "oracle_mutant", "exec"), mutant.__dict__)
    with pytest.raises(Exception):
        battery(mutant)
