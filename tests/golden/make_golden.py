"""Writes tests/golden/cfg0_oracle_trajectory.txt: per-step fingerprints of the float64
oracle on the cfg0 workload (256 x 512, r = 16, 10 chained steps, both modes).

Calls only `oracle/` and the seeded input generators; run it again only when the oracle's
arithmetic or the input recipe is changed on purpose:

    python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import orthdion_oracle as orc                      # noqa: E402
from paper_2605_16341_b200 import workloads as wl              # noqa: E402


def trajectory(mode, steps=10, seed=0):
    w = wl.workload("cfg0")
    spec = w.matrices[0]
    X, M, Q = wl.initial_state(spec, seed, 0)
    X, M, Q = X.double().numpy(), M.double().numpy(), Q.double().numpy()
    rows = []
    for t in range(steps):
        G = wl.gradient(w, spec, seed, 0, t, None).double().numpy()
        out = orc.step(X, M, G, Q, eta=w.eta, mu=w.mu, wd=w.wd, mode=mode)
        X, M, Q = out["X"], out["M"], out["Q"]
        rows.append((t, np.linalg.norm(X), np.linalg.norm(M), float(np.sum(out["B"] * out["D"])),
                     orc.nu(Q)))
    return rows


def main():
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "cfg0_oracle_trajectory.txt")
    with open(path, "w") as f:
        f.write("# oracle fingerprints on cfg0 (seed 0): mode step |X|_F |M|_F <B,PQ^T> nu\n")
        f.write("# written by tests/golden/make_golden.py from oracle/ only\n")
        for mode, name in ((orc.ORTH, "ORTH"), (orc.COLNORM, "COLNORM")):
            for t, nx, nm, ip, v in trajectory(mode):
                f.write(f"{name} {t} {nx:.15e} {nm:.15e} {ip:.15e} {v:.15e}\n")
    print("wrote", path)


if __name__ == "__main__":
    main()
