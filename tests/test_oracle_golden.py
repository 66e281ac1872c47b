"""The oracle's cfg0 trajectory must not drift from the committed fingerprints."""
import importlib.util
import os

import numpy as np

from oracle import orthdion_oracle as orc

HERE = os.path.dirname(os.path.abspath(__file__))


def _load_maker():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_cfg0_trajectory_matches_committed_fingerprints():
    stored = {}
    with open(os.path.join(HERE, "golden", "cfg0_oracle_trajectory.txt")) as f:
        for line in f:
            if line.startswith("#"):
                continue
            name, t, *vals = line.split()
            stored[(name, int(t))] = np.array([float(v) for v in vals])
    maker = _load_maker()
    for mode, name in ((orc.ORTH, "ORTH"), (orc.COLNORM, "COLNORM")):
        for t, *vals in maker.trajectory(mode):
            assert np.allclose(np.array(vals), stored[(name, t)], rtol=1e-9), (name, t)
    # Lemma 4.3: the residual norms of the two modes coincide step by step
    for t in range(10):
        assert abs(stored[("ORTH", t)][1] - stored[("COLNORM", t)][1]) < 1e-9 * stored[("ORTH", t)][1]
        assert abs(stored[("ORTH", t)][3] - 1.0) < 1e-12 and stored[("COLNORM", t)][3] > 1.0
