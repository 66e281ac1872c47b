"""The C-ABI library loads without a GPU, exports every symbol the header declares and
rejects bad arguments on the host."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2605_16341_b200 import binding
    if not os.path.exists(binding.LIB_PATH):
        binding.build_library()
    return binding.lib()


def declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(orthdion_[a-z_0-9]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported(L):
    from paper_2605_16341_b200 import binding
    names = declared_symbols()
    assert len(names) >= 15
    for n in names:
        assert hasattr(L, n), n
    assert set(binding.EXPORTED) == names


def test_host_argument_checks(L):
    from paper_2605_16341_b200 import binding as b
    h = ctypes.c_void_p()
    assert L.orthdion_create(ctypes.byref(h), 64, 64, 0, 0.95, 0.01, 0.0, 0) == -2      # r < 1
    assert L.orthdion_create(ctypes.byref(h), 64, 32, 48, 0.95, 0.01, 0.0, 0) == -2     # r > min(m, n)
    assert L.orthdion_create(ctypes.byref(h), 64, 64, 16, 0.95, 0.01, 0.0, 7) == -1     # bad mode
    assert L.orthdion_create(None, 64, 64, 16, 0.95, 0.01, 0.0, 0) == -3
    assert L.orthdion_create(ctypes.byref(h), 256, 512, 16, 0.95, 0.01, 0.0, 0) == 0
    assert L.orthdion_set_dtypes(h, 5, 0) == -1
    assert L.orthdion_set_dtypes(h, 0, 0) == 0
    assert L.orthdion_set_engine(h, 9) == -1
    assert L.orthdion_set_passes(h, 0, 2) == -1
    assert L.orthdion_set_passes(h, 0, 3) == 0
    ws = L.orthdion_workspace_bytes(h)
    assert ws >= 4 * (256 + 512) * 16
    # null pointers are rejected before anything is enqueued
    assert L.orthdion_step(h, None, None, None, None, None, 0, None) == -3
    assert L.orthdion_set_concurrency(0) == -1 and L.orthdion_set_concurrency(9) == -1
    assert L.orthdion_set_concurrency(4) == 0   # the default
    assert L.orthdion_destroy(h) == 0
    assert L.orthdion_destroy(h) == -1          # stale handle is recognised
    assert b.orthdion_version().startswith("orthdion")


def test_grouped_workspace_is_at_least_the_sum_of_factors(L):
    from paper_2605_16341_b200 import binding as b
    hs = [b.orthdion_create(128, 256, 16, 0.95, 0.01, 0.0, 0), b.orthdion_create(256, 128, 32, 0.95, 0.01, 0.0, 1)]
    need = b.orthdion_workspace_bytes_grouped(hs)
    assert need >= 4 * ((128 + 256) * 16 + (256 + 128) * 32)
    assert need >= max(b.orthdion_workspace_bytes(h) for h in hs)
    for h in hs:
        b.orthdion_destroy(h)
