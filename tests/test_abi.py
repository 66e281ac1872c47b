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


def test_default_pass_counts_follow_dtypes_and_feedback_form(L):
    """The pass counts of the fused feedback/update product follow the plan until the caller fixes
    them: one fp16 pass each for bf16 weights in the momentum form (|b| <= 0.1 |a|), three bf16
    passes for P R^T in the residual form a = b and for fp32 weights.  The fp16 form shows in the
    workspace: P, R and Q then carry a third operand plane (2 bytes per entry)."""
    m, n, r = 512, 768, 64
    planes = 2 * (m + 2 * n) * r                      # bytes of the fp16 planes (rows are multiples of 128)

    def plan():
        h = ctypes.c_void_p()
        assert L.orthdion_create(ctypes.byref(h), m, n, r, ctypes.c_float(0.95), ctypes.c_float(0.01),
                                 ctypes.c_float(0.0), 0) == 0
        return h

    h = plan()
    fused = L.orthdion_workspace_bytes(h)             # defaults: bf16 weights, momentum form (a = 1, b = 0.05): 1, 1
    assert L.orthdion_set_dtypes(h, 0, 0) == 0        # fp32 weights and gradients: 3, 3
    base = L.orthdion_workspace_bytes(h)
    assert fused - base == planes
    assert L.orthdion_set_dtypes(h, 1, 1) == 0
    assert L.orthdion_workspace_bytes(h) == fused
    assert L.orthdion_set_ef(h, ctypes.c_float(0.95), ctypes.c_float(0.95)) == 0      # residual form: 3, 1
    assert L.orthdion_workspace_bytes(h) == base
    assert L.orthdion_set_ef(h, ctypes.c_float(1.0), ctypes.c_float(0.05)) == 0
    assert L.orthdion_workspace_bytes(h) == fused
    assert L.orthdion_set_passes(h, 2, 3) == 0        # fixed by the caller: stays through later changes
    assert L.orthdion_workspace_bytes(h) == base
    assert L.orthdion_set_dtypes(h, 1, 1) == 0
    assert L.orthdion_workspace_bytes(h) == base
    assert L.orthdion_set_passes(h, 2, 0) == 0        # handed back to the rule
    assert L.orthdion_workspace_bytes(h) == fused
    assert L.orthdion_set_dtypes(h, 0, 1) == 0        # fp32 weights again
    assert L.orthdion_workspace_bytes(h) == base
    assert L.orthdion_set_passes(h, 2, 1) == 0 and L.orthdion_set_passes(h, 3, 1) == 0
    assert L.orthdion_workspace_bytes(h) == fused     # asked for explicitly
    assert L.orthdion_destroy(h) == 0
