"""orthdion_step_noalloc: the step for callers that may not allocate device memory.

Some callers of this library cannot call cudaMalloc at the point where they step the optimizer:
code inside a stream capture, framework hooks that are forbidden to touch the allocator, processes
with a pre-sized, locked memory pool.  For them the library carries its scratch in a fixed device
array of its own.  This test drives that entry point through the C ABI and checks that it gives
what orthdion_step gives on the same inputs, and what the float64 oracle gives, on two calls in a
row (the second call finds the array full of the first call's leftovers and must not be disturbed
by them).  Allocation is watched from two sides: torch's allocator statistics, and the free device
memory the CUDA runtime reports around the second call (a cudaMalloc inside the library would be
invisible to torch; the first call is left out of that check because the driver loads kernels
lazily on first use).

The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

from oracle import orthdion_oracle as orc
from paper_2605_16341_b200 import binding as od
from paper_2605_16341_b200 import workloads as wl

from parity_util import TOL_CHAIN, TOL_STEP, f64, rel

pytestmark = pytest.mark.gpu


def _problem(m, n, r, dtype, seed):
    g = torch.Generator().manual_seed(seed)
    X = (0.02 * torch.randn(m, n, generator=g)).to(dtype)
    M = 0.3 * torch.randn(m, n, generator=g)
    Gs = [torch.randn(m, n, generator=g).to(dtype) for _ in range(2)]
    Q = wl.random_orthonormal(n, r, g)
    return X, M, Gs, Q


@pytest.mark.parametrize("mode", [od.MODE_ORTH, od.MODE_COLNORM])
@pytest.mark.parametrize("shape,dtype", [((520, 384, 64), torch.bfloat16), ((200, 328, 24), torch.float32)])
def test_noalloc_matches_step_on_two_calls_in_a_row(shape, dtype, mode):
    m, n, r = shape
    X, M, Gs, Q = _problem(m, n, r, dtype, seed=m + n + r)
    h = od.orthdion_create(m, n, r, 0.95, 0.01, 0.0, mode)
    od.orthdion_set_dtypes(h, dtype, dtype)
    assert od.orthdion_workspace_bytes(h) <= od.NOALLOC_SCRATCH_BYTES
    ws = od.alloc_workspace(od.orthdion_workspace_bytes(h))
    Xa, Ma, Qa = X.cuda(), M.cuda(), Q.cuda()           # stepped by orthdion_step
    Xb, Mb, Qb = X.cuda(), M.cuda(), Q.cuda()           # stepped by orthdion_step_noalloc
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    Xo, Mo, Qo = f64(X), f64(M), f64(Q)                 # stepped by the oracle
    omode = orc.ORTH if mode == od.MODE_ORTH else orc.COLNORM
    for t in range(2):
        G = Gs[t].cuda()
        od.orthdion_step(h, Xa, Ma, G, Qa, ws)
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated()
        free_before = torch.cuda.mem_get_info()[0]
        od.orthdion_step_noalloc(h, Xb, Mb, G, Qb, status)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        if t == 1:
            assert torch.cuda.mem_get_info()[0] >= free_before
        assert status.item() == od.orthdion_last_status([h], ws)[0] == 0
        assert rel(f64(Mb), f64(Ma)) <= TOL_STEP
        assert rel(f64(Qb), f64(Qa)) <= TOL_STEP
        assert rel(f64(Xb) - f64(X), f64(Xa) - f64(X)) <= TOL_STEP
        # against the oracle, which carries its own state over the two steps
        ref = orc.step(Xo, Mo, f64(Gs[t]), Qo, eta=0.01, mu=0.95, mode=omode)
        tol = TOL_STEP if t == 0 else TOL_CHAIN
        assert rel(f64(Mb), ref["M"]) <= tol
        assert rel(f64(Qb), ref["Q"]) <= tol
        if dtype == torch.float32:
            assert rel(f64(Xb) - Xo, ref["X"] - Xo) <= tol
            Xo = ref["X"]
        else:
            # bf16 weights: the stored value is the oracle's, rounded, to one bf16 step
            x_ref = orc.round_to_bf16(ref["X"]).astype(np.float64)
            assert np.abs(f64(Xb) - x_ref).max() <= np.abs(x_ref).max() * 2.0 ** -7
            Xo = x_ref
        Mo, Qo = ref["M"], ref["Q"]
    od.orthdion_destroy(h)


def test_noalloc_rejects_plans_beyond_the_built_in_scratch():
    h = od.orthdion_create(8192, 8192, 512, 0.95, 0.01, 0.0, od.MODE_ORTH)
    assert od.orthdion_workspace_bytes(h) > od.NOALLOC_SCRATCH_BYTES
    dummy = torch.zeros(64, device="cuda")
    with pytest.raises(od.OrthDionError) as e:
        od.orthdion_step_noalloc(h, dummy, dummy, dummy, dummy)
    assert e.value.code == -4
    od.orthdion_destroy(h)
