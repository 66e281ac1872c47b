"""ctypes binding of liborthdion.so: same entry points as include/orthdion.h, argument
marshalling only.  Tensors are torch CUDA tensors (torch supplies device memory and streams);
every step of the optimizer path runs in the library's own kernels.

The shared library is built in-tree by `__graft_entry__.build()` (or `build_library()` below).
If it is missing, any call raises: there is no CPU or PyTorch fallback.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liborthdion.so")
CSRC = os.path.join(_HERE, "csrc")

MODE_ORTH, MODE_COLNORM = 0, 1
DTYPE_F32, DTYPE_BF16 = 0, 1
ENGINE_TENSOR, ENGINE_SIMT = 0, 1

STATUS_SHIFTED_LEFT, STATUS_SHIFTED_RIGHT, STATUS_RANK_DEFICIENT = 1, 2, 4
STATUS_NONFINITE, STATUS_ZERO_COLUMN, STATUS_WAIT_LIMIT = 8, 16, 32

ERRORS = {0: "OK", -1: "INVALID_ARG", -2: "RANK", -3: "NULL", -4: "WORKSPACE", -5: "CUDA", -6: "ALIGNMENT"}

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "--shared", "-Xcompiler", "-fPIC"]


class OrthDionError(RuntimeError):
    def __init__(self, code, where):
        super().__init__(f"{where} failed: {ERRORS.get(code, code)} ({code})")
        self.code = code


def build_library(verbose: bool = False) -> str:
    """Compile csrc/orthdion.cu for sm_100a into liborthdion.so next to this file."""
    src = os.path.join(CSRC, "orthdion.cu")
    cmd = ["nvcc", *NVCC_FLAGS, "-o", LIB_PATH, src]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.run(cmd, check=True)
    return LIB_PATH


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            f"{LIB_PATH} is missing: build it with __graft_entry__.build(); there is no fallback path")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, f32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float, ctypes.c_size_t
    pvp = ctypes.POINTER(vp)
    L.orthdion_create.argtypes = [pvp, i64, i64, i32, f32, f32, f32, i32]
    L.orthdion_destroy.argtypes = [vp]
    L.orthdion_set_dtypes.argtypes = [vp, i32, i32]
    L.orthdion_set_lr.argtypes = [vp, f32]
    L.orthdion_set_scale.argtypes = [vp, f32]
    L.orthdion_set_ef.argtypes = [vp, f32, f32]
    L.orthdion_set_engine.argtypes = [vp, i32]
    L.orthdion_set_passes.argtypes = [vp, i32, i32]
    L.orthdion_workspace_bytes.argtypes = [vp]
    L.orthdion_workspace_bytes.restype = sz
    L.orthdion_workspace_bytes_grouped.argtypes = [pvp, i32]
    L.orthdion_workspace_bytes_grouped.restype = sz
    L.orthdion_step.argtypes = [vp, vp, vp, vp, vp, vp, sz, vp]
    L.orthdion_step_grouped.argtypes = [pvp, i32, pvp, pvp, pvp, pvp, vp, sz, vp]
    L.orthdion_step_noalloc.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    L.orthdion_get_factors.argtypes = [pvp, i32, i32, vp, pvp, pvp]
    L.orthdion_last_status.argtypes = [pvp, i32, vp, vp, ctypes.POINTER(i32)]
    L.orthdion_set_concurrency.argtypes = [i32]
    L.orthdion_shard_phase.argtypes = [vp, i32, vp, vp, vp, vp, vp, sz, vp]
    L.orthdion_shard_reduce_buffer.argtypes = [vp, i32, vp, pvp, ctypes.POINTER(i64)]
    L.orthdion_set_diagnostics.argtypes = [vp, i32]
    L.orthdion_last_diagnostics.argtypes = [pvp, i32, vp, vp, ctypes.POINTER(ctypes.c_float)]
    dbl = ctypes.c_double
    L.orthdion_rank_policy.argtypes = [dbl, i32, dbl, i32, i32, dbl, dbl, i32, ctypes.POINTER(dbl),
                                       ctypes.POINTER(i32)]
    L.orthdion_resize_factor.argtypes = [vp, i64, i32, vp, i32, vp, vp]
    L.orthdion_version.restype = ctypes.c_char_p
    L.orthdion_launch_count.restype = i64
    L.orthdion_profile_begin.argtypes = [i32]
    L.orthdion_profile_begin.restype = i32
    L.orthdion_profile_end.argtypes = [i32, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(i64)]
    L.orthdion_profile_end.restype = i32
    L.orthdion_stage_count.restype = i32
    L.orthdion_stage_name.argtypes = [i32]
    L.orthdion_stage_name.restype = ctypes.c_char_p
    for name in ("create", "destroy", "set_dtypes", "set_lr", "set_scale", "set_ef", "set_engine",
                 "set_passes", "step", "step_grouped", "step_noalloc", "get_factors", "last_status",
                 "set_diagnostics", "last_diagnostics", "rank_policy", "resize_factor", "set_concurrency", "shard_phase", "shard_reduce_buffer"):
        getattr(L, "orthdion_" + name).restype = i32
    _lib = L
    return L


EXPORTED = ["orthdion_create", "orthdion_destroy", "orthdion_set_dtypes", "orthdion_set_lr",
            "orthdion_set_scale", "orthdion_set_ef", "orthdion_set_engine", "orthdion_set_passes",
            "orthdion_workspace_bytes", "orthdion_workspace_bytes_grouped", "orthdion_step",
            "orthdion_step_grouped", "orthdion_step_noalloc", "orthdion_get_factors", "orthdion_last_status",
            "orthdion_set_concurrency", "orthdion_shard_phase", "orthdion_shard_reduce_buffer", "orthdion_set_diagnostics", "orthdion_last_diagnostics", "orthdion_rank_policy",
            "orthdion_resize_factor", "orthdion_version",
            "orthdion_launch_count", "orthdion_profile_begin", "orthdion_profile_end", "orthdion_stage_count",
            "orthdion_stage_name"]


def _check(code, where):
    if code != 0:
        raise OrthDionError(code, where)


def _dt(t: torch.dtype) -> int:
    if t == torch.float32:
        return DTYPE_F32
    if t == torch.bfloat16:
        return DTYPE_BF16
    raise TypeError(f"unsupported dtype {t}")


def _stream_ptr(stream) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


# ---------------------------------------------------------------------------------------------
def orthdion_create(m, n, r, mu, eta, wd, mode) -> int:
    h = ctypes.c_void_p()
    _check(lib().orthdion_create(ctypes.byref(h), m, n, r, mu, eta, wd, mode), "orthdion_create")
    return h.value


def orthdion_destroy(h):
    _check(lib().orthdion_destroy(h), "orthdion_destroy")


def orthdion_set_dtypes(h, x_dtype, g_dtype):
    _check(lib().orthdion_set_dtypes(h, _dt(x_dtype) if isinstance(x_dtype, torch.dtype) else x_dtype,
                                     _dt(g_dtype) if isinstance(g_dtype, torch.dtype) else g_dtype),
           "orthdion_set_dtypes")


def orthdion_set_lr(h, eta):
    _check(lib().orthdion_set_lr(h, eta), "orthdion_set_lr")


def orthdion_set_scale(h, scale):
    _check(lib().orthdion_set_scale(h, scale), "orthdion_set_scale")


def orthdion_set_ef(h, a, b):
    _check(lib().orthdion_set_ef(h, a, b), "orthdion_set_ef")


def orthdion_set_engine(h, engine):
    _check(lib().orthdion_set_engine(h, engine), "orthdion_set_engine")


def orthdion_set_passes(h, which, passes):
    _check(lib().orthdion_set_passes(h, which, passes), "orthdion_set_passes")


def orthdion_workspace_bytes(h) -> int:
    return lib().orthdion_workspace_bytes(h)


def _harr(hs):
    return (ctypes.c_void_p * len(hs))(*hs)


def orthdion_workspace_bytes_grouped(hs) -> int:
    return lib().orthdion_workspace_bytes_grouped(_harr(hs), len(hs))


def _dev_ptr(t: torch.Tensor, name: str) -> int:
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return t.data_ptr()


def orthdion_step(h, X, M, G, Q, workspace, stream=None):
    """One step for one matrix.  X, M, G, Q, workspace: CUDA tensors (workspace: uint8)."""
    _check(lib().orthdion_step(h, _dev_ptr(X, "X"), _dev_ptr(M, "M"), _dev_ptr(G, "G"), _dev_ptr(Q, "Q"),
                               _dev_ptr(workspace, "workspace"), workspace.numel() * workspace.element_size(),
                               _stream_ptr(stream)), "orthdion_step")


NOALLOC_SCRATCH_BYTES = 64 << 20


def orthdion_step_noalloc(h, X, M, G, Q, status=None, stream=None):
    """One step for one matrix with the library's built-in scratch array: no workspace argument
    and no device allocation anywhere in the call (for callers that must not allocate, e.g. while
    a stream is being captured or when the memory pool is locked).  `status`, if given, is a
    one-element int32 CUDA tensor that receives the status flags in stream order.  Plans that
    need more than NOALLOC_SCRATCH_BYTES are rejected (OrthDionError WORKSPACE).  Calls share
    the array: do not let two of them overlap on the GPU."""
    sp = 0 if status is None else _dev_ptr(status, "status")
    _check(lib().orthdion_step_noalloc(h, _dev_ptr(X, "X"), _dev_ptr(M, "M"), _dev_ptr(G, "G"), _dev_ptr(Q, "Q"),
                                       sp, _stream_ptr(stream)), "orthdion_step_noalloc")


class PointerTable:
    """Host arrays of device pointers for orthdion_step_grouped, built once and reused."""

    def __init__(self, hs, Xs, Ms, Gs, Qs):
        n = len(hs)
        assert len(Xs) == len(Ms) == len(Gs) == len(Qs) == n
        arr = ctypes.c_void_p * n
        self.n = n
        self.hs = arr(*hs)
        self.X = arr(*[_dev_ptr(t, "X") for t in Xs])
        self.M = arr(*[_dev_ptr(t, "M") for t in Ms])
        self.G = arr(*[_dev_ptr(t, "G") for t in Gs])
        self.Q = arr(*[_dev_ptr(t, "Q") for t in Qs])
        self._keep = (Xs, Ms, Gs, Qs)


def orthdion_step_grouped(table: PointerTable, workspace, stream=None):
    _check(lib().orthdion_step_grouped(table.hs, table.n, table.X, table.M, table.G, table.Q,
                                       _dev_ptr(workspace, "workspace"),
                                       workspace.numel() * workspace.element_size(), _stream_ptr(stream)),
           "orthdion_step_grouped")


def orthdion_shard_phase(h, phase, X, M, G, Q, workspace, stream=None):
    """One local phase of the column-sharded step (X, M, G: this rank's columns; Q: its rows)."""
    _check(lib().orthdion_shard_phase(h, phase, _dev_ptr(X, "X"), _dev_ptr(M, "M"), _dev_ptr(G, "G"), _dev_ptr(Q, "Q"),
                                      _dev_ptr(workspace, "workspace"), workspace.numel() * workspace.element_size(),
                                      _stream_ptr(stream)), "orthdion_shard_phase")


def orthdion_shard_reduce_buffer(h, phase, workspace) -> torch.Tensor:
    """The fp32 buffer inside `workspace` that has to be summed over the ranks after `phase`
    (a flat torch view: all-reduce it in place)."""
    buf, cnt = ctypes.c_void_p(), ctypes.c_int64()
    _check(lib().orthdion_shard_reduce_buffer(h, phase, _dev_ptr(workspace, "workspace"), ctypes.byref(buf),
                                              ctypes.byref(cnt)), "orthdion_shard_reduce_buffer")
    off = (buf.value - workspace.data_ptr()) // 4
    return workspace.view(torch.float32)[off:off + cnt.value]


def orthdion_set_concurrency(lanes: int):
    """Number of internal streams a grouped call spreads its launch batches over (1: none)."""
    _check(lib().orthdion_set_concurrency(lanes), "orthdion_set_concurrency")


def orthdion_get_factors(hs, index, workspace, shapes):
    """Returns torch views (P m x r, R n x r) of the factors of matrix `index` inside `workspace`.
    shapes = (m, n, r) of that matrix."""
    P, R = ctypes.c_void_p(), ctypes.c_void_p()
    _check(lib().orthdion_get_factors(_harr(hs), len(hs), index, _dev_ptr(workspace, "workspace"),
                                      ctypes.byref(P), ctypes.byref(R)), "orthdion_get_factors")
    m, n, r = shapes
    base = workspace.data_ptr()
    wf = workspace.view(torch.float32)
    po, ro = (P.value - base) // 4, (R.value - base) // 4
    return wf[po:po + m * r].view(m, r), wf[ro:ro + n * r].view(n, r)


def orthdion_last_status(hs, workspace, stream=None):
    flags = (ctypes.c_int32 * len(hs))()
    _check(lib().orthdion_last_status(_harr(hs), len(hs), _dev_ptr(workspace, "workspace"),
                                      _stream_ptr(stream), flags), "orthdion_last_status")
    return list(flags)


DIAG_FLOATS = 8
DIAG_NAMES = ("nu", "erank", "tr_t2", "norm_r", "norm_m", "norm_g", "norm_b", "iterations")


def orthdion_set_diagnostics(h, mask: int):
    _check(lib().orthdion_set_diagnostics(h, mask), "orthdion_set_diagnostics")


def orthdion_last_diagnostics(hs, workspace, stream=None):
    """One dict per matrix (keys DIAG_NAMES) from the diagnostic records of the last step."""
    out = (ctypes.c_float * (DIAG_FLOATS * len(hs)))()
    _check(lib().orthdion_last_diagnostics(_harr(hs), len(hs), _dev_ptr(workspace, "workspace"),
                                           _stream_ptr(stream), out), "orthdion_last_diagnostics")
    return [dict(zip(DIAG_NAMES, out[i * DIAG_FLOATS:(i + 1) * DIAG_FLOATS])) for i in range(len(hs))]


def orthdion_rank_policy(e_t, r_t, ema_prev, r_min, r_max, alpha, gamma, multiple=8):
    """Returns (ema_t, r_next) of the rank-selection rule (host arithmetic inside the library)."""
    ema, r_next = ctypes.c_double(), ctypes.c_int32()
    _check(lib().orthdion_rank_policy(e_t, r_t, ema_prev, r_min, r_max, alpha, gamma, multiple,
                                      ctypes.byref(ema), ctypes.byref(r_next)), "orthdion_rank_policy")
    return ema.value, r_next.value


def orthdion_resize_factor(Q_old, Q_new, pad=None, stream=None):
    n, r_old = Q_old.shape
    r_new = Q_new.shape[1]
    assert Q_new.shape[0] == n and Q_old.dtype == Q_new.dtype == torch.float32
    _check(lib().orthdion_resize_factor(_dev_ptr(Q_old, "Q_old"), n, r_old, _dev_ptr(Q_new, "Q_new"), r_new,
                                        _dev_ptr(pad, "pad") if pad is not None else None,
                                        _stream_ptr(stream)), "orthdion_resize_factor")


def orthdion_launch_count() -> int:
    return lib().orthdion_launch_count()


def orthdion_profile_begin(max_launches: int):
    _check(lib().orthdion_profile_begin(max_launches), "orthdion_profile_begin")


def orthdion_profile_end() -> dict:
    """{stage name: (milliseconds, launches)} for the launches recorded since profile_begin."""
    n = lib().orthdion_stage_count()
    ms = (ctypes.c_double * n)()
    cnt = (ctypes.c_int64 * n)()
    _check(lib().orthdion_profile_end(n, ms, cnt), "orthdion_profile_end")
    return {lib().orthdion_stage_name(i).decode(): (ms[i], cnt[i]) for i in range(n)}


def orthdion_version() -> str:
    return lib().orthdion_version().decode()


def alloc_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """A 256-byte aligned uint8 CUDA tensor (torch's caching allocator aligns to 512 bytes)."""
    t = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)
    assert t.data_ptr() % 256 == 0
    return t
