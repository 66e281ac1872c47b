"""Seeded synthetic inputs for the optimizer-step workloads.

This module only draws random numbers and shapes them; it contains none of the
optimizer's arithmetic and imports neither the CUDA binding nor the CPU oracle, so both
sides can be fed the very same tensors.  Orthonormal bases used to *build inputs* come
from the library QR of torch (an input recipe, not a step of the method).

Workloads (all synthetic; they stand in for LLM pre-training gradients, which the paper
measures on but which cannot be regenerated here):

  cfg0  one 256 x 512 fp32 matrix, r = 16, i.i.d. N(0,1) gradients
  cfg1  one 4096 x 4096 matrix, bf16 X/G, r = 256, low-rank-plus-noise gradients
  cfg2  one 11008 x 4096 matrix, rank sweep, gradients as cfg1
  cfg3  1.1B Llama-style model, 22 layers x 7 matrices, r = 512, noise + rank-64 spike
  cfg4  8B Llama-style model, 32 layers x 7 matrices, r = 512, gradients as cfg3
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import torch


@dataclass(frozen=True)
class MatrixSpec:
    name: str
    m: int
    n: int
    r: int
    x_dtype: torch.dtype = torch.bfloat16
    g_dtype: torch.dtype = torch.bfloat16

    @property
    def numel(self) -> int:
        return self.m * self.n


@dataclass(frozen=True)
class Workload:
    name: str
    matrices: tuple
    grad: str                      # "gaussian" | "lowrank_noise" | "noise_spike"
    mu: float = 0.95
    eta: float = 0.01
    wd: float = 0.0
    grad_params: dict = field(default_factory=dict)

    @property
    def numel(self) -> int:
        return sum(s.numel for s in self.matrices)


def _llama_layers(layers, d, dkv, dff, r):
    out = []
    for l in range(layers):
        out += [MatrixSpec(f"l{l}.q", d, d, r), MatrixSpec(f"l{l}.k", dkv, d, r),
                MatrixSpec(f"l{l}.v", dkv, d, r), MatrixSpec(f"l{l}.o", d, d, r),
                MatrixSpec(f"l{l}.gate", dff, d, r), MatrixSpec(f"l{l}.up", dff, d, r),
                MatrixSpec(f"l{l}.down", d, dff, r)]
    return tuple(out)


def workload(name: str, *, r: int | None = None, layers: int | None = None) -> Workload:
    """Return one of the named workloads.  `r` overrides the rank (cfg2's sweep);
    `layers` truncates the grouped models (for small test cases of the same shape mix)."""
    f32 = torch.float32
    if name == "cfg0":
        return Workload("cfg0", (MatrixSpec("w", 256, 512, r or 16, f32, f32),), "gaussian")
    if name == "cfg1":
        return Workload("cfg1", (MatrixSpec("w", 4096, 4096, r or 256),), "lowrank_noise",
                        grad_params=dict(k=1024, noise=0.1))
    if name == "cfg2":
        return Workload("cfg2", (MatrixSpec("up", 11008, 4096, r or 256),), "lowrank_noise",
                        grad_params=dict(k=1024, noise=0.1))
    if name == "cfg3":
        return Workload("cfg3", _llama_layers(layers or 22, 2048, 2048, 5632, r or 512),
                        "noise_spike", grad_params=dict(k=64, factor=10.0))
    if name == "cfg4":
        return Workload("cfg4", _llama_layers(layers or 32, 4096, 1024, 14336, r or 512),
                        "noise_spike", grad_params=dict(k=64, factor=10.0))
    raise KeyError(name)


# ---------------------------------------------------------------------------------
def _gen(seed: int, *ids: int, device="cpu") -> torch.Generator:
    """A generator keyed by (seed, ids...).  The key is folded with a fixed odd-multiplier
    hash so that neighbouring ids give unrelated streams."""
    h = (seed * 0x9E3779B97F4A7C15 + 0x1234567) & 0xFFFFFFFFFFFFFFFF
    for i in ids:
        h = ((h ^ (i + 0x9E3779B97F4A7C15)) * 0xBF58476D1CE4E5B9) & 0xFFFFFFFFFFFFFFFF
        h ^= h >> 31
    g = torch.Generator(device=device)
    g.manual_seed(h & 0x7FFFFFFFFFFFFFFF)
    return g


def _randn(shape, gen, device):
    return torch.randn(shape, generator=gen, device=device, dtype=torch.float32)


def random_orthonormal(rows: int, cols: int, gen, device="cpu") -> torch.Tensor:
    """rows x cols matrix with orthonormal columns: library QR of a Gaussian matrix, signs
    fixed so the triangular factor has a positive diagonal.  fp32 result (fp64 QR on CPU)."""
    a = _randn((rows, cols), gen, device)
    if str(device) == "cpu":
        q, t = torch.linalg.qr(a.double(), mode="reduced")
    else:
        q, t = torch.linalg.qr(a, mode="reduced")
    d = torch.sign(torch.diagonal(t))
    d[d == 0] = 1
    return (q * d[None, :]).float().contiguous()


TENSOR_X, TENSOR_Q, TENSOR_G, TENSOR_U, TENSOR_V = 1, 2, 3, 4, 5


def initial_state(spec: MatrixSpec, seed: int, matrix_id: int, device="cpu"):
    """X_0 ~ N(0, 0.02^2) in its storage dtype, M_0 = 0 (fp32), Q_0 = orthonormalised
    Gaussian n x r (fp32)."""
    X = (0.02 * _randn((spec.m, spec.n), _gen(seed, matrix_id, TENSOR_X, device=device), device)
         ).to(spec.x_dtype)
    M = torch.zeros((spec.m, spec.n), dtype=torch.float32, device=device)
    Q = random_orthonormal(spec.n, spec.r, _gen(seed, matrix_id, TENSOR_Q, device=device), device)
    return X, M, Q


def grad_basis(wl: Workload, spec: MatrixSpec, seed: int, matrix_id: int, device="cpu"):
    """The fixed (across steps) orthonormal factors U (m x k), V (n x k) of the structured
    part of the gradient; None for purely Gaussian gradients."""
    if wl.grad == "gaussian":
        return None
    k = min(wl.grad_params["k"], spec.m, spec.n)
    U = random_orthonormal(spec.m, k, _gen(seed, matrix_id, TENSOR_U, device=device), device)
    V = random_orthonormal(spec.n, k, _gen(seed, matrix_id, TENSOR_V, device=device), device)
    return U, V


def gradient(wl: Workload, spec: MatrixSpec, seed: int, matrix_id: int, step: int, basis,
             device="cpu") -> torch.Tensor:
    """G_t for one matrix, rounded to its storage dtype (round-to-nearest-even)."""
    noise = _randn((spec.m, spec.n), _gen(seed, matrix_id, TENSOR_G, step, device=device), device)
    if wl.grad == "gaussian":
        g = noise
    elif wl.grad == "lowrank_noise":
        # G = U diag(1/i) V^T + noise_std * N(0,1)
        U, V = basis
        k = U.shape[1]
        s = 1.0 / torch.arange(1, k + 1, device=device, dtype=torch.float32)
        g = (U * s[None, :]) @ V.T + wl.grad_params["noise"] * noise
    elif wl.grad == "noise_spike":
        # G = N(0,1)/sqrt(fan_in) + s * sum_k u_k v_k^T, every spike singular value
        # s = factor * (sqrt(m)+sqrt(n))/sqrt(n), i.e. `factor` times the noise's top one.
        U, V = basis
        m, n = spec.m, spec.n
        s = wl.grad_params["factor"] * (math.sqrt(m) + math.sqrt(n)) / math.sqrt(n)
        g = noise / math.sqrt(n) + s * (U @ V.T)
    else:
        raise KeyError(wl.grad)
    return g.to(spec.g_dtype).contiguous()


def shape_classes(matrices):
    """Group matrix indices by (m, n, r, x_dtype, g_dtype), keeping first-seen order."""
    classes: dict = {}
    for i, s in enumerate(matrices):
        classes.setdefault((s.m, s.n, s.r, s.x_dtype, s.g_dtype), []).append(i)
    return classes
