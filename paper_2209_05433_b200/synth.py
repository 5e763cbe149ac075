"""Seeded synthetic inputs shaped like the paper's transformer workloads.

This module holds none of the FP8 method's arithmetic: it only makes wide
(fp32 / bf16) tensors.  The same tensors feed the CUDA library and the CPU
checker, so neither side ever sees the other's output as an input.

Every element is a pure function of (seed, tensor id, element index): a
splitmix64-style counter hash gives uniforms, Box-Muller gives normals, the
inverse CDF gives Laplace draws and a ratio of normals gives Student-t with 3
degrees of freedom.  Generation is chunked so that 2^30-element tensors can be
made directly on the device that will consume them.
"""
from __future__ import annotations

import math

import torch

_M1 = 0xBF58476D1CE4E5B9 - (1 << 64)
_M2 = 0x94D049BB133111EB - (1 << 64)
_GOLD = 0x9E3779B97F4A7C15 - (1 << 64)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """logical shift right of int64 lanes"""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix(x: torch.Tensor) -> torch.Tensor:
    x = x ^ _lsr(x, 30)
    x = x * _M1
    x = x ^ _lsr(x, 27)
    x = x * _M2
    x = x ^ _lsr(x, 31)
    return x


def _key(seed: int, tensor_id: int, stream: int) -> int:
    k = (seed * 0x632BE59BD9B4E019 + tensor_id * 0xD1342543DE82EF95 + stream * 0x2545F4914F6CDD1D + 0x1234567) % (1 << 64)
    return k - (1 << 64) if k >= (1 << 63) else k


def uniform(seed: int, tensor_id: int, stream: int, idx: torch.Tensor) -> torch.Tensor:
    """float32 uniforms in (0, 1): (23 random bits + 1/2) / 2^23, exact in fp32, never 0 or 1."""
    h = _mix(_mix(idx * _GOLD + _key(seed, tensor_id, stream)))
    top = _lsr(h, 41)                                  # 23 bits
    return (top.to(torch.float32) + 0.5) * (1.0 / 8388608.0)


def normal(seed, tensor_id, stream, idx):
    u1 = uniform(seed, tensor_id, 2 * stream, idx)
    u2 = uniform(seed, tensor_id, 2 * stream + 1, idx)
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)


def laplace(seed, tensor_id, stream, idx, b: float):
    u = uniform(seed, tensor_id, stream, idx) - 0.5
    return -b * torch.sign(u) * torch.log1p(-2.0 * torch.abs(u))


def student_t3(seed, tensor_id, stream, idx):
    z0 = normal(seed, tensor_id, stream, idx)
    s = (normal(seed, tensor_id, stream + 1, idx) ** 2 + normal(seed, tensor_id, stream + 2, idx) ** 2
         + normal(seed, tensor_id, stream + 3, idx) ** 2)
    return z0 / torch.sqrt(s / 3.0)


def _generate(n: int, fn, dtype, device, chunk: int = 1 << 24) -> torch.Tensor:
    out = torch.empty(n, dtype=dtype, device=device)
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        idx = torch.arange(lo, hi, dtype=torch.int64, device=device)
        out[lo:hi] = fn(idx).to(dtype)
    return out


# tensor ids
X_ID, W_ID, DY_ID, A_ID, B_ID, T_ID = 1, 2, 3, 4, 5, 6


def normal_with_scaled_outliers(n, seed, tensor_id, frac, factor, dtype=torch.float32, device="cpu"):
    """N(0,1); an i.i.d. `frac` of the entries multiplied by `factor` (tiny-case recipe)."""
    def fn(idx):
        z = normal(seed, tensor_id, 0, idx)
        pick = uniform(seed, tensor_id, 8, idx) < frac
        return torch.where(pick, z * factor, z)
    return _generate(n, fn, dtype, device)


def normal_laplace_mixture(n, seed, tensor_id, frac=1e-3, b=50.0, dtype=torch.bfloat16, device="cpu"):
    """each element independently Laplace(0,b) with probability `frac`, else N(0,1) (bandwidth sweep recipe)."""
    def fn(idx):
        z = normal(seed, tensor_id, 0, idx)
        pick = uniform(seed, tensor_id, 8, idx) < frac
        return torch.where(pick, laplace(seed, tensor_id, 9, idx, b), z)
    return _generate(n, fn, dtype, device)


def activations(n, seed, tensor_id=X_ID, frac=1e-3, lo=20.0, hi=100.0, dtype=torch.bfloat16, device="cpu"):
    """N(0,1) with an i.i.d. `frac` of positions replaced by a value of magnitude U[lo,hi] and random sign."""
    def fn(idx):
        z = normal(seed, tensor_id, 0, idx)
        pick = uniform(seed, tensor_id, 8, idx) < frac
        mag = lo + (hi - lo) * uniform(seed, tensor_id, 9, idx)
        sgn = torch.where(uniform(seed, tensor_id, 10, idx) < 0.5, -1.0, 1.0)
        return torch.where(pick, mag * sgn, z)
    return _generate(n, fn, dtype, device)


def weights(n, seed, sigma, tensor_id=W_ID, dtype=torch.bfloat16, device="cpu"):
    return _generate(n, lambda idx: sigma * normal(seed, tensor_id, 0, idx), dtype, device)


def gradients(n, seed, scale=1e-4, tensor_id=DY_ID, dtype=torch.bfloat16, device="cpu"):
    """heavy-tailed output gradients: scale * Student-t(nu=3)."""
    return _generate(n, lambda idx: scale * student_t3(seed, tensor_id, 0, idx), dtype, device)


# The five workloads (shapes only; tensors are made by the functions above).
CONFIGS = {
    1: dict(name="tiny codec+GEMM", seed=0, M=256, N=256, K=256),
    2: dict(name="quantize bandwidth sweep", seed=1, sizes=[1 << 20, 1 << 24, 1 << 28, 1 << 30]),
    3: dict(name="transformer forward linear, hidden 4096", seed=3, tokens=8192, d_in=4096, d_out=16384, w_sigma=0.02),
    4: dict(name="transformer backward, hidden 4096", seed=4, tokens=8192, d_in=4096, d_out=16384, w_sigma=0.02),
    5: dict(name="FFN layer, hidden 12288", seed=5, tokens=8192, d_in=12288, d_out=49152, w_sigma=0.006),
}
