"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

This module holds no arithmetic of the quantization method: it only draws numbers.  The paper
measures on LLM weights and activations that are not available offline; these generators stand in
for them with tensors of the same shapes and rough value distributions:

* ``normal``          i.i.d. N(0, sigma^2)              (numerical study; 1024x1024 fp32 case)
* ``student_t``       scale * t_nu                      (weight-shaped tensors, heavy tails)
* ``outlier_columns`` N(0,1) rows, 1 % of columns x50   (activation-shaped tensors)
* ``laplace``         Laplace(0, 1)                     (bulk scale-search case)
* ``sigma_sweep``     N(0, sigma^2) segments, 151 sigmas (the numerical study's sampling protocol)
* ``adversarial``     short-mantissa values, zeros, signed zeros, denormals, tiny and huge blocks

Every generator takes a seed and a device and returns a flat torch tensor; the same call on the
same device type returns the same bytes.  ``to_numpy_bits`` turns a tensor into what the CPU
oracle reads (float32 array, or uint16 array of bf16 bit patterns).
"""
from __future__ import annotations

import numpy as np
import torch


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _cast(x: torch.Tensor, dtype: torch.dtype) -> torch.Tensor:
    return x.to(dtype).contiguous()


def normal(n: int, seed: int, sigma: float = 1.0, dtype=torch.float32, device="cpu") -> torch.Tensor:
    x = torch.randn(n, generator=_gen(seed, device), device=device, dtype=torch.float32)
    return _cast(x * sigma, dtype)


def student_t(n: int, nu: int, scale: float, seed: int, dtype=torch.bfloat16, device="cpu",
              chunk: int = 1 << 26) -> torch.Tensor:
    """scale * Z / sqrt(chi2_nu / nu), chi2_nu as a sum of nu squared normals; drawn in chunks."""
    g = _gen(seed, device)
    out = torch.empty(n, dtype=dtype, device=device)
    for s in range(0, n, chunk):
        m = min(chunk, n - s)
        z = torch.randn(m, generator=g, device=device, dtype=torch.float32)
        chi = torch.zeros(m, device=device, dtype=torch.float32)
        for _ in range(nu):
            chi += torch.randn(m, generator=g, device=device, dtype=torch.float32) ** 2
        out[s:s + m] = (z * torch.rsqrt(chi / nu) * scale).to(dtype)
    return out


def laplace(n: int, seed: int, dtype=torch.float32, device="cpu", chunk: int = 1 << 26) -> torch.Tensor:
    """Laplace(0,1) by inverse CDF of a uniform draw."""
    g = _gen(seed, device)
    out = torch.empty(n, dtype=dtype, device=device)
    for s in range(0, n, chunk):
        m = min(chunk, n - s)
        u = torch.rand(m, generator=g, device=device, dtype=torch.float32) - 0.5
        x = -torch.sign(u) * torch.log1p(-2.0 * u.abs().clamp(max=0.5 - 1e-7))
        out[s:s + m] = x.to(dtype)
    return out


def outlier_columns(rows: int, cols: int, seed: int, frac: float = 0.01, gain: float = 50.0,
                    dtype=torch.bfloat16, device="cpu") -> torch.Tensor:
    """N(0,1) matrix with round(frac*cols) seeded columns multiplied by `gain`; returned flat."""
    g = _gen(seed, device)
    x = torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32)
    k = max(1, int(round(frac * cols)))
    idx = torch.randperm(cols, generator=g, device=device)[:k]
    x[:, idx] *= gain
    return _cast(x.reshape(-1), dtype)


def adversarial(n: int, seed: int, dtype=torch.float32) -> torch.Tensor:
    """CPU-only mix that provokes rounding ties and range edges.

    Runs of 64 elements, each run of one kind: short-mantissa values k/8 * 2^e (these land exactly
    on rounding midpoints after scaling), the same one float below/above, all zeros, signed zeros
    with a few tiny values, denormals, very small magnitudes (2^-20..2^-8), very large magnitudes
    (2^10..2^40), random bit patterns of moderate exponent, and plain normals.
    """
    rng = np.random.default_rng(seed)
    n_runs = (n + 63) // 64
    out = np.empty(n_runs * 64, dtype=np.float32)
    for r in range(n_runs):
        kind = r % 10
        sign = rng.choice(np.array([-1.0, 1.0], dtype=np.float32), 64)
        if kind in (0, 1, 2):
            k = rng.integers(0, 97, 64).astype(np.float32)
            e = int(rng.integers(-12, 6))
            v = np.ldexp(k / np.float32(8.0), e).astype(np.float32)
            if kind == 1:
                v = np.nextafter(v, np.float32(0.0))
            if kind == 2:
                v = np.nextafter(v, np.float32(np.inf))
        elif kind == 3:
            v = np.zeros(64, dtype=np.float32)
        elif kind == 4:
            v = np.zeros(64, dtype=np.float32)
            j = rng.integers(0, 64, 4)
            v[j] = np.ldexp(np.float32(1.0), rng.integers(-30, -5, 4)).astype(np.float32)
        elif kind == 5:
            v = (rng.integers(0, 1 << 23, 64).astype(np.uint32)).view(np.float32)  # denormals
        elif kind == 6:
            v = np.ldexp(rng.random(64, dtype=np.float32) + np.float32(1.0), rng.integers(-20, -8, 64)).astype(np.float32)
        elif kind == 7:
            v = np.ldexp(rng.random(64, dtype=np.float32) + np.float32(1.0), rng.integers(10, 40, 64)).astype(np.float32)
        elif kind == 8:
            bits = rng.integers(0, 1 << 23, 64).astype(np.uint32) | (rng.integers(110, 135, 64).astype(np.uint32) << 23)
            v = bits.view(np.float32)
        else:
            v = rng.standard_normal(64).astype(np.float32)
        out[r * 64:(r + 1) * 64] = v * sign
    return _cast(torch.from_numpy(out[:n].copy()), dtype)


def sigma_grid(n_sigma: int = 151, lo: float = 0.0005, hi: float = 0.05) -> torch.Tensor:
    """The standard deviations of the numerical study: n_sigma evenly spaced points in [lo, hi] (float64)."""
    return torch.linspace(lo, hi, n_sigma, dtype=torch.float64)


def sigma_sweep(elems_per_sigma: int, seed: int, n_sigma: int = 151, lo: float = 0.0005, hi: float = 0.05,
                dtype=torch.float32, device="cpu", chunk_sigmas: int = 8) -> torch.Tensor:
    """Concatenation of n_sigma segments of elems_per_sigma i.i.d. N(0, sigma_k^2) samples, sigma_k from
    ``sigma_grid`` (numerical study: 50,000 x block_size samples per sigma)."""
    g = _gen(seed, device)
    sig = sigma_grid(n_sigma, lo, hi).to(torch.float32).to(device)
    out = torch.empty(n_sigma * elems_per_sigma, dtype=dtype, device=device)
    for s in range(0, n_sigma, chunk_sigmas):
        k = min(chunk_sigmas, n_sigma - s)
        z = torch.randn(k, elems_per_sigma, generator=g, device=device, dtype=torch.float32)
        out[s * elems_per_sigma:(s + k) * elems_per_sigma] = (z * sig[s:s + k, None]).reshape(-1).to(dtype)
    return out


def to_numpy_bits(x: torch.Tensor) -> np.ndarray:
    """float32 tensor -> float32 array; bf16 tensor -> uint16 array of its bit patterns (host copy)."""
    x = x.detach().reshape(-1).cpu().contiguous()
    if x.dtype == torch.float32:
        return x.numpy()
    if x.dtype == torch.bfloat16:
        return x.view(torch.uint16).numpy()
    raise TypeError(f"unsupported dtype {x.dtype}")


# Matrix shapes of an 8B-parameter Llama-style decoder layer: (name, rows, cols); fan_in = cols.
LLAMA8B_LAYER_SHAPES = (
    ("q", 4096, 4096), ("k", 1024, 4096), ("v", 1024, 4096), ("o", 4096, 4096),
    ("gate", 14336, 4096), ("up", 14336, 4096), ("down", 4096, 14336),
)
LLAMA8B_LAYERS = 32
