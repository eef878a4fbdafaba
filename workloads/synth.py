"""Seeded synthetic-input generator shared by the tests, the benchmark and the smoke check.

This module holds NO attention arithmetic: it only produces reproducible numbers.
Everything is counter based: a value is a pure function of (seed, stream, coordinates),
built from 32-bit integer mixing and one table lookup, so the same code gives the same
bits on the CPU (for the fp64 oracle) and on a CUDA device (to fill a large KvPage pool
without staging it through host memory).  Integer work is done in int64 tensors masked to
32 bits, which torch evaluates identically on every device.

Value recipe: a 32-bit hash of the coordinates selects one of 65,536 equally likely
standard-normal quantiles z_i = Phi^-1((i + 0.5) / 65536); the quantile table is computed
once in fp64 on the CPU and rounded to the element type (bf16 or fp32).  The elements are
therefore i.i.d. N(0,1) up to the 16-bit quantisation of the quantile index.
"""
from __future__ import annotations

import functools

import numpy as np
import torch

M32 = 0xFFFFFFFF
_GOLD = 0x9E3779B9
_C1 = 0x85EBCA6B
_C2 = 0xC2B2AE35


def mix32(x):
    """32-bit avalanche finaliser (multiply/xor-shift) on int64 tensors or Python ints."""
    x = x ^ (x >> 16)
    x = (x * _C1) & M32
    x = x ^ (x >> 13)
    x = (x * _C2) & M32
    x = x ^ (x >> 16)
    return x


def hash_coords(seed: int, stream: int, *coords):
    """Chain-hash integer coordinates (Python ints or broadcastable int64 tensors) to u32.

    Early coordinates may be small tensors; broadcasting makes only the last steps run at
    full size.  The result is an int64 tensor (or int) holding a value in [0, 2^32).
    """
    h = mix32(((seed & M32) ^ ((stream * _GOLD) & M32)) & M32)
    for c in coords:
        h = mix32(((h ^ (c & M32)) + _GOLD) & M32)
    return h


@functools.lru_cache(maxsize=None)
def _quantiles_f64() -> torch.Tensor:
    i = torch.arange(65536, dtype=torch.float64)
    return torch.special.ndtri((i + 0.5) / 65536.0)


@functools.lru_cache(maxsize=None)
def normal_table(dtype: str, device: str = "cpu") -> torch.Tensor:
    """65,536 standard-normal quantiles rounded to `dtype` ("bf16" or "f32")."""
    z = _quantiles_f64().to(torch.float32)
    if dtype == "bf16":
        z = z.to(torch.bfloat16)
    elif dtype != "f32":
        raise ValueError(dtype)
    return z.to(device)


def normal_from_hash(h: torch.Tensor, dtype: str) -> torch.Tensor:
    """Map u32 hashes (int64 tensor) to N(0,1) elements of `dtype` on h's device."""
    table = normal_table(dtype, str(h.device))
    return table[(h >> 16)]


def normal_tensor(seed: int, stream: int, shape, dtype: str, device="cpu", lead=()) -> torch.Tensor:
    """An N(0,1) tensor of `shape`; element hash = hash(seed, stream, *lead, flat index)."""
    n = int(np.prod(shape)) if len(shape) else 1
    idx = torch.arange(n, dtype=torch.int64, device=device)
    h = hash_coords(seed, stream, *lead, idx)
    return normal_from_hash(h, dtype).reshape(shape)


def uniform_ints(seed: int, stream: int, n: int, lo: int, hi: int) -> np.ndarray:
    """n integers, inclusive-uniform in [lo, hi] (modulo bias < 2^-16 for spans < 2^16)."""
    idx = torch.arange(n, dtype=torch.int64)
    h = hash_coords(seed, stream, idx)
    return (lo + (h % (hi - lo + 1))).numpy().astype(np.int64)


def uniform_unit(seed: int, stream: int, shape, lead=()) -> np.ndarray:
    """Uniform floats in [0,1) with 32-bit resolution (for Bernoulli masks)."""
    n = int(np.prod(shape)) if len(shape) else 1
    idx = torch.arange(n, dtype=torch.int64)
    h = hash_coords(seed, stream, *lead, idx)
    return (h.to(torch.float64) / 4294967296.0).numpy().reshape(shape)


def permutation(seed: int, stream: int, n: int) -> np.ndarray:
    """A seeded permutation of range(n): stable argsort of per-index hashes."""
    idx = torch.arange(n, dtype=torch.int64)
    h = hash_coords(seed, stream, idx)
    return torch.argsort(h * n + idx).numpy().astype(np.int64)  # key is unique


def kv_rows(seed: int, which: int, owner, pos: torch.Tensor, n_kv_heads: int, head_dim: int,
            dtype: str) -> torch.Tensor:
    """Context K (which=0) or V (which=1) rows keyed by (owner, logical position, head, d).

    `owner` and `pos` are int64 tensors of equal shape [n] (owner may be an int); the
    result is [n, n_kv_heads, head_dim] on pos.device.  Keys never mention the physical
    page or the page size, so the same logical sequence can be laid out in any paging.
    """
    dev = pos.device
    if not torch.is_tensor(owner):
        owner = torch.full_like(pos, int(owner))
    row = hash_coords(seed, 100 + which, owner, pos)                      # [n]
    head = torch.arange(n_kv_heads, dtype=torch.int64, device=dev)
    d = torch.arange(head_dim, dtype=torch.int64, device=dev)
    h = mix32(((row[:, None] ^ (head[None, :] * 0x01000193 & M32)) + _GOLD) & M32)   # [n,H]
    h = mix32(((h[:, :, None] ^ d[None, None, :]) + _GOLD) & M32)                    # [n,H,D]
    return normal_from_hash(h, dtype)


def to_numpy_bits(t: torch.Tensor) -> np.ndarray:
    """Host numpy view of a tensor: bf16 -> uint16 bit patterns, fp32 -> float32."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()
