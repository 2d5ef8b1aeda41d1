"""Seeded fp32 feature matrices with N(0, 1) entries (Box-Muller).

Element (i, f) of an [n, F] matrix is a function of (seed, i * F + f) only, so
any row range can be generated on its own.  The transcendental functions may
differ in the last place between devices; callers that compare two
implementations generate the matrix once and hand the same tensor to both.

This module holds no arithmetic of the propagation method itself.
"""
from __future__ import annotations

import math

import torch

from . import rng

STREAM_FEATURES = 3


def normal_rows(row_lo: int, row_hi: int, feat_dim: int, seed: int, device="cpu",
                out: torch.Tensor | None = None) -> torch.Tensor:
    """Rows [row_lo, row_hi) of the seeded N(0,1) matrix, fp32, row-major."""
    key = rng.stream_key(seed, STREAM_FEATURES)
    count = (row_hi - row_lo) * feat_dim
    counter = torch.arange(row_lo * feat_dim, row_lo * feat_dim + count, dtype=torch.int64, device=device)
    bits = rng.mix64(key, counter)
    del counter
    # 24-bit uniforms: u1 in (0, 1], u2 in [0, 1)
    u1 = ((rng.hi32(bits) >> 8) + 1).to(torch.float64) * (1.0 / (1 << 24))
    u2 = (rng.lo32(bits) >> 8).to(torch.float64) * (1.0 / (1 << 24))
    del bits
    z = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
    z = z.to(torch.float32).reshape(row_hi - row_lo, feat_dim)
    if out is not None:
        out.copy_(z)
        return out
    return z


def normal_matrix(n: int, feat_dim: int, seed: int, device="cpu", ld: int | None = None,
                  chunk_rows: int = 1 << 18, pin: bool = False) -> torch.Tensor:
    """The whole [n, F] matrix; with ld > F the result is a view of an [n, ld] buffer
    whose padding columns are zero."""
    ld = feat_dim if ld is None else ld
    assert ld >= feat_dim
    if pin:
        buf = torch.zeros((n, ld), dtype=torch.float32, pin_memory=True)
    else:
        buf = torch.zeros((n, ld), dtype=torch.float32, device=device)
    gen_device = device
    for lo in range(0, n, chunk_rows):
        hi = min(n, lo + chunk_rows)
        buf[lo:hi, :feat_dim].copy_(normal_rows(lo, hi, feat_dim, seed, gen_device))
    return buf[:, :feat_dim]
