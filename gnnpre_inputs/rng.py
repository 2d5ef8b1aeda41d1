"""Counter-based random bits for the synthetic inputs.

Every random quantity is a pure function of (seed, stream, counter), so a
graph or a feature matrix comes out the same for any chunking, thread count or
device.  The mixer is the public-domain SplitMix64 finaliser (Steele, Lea,
Flood: "Fast splittable pseudorandom number generators", OOPSLA 2014) applied
to a Weyl sequence; all arithmetic is wrapping 64-bit integer arithmetic, which
torch evaluates identically on CPU and CUDA tensors.

This module holds no arithmetic of the propagation method itself.
"""
from __future__ import annotations

import torch

_MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_MUL1 = 0xBF58476D1CE4E5B9
_MUL2 = 0x94D049BB133111EB


def _signed(v: int) -> int:
    """Two's-complement view of a 64-bit pattern as a Python int in int64 range."""
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


def _mix_py(z: int) -> int:
    z &= _MASK64
    z = ((z ^ (z >> 30)) * _MUL1) & _MASK64
    z = ((z ^ (z >> 27)) * _MUL2) & _MASK64
    return z ^ (z >> 31)


def stream_key(seed: int, stream: int) -> int:
    """Fold (seed, stream) into one 64-bit key (unsigned Python int)."""
    return _mix_py(_mix_py(seed + _GOLDEN) ^ ((stream + 1) * _GOLDEN))


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    # torch's >> on int64 is arithmetic; mask the sign extension away.
    return (z >> s) & ((1 << (64 - s)) - 1)


def mix64(key: int, counter: torch.Tensor) -> torch.Tensor:
    """64 random bits per counter value, as an int64 tensor (bit pattern)."""
    assert counter.dtype == torch.int64
    z = counter * _signed(_GOLDEN) + _signed(key)
    z = (z ^ _lsr(z, 30)) * _signed(_MUL1)
    z = (z ^ _lsr(z, 27)) * _signed(_MUL2)
    return z ^ _lsr(z, 31)


def hi32(bits: torch.Tensor) -> torch.Tensor:
    """Upper 32 bits as a non-negative int64."""
    return _lsr(bits, 32)


def lo32(bits: torch.Tensor) -> torch.Tensor:
    """Lower 32 bits as a non-negative int64."""
    return bits & 0xFFFFFFFF


def below(u32: torch.Tensor, n: int) -> torch.Tensor:
    """Map a 32-bit uniform to [0, n) by multiply-shift (n < 2**31)."""
    return (u32 * n) >> 32
