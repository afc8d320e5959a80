"""Counter-based random numbers for the synthetic workloads.

Every value is a pure function of (seed, stream, index): a 64-bit splitmix-style
finaliser applied to a key derived from (seed, stream) plus a Weyl step per
index.  Nothing here belongs to the decoding method; the module only produces
inputs (weights, prompts, forced drafts) that are then handed, as the same
bytes, to the CPU oracle and to the CUDA library.

Two implementations of the same integer function are kept: plain Python ints
(`mix64`, `hash_at`) for the sequential prompt sources, and torch int64 tensor
ops (`hash_tensor`) for bulk weight generation on either the CPU or a GPU.
`tests/test_workloads.py` checks that they agree bit for bit.
"""
from __future__ import annotations

import math

import torch

MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB


def mix64(z: int) -> int:
    """splitmix64 output function on a Python int (64-bit wraparound)."""
    z &= MASK64
    z = ((z ^ (z >> 30)) * _M1) & MASK64
    z = ((z ^ (z >> 27)) * _M2) & MASK64
    return z ^ (z >> 31)


def stream_key(seed: int, stream: int) -> int:
    return mix64(mix64(seed & MASK64) + ((stream & MASK64) * _GOLDEN))


def hash_at(seed: int, stream: int, index: int) -> int:
    """The 64-bit value of (seed, stream) at position `index`."""
    return mix64(stream_key(seed, stream) + ((index + 1) * _GOLDEN))


def uniform_at(seed: int, stream: int, index: int) -> float:
    """Uniform in [0, 1): the top 24 bits of the hash over 2**24."""
    return (hash_at(seed, stream, index) >> 40) / float(1 << 24)


def randint_at(seed: int, stream: int, index: int, lo: int, hi: int) -> int:
    """Integer in [lo, hi] (inclusive) from the hash (modulo reduction)."""
    return lo + hash_at(seed, stream, index) % (hi - lo + 1)


# ----------------------------------------------------------------------------
# torch (bulk) version
# ----------------------------------------------------------------------------

def _signed(v: int) -> int:
    v &= MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of an int64 tensor holding uint64 bit patterns."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def _mix64_t(z: torch.Tensor) -> torch.Tensor:
    z = (z ^ _lsr(z, 30)) * _signed(_M1)
    z = (z ^ _lsr(z, 27)) * _signed(_M2)
    return z ^ _lsr(z, 31)


def hash_tensor(seed: int, stream: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """int64 tensor holding the uint64 bit patterns hash_at(seed, stream, start + i)."""
    idx = torch.arange(start + 1, start + count + 1, dtype=torch.int64, device=device)
    z = idx * _signed(_GOLDEN) + _signed(stream_key(seed, stream))
    return _mix64_t(z)


def normal_tensor(seed: int, stream: int, count: int, std: float, device="cpu",
                  chunk: int = 1 << 24) -> torch.Tensor:
    """`count` fp32 samples of N(0, std^2) by Box-Muller, one hash per sample.

    u1 = (bits 63..40 + 1) / 2^24 in (0, 1], u2 = bits 39..16 / 2^24 in [0, 1).
    The transcendental functions are the device's own, so a tensor is generated
    once and the resulting bytes are what both sides of a comparison receive.
    """
    out = torch.empty(count, dtype=torch.float32, device=device)
    for s in range(0, count, chunk):
        n = min(chunk, count - s)
        h = hash_tensor(seed, stream, s, n, device)
        u1 = (_lsr(h, 40) + 1).to(torch.float32) * (1.0 / (1 << 24))
        u2 = (_lsr(h, 16) & 0xFFFFFF).to(torch.float32) * (1.0 / (1 << 24))
        r = torch.sqrt(-2.0 * torch.log(u1))
        out[s:s + n] = r * torch.cos((2.0 * math.pi) * u2) * std
    return out
