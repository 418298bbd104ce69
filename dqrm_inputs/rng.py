"""Counter-based random numbers for the synthetic DQRM workloads.

Every value is a pure function of (seed, stream, substream, counter), so any
element of any input can be regenerated in isolation: a test can rebuild one
row of a 12 GB table on the host without materialising the table.

The generator is the SplitMix64 output function (Steele, Lea & Flood, "Fast
splittable pseudorandom number generators", OOPSLA 2014) applied to
``key + GOLDEN * (counter + 1)``; the key itself is derived by chaining the
same function over (seed, stream, substream).

Two array back-ends produce identical bits: numpy (``uint64``) on the host and
torch (``int64`` two's-complement arithmetic) on any torch device.  This module
contains no arithmetic of the quantisation method; it only makes inputs.
"""
from __future__ import annotations

import numpy as np

_M64 = (1 << 64) - 1
GOLDEN = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB

# stream ids (one per kind of input)
STREAM_ROWS = 1      # table row counts
STREAM_TABLE = 2     # table initial values     (substream = table id)
STREAM_INDEX = 3     # lookup indices           (substream = step * 4096 + table id)
STREAM_BAGLEN = 4    # bag lengths              (substream = step * 4096 + table id)
STREAM_GRAD = 5      # upstream gradients       (substream = step)


def _mix_py(z: int) -> int:
    z &= _M64
    z = ((z ^ (z >> 30)) * _C1) & _M64
    z = ((z ^ (z >> 27)) * _C2) & _M64
    return z ^ (z >> 31)


def make_key(seed: int, stream: int, substream: int = 0) -> int:
    """64-bit key for one random stream (plain Python integers)."""
    k = _mix_py(seed + GOLDEN)
    k = _mix_py(k ^ ((stream * GOLDEN) & _M64))
    k = _mix_py(k ^ ((substream * _C1 + 1) & _M64))
    return k


# ----------------------------------------------------------------------------
# numpy back-end
# ----------------------------------------------------------------------------
def bits_np(key: int, counter: np.ndarray) -> np.ndarray:
    """64 random bits per counter value (numpy uint64)."""
    c = np.asarray(counter).astype(np.uint64)
    with np.errstate(over="ignore"):
        z = np.uint64(key) + np.uint64(GOLDEN) * (c + np.uint64(1))
        z = (z ^ (z >> np.uint64(30))) * np.uint64(_C1)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(_C2)
        z = z ^ (z >> np.uint64(31))
    return z


def uniform_np(key: int, counter: np.ndarray) -> np.ndarray:
    """float64 in [0, 1) with 53 random bits."""
    return (bits_np(key, counter) >> np.uint64(11)).astype(np.float64) * (2.0 ** -53)


# ----------------------------------------------------------------------------
# torch back-end (same bits; int64 wraps like uint64, shifts are made logical)
# ----------------------------------------------------------------------------
def _s64(v: int) -> int:
    v &= _M64
    return v - (1 << 64) if v >= (1 << 63) else v


def _lsr(z, k: int):
    return (z >> k) & ((1 << (64 - k)) - 1)


def bits_torch(key: int, counter):
    """64 random bits per counter value as torch int64 (bit pattern of the uint64)."""
    import torch

    c = counter.to(torch.int64)
    z = c.add(1).mul_(_s64(GOLDEN)).add_(_s64(key))
    z = (z ^ _lsr(z, 30)) * _s64(_C1)
    z = (z ^ _lsr(z, 27)) * _s64(_C2)
    z = z ^ _lsr(z, 31)
    return z


def uniform_torch(key: int, counter):
    import torch

    return _lsr(bits_torch(key, counter), 11).to(torch.float64) * (2.0 ** -53)
