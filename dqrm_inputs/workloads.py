"""Seeded synthetic workloads with the shapes of the DQRM experiments.

The paper trains on Criteo Kaggle (26 tables, feature size 16) and Criteo
Terabyte (26 tables, feature size 64) (Table "DLRM model architecture
configurations").  Neither dataset is used here: these generators only
reproduce table counts, feature sizes, row-count spread, batch sizes, index
skew and bag-length mix.  Nothing in this file quantises, pools or updates.

Layout conventions shared by every consumer:
  * tables live in one arena ``[sum(rows), D]`` float32; ``row_off[t]`` is the
    first arena row of table ``t``.
  * ``indices`` are row numbers within their table, table-major: all lookups
    of table 0 (sample 0, 1, ...), then table 1, ...
  * bag ``g = t * B + i`` owns ``indices[offsets[g]:offsets[g+1]]``.
  * ``grad_out`` and pooled outputs are ``[B, T, D]`` float32.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import List, Optional

import numpy as np

from . import rng


@dataclass(frozen=True)
class Workload:
    name: str
    rows: tuple            # rows per table
    D: int                 # embedding feature size
    B: int                 # samples per step
    alpha: Optional[float]  # Zipf exponent; None = uniform indices
    bits: int = 4          # weight fake-quant bit width
    period: int = 100      # scale refresh period (steps)
    iters: int = 100
    bag_mean: Optional[float] = None   # None = one index per bag; else Poisson mean
    bag_max: int = 64
    lr: float = 0.1
    grad_sigma: float = 0.1            # N(0, 0.01): variance 0.01
    seed: int = 0
    scatter_ranks: bool = True         # spread hot Zipf ranks over the table

    @property
    def T(self) -> int:
        return len(self.rows)

    @property
    def total_rows(self) -> int:
        return int(sum(self.rows))

    def row_off(self) -> np.ndarray:
        off = np.zeros(self.T + 1, dtype=np.int64)
        off[1:] = np.cumsum(np.asarray(self.rows, dtype=np.int64))
        return off

    def table_bytes(self) -> int:
        return self.total_rows * self.D * 4

    def with_batch(self, B: int) -> "Workload":
        return replace(self, B=B, name=f"{self.name.split('_b')[0]}_b{B}")


def log_uniform_rows(T: int, lo: float, hi: float, target: float, seed: int) -> tuple:
    """Row counts drawn log-uniformly in [lo, hi], rescaled to sum to ~target."""
    key = rng.make_key(seed, rng.STREAM_ROWS)
    u = rng.uniform_np(key, np.arange(T))
    r = np.exp(math.log(lo) + u * (math.log(hi) - math.log(lo)))
    f = target / r.sum()
    return tuple(int(max(4, round(f * x))) for x in r)


def tiny() -> Workload:
    return Workload("tiny", (1000, 5000, 20000, 100000), D=16, B=128, alpha=1.05,
                    bits=4, period=10, iters=100)


def kaggle(B: int = 16384) -> Workload:
    rows = log_uniform_rows(26, 4.0, 1.0e7, 33.8e6, seed=0)
    return Workload(f"kaggle_b{B}", rows, D=16, B=B, alpha=1.05, bits=4, period=100, iters=1000)


def terabyte(B: int = 32768) -> Workload:
    rows = log_uniform_rows(26, 4.0, 4.0e7, 49.0e6, seed=0)
    return Workload(f"terabyte_b{B}", rows, D=64, B=B, alpha=1.1, bits=4, period=100, iters=200)


def multihot(B: int = 16384) -> Workload:
    return Workload(f"multihot_b{B}", (1_000_000,) * 26, D=64, B=B, alpha=1.2, bits=4,
                    period=100, iters=200, bag_mean=20.0)


def sweep(D: int = 16, bits: int = 4, zipf: bool = False, rows: int = 10_000_000,
          B: int = 65536) -> Workload:
    tag = "zipf" if zipf else "uniform"
    return Workload(f"sweep_d{D}_b{bits}_{tag}", (rows,), D=D, B=B,
                    alpha=1.2 if zipf else None, bits=bits, period=100, iters=100)


def scaled_down(wl: Workload, total_rows: int, B: int, name: Optional[str] = None) -> Workload:
    """Same table-count, skew and row-count spread with fewer rows and samples."""
    f = total_rows / wl.total_rows
    rows = tuple(int(max(4, round(f * r))) for r in wl.rows)
    return replace(wl, rows=rows, B=B, name=name or f"{wl.name}_small")


BY_NAME = {
    "tiny": tiny,
    "kaggle_b128": lambda: kaggle(128),
    "kaggle_b16384": lambda: kaggle(16384),
    "terabyte_b2048": lambda: terabyte(2048),
    "terabyte_b32768": lambda: terabyte(32768),
    "multihot_b16384": lambda: multihot(16384),
}


# ----------------------------------------------------------------------------
# tables
# ----------------------------------------------------------------------------
def table_rows_np(wl: Workload, t: int, row_lo: int, row_hi: int) -> np.ndarray:
    """Initial values of rows [row_lo, row_hi) of table t: U(-1/sqrt(R), 1/sqrt(R))."""
    R = wl.rows[t]
    a = 1.0 / math.sqrt(R)
    key = rng.make_key(wl.seed, rng.STREAM_TABLE, t)
    ctr = np.arange(row_lo * wl.D, row_hi * wl.D, dtype=np.uint64)
    u = rng.uniform_np(key, ctr)
    return ((2.0 * u - 1.0) * a).astype(np.float32).reshape(row_hi - row_lo, wl.D)


def table_rows_at_np(wl: Workload, t: int, rows: np.ndarray) -> np.ndarray:
    """Initial values of the listed rows of table t (any order, repeats allowed)."""
    R = wl.rows[t]
    a = 1.0 / math.sqrt(R)
    key = rng.make_key(wl.seed, rng.STREAM_TABLE, t)
    rows = np.asarray(rows, dtype=np.uint64)
    ctr = rows[:, None] * np.uint64(wl.D) + np.arange(wl.D, dtype=np.uint64)[None, :]
    u = rng.uniform_np(key, ctr)
    return ((2.0 * u - 1.0) * a).astype(np.float32)


def tables_np(wl: Workload) -> np.ndarray:
    """Whole arena on the host (small workloads only)."""
    out = np.empty((wl.total_rows, wl.D), dtype=np.float32)
    off = wl.row_off()
    for t in range(wl.T):
        out[off[t]:off[t + 1]] = table_rows_np(wl, t, 0, wl.rows[t])
    return out


def tables_torch(wl: Workload, device, chunk_rows: int = 1 << 20):
    """Whole arena generated on a torch device, bit-identical to ``tables_np``."""
    import torch

    out = torch.empty((wl.total_rows, wl.D), dtype=torch.float32, device=device)
    off = wl.row_off()
    for t in range(wl.T):
        R = wl.rows[t]
        a = 1.0 / math.sqrt(R)
        key = rng.make_key(wl.seed, rng.STREAM_TABLE, t)
        for lo in range(0, R, chunk_rows):
            hi = min(R, lo + chunk_rows)
            ctr = torch.arange(lo * wl.D, hi * wl.D, dtype=torch.int64, device=device)
            u = rng.uniform_torch(key, ctr)
            vals = ((2.0 * u - 1.0) * a).to(torch.float32)
            out[off[t] + lo: off[t] + hi] = vals.view(hi - lo, wl.D)
    return out


# ----------------------------------------------------------------------------
# indices
# ----------------------------------------------------------------------------
def _coprime_stride(R: int) -> int:
    a = max(1, math.ceil(0.618 * R))
    while math.gcd(a, R) != 1:
        a += 1
    return a


class IndexSampler:
    """Finite Zipf(alpha) over R rows by inversion of the exact cumulative table,
    or uniform when alpha is None.  Rank k (0 = hottest) maps to row
    ``(k * A) mod R`` with A coprime to R so that hot rows are not neighbours."""

    def __init__(self, R: int, alpha: Optional[float], scatter: bool = True):
        self.R = R
        self.alpha = alpha
        self.A = _coprime_stride(R) if scatter else 1
        if alpha is not None:
            w = np.arange(1, R + 1, dtype=np.float64) ** (-alpha)
            self.cum = np.cumsum(w)
        else:
            self.cum = None

    def sample(self, u: np.ndarray) -> np.ndarray:
        if self.cum is None:
            k = np.minimum((u * self.R).astype(np.int64), self.R - 1)
            return k.astype(np.int32)
        k = np.searchsorted(self.cum, u * self.cum[-1], side="right")
        k = np.minimum(k, self.R - 1).astype(np.int64)
        return ((k * self.A) % self.R).astype(np.int32)


def make_samplers(wl: Workload) -> List[IndexSampler]:
    cache = {}
    out = []
    for R in wl.rows:
        if R not in cache:
            cache[R] = IndexSampler(R, wl.alpha, wl.scatter_ranks)
        out.append(cache[R])
    return out


def _poisson_cdf(mean: float, kmax: int = 256) -> np.ndarray:
    k = np.arange(kmax, dtype=np.float64)
    logp = -mean + k * math.log(mean) - np.array([math.lgamma(x + 1.0) for x in k])
    return np.cumsum(np.exp(logp))


def bag_lengths(wl: Workload, step: int, t: int) -> np.ndarray:
    if wl.bag_mean is None:
        return np.ones(wl.B, dtype=np.int64)
    key = rng.make_key(wl.seed, rng.STREAM_BAGLEN, step * 4096 + t)
    u = rng.uniform_np(key, np.arange(wl.B))
    n = np.searchsorted(_poisson_cdf(wl.bag_mean), u, side="right")
    return np.clip(n, 1, wl.bag_max).astype(np.int64)


def make_batch(wl: Workload, step: int, samplers: Optional[List[IndexSampler]] = None):
    """Returns (indices int32 [L], offsets int32 [T*B+1]) for one step."""
    samplers = samplers or make_samplers(wl)
    idx_parts = []
    lens = []
    for t in range(wl.T):
        n = bag_lengths(wl, step, t)
        lens.append(n)
        cnt = int(n.sum())
        key = rng.make_key(wl.seed, rng.STREAM_INDEX, step * 4096 + t)
        u = rng.uniform_np(key, np.arange(cnt))
        idx_parts.append(samplers[t].sample(u))
    indices = np.concatenate(idx_parts).astype(np.int32)
    offsets = np.zeros(wl.T * wl.B + 1, dtype=np.int64)
    offsets[1:] = np.cumsum(np.concatenate(lens))
    assert offsets[-1] == indices.shape[0] and offsets[-1] < 2 ** 31
    return indices, offsets.astype(np.int32)


# ----------------------------------------------------------------------------
# upstream gradient
# ----------------------------------------------------------------------------
def grad_out_np(wl: Workload, step: int) -> np.ndarray:
    """[B, T, D] float32 ~ N(0, grad_sigma^2) by Box-Muller in double."""
    n = wl.B * wl.T * wl.D
    key = rng.make_key(wl.seed, rng.STREAM_GRAD, step)
    i = np.arange(n, dtype=np.uint64)
    u1 = 1.0 - rng.uniform_np(key, 2 * i)            # (0, 1]
    u2 = rng.uniform_np(key, 2 * i + 1)
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * math.pi * u2)
    return (z * wl.grad_sigma).astype(np.float32).reshape(wl.B, wl.T, wl.D)


def grad_out_torch(wl: Workload, step: int, device):
    """Same law generated on a torch device (transcendentals differ in the last
    bits from numpy's, so parity tests use ``grad_out_np``; timing runs may use this)."""
    import torch

    n = wl.B * wl.T * wl.D
    key = rng.make_key(wl.seed, rng.STREAM_GRAD, step)
    i = torch.arange(n, dtype=torch.int64, device=device)
    u1 = 1.0 - rng.uniform_torch(key, 2 * i)
    u2 = rng.uniform_torch(key, 2 * i + 1)
    z = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos(2.0 * math.pi * u2)
    return (z * wl.grad_sigma).to(torch.float32).view(wl.B, wl.T, wl.D)
