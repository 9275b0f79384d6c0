"""Seeded synthetic workloads shaped like the paper's DLRM embedding traffic.

This module only *generates inputs* (table shapes, index streams, initial weights,
upstream gradients).  It contains none of the method's arithmetic and imports neither
the CUDA binding nor the CPU oracle; both consume the arrays produced here.

Shapes follow the paper's workload description: embedding dims 64-256, pooling
factors from 1 to ~100 with an average of 18-33 (Table 2), tens to hundreds of
tables, small-hot / large-cold tables (Section 3.1), power-law index reuse with very low
spatial locality (Section 3.2).
"""
from __future__ import annotations

import dataclasses
import math
import os
from typing import List, Optional, Sequence

import numpy as np

FP32 = 0
FP16 = 1

_MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_MIX1 = 0xBF58476D1CE4E5B9
_MIX2 = 0x94D049BB133111EB


@dataclasses.dataclass
class TableSpec:
    rows: int           # E_t (hash size H of the paper)
    dim: int            # D_t
    pooling: float      # mean bag length L_t
    alpha: float        # Zipf exponent; 0 = uniform ids
    perm_a: int = 1     # rank -> row scatter: row = (perm_a * (rank-1) + perm_c) mod rows
    perm_c: int = 0


@dataclasses.dataclass
class ModelSpec:
    name: str
    tables: List[TableSpec]
    dtype: int                  # FP32 / FP16 weight storage
    batch: int                  # B
    bag_dist: str               # "fixed" or "poisson"
    seed: int = 0
    lr: float = 0.01
    eps: float = 1e-8
    # cached configurations
    cached: bool = False        # rows live in host memory behind an HBM cache
    cache_fraction: float = 0.0  # cache slots / rows, per dim group
    reuse_prob: float = 0.0     # temporal reuse: probability of copying an older index
    reuse_window: int = 0       # ... from the previous `reuse_window` batches
    n_batches: int = 1
    note: str = ""

    # ---- derived layout (table-major) ----
    @property
    def T(self) -> int:
        return len(self.tables)

    @property
    def rows(self) -> np.ndarray:
        return np.array([t.rows for t in self.tables], dtype=np.int64)

    @property
    def dims(self) -> np.ndarray:
        return np.array([t.dim for t in self.tables], dtype=np.int32)

    @property
    def row_offset(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.rows)]).astype(np.int64)

    @property
    def out_offset(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.dims)]).astype(np.int32)

    @property
    def weight_offset(self) -> np.ndarray:
        """Element offset of table t in one flat weight buffer (tables back to back)."""
        sizes = self.rows * self.dims.astype(np.int64)
        return np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)

    @property
    def total_dim(self) -> int:
        return int(self.dims.sum())

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == FP32 else 2

    @property
    def weight_bytes(self) -> int:
        return int(self.weight_offset[-1]) * self.elem_bytes

    def dim_groups(self):
        """Contiguous table ranges [(dim, t_begin, t_end)] sharing one embedding dim.

        Cached configurations keep one cache per distinct dim; tables are ordered by dim
        by the config builders so that each group is a contiguous range."""
        groups = []
        t0 = 0
        d = self.dims
        for t in range(1, self.T + 1):
            if t == self.T or d[t] != d[t0]:
                groups.append((int(d[t0]), t0, t))
                t0 = t
        return groups


# --------------------------------------------------------------------------------------
# counter-based initial weights (numpy and torch twins of one generator)
# --------------------------------------------------------------------------------------

def _splitmix64_np(x: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser (Steele, Lea, Flood 2014) on uint64 arrays; wraps mod 2^64."""
    x = (x + np.uint64(_GOLDEN)).astype(np.uint64)
    x = (x ^ (x >> np.uint64(30))) * np.uint64(_MIX1)
    x = (x ^ (x >> np.uint64(27))) * np.uint64(_MIX2)
    return x ^ (x >> np.uint64(31))


def _seed_word(seed: int, table: int) -> int:
    return ((seed * 0x100000001B3) ^ (table * 0x9E3779B1) ^ 0x5851F42D4C957F2D) & _MASK64


def weights_numpy(spec: ModelSpec, t: int, rows: Optional[np.ndarray] = None) -> np.ndarray:
    """Initial weights of table t (all rows, or the selected `rows`), storage dtype.

    W0[r, d] = (u24(splitmix64(seed_word + r*D + d)) / 2^24 - 1/2) * 0.1, evaluated in
    fp32 (every step exact except the final multiply), then cast to the storage dtype.
    Any row can be produced on demand, so large host tables never need a host copy on
    the checking side."""
    tab = spec.tables[t]
    if rows is None:
        rows = np.arange(tab.rows, dtype=np.int64)
    rows = np.asarray(rows, dtype=np.int64)
    ctr = (rows.astype(np.uint64)[:, None] * np.uint64(tab.dim)
           + np.arange(tab.dim, dtype=np.uint64)[None, :])
    with np.errstate(over="ignore"):
        h = _splitmix64_np(ctr + np.uint64(_seed_word(spec.seed, t)))
    u = (h >> np.uint64(40)).astype(np.float32) * np.float32(1.0 / (1 << 24))
    w = (u - np.float32(0.5)) * np.float32(0.1)
    return w.astype(np.float16 if spec.dtype == FP16 else np.float32)


def weights_torch(spec: ModelSpec, t: int, device, row_begin: int = 0,
                  row_end: Optional[int] = None, chunk_rows: int = 1 << 20):
    """Same generator as `weights_numpy`, evaluated with torch ops on `device`.

    Returns a [rows, D] tensor in the storage dtype.  Used to fill multi-GB tables on the
    device (or in pinned host memory) without a slow host loop."""
    import torch

    tab = spec.tables[t]
    if row_end is None:
        row_end = tab.rows
    out_dtype = torch.float16 if spec.dtype == FP16 else torch.float32
    out = torch.empty((row_end - row_begin, tab.dim), dtype=out_dtype, device=device)
    sw = _seed_word(spec.seed, t)

    def s64(v):  # python int (mod 2^64) -> signed 64-bit value torch accepts
        v &= _MASK64
        return v - (1 << 64) if v >= (1 << 63) else v

    def lsr(x, k):  # logical shift right on int64 tensors
        return (x >> k) & ((1 << (64 - k)) - 1)

    d = torch.arange(tab.dim, dtype=torch.int64, device=device)[None, :]
    for r0 in range(row_begin, row_end, chunk_rows):
        r1 = min(r0 + chunk_rows, row_end)
        r = torch.arange(r0, r1, dtype=torch.int64, device=device)[:, None]
        x = r * tab.dim + d + s64(sw)
        x = x + s64(_GOLDEN)
        x = (x ^ lsr(x, 30)) * s64(_MIX1)
        x = (x ^ lsr(x, 27)) * s64(_MIX2)
        x = x ^ lsr(x, 31)
        u = lsr(x, 40).to(torch.float32) * (1.0 / (1 << 24))
        w = (u - 0.5) * torch.tensor(0.1, dtype=torch.float32, device=device)
        out[r0 - row_begin:r1 - row_begin] = w.to(out_dtype)
    return out


def all_weights_numpy(spec: ModelSpec) -> np.ndarray:
    """Flat weight buffer (tables back to back) on the host; small configs only."""
    parts = [weights_numpy(spec, t).reshape(-1) for t in range(spec.T)]
    return np.concatenate(parts)


# --------------------------------------------------------------------------------------
# index streams
# --------------------------------------------------------------------------------------

def zipf_ranks(u: np.ndarray, E: int, alpha: float) -> np.ndarray:
    """Bounded power-law ranks in [1, E] by inverting the continuous CDF on u ~ U(0,1)."""
    if alpha == 0.0:
        r = np.floor(u * E).astype(np.int64) + 1
    elif abs(alpha - 1.0) < 1e-12:
        r = np.floor(np.power(float(E + 1), u)).astype(np.int64)
    else:
        e = 1.0 - alpha
        r = np.floor(np.power((math.pow(E + 1.0, e) - 1.0) * u + 1.0, 1.0 / e)).astype(np.int64)
    return np.clip(r, 1, E)


def _coprime_multiplier(E: int) -> int:
    a = int(E * 0.6180339887498949) | 1
    while math.gcd(a, E) != 1:
        a += 2
    return a % E if E > 1 else 0


def _finish_tables(tables: Sequence[TableSpec], rng: np.random.Generator) -> List[TableSpec]:
    out = []
    for tab in tables:
        a = _coprime_multiplier(tab.rows)
        c = int(rng.integers(0, tab.rows))
        out.append(dataclasses.replace(tab, perm_a=a, perm_c=c))
    return out


def draw_rows(tab: TableSpec, rng: np.random.Generator, n: int) -> np.ndarray:
    """n fresh row ids of one table: Zipf rank scattered over the table by an affine map."""
    u = rng.random(n)
    rank = zipf_ranks(u, tab.rows, tab.alpha)
    if tab.alpha == 0.0:
        return rank - 1
    return (tab.perm_a * (rank - 1) + tab.perm_c) % tab.rows


def bag_lengths(spec: ModelSpec, tab: TableSpec, rng: np.random.Generator) -> np.ndarray:
    if spec.bag_dist == "fixed":
        return np.full(spec.batch, int(round(tab.pooling)), dtype=np.int64)
    return rng.poisson(tab.pooling, size=spec.batch).astype(np.int64)


class BatchStream:
    """Consecutive batches of one model; keeps the per-table history temporal reuse needs.

    Table t of batch k draws from `default_rng([seed, 7919, k, t])`, so the tables of a batch are independent
    of one another (large batches are generated by a few threads, with the same result) and batch k of a
    stream is reproducible only as part of the stream when reuse is on (it copies indices of earlier batches)."""

    PARALLEL_FROM = 2_000_000       # expected lookups per batch from which the tables are drawn by threads

    def __init__(self, spec: ModelSpec):
        self.spec = spec
        self.k = 0
        self.history: List[List[np.ndarray]] = []   # last `reuse_window` batches, per table
        expected = spec.batch * sum(t.pooling for t in spec.tables)
        self._pool = None
        if expected >= self.PARALLEL_FROM and spec.T > 1:
            from concurrent.futures import ThreadPoolExecutor
            self._pool = ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1, spec.T))

    def _table(self, t: int):
        spec, tab = self.spec, self.spec.tables[t]
        rng = np.random.default_rng([spec.seed, 7919, self.k, t])
        lens = bag_lengths(spec, tab, rng)
        n = int(lens.sum())
        idx = draw_rows(tab, rng, n)
        if spec.reuse_prob > 0.0 and self.history:
            parts = [h[t] for h in self.history]
            size = sum(p.size for p in parts)
            if size:
                reuse = rng.random(n) < spec.reuse_prob
                pick = rng.integers(0, size, size=n)
                # index `pick` of the previous batches' indices laid end to end, oldest first
                ends = np.cumsum([p.size for p in parts])
                which = np.searchsorted(ends, pick, side="right")
                old = np.empty(n, dtype=np.int64)
                for j, p in enumerate(parts):
                    sel = which == j
                    if sel.any():
                        old[sel] = p[pick[sel] - (ends[j] - p.size)]
                idx = np.where(reuse, old, idx)
        return idx, lens

    def next(self):
        spec = self.spec
        if self._pool is not None:
            res = list(self._pool.map(self._table, range(spec.T)))
        else:
            res = [self._table(t) for t in range(spec.T)]
        per_table = [r[0] for r in res]
        if spec.reuse_window > 0:
            self.history.append(per_table)
            if len(self.history) > spec.reuse_window:
                self.history.pop(0)
        indices = np.concatenate(per_table).astype(np.int64) if per_table else np.zeros(0, np.int64)
        lens = np.concatenate([r[1] for r in res])
        offsets = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
        self.k += 1
        return indices, offsets


def gen_batch(spec: ModelSpec, k: int = 0):
    """Batch k of a model without temporal reuse (indices int64 [N], offsets int64 [T*B+1]).

    `offsets` is CSR over bag id t*B + b (table-major)."""
    assert spec.reuse_prob == 0.0, "use BatchStream for configurations with temporal reuse"
    s = BatchStream(spec)
    s.k = k
    return s.next()


def gen_grad(spec: ModelSpec, k: int = 0, scale: float = 0.1) -> np.ndarray:
    """Upstream gradient of the pooled output, fp32 [B, sum(D)], N(0, scale^2)."""
    rng = np.random.default_rng([spec.seed, 104729, k])
    return (rng.standard_normal((spec.batch, spec.total_dim), dtype=np.float32)
            * np.float32(scale))


# --------------------------------------------------------------------------------------
# the five configurations
# --------------------------------------------------------------------------------------

def config1(seed: int = 0) -> ModelSpec:
    """4 tables x 10,000 rows x dim 64 fp32, batch 512, fixed pooling 20, uniform ids."""
    tabs = [TableSpec(rows=10_000, dim=64, pooling=20, alpha=0.0) for _ in range(4)]
    return ModelSpec("cfg1", tabs, FP32, 512, "fixed", seed=seed)


def config2(seed: int = 0, row_scale: float = 1.0, batch: int = 8192, tables: int = 26) -> ModelSpec:
    """26 tables x 1M rows x dim 128 fp16, batch 8192, Poisson(30) bags, Zipf 1.05."""
    rng = np.random.default_rng([seed, 2])
    E = max(64, int(1_000_000 * row_scale))
    tabs = [TableSpec(rows=E, dim=128, pooling=30, alpha=1.05) for _ in range(tables)]
    return ModelSpec("cfg2", _finish_tables(tabs, rng), FP16, batch, "poisson", seed=seed)


def _hetero_tables(rng: np.random.Generator, T: int, row_scale: float) -> List[TableSpec]:
    u = rng.random(T)
    n = rng.standard_normal(T)
    dims = rng.choice(np.array([64, 128, 256]), size=T)
    alphas = rng.uniform(0.8, 1.3, size=T)
    v = np.clip(u + 0.15 * n, 0.0, 1.0)
    tabs = []
    for t in range(T):
        E = max(32, int(math.floor(10.0 ** (4.0 + 3.0 * u[t]) * row_scale)))
        L = 10.0 ** (2.0 * (1.0 - v[t]))
        tabs.append(TableSpec(rows=E, dim=int(dims[t]), pooling=float(L), alpha=float(alphas[t])))
    tabs.sort(key=lambda s: s.dim)      # stable: one contiguous table range per dim
    return _finish_tables(tabs, rng)


def config3(seed: int = 0, row_scale: float = 1.0, batch: int = 16384, tables: int = 64) -> ModelSpec:
    """64 heterogeneous tables: rows log-uniform 1e4-1e7, dim 64/128/256, pooling 1-100
    anti-correlated with size, Zipf 0.8-1.3, fp16, batch 16384, all in HBM."""
    rng = np.random.default_rng([seed, 3])
    return ModelSpec("cfg3", _hetero_tables(rng, tables, row_scale), FP16, batch, "poisson", seed=seed)


BENCH_CFG4_BUDGET_GB = 20.0     # HBM budget bench.py runs configuration 4 at (80 GB of host rows)


def config4(seed: int = 0, hbm_budget_gb: Optional[float] = None, batch: int = 16384,
            tables: int = 64, n_batches: int = 200) -> ModelSpec:
    """The config-3 mix with every table's rows scaled so total weights = 4 x an HBM budget
    (default 40 GB, override MTRAINS_HBM_BUDGET_GB); rows in pinned host memory behind
    32-way LRU caches holding 10% of rows; 70% of indices resampled from the last 8 batches."""
    if hbm_budget_gb is None:
        hbm_budget_gb = float(os.environ.get("MTRAINS_HBM_BUDGET_GB", "40"))
    rng = np.random.default_rng([seed, 3])
    base = _hetero_tables(rng, tables, 1.0)
    base_bytes = sum(t.rows * t.dim * 2 for t in base)
    factor = 4.0 * hbm_budget_gb * 1e9 / base_bytes
    tabs = [dataclasses.replace(t, rows=max(32, int(t.rows * factor))) for t in base]
    tabs = _finish_tables(tabs, np.random.default_rng([seed, 4]))
    return ModelSpec("cfg4", tabs, FP16, batch, "poisson", seed=seed, cached=True,
                     cache_fraction=0.10, reuse_prob=0.7, reuse_window=8, n_batches=n_batches,
                     note=f"hbm_budget_gb={hbm_budget_gb:g}")


def config5(seed: int = 0, rows: int = 50_000_000, batch: int = 16384, pooling: int = 50,
            alpha: float = 1.0, cache_fraction: float = 0.10, n_batches: int = 60) -> ModelSpec:
    """One 50M-row x dim 128 fp16 table behind a cache; one point of the throughput sweep."""
    rng = np.random.default_rng([seed, 5])
    tabs = _finish_tables([TableSpec(rows=rows, dim=128, pooling=pooling, alpha=alpha)], rng)
    return ModelSpec("cfg5", tabs, FP16, batch, "fixed", seed=seed, cached=True,
                     cache_fraction=cache_fraction, n_batches=n_batches)


def cache_sets_for(rows_in_group: int, fraction: float, ways: int = 32) -> int:
    """Number of sets of a cache holding `fraction` of a table group's rows."""
    return max(1, int(math.ceil(rows_in_group * fraction / ways)))
