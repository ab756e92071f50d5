"""Seeded synthetic inputs for the BLS distributed embedding lookup.

This module only *generates inputs* (table values, sparse IDs, bag offsets,
workload shapes).  It contains none of the method's arithmetic: no owner map,
no routing, no pooling, no slot ring.  Both the CPU oracle's tests and the CUDA
path's tests and benchmark draw their inputs from here so that the two sides
see identical data.

Workload shapes follow the paper's experimental section: 26 tables with up to
about 1e6 rows and one ID per table per sample stand in for the click-log
datasets (Section V-F), and bags of 1..100 IDs per table stand in for the
heterogeneous-message-size setting (Section V-E, setting 1).  No dataset item
is reproduced; everything is drawn from seeded generators.

Input layout (shared by every consumer):
  * P logical ranks, T tables, local batch b, global batch B = P*b.
  * A bag is (src, t, s): sample s of requester rank src, table t.  Bags are
    ordered (src, t, s), so the flat bag index is g = (src*T + t)*b + s.
  * ``offsets`` is int32 [G+1] (exclusive prefix of bag lengths, G = P*T*b)
    and ``ids`` is int32 [L], flat in bag order.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Tuple

import numpy as np

__all__ = [
    "TableSpec", "Workload", "workload", "tiny_workload", "table_rows",
    "table_values", "hash_rows", "make_iteration", "table_permutation",
    "HASH_SCALE_F32",
]

_MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
# sum of four independent uniform 16-bit integers has mean 4*32767.5 and
# variance 4*(65536^2-1)/12; the scale brings it to (about) unit variance.
_HASH_MEAN = 131070
HASH_SCALE_F32 = np.float32(1.0 / np.sqrt(4.0 * (65536.0 ** 2 - 1.0) / 12.0))

_DT_BYTES = {"f32": 4, "bf16": 2, "f16": 2}


@dataclass(frozen=True)
class TableSpec:
    rows: int
    dim: int
    dtype: str          # "f32" | "bf16" | "f16"  (storage type)
    kind: str           # "normal" (numpy standard_normal) | "hash" (counter hash)
    seed: int
    index: int          # table number t


@dataclass(frozen=True)
class Workload:
    name: str
    number: int                 # 1..5 for the five benchmark shapes, 0 for ad-hoc
    tables: Tuple[TableSpec, ...]
    P: int
    partition: str              # "table_rr" | "row_block"
    local_batch: int
    lengths: str                # "one" | "poisson20c" | "poisson10" | "pareto15c" | "mixed"
    id_dist: str                # "uniform" | "zipf"
    zipf_s: float
    hot_ranges: Tuple[Tuple[int, int], ...]   # tables 0..7: the hottest rows land alternately in these row ranges; () = anywhere
    iterations: int
    ks: Tuple[int, ...]
    seed: int

    @property
    def T(self) -> int:
        return len(self.tables)

    @property
    def global_batch(self) -> int:
        return self.P * self.local_batch

    @property
    def n_bags(self) -> int:
        return self.P * self.T * self.local_batch

    def table_bytes(self) -> int:
        return sum(t.rows * t.dim * _DT_BYTES[t.dtype] for t in self.tables)


# --------------------------------------------------------------------------
# workload shapes
# --------------------------------------------------------------------------
def _specs(rows, dim, dtype, kind, seed):
    return tuple(TableSpec(int(r), dim, dtype, kind, seed, i) for i, r in enumerate(rows))


def workload(number: int, rows_scale: float = 1.0, batch_scale: float = 1.0) -> Workload:
    """The five benchmark shapes.  ``rows_scale``/``batch_scale`` < 1 shrink
    table heights and the batch for CPU-sized parity cases; 1.0 is full size."""
    def rs(n):
        return max(8, int(round(n * rows_scale)))

    def bs(n, P):
        return max(1, int(round(n * batch_scale / P)))

    if number == 1:
        P = 4
        tables = _specs([rs(10_000)] * 8, 16, "f32", "normal", 0)
        return Workload("cfg1_onehot_8x10k_d16", 1, tables, P, "table_rr", bs(256, P),
                        "one", "uniform", 0.0, (), 10, (0, 2), 1000)
    if number == 2:
        P = 8
        rng = np.random.Generator(np.random.PCG64(2001))
        rows = np.floor(10.0 ** rng.uniform(3.0, 6.0, size=26)).astype(np.int64)
        tables = _specs([rs(r) for r in rows], 16, "f32", "normal", 2000)
        return Workload("cfg2_onehot_26xlogu_d16", 2, tables, P, "table_rr", bs(2048, P),
                        "one", "uniform", 0.0, (), 100, (0, 1, 4), 2000)
    if number == 3:
        P = 8
        tables = _specs([rs(1_000_000)] * 26, 64, "f32", "hash", 3000)
        return Workload("cfg3_zipf_multihot_26x1m_d64", 3, tables, P, "table_rr", bs(16384, P),
                        "poisson20c", "zipf", 1.05, (), 100, (0, 1, 4), 3000)
    if number == 4:
        P = 16
        n = rs(2_000_000)
        tables = _specs([n] * 64, 128, "bf16", "hash", 4000)
        # "the 8 hottest tables' hot rows placed on 2 ranks": the first and the second sixteenth of the rows
        sixteenth = max(1, n // 16)
        return Workload("cfg4_unbalanced_rowwise_64x2m_d128_bf16", 4, tables, P, "row_block",
                        bs(32768, P), "poisson10", "zipf", 1.2,
                        ((0, sixteenth), (sixteenth, min(n, 2 * sixteenth))), 200, (0, 1, 2, 8), 4000)
    if number == 5:
        P = 32
        tables = _specs([rs(5_000_000)] * 100, 64, "f16", "hash", 5000)
        return Workload("cfg5_large_100x5m_d64_f16", 5, tables, P, "table_rr", bs(65536, P),
                        "pareto15c", "zipf", 1.1, (), 100, (4,), 5000)
    raise ValueError("workload number must be 1..5")


def tiny_workload(T=3, P=2, b=2, rows=7, dim=4, dtype="f32", partition="table_rr",
                  lengths="mixed", seed=7, id_dist="uniform", zipf_s=0.0) -> Workload:
    """Ad-hoc small shapes for brute-force and edge-case tests."""
    rows_l = rows if isinstance(rows, (list, tuple)) else [rows] * T
    tables = _specs(rows_l, dim, dtype, "normal", seed)
    return Workload(f"tiny_T{T}_P{P}_b{b}", 0, tables, P, partition, b, lengths, id_dist,
                    zipf_s, (), 4, (0, 1, 2), seed)


# --------------------------------------------------------------------------
# table values
# --------------------------------------------------------------------------
def _splitmix64(x: np.ndarray) -> np.ndarray:
    """Output function of the SplitMix64 generator (Steele, Lea, Flood 2014)
    applied to an already-advanced state ``x`` (uint64 array)."""
    z = x.copy()
    z ^= z >> np.uint64(30)
    z *= np.uint64(0xBF58476D1CE4E5B9)
    z ^= z >> np.uint64(27)
    z *= np.uint64(0x94D049BB133111EB)
    z ^= z >> np.uint64(31)
    return z


def _f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    u = x.astype(np.float32).view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    u = u + np.uint64(0x7FFF) + lsb
    return (u >> np.uint64(16)).astype(np.uint16)


def hash_rows(seed: int, t: int, row_idx: np.ndarray, dim: int, dtype: str) -> np.ndarray:
    """Counter-hash table values for the given rows of table ``t``.

    Element (row, c) is: the (counter+1)-th SplitMix64 output for seed ``seed``
    with counter = t<<48 | row<<16 | c; its four 16-bit fields are summed, the
    mean 131070 is subtracted (an exact integer), the result is converted to
    fp32 (exact) and multiplied once by ``HASH_SCALE_F32`` in fp32, then rounded
    to the storage type.  Returns fp32, or uint16 bit patterns for bf16, or
    float16.
    """
    rows = np.asarray(row_idx, dtype=np.uint64).reshape(-1, 1)
    c = np.arange(dim, dtype=np.uint64).reshape(1, -1)
    counter = (np.uint64(t) << np.uint64(48)) | (rows << np.uint64(16)) | c
    with np.errstate(over="ignore"):
        state = np.uint64(seed & _MASK64) + (counter + np.uint64(1)) * np.uint64(_GOLDEN)
        z = _splitmix64(state)
    m = np.uint64(0xFFFF)
    s = ((z & m) + ((z >> np.uint64(16)) & m) + ((z >> np.uint64(32)) & m)
         + ((z >> np.uint64(48)) & m)).astype(np.int64) - _HASH_MEAN
    v = s.astype(np.float32) * HASH_SCALE_F32
    if dtype == "f32":
        return v
    if dtype == "f16":
        return v.astype(np.float16)
    if dtype == "bf16":
        return _f32_to_bf16_bits(v)
    raise ValueError(dtype)


def table_rows(spec: TableSpec, row_idx: np.ndarray) -> np.ndarray:
    """Values of selected rows (hash tables only; normal tables are materialised)."""
    if spec.kind != "hash":
        raise ValueError("row-on-demand needs a hash table; materialise normal tables")
    return hash_rows(spec.seed, spec.index, row_idx, spec.dim, spec.dtype)


def table_values(spec: TableSpec) -> np.ndarray:
    """Materialise a whole table on the host (small/medium tables only).

    fp32 -> float32 array; f16 -> float16 array; bf16 -> uint16 bit patterns.
    """
    if spec.kind == "hash":
        out = []
        step = 1 << 16
        for lo in range(0, spec.rows, step):
            out.append(hash_rows(spec.seed, spec.index,
                                 np.arange(lo, min(spec.rows, lo + step)), spec.dim, spec.dtype))
        return np.concatenate(out, axis=0)
    rng = np.random.Generator(np.random.PCG64([spec.seed, 0, spec.index]))
    v = rng.standard_normal((spec.rows, spec.dim), dtype=np.float32)
    if spec.dtype == "f32":
        return v
    if spec.dtype == "f16":
        return v.astype(np.float16)
    return _f32_to_bf16_bits(v)


# --------------------------------------------------------------------------
# sparse inputs: bag lengths and IDs
# --------------------------------------------------------------------------
_perm_cache: dict = {}
_cdf_cache: dict = {}


def table_permutation(w: Workload, t: int) -> np.ndarray:
    """Random map from popularity rank (0 = hottest) to row number for table t.

    When the workload names row ranges for its hot rows (``hot_ranges``, two of
    them), tables 0..7 place popularity ranks 0..4095 alternately into the first
    and the second range; every other rank/table is uniformly random.
    """
    key = (w.name, w.tables[t].rows, t, w.seed)
    if key in _perm_cache:
        return _perm_cache[key]
    n = w.tables[t].rows
    rng = np.random.Generator(np.random.PCG64([w.seed, 1, t]))
    perm = rng.permutation(n).astype(np.int32)
    if len(w.hot_ranges) == 2 and t < 8:
        (lo0, hi0), (lo1, hi1) = w.hot_ranges
        nhot = min(4096, n // 4, (hi0 - lo0) + (hi1 - lo1))
        if nhot >= 2 and hi1 > lo1:
            # positions (rows) the hot ranks must land on: alternate first range / second range
            half = (nhot + 1) // 2
            r0 = lo0 + rng.choice(hi0 - lo0, size=half, replace=False)
            r1 = lo1 + rng.choice(hi1 - lo1, size=nhot - half, replace=False)
            target = np.empty(nhot, dtype=np.int64)
            target[0::2] = r0
            target[1::2] = r1[: len(target[1::2])]
            inv = np.empty(n, dtype=np.int64)
            inv[perm] = np.arange(n)
            for rank in range(nhot):          # swap so that perm[rank] == target[rank]
                cur = perm[rank]
                want = target[rank]
                if cur == want:
                    continue
                other = inv[want]
                perm[rank], perm[other] = want, cur
                inv[want], inv[cur] = rank, other
    _perm_cache[key] = perm
    return perm


def _zipf_cdf(n: int, s: float) -> np.ndarray:
    key = (n, s)
    if key not in _cdf_cache:
        p = np.arange(1, n + 1, dtype=np.float64) ** (-s)
        c = np.cumsum(p)
        _cdf_cache[key] = c / c[-1]
    return _cdf_cache[key]


def _bag_lengths(w: Workload, rng: np.random.Generator, n: int) -> np.ndarray:
    if w.lengths == "one":
        return np.ones(n, dtype=np.int64)
    if w.lengths == "poisson20c":
        return np.clip(rng.poisson(20.0, size=n), 1, 100).astype(np.int64)
    if w.lengths == "poisson10":                      # zero-length bags allowed
        return rng.poisson(10.0, size=n).astype(np.int64)
    if w.lengths == "pareto15c":
        u = rng.random(n)
        return np.minimum(100, np.floor((1.0 - u) ** (-1.0 / 1.5))).astype(np.int64)
    if w.lengths == "extremes":                       # empty, single and maximum-length (100) bags
        return rng.choice(np.array([0, 1, 100]), size=n).astype(np.int64)
    if w.lengths == "mixed":                          # 0..5 with empties, for edge cases
        return rng.integers(0, 6, size=n).astype(np.int64)
    raise ValueError(w.lengths)


def make_iteration(w: Workload, it: int) -> Tuple[np.ndarray, np.ndarray]:
    """IDs and offsets of iteration ``it``: (ids int32 [L], offsets int32 [G+1])."""
    P, T, b = w.P, w.T, w.local_batch
    G = P * T * b
    rng_len = np.random.Generator(np.random.PCG64([w.seed, 2, it]))
    rng_ids = np.random.Generator(np.random.PCG64([w.seed, 3, it]))
    lens = _bag_lengths(w, rng_len, G)
    offsets = np.zeros(G + 1, dtype=np.int64)
    np.cumsum(lens, out=offsets[1:])
    L = int(offsets[-1])
    if L >= 2 ** 31:
        raise ValueError("iteration too large for int32 offsets")
    u = rng_ids.random(L)
    ids = np.empty(L, dtype=np.int32)
    same = len({tb.rows for tb in w.tables}) == 1
    rank_all = None
    if w.id_dist == "zipf" and same:
        rank_all = np.searchsorted(_zipf_cdf(w.tables[0].rows, w.zipf_s), u, side="left")
        np.minimum(rank_all, w.tables[0].rows - 1, out=rank_all)
    chunk = offsets[::b]                              # boundaries of (src, t) chunks
    for src in range(P):
        for t in range(T):
            lo, hi = int(chunk[src * T + t]), int(chunk[src * T + t + 1])
            if hi == lo:
                continue
            n = w.tables[t].rows
            if w.id_dist == "uniform":
                ids[lo:hi] = np.minimum((u[lo:hi] * n).astype(np.int64), n - 1)
            else:
                if rank_all is not None:
                    r = rank_all[lo:hi]
                else:
                    r = np.minimum(np.searchsorted(_zipf_cdf(n, w.zipf_s), u[lo:hi]), n - 1)
                ids[lo:hi] = table_permutation(w, t)[r]
    return ids, offsets.astype(np.int32)
