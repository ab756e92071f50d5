"""CPU oracle (test infrastructure only): ctypes binding of ``bls_oracle.c``.

Nothing under ``oracle/`` may be imported by the product package; it exists so
that tests, the smoke check and the benchmark's CPU-baseline leg can state what
the hot path must compute.  It shares no code with the CUDA library.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bls_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

PART = {"table_rr": 0, "row_block": 1}
DTYPE = {"f32": 0, "bf16": 1, "f16": 2}


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (idempotent)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


class _Table(C.Structure):
    _fields_ = [("data", C.c_void_p), ("rows", C.c_int64), ("dim", C.c_int32),
                ("dtype", C.c_int32), ("seed", C.c_uint64), ("index", C.c_int32)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_subbags_per_pair.restype = C.c_int64
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _tables(specs, data: Optional[Sequence[Optional[np.ndarray]]]):
    arr = (_Table * len(specs))()
    keep = []
    for i, s in enumerate(specs):
        d = None if data is None else data[i]
        if d is not None:
            d = np.ascontiguousarray(d)
            keep.append(d)
        arr[i] = _Table(None if d is None else d.ctypes.data, s.rows, s.dim, DTYPE[s.dtype],
                        s.seed & ((1 << 64) - 1), s.index)
    return arr, keep


def subbags_per_pair(part: str, P: int, T: int, b: int, dst: int) -> int:
    return int(lib().oracle_subbags_per_pair(PART[part], P, T, b, dst))


def route(P: int, T: int, b: int, part: str, rows: Sequence[int], ids: np.ndarray,
          offsets: np.ndarray, nthreads: int = 1) -> dict:
    """Routing artefacts of one iteration (step 1); see ``oracle_route`` in the C file."""
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    offsets = np.ascontiguousarray(offsets, dtype=np.int32)
    rows_a = np.ascontiguousarray(rows, dtype=np.int64)
    L = int(offsets[-1])
    n_sub = sum(P * subbags_per_pair(part, P, T, b, d) for d in range(P))
    out = {
        "sendcounts": np.zeros((P, P), np.int32), "sdispls": np.zeros((P, P), np.int32),
        "recvcounts": np.zeros((P, P), np.int32), "rdispls": np.zeros((P, P), np.int32),
        "sendbuf": np.full(L, -1, np.int32), "recvbuf": np.full(L, -1, np.int32),
        "sublen": np.full(n_sub, -1, np.int32),
    }
    rc = lib().oracle_route(P, T, b, PART[part], _p(rows_a), _p(ids), _p(offsets),
                            _p(out["sendcounts"]), _p(out["sdispls"]), _p(out["recvcounts"]),
                            _p(out["rdispls"]), _p(out["sendbuf"]), _p(out["recvbuf"]),
                            _p(out["sublen"]), nthreads)
    if rc != 0:
        raise ValueError("oracle_route: id out of range or offsets not monotone")
    return out


def pool_definition(P: int, T: int, b: int, specs, data, ids: np.ndarray, offsets: np.ndarray,
                    sel: Optional[np.ndarray] = None, nthreads: int = 1) -> np.ndarray:
    """Pooled output by the plain definition: out[src][s][t][:] (or [len(sel)][D])."""
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    offsets = np.ascontiguousarray(offsets, dtype=np.int32)
    tabs, keep = _tables(specs, data)
    D = specs[0].dim
    if sel is None:
        out = np.zeros((P, b, T, D), np.float32)
        n_sel, selp = 0, None
    else:
        sel = np.ascontiguousarray(sel, dtype=np.int64)
        out = np.zeros((len(sel), D), np.float32)
        n_sel, selp = len(sel), _p(sel)
    rc = lib().oracle_pool_definition(P, T, b, tabs, _p(ids), _p(offsets), C.c_int64(n_sel), selp,
                                      _p(out), nthreads)
    assert rc == 0
    return out


def pool_routed(P: int, T: int, b: int, part: str, specs, data, art: dict) -> np.ndarray:
    """Pooled output by following the routed buffers (steps 2 and 3)."""
    tabs, keep = _tables(specs, data)
    D = specs[0].dim
    out = np.zeros((P, b, T, D), np.float32)
    rc = lib().oracle_pool_routed(P, T, b, PART[part], tabs, _p(art["recvbuf"]),
                                  _p(art["recvcounts"]), _p(art["rdispls"]), _p(art["sublen"]), _p(out))
    if rc != 0:
        raise ValueError(f"oracle_pool_routed failed ({rc}): sub-bag lengths do not add up")
    return out


def fill_table(spec, row_lo: int = 0, nrows: Optional[int] = None, nthreads: int = 1) -> np.ndarray:
    """Materialise rows of a counter-hash table (fp32 array or uint16 bit patterns)."""
    nrows = spec.rows - row_lo if nrows is None else nrows
    out = np.empty((nrows, spec.dim), np.float32 if spec.dtype == "f32" else np.uint16)
    lib().oracle_fill_table(C.c_uint64(spec.seed & ((1 << 64) - 1)), spec.index, C.c_int64(row_lo),
                            C.c_int64(nrows), spec.dim, DTYPE[spec.dtype], _p(out), nthreads)
    return out


def vector_rel_err(got: np.ndarray, want: np.ndarray) -> float:
    """Headline error figure: per output vector, max_c|g-o| / max_c|o|, maximised
    over vectors (vectors whose reference is all zero must match exactly)."""
    g = np.asarray(got, np.float64).reshape(-1, got.shape[-1])
    o = np.asarray(want, np.float64).reshape(-1, want.shape[-1])
    num = np.abs(g - o).max(axis=1)
    den = np.abs(o).max(axis=1)
    zero = den == 0
    if np.any(num[zero] != 0):
        return float("inf")
    if np.all(zero):
        return 0.0
    return float((num[~zero] / den[~zero]).max())
