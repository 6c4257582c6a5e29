"""CPU ORACLE -- TEST INFRASTRUCTURE ONLY (tests/, the smoke check and the benchmark's
cpu_baseline leg).  The product path never imports this package.

Thin ctypes wrapper over ``ref_spmspv.c``: the textbook push and pull SpMSpV loops of
Algorithm 1 (Section 2.1) in fp64, a queue BFS, and the dense-output decode variant
(Section 4.3), and the (min, +) product with a Bellman-Ford search.  The C file is compiled with gcc on first use (``build()``).  Shares no code
with the CUDA library and does not import it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ref_spmspv.c")
_LIB = os.path.join(_HERE, "libref_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle (plain gcc -O2, no OpenMP: single-threaded by construction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.ref_pull.restype = ctypes.c_int64
        _lib.ref_push.restype = ctypes.c_int64
        _lib.ref_bfs.restype = ctypes.c_int64
        _lib.ref_csr_to_csc.restype = None
        _lib.ref_decode.restype = None
        _lib.ref_minplus.restype = ctypes.c_int64
        _lib.ref_sssp.restype = ctypes.c_int64
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _i64(v):
    return ctypes.c_int64(int(v))


def _prep(a, dt):
    return None if a is None else np.ascontiguousarray(a, dtype=dt)


class RefMatrix:
    """CSR arrays plus the oracle's own CSC transposition (built lazily)."""

    def __init__(self, m, n, row_ptr, col_idx, val=None):
        self.m, self.n = int(m), int(n)
        self.row_ptr = _prep(row_ptr, np.int64)
        self.col_idx = _prep(col_idx, np.int32)
        self.val = _prep(val, np.float32)
        self._csc = None

    @property
    def nnz(self):
        return int(self.row_ptr[-1])

    def csc(self):
        if self._csc is None:
            col_ptr = np.zeros(self.n + 1, dtype=np.int64)
            row_idx = np.empty(max(self.nnz, 1), dtype=np.int32)
            cval = None if self.val is None else np.empty(max(self.nnz, 1), dtype=np.float32)
            _load().ref_csr_to_csc(_i64(self.m), _i64(self.n), _p(self.row_ptr), _p(self.col_idx),
                                   _p(self.val), _p(col_ptr), _p(row_idx), _p(cval))
            self._csc = (col_ptr, row_idx, cval)
        return self._csc


def _result(cnt, y_idx, y_val, y_scale):
    if cnt < 0:
        raise MemoryError("oracle allocation failed")
    return y_idx[:cnt].copy(), y_val[:cnt].copy(), y_scale[:cnt].copy()


def ref_pull(A: RefMatrix, x_idx, x_val=None):
    """Algorithm 1 (pull).  Returns (y_idx int32 ascending, y_val fp64, y_scale fp64).
    x_val None (or a pattern matrix) -> Boolean: y_val counts hits, use y_idx only."""
    x_idx = _prep(x_idx, np.int32)
    x_val = _prep(x_val, np.float32)
    y_idx = np.empty(A.m, dtype=np.int32)
    y_val = np.empty(A.m, dtype=np.float64)
    y_scale = np.empty(A.m, dtype=np.float64)
    cnt = _load().ref_pull(_i64(A.m), _i64(A.n), _p(A.row_ptr), _p(A.col_idx), _p(A.val),
                           _i64(x_idx.size), _p(x_idx), _p(x_val), _p(y_idx), _p(y_val),
                           _p(y_scale))
    return _result(cnt, y_idx, y_val, y_scale)


def ref_push(A: RefMatrix, x_idx, x_val=None):
    """Algorithm 1 (push) over the oracle's CSC copy.  Same return convention as ref_pull."""
    x_idx = _prep(x_idx, np.int32)
    x_val = _prep(x_val, np.float32)
    col_ptr, row_idx, cval = A.csc()
    y_idx = np.empty(A.m, dtype=np.int32)
    y_val = np.empty(A.m, dtype=np.float64)
    y_scale = np.empty(A.m, dtype=np.float64)
    cnt = _load().ref_push(_i64(A.m), _i64(A.n), _p(col_ptr), _p(row_idx), _p(cval),
                           _i64(x_idx.size), _p(x_idx), _p(x_val), _p(y_idx), _p(y_val),
                           _p(y_scale))
    return _result(cnt, y_idx, y_val, y_scale)


def ref_bfs(A: RefMatrix, src: int) -> np.ndarray:
    """Queue BFS; A[i][j] stored = edge j -> i.  int32 levels, source 0, unreachable -1."""
    if A.m != A.n:
        raise ValueError("BFS needs a square matrix")
    col_ptr, row_idx, _ = A.csc()
    levels = np.empty(A.n, dtype=np.int32)
    _load().ref_bfs(_i64(A.n), _p(col_ptr), _p(row_idx), ctypes.c_int32(int(src)), _p(levels))
    return levels


def ref_bfs_levelsync(A: RefMatrix, src: int) -> np.ndarray:
    """BFS as the paper states it (Section 4.2): each level is one Boolean SpMSpV with the
    frontier as x, already visited vertices are stripped from the result, until the frontier
    is empty.  Cross-check for ref_bfs."""
    levels = np.full(A.n, -1, dtype=np.int32)
    levels[src] = 0
    frontier = np.asarray([src], dtype=np.int32)
    depth = 0
    pattern = RefMatrix(A.m, A.n, A.row_ptr, A.col_idx, None)
    while frontier.size:
        depth += 1
        y_idx, _, _ = ref_push(pattern, frontier, None)
        nxt = y_idx[levels[y_idx] < 0]
        levels[nxt] = depth
        frontier = nxt
    return levels


def ref_decode(A: RefMatrix, x_dense):
    """Dense-in, dense-out layer y = W x; zeros of x are structurally absent.  Returns
    (y fp64 length m, scale fp64 length m)."""
    x = _prep(x_dense, np.float32)
    y = np.empty(A.m, dtype=np.float64)
    s = np.empty(A.m, dtype=np.float64)
    _load().ref_decode(_i64(A.m), _i64(A.n), _p(A.row_ptr), _p(A.col_idx), _p(A.val), _p(x),
                       _p(y), _p(s))
    return y, s


def ref_minplus(A: RefMatrix, x_idx, x_val=None):
    """(min, +) SpMSpV: y_i = min_j (A[i][j] + x_j) over stored A[i][j] and listed x_j.
    x_val None -> every listed entry is 0; a pattern matrix -> every weight is 1.
    Returns (y_idx int32 ascending, y_val fp64)."""
    x_idx = _prep(x_idx, np.int32)
    x_val = _prep(x_val, np.float32)
    y_idx = np.empty(A.m, dtype=np.int32)
    y_val = np.empty(A.m, dtype=np.float64)
    cnt = _load().ref_minplus(_i64(A.m), _i64(A.n), _p(A.row_ptr), _p(A.col_idx), _p(A.val),
                              _i64(x_idx.size), _p(x_idx), _p(x_val), _p(y_idx), _p(y_val))
    if cnt < 0:
        raise MemoryError("oracle allocation failed")
    return y_idx[:cnt].copy(), y_val[:cnt].copy()


def ref_sssp(A: RefMatrix, src: int) -> np.ndarray:
    """Bellman-Ford sweeps; A[i][j] stored = edge j -> i of weight A[i][j] (1 for a pattern
    matrix).  fp64 distances, source 0, unreachable +inf."""
    if A.m != A.n:
        raise ValueError("SSSP needs a square matrix")
    col_ptr, row_idx, cval = A.csc()
    dist = np.empty(A.n, dtype=np.float64)
    sweeps = _load().ref_sssp(_i64(A.n), _p(col_ptr), _p(row_idx), _p(cval), ctypes.c_int32(int(src)), _p(dist))
    if sweeps < 0:
        raise ValueError("negative cycle")
    return dist


def ref_sssp_frontier(A: RefMatrix, src: int) -> np.ndarray:
    """The same search as the iteration of (min, +) SpMSpV steps a frontier-driven driver
    makes: x = the vertices whose distance improved in the last step, with their distances;
    y = A (min,+) x; every y_i below dist_i replaces it and puts i on the next frontier.
    Cross-check for ref_sssp."""
    dist = np.full(A.n, np.inf, dtype=np.float64)
    dist[src] = 0.0
    frontier = np.asarray([src], dtype=np.int32)
    steps = 0
    while frontier.size:
        steps += 1
        if steps > A.n + 1:
            raise ValueError("negative cycle")
        y_idx, y_val = ref_minplus(A, frontier, dist[frontier].astype(np.float32))
        better = y_val < dist[y_idx]
        dist[y_idx[better]] = y_val[better]
        frontier = y_idx[better]
    return dist
