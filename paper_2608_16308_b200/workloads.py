"""Seeded synthetic inputs shaped like the paper's workloads (Section 5.1 lists the real ones:
SuiteSparse matrices, symmetric graphs and three pruned LLMs, none of which are available
offline).  This module holds input generation only -- none of the method's arithmetic --
so both the CPU oracle's tests and the CUDA path's tests/benchmark may use it.

Randomness is counter based: every random number is a pure function of
(seed, stream id, element index), so any element can be regenerated independently and the
result does not depend on numpy's PRNG version.

All matrices are returned as CSR: ``row_ptr`` int64 (m+1), ``col_idx`` int32 sorted within a
row, ``val`` float32 (or None for pattern matrices).  Values are always assigned after the
structure is final, in sorted (row, col) order.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np

_U64 = np.uint64
_GOLD = _U64(0x9E3779B97F4A7C15)
_M1 = _U64(0xBF58476D1CE4E5B9)
_M2 = _U64(0x94D049BB133111EB)


def _mix64(x: np.ndarray) -> np.ndarray:
    """64-bit finaliser (splitmix64's output function) applied element-wise."""
    x = x.astype(_U64, copy=True)
    x ^= x >> _U64(30)
    x *= _M1
    x ^= x >> _U64(27)
    x *= _M2
    x ^= x >> _U64(31)
    return x


def rand_u64(seed: int, stream: int, idx) -> np.ndarray:
    """Uniform 64-bit integers, a pure function of (seed, stream, idx)."""
    with np.errstate(over="ignore"):
        idx = np.asarray(idx, dtype=_U64)
        key = _mix64(np.asarray([(seed * 0x632BE59BD9B4E019 + stream * 0xD1342543DE82EF95 + 1)
                                 & 0xFFFFFFFFFFFFFFFF], dtype=_U64))[0]
        return _mix64(idx * _GOLD + key)


def rand_f32(seed: int, stream: int, idx) -> np.ndarray:
    """Uniform float32 in [0, 1) from the top 24 bits."""
    return ((rand_u64(seed, stream, idx) >> _U64(40)).astype(np.float32)
            * np.float32(1.0 / (1 << 24)))


def rand_f64(seed: int, stream: int, idx) -> np.ndarray:
    """Uniform float64 in [0, 1) from the top 53 bits."""
    return (rand_u64(seed, stream, idx) >> _U64(11)).astype(np.float64) * (1.0 / (1 << 53))


def rand_below(seed: int, stream: int, idx, n: int) -> np.ndarray:
    """Uniform integers in [0, n) (n < 2**32) by multiply-shift on the top 32 bits."""
    hi = rand_u64(seed, stream, idx) >> _U64(32)
    return ((hi * _U64(n)) >> _U64(32)).astype(np.int64)


def rand_normal_f32(seed: int, stream: int, idx) -> np.ndarray:
    """Standard normals by Box-Muller on two independent uniform streams."""
    idx = np.asarray(idx, dtype=_U64)
    u1 = 1.0 - rand_f64(seed, stream, idx * _U64(2))          # (0, 1]
    u2 = rand_f64(seed, stream, idx * _U64(2) + _U64(1))
    return (np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)).astype(np.float32)


def distinct_indices(seed: int, stream: int, n: int, k: int) -> np.ndarray:
    """k distinct uniform indices in [0, n): sequential draws, a draw equal to an earlier
    accepted index is rejected.  Returned in draw order."""
    if k > n:
        raise ValueError("k > n")
    out = np.empty(k, dtype=np.int64)
    seen = np.zeros(n, dtype=bool)
    got, ctr = 0, 0
    while got < k:
        batch = max(1024, 2 * (k - got))
        cand = rand_below(seed, stream, np.arange(ctr, ctr + batch, dtype=np.uint64), n)
        ctr += batch
        _, first = np.unique(cand, return_index=True)
        keep = np.zeros(batch, dtype=bool)
        keep[first] = True
        keep &= ~seen[cand]
        acc = cand[keep][: k - got]
        out[got:got + acc.size] = acc
        seen[acc] = True
        got += acc.size
    return out


@dataclass
class CSR:
    m: int
    n: int
    row_ptr: np.ndarray            # int64, m+1
    col_idx: np.ndarray            # int32, nnz
    val: Optional[np.ndarray]      # float32 nnz, or None (pattern)

    @property
    def nnz(self) -> int:
        return int(self.row_ptr[-1])

    def rows(self) -> np.ndarray:
        """Row index of every stored entry (int32)."""
        return np.repeat(np.arange(self.m, dtype=np.int32), np.diff(self.row_ptr))


@dataclass
class SparseVec:
    n: int
    idx: np.ndarray                # int32, distinct, arbitrary order
    val: Optional[np.ndarray]      # float32 or None


def sorted_unique(keys: np.ndarray) -> np.ndarray:
    """Sorted distinct values (sort + neighbour compare; much faster than np.unique here)."""
    keys = np.sort(keys)
    if keys.size == 0:
        return keys
    keep = np.empty(keys.size, dtype=bool)
    keep[0] = True
    np.not_equal(keys[1:], keys[:-1], out=keep[1:])
    return keys[keep]


def csr_from_sorted_keys(m: int, n: int, keys: np.ndarray) -> tuple[np.ndarray, np.ndarray]:
    """keys = row*n + col, sorted and unique -> (row_ptr int64, col_idx int32)."""
    rows = keys // n
    cols = (keys - rows * n).astype(np.int32)
    counts = np.bincount(rows, minlength=m)
    row_ptr = np.zeros(m + 1, dtype=np.int64)
    np.cumsum(counts, out=row_ptr[1:])
    return row_ptr, cols


def _values_uniform(seed: int, stream: int, nnz: int, lo: float, hi: float) -> np.ndarray:
    out = np.empty(nnz, dtype=np.float32)
    step = 1 << 24
    for s in range(0, nnz, step):
        e = min(nnz, s + step)
        u = rand_f32(seed, stream, np.arange(s, e, dtype=np.uint64))
        out[s:e] = np.float32(lo) + np.float32(hi - lo) * u
    return out


def sparse_x(seed: int, stream: int, n: int, k: int, values: bool = True) -> SparseVec:
    """k distinct uniform positions, float32 values U(-1, 1) (never exactly 0)."""
    idx = distinct_indices(seed, stream, n, k).astype(np.int32)
    val = None
    if values:
        val = _values_uniform(seed, stream + 1000, k, -1.0, 1.0)
        val[val == 0.0] = np.float32(0.5)
    return SparseVec(n, idx, val)


# ----------------------------------------------------------------------------------------
# Config 0: uniform random matrix, fixed number of nonzeros per row
# ----------------------------------------------------------------------------------------
def uniform_rows(n: int = 16384, per_row: int = 8, seed: int = 0) -> CSR:
    """n x n, exactly `per_row` distinct uniformly random columns in every row; U(-1,1)."""
    tries = per_row * 3
    rows = np.arange(n, dtype=np.uint64)
    cols = np.empty((n, per_row), dtype=np.int64)
    for r0 in range(0, n, 65536):
        r1 = min(n, r0 + 65536)
        ctr = rows[r0:r1, None] * np.uint64(1 << 16) + np.arange(tries, dtype=np.uint64)[None, :]
        cand = rand_below(seed, 0, ctr, n)
        dup = np.zeros(cand.shape, dtype=bool)
        for t in range(1, tries):
            dup[:, t] = (cand[:, :t] == cand[:, t:t + 1]).any(axis=1)
        rank = np.cumsum(~dup, axis=1)
        take = (~dup) & (rank <= per_row)
        if not (take.sum(axis=1) == per_row).all():
            raise RuntimeError("not enough distinct draws; raise `tries`")
        cols[r0:r1] = cand[take].reshape(r1 - r0, per_row)
    cols.sort(axis=1)
    row_ptr = np.arange(0, (n + 1) * per_row, per_row, dtype=np.int64)
    col_idx = cols.reshape(-1).astype(np.int32)
    val = _values_uniform(seed, 1, col_idx.size, -1.0, 1.0)
    return CSR(n, n, row_ptr, col_idx, val)


# ----------------------------------------------------------------------------------------
# Configs 1 and 3: R-MAT
# ----------------------------------------------------------------------------------------
def rmat_keys(scale: int, edge_factor: int, seed: int,
              probs=(0.57, 0.19, 0.19, 0.05)) -> np.ndarray:
    """Raw R-MAT edge draws as keys row*n + col (int64), duplicates and self loops kept."""
    n = 1 << scale
    ne = edge_factor * n
    a, b, c, _ = probs
    t1, t2, t3 = a, a + b, a + b + c
    keys = np.empty(ne, dtype=np.int64)
    # integer thresholds on 32-bit uniform chunks; two levels are drawn from each 64-bit hash
    q1, q2, q3 = (np.uint32(int(t * 4294967296.0)) for t in (t1, t2, t3))
    step = 1 << 22
    for s in range(0, ne, step):
        e = min(ne, s + step)
        idx = np.arange(s, e, dtype=np.uint64)
        row = np.zeros(e - s, dtype=np.int64)
        col = np.zeros(e - s, dtype=np.int64)
        for lvl in range(scale):
            if lvl % 2 == 0:
                h = rand_u64(seed, 16 + lvl // 2, idx)
                u = (h >> _U64(32)).astype(np.uint32)
            else:
                u = h.astype(np.uint32)          # low 32 bits
            rbit = u >= q2                       # quadrants c and d are the lower half
            cbit = ((u >= q1) & ~rbit) | (u >= q3)
            row <<= 1
            row |= rbit
            col <<= 1
            col |= cbit
        keys[s:e] = row * n + col
    return keys


def vertex_permutation(n: int, seed: int, stream: int = 9) -> np.ndarray:
    """A seeded permutation of 0..n-1 (argsort of counter-based random keys, ties by index)."""
    return np.argsort(rand_u64(seed, stream, np.arange(n, dtype=np.uint64)), kind="stable").astype(np.int64)


def rmat(scale: int = 20, edge_factor: int = 16, seed: int = 1, values: bool = True,
         symmetrise: bool = False, relabel: bool = False) -> CSR:
    """R-MAT power-law matrix; duplicates merged.  With `symmetrise`, self loops are dropped
    and every edge gets its reverse (the BFS graph of the paper's DB-BFS experiments is
    symmetric, Section 5.1).  With `relabel`, rows and columns are renumbered by one seeded
    permutation (the Graph500 habit): the hubs no longer sit next to each other at the low
    indices.  The configurations of the paper's workloads use no relabelling."""
    n = 1 << scale
    keys = rmat_keys(scale, edge_factor, seed)
    if relabel:
        perm = vertex_permutation(n, seed)
        r = keys // n
        keys = perm[r] * n + perm[keys - r * n]
        del r, perm
    if symmetrise:
        r = keys // n
        c = keys - r * n
        keep = r != c
        r, c = r[keep], c[keep]
        keys = np.concatenate([r * n + c, c * n + r])
        del r, c
    keys = sorted_unique(keys)
    row_ptr, col_idx = csr_from_sorted_keys(n, n, keys)
    del keys
    val = _values_uniform(seed, 2, col_idx.size, -1.0, 1.0) if values else None
    return CSR(n, n, row_ptr, col_idx, val)


def rmat_x(n: int, fraction: float, point: int) -> SparseVec:
    """Input vector of the sparsity sweep: round(n*fraction) distinct uniform positions."""
    k = int(np.floor(n * fraction + 0.5))
    return sparse_x(100 + point, 0, n, k)


RMAT_SWEEP = (1e-5, 1e-4, 1e-3, 1e-2, 1e-1, 0.5)


def bfs_sources(g: CSR, count: int = 16, seed: int = 4) -> np.ndarray:
    """The first `count` vertices with degree > 0 from a seeded uniform stream."""
    deg = np.diff(g.row_ptr)
    out, seen, ctr = [], set(), 0
    while len(out) < count:
        cand = rand_below(seed, 0, np.arange(ctr, ctr + 256, dtype=np.uint64), g.n)
        ctr += 256
        for v in cand:
            v = int(v)
            if deg[v] > 0 and v not in seen:
                seen.add(v)
                out.append(v)
                if len(out) == count:
                    break
    return np.asarray(out, dtype=np.int32)


# ----------------------------------------------------------------------------------------
# Config 2: 27-point stencil on a d^3 grid, clustered x
# ----------------------------------------------------------------------------------------
def stencil27(d: int = 160, seed: int = 2, values: bool = True) -> CSR:
    """Grid index = x + d*(y + d*z); entry (i, j) for every in-grid j with Chebyshev
    distance <= 1 (diagonal included).  Off-diagonals U(0.5, 1.5), diagonal 27."""
    n = d * d * d
    ar = np.arange(d, dtype=np.int32)
    z, y, x = np.meshgrid(ar, ar, ar, indexing="ij")
    x, y, z = x.reshape(-1), y.reshape(-1), z.reshape(-1)
    cols = np.full((n, 27), -1, dtype=np.int32)
    k = 0
    for dz in (-1, 0, 1):
        okz = (z + dz >= 0) & (z + dz < d)
        for dy in (-1, 0, 1):
            oky = okz & (y + dy >= 0) & (y + dy < d)
            for dx in (-1, 0, 1):
                ok = oky & (x + dx >= 0) & (x + dx < d)
                off = dx + d * (dy + d * dz)
                cols[ok, k] = np.arange(n, dtype=np.int32)[ok] + off
                k += 1
    valid = cols >= 0
    counts = valid.sum(axis=1)
    row_ptr = np.zeros(n + 1, dtype=np.int64)
    np.cumsum(counts, out=row_ptr[1:])
    col_idx = cols[valid]
    del cols, valid
    val = None
    if values:
        val = _values_uniform(seed, 1, col_idx.size, 0.5, 1.5)
        rows = np.repeat(np.arange(n, dtype=np.int32), counts)
        val[rows == col_idx] = np.float32(27.0)
    return CSR(n, n, row_ptr, col_idx, val)


def clustered_x(n: int, runs: int, run_len: int = 64, seed: int = 2, stream: int = 7
                ) -> SparseVec:
    """`runs` runs of `run_len` consecutive indices; starts uniform in [0, n-run_len]; a start
    is redrawn if its run overlaps an earlier one.  Runs are not aligned to vector blocks."""
    used = np.zeros(n, dtype=bool)
    starts, ctr = [], 0
    while len(starts) < runs:
        cand = rand_below(seed, stream, np.arange(ctr, ctr + 4096, dtype=np.uint64),
                          n - run_len + 1)
        ctr += 4096
        for s in cand:
            s = int(s)
            if not used[s:s + run_len].any():
                used[s:s + run_len] = True
                starts.append(s)
                if len(starts) == runs:
                    break
    idx = (np.asarray(starts, dtype=np.int64)[:, None] + np.arange(run_len)[None, :]).reshape(-1)
    val = _values_uniform(seed, stream + 1000, idx.size, -1.0, 1.0)
    val[val == 0.0] = np.float32(0.5)
    return SparseVec(n, idx.astype(np.int32), val)


# ----------------------------------------------------------------------------------------
# Config 4: single-token linear layers (bf16 weights, magnitude pruned; ReLU activations)
# ----------------------------------------------------------------------------------------
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bfloat16, returned as uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


DECODE_SHAPES = ((12288, 4096), (11008, 4096), (4096, 11008))


def pruned_weight(m: int, n: int, prune: float, seed: int = 5, stream: int = 0) -> CSR:
    """N(0, 0.02) weights; the floor(prune*m*n) smallest |w| (fp32, ties to the lower linear
    index) are removed; survivors rounded to bf16.  `val` holds the bf16 values widened back
    to float32 (exactly representable)."""
    tot = m * n
    w = np.empty(tot, dtype=np.float32)
    step = 1 << 23
    for s in range(0, tot, step):
        e = min(tot, s + step)
        w[s:e] = np.float32(0.02) * rand_normal_f32(seed, stream, np.arange(s, e, dtype=np.uint64))
    k = int(np.floor(prune * tot))
    keep = np.ones(tot, dtype=bool)
    if k > 0:
        aw = np.abs(w)
        thr = np.partition(aw, k - 1)[k - 1]
        below = aw < thr
        keep[below] = False
        need = k - int(below.sum())
        ties = np.flatnonzero(aw == thr)
        keep[ties[:need]] = False
    keep2 = keep.reshape(m, n)
    counts = keep2.sum(axis=1)
    row_ptr = np.zeros(m + 1, dtype=np.int64)
    np.cumsum(counts, out=row_ptr[1:])
    col_idx = np.nonzero(keep2)[1].astype(np.int32)
    val = bf16_bits_to_f32(f32_to_bf16_bits(w[keep]))
    return CSR(m, n, row_ptr, col_idx, val)


def relu_activation(n: int, zero_fraction: float, seed: int = 5, stream: int = 50) -> np.ndarray:
    """Dense activation x = ReLU(N(mu, 1)) rounded to bf16 (returned widened to float32), with
    mu = -Phi^{-1}(zero_fraction) so that about `zero_fraction` of the entries are zero."""
    mu = {0.7: -0.5244005127080407, 0.9: -1.2815515655446004}.get(zero_fraction)
    if mu is None:
        from statistics import NormalDist
        mu = -NormalDist().inv_cdf(zero_fraction)
    z = rand_normal_f32(seed, stream, np.arange(n, dtype=np.uint64)) + np.float32(mu)
    x = np.maximum(z, np.float32(0.0))
    return bf16_bits_to_f32(f32_to_bf16_bits(x))


# ----------------------------------------------------------------------------------------
# Small random matrices for unit tests
# ----------------------------------------------------------------------------------------
def random_sparse(m: int, n: int, nnz: int, seed: int, values: bool = True,
                  integer_values: bool = False) -> CSR:
    """Up to nnz uniformly placed entries (duplicates merged)."""
    keys = rand_below(seed, 0, np.arange(nnz, dtype=np.uint64), m) * n \
        + rand_below(seed, 1, np.arange(nnz, dtype=np.uint64), n)
    keys = sorted_unique(keys)
    row_ptr, col_idx = csr_from_sorted_keys(m, n, keys)
    val = None
    if values:
        if integer_values:
            val = (rand_below(seed, 2, np.arange(keys.size, dtype=np.uint64), 17) - 8
                   ).astype(np.float32)
        else:
            val = _values_uniform(seed, 2, keys.size, -1.0, 1.0)
    return CSR(m, n, row_ptr, col_idx, val)


def csr_from_dense(a: np.ndarray, keep_zeros_mask: Optional[np.ndarray] = None) -> CSR:
    """CSR of the entries where `keep_zeros_mask` (default: a != 0) is true."""
    mask = (a != 0) if keep_zeros_mask is None else keep_zeros_mask
    m, n = a.shape
    counts = mask.sum(axis=1)
    row_ptr = np.zeros(m + 1, dtype=np.int64)
    np.cumsum(counts, out=row_ptr[1:])
    col_idx = np.nonzero(mask)[1].astype(np.int32)
    return CSR(m, n, row_ptr, col_idx, a[mask].astype(np.float32))
