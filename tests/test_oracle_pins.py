"""Pins for the CPU oracle: checks against things that are not the oracle itself -- brute-force
dense products, closed forms, invariants and textbook special cases -- chosen so that a dropped
term, a wrong sign or index, or a transposed operand fails at least one of them."""
import numpy as np
import pytest

import oracle
from paper_2608_16308_b200 import workloads as wl


def _mat(csr):
    return oracle.RefMatrix(csr.m, csr.n, csr.row_ptr, csr.col_idx, csr.val)


def _dense(csr):
    a = np.zeros((csr.m, csr.n), dtype=np.float64)
    s = np.zeros((csr.m, csr.n), dtype=bool)
    r = csr.rows()
    a[r, csr.col_idx] = csr.val if csr.val is not None else 1.0
    s[r, csr.col_idx] = True
    return a, s


@pytest.mark.parametrize("m,n,nnz,k,seed", [(1, 1, 1, 1, 0), (7, 5, 12, 3, 1), (33, 64, 300, 9, 2),
                                            (64, 64, 900, 64, 3), (64, 17, 40, 1, 4),
                                            (50, 50, 60, 0, 5)])
def test_brute_force_dense(m, n, nnz, k, seed):
    """Algorithm 1 vs a dense fp64 mat-vec with explicit structural masks (numpy), including
    empty rows/columns and an empty x."""
    csr = wl.random_sparse(m, n, nnz, seed)
    x = wl.sparse_x(seed + 50, 0, n, k)
    a, s = _dense(csr)
    xd = np.zeros(n)
    xp = np.zeros(n, dtype=bool)
    xd[x.idx] = x.val
    xp[x.idx] = True
    want_val = a @ xd
    want_hit = (s.astype(np.int64) @ xp.astype(np.int64)) > 0
    want_scale = np.abs(a) @ np.abs(xd)
    for fn in (oracle.ref_pull, oracle.ref_push):
        yi, yv, ys = fn(_mat(csr), x.idx, x.val)
        assert np.array_equal(yi, np.flatnonzero(want_hit))
        assert np.allclose(yv, want_val[yi], rtol=0, atol=1e-12)
        assert np.allclose(ys, want_scale[yi], rtol=0, atol=1e-12)


def test_structural_hit_with_numeric_cancellation():
    """Row 0 sums 1*2 + (-2)*1 = 0 but is structurally hit; row 1 meets no listed x."""
    a = np.array([[1.0, -2.0, 0.0], [0.0, 0.0, 5.0], [0.0, 3.0, 0.0]], dtype=np.float32)
    csr = wl.csr_from_dense(a)
    for fn in (oracle.ref_pull, oracle.ref_push):
        yi, yv, ys = fn(_mat(csr), np.array([1, 0], np.int32), np.array([1.0, 2.0], np.float32))
        assert yi.tolist() == [0, 2]
        assert yv.tolist() == [0.0, 3.0]
        assert ys.tolist() == [4.0, 3.0]


def test_explicit_zero_entry_is_structural():
    a = np.array([[0.0, 1.0], [1.0, 0.0]], dtype=np.float32)
    keep = np.array([[True, True], [False, False]])
    csr = wl.csr_from_dense(a, keep)
    yi, yv, _ = oracle.ref_pull(_mat(csr), np.array([0], np.int32), np.array([3.0], np.float32))
    assert yi.tolist() == [0] and yv.tolist() == [0.0]


def test_identity_returns_x():
    n = 100
    csr = wl.CSR(n, n, np.arange(n + 1, dtype=np.int64), np.arange(n, dtype=np.int32),
                 np.ones(n, np.float32))
    x = wl.sparse_x(9, 0, n, 17)
    order = np.argsort(x.idx)
    for fn in (oracle.ref_pull, oracle.ref_push):
        yi, yv, _ = fn(_mat(csr), x.idx, x.val)
        assert np.array_equal(yi, x.idx[order])
        assert np.array_equal(yv, x.val[order].astype(np.float64))


def test_permutation_matrix_is_bit_exact_and_not_transposed():
    """A[p[j]][j] = 1: y[p[j]] = x[j].  A transposed operand would give y[j] = x[p[j]]."""
    n = 257
    p = wl.distinct_indices(3, 0, n, n)          # a permutation
    rows, cols = p, np.arange(n)
    order = np.argsort(rows)
    csr = wl.CSR(n, n, np.arange(n + 1, dtype=np.int64), cols[order].astype(np.int32),
                 np.ones(n, np.float32))
    x = wl.sparse_x(11, 0, n, 40)
    want = {int(p[j]): float(v) for j, v in zip(x.idx, x.val)}
    for fn in (oracle.ref_pull, oracle.ref_push):
        yi, yv, _ = fn(_mat(csr), x.idx, x.val)
        assert yi.tolist() == sorted(want)
        assert yv.tolist() == [want[i] for i in sorted(want)]


def test_linearity_exact_on_small_integers():
    """A(x1 + x2) = A x1 + A x2 exactly when all values are small integers."""
    m, n = 300, 200
    csr = wl.random_sparse(m, n, 4000, 7, integer_values=True)
    A = _mat(csr)
    i1 = wl.distinct_indices(1, 0, n, 30)
    i2 = wl.distinct_indices(2, 0, n, 50)
    v1 = (wl.rand_below(1, 5, np.arange(30, dtype=np.uint64), 17) - 8).astype(np.float32)
    v2 = (wl.rand_below(2, 5, np.arange(50, dtype=np.uint64), 17) - 8).astype(np.float32)
    xs = np.zeros(n)
    xs[i1] += v1
    xs[i2] += v2
    iu = np.union1d(i1, i2)
    for fn in (oracle.ref_pull, oracle.ref_push):
        ya = np.zeros(m); yb = np.zeros(m); yc = np.zeros(m)
        yi, yv, _ = fn(A, i1, v1); ya[yi] = yv
        yi, yv, _ = fn(A, i2, v2); yb[yi] = yv
        yi, yv, _ = fn(A, iu, xs[iu].astype(np.float32)); yc[yi] = yv
        assert np.array_equal(ya + yb, yc)


def test_pull_equals_push_on_larger_random():
    csr = wl.random_sparse(5000, 4000, 60000, 21)
    x = wl.sparse_x(22, 0, 4000, 700)
    a = oracle.ref_pull(_mat(csr), x.idx, x.val)
    b = oracle.ref_push(_mat(csr), x.idx, x.val)
    assert np.array_equal(a[0], b[0])
    assert np.allclose(a[1], b[1], rtol=0, atol=1e-12)
    assert np.allclose(a[2], b[2], rtol=0, atol=1e-12)


def test_boolean_mode_matches_structure():
    csr = wl.random_sparse(200, 300, 1500, 31, values=False)
    x = wl.sparse_x(32, 0, 300, 25, values=False)
    _, s = _dense(csr)
    xp = np.zeros(300, dtype=bool)
    xp[x.idx] = True
    want = np.flatnonzero((s.astype(np.int64) @ xp.astype(np.int64)) > 0)
    assert np.array_equal(oracle.ref_pull(_mat(csr), x.idx)[0], want)
    assert np.array_equal(oracle.ref_push(_mat(csr), x.idx)[0], want)


# ------------------------------------------------------------------------------ BFS
def _graph(n, edges):
    """edges (u, v) meaning u -> v, i.e. stored entry A[v][u]."""
    a = np.zeros((n, n), dtype=np.float32)
    for u, v in edges:
        a[v, u] = 1.0
    return _mat(wl.csr_from_dense(a))


def test_bfs_path_graph():
    n = 50
    g = _graph(n, [(i, i + 1) for i in range(n - 1)] + [(i + 1, i) for i in range(n - 1)])
    assert oracle.ref_bfs(g, 0).tolist() == list(range(n))
    assert oracle.ref_bfs(g, 20).tolist() == [abs(i - 20) for i in range(n)]


def test_bfs_star_and_two_components():
    g = _graph(7, [(0, i) for i in range(1, 5)] + [(i, 0) for i in range(1, 5)] + [(5, 6), (6, 5)])
    assert oracle.ref_bfs(g, 0).tolist() == [0, 1, 1, 1, 1, -1, -1]
    assert oracle.ref_bfs(g, 3).tolist() == [1, 2, 2, 0, 2, -1, -1]
    assert oracle.ref_bfs(g, 5).tolist() == [-1, -1, -1, -1, -1, 0, 1]


def test_bfs_directed_cycle_pins_edge_orientation():
    """0 -> 1 -> 2 -> 0 stored as A[1][0], A[2][1], A[0][2]: from 0 the levels are 0, 1, 2;
    with the opposite orientation they would be 0, 2, 1."""
    g = _graph(3, [(0, 1), (1, 2), (2, 0)])
    assert oracle.ref_bfs(g, 0).tolist() == [0, 1, 2]
    assert oracle.ref_bfs_levelsync(g, 0).tolist() == [0, 1, 2]


def test_bfs_isolated_source():
    g = _graph(4, [(1, 2), (2, 1)])
    assert oracle.ref_bfs(g, 0).tolist() == [0, -1, -1, -1]


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_queue_bfs_equals_levelsync_spmspv_bfs(seed):
    csr = wl.random_sparse(400, 400, 900, 40 + seed, values=False)
    g = _mat(csr)
    for src in (0, 17, 399):
        assert np.array_equal(oracle.ref_bfs(g, src), oracle.ref_bfs_levelsync(g, src))


def test_bfs_chebyshev_closed_form_on_grid_graph():
    """On the 27-point grid graph the BFS level of v is max(|dx|,|dy|,|dz|) from the source."""
    d = 24
    csr = wl.stencil27(d, values=False)
    g = _mat(csr)
    ar = np.arange(d)
    z, y, x = np.meshgrid(ar, ar, ar, indexing="ij")
    for sx, sy, sz in ((0, 0, 0), (5, 17, 11), (23, 0, 12)):
        src = sx + d * (sy + d * sz)
        want = np.maximum(np.maximum(abs(x - sx), abs(y - sy)), abs(z - sz)).reshape(-1)
        assert np.array_equal(oracle.ref_bfs(g, src), want.astype(np.int32))


# ------------------------------------------------------------------------------ decode
def test_decode_equals_dense_gemv_on_bf16_operands():
    w = wl.pruned_weight(96, 80, 0.5, seed=5, stream=3)
    x = wl.relu_activation(80, 0.7, seed=5, stream=51)
    a, _ = _dense(w)
    y, s = oracle.ref_decode(_mat(w), x)
    assert np.allclose(y, a @ x.astype(np.float64), rtol=0, atol=1e-15)
    assert np.allclose(s, np.abs(a) @ np.abs(x.astype(np.float64)), rtol=0, atol=1e-15)


def test_decode_small_integers_exact_and_negative_zero_is_zero():
    a = np.array([[1, 2, 0, 4], [0, 0, 3, 0], [5, 0, 0, 0]], dtype=np.float32)
    x = np.array([2.0, -0.0, 0.0, 1.0], dtype=np.float32)
    y, s = oracle.ref_decode(_mat(wl.csr_from_dense(a)), x)
    assert y.tolist() == [6.0, 0.0, 10.0]
    assert s.tolist() == [6.0, 0.0, 10.0]


# ---- (min, +) product and shortest paths -------------------------------------------------

@pytest.mark.parametrize("m,n,nnz,k,seed", [(1, 1, 1, 1, 0), (7, 5, 12, 3, 1), (33, 64, 300, 9, 2),
                                            (64, 64, 900, 64, 3), (50, 50, 60, 0, 5)])
def test_minplus_brute_force_dense(m, n, nnz, k, seed):
    """(min, +) product vs the definition on a dense copy with explicit structure masks (numpy):
    absent entries are +inf, not 0; rows with no (stored, listed) pair are absent."""
    csr = wl.random_sparse(m, n, nnz, seed)
    a, s = _dense(csr)
    rng = np.random.default_rng(100 + seed)
    x_idx = np.sort(rng.choice(n, size=k, replace=False)).astype(np.int32)
    x_val = rng.standard_normal(k).astype(np.float32)
    y_idx, y_val = oracle.ref_minplus(_mat(csr), x_idx, x_val)
    big = np.where(s[:, x_idx], a[:, x_idx] + x_val.astype(np.float64)[None, :], np.inf) if k else np.full((m, 0), np.inf)
    want_rows = np.flatnonzero(s[:, x_idx].any(axis=1)) if k else np.zeros(0, dtype=np.int64)
    assert np.array_equal(y_idx, want_rows)
    if k:
        assert np.array_equal(y_val, big.min(axis=1)[want_rows])


def test_minplus_single_zero_entry_returns_the_column():
    """x = {j: 0}: y is column j of A, stored zeros and negative weights included (a listed 0
    takes part; with 0 read as "absent" the result would be empty)."""
    a = np.zeros((5, 4))
    a[0, 2], a[3, 2], a[4, 2], a[1, 1] = 2.5, -1.0, 7.0, 3.0
    csr = wl.csr_from_dense(a)
    y_idx, y_val = oracle.ref_minplus(_mat(csr), np.asarray([2], np.int32), np.asarray([0.0], np.float32))
    assert y_idx.tolist() == [0, 3, 4] and y_val.tolist() == [2.5, -1.0, 7.0]
    # the minimum, not the sum and not the last one: two listed columns meet row 0
    a[0, 1] = 1.0
    csr = wl.csr_from_dense(a)
    y_idx, y_val = oracle.ref_minplus(_mat(csr), np.asarray([1, 2], np.int32), np.asarray([0.25, 0.0], np.float32))
    assert y_idx.tolist() == [0, 1, 3, 4] and y_val.tolist() == [1.25, 3.25, -1.0, 7.0]


def _weighted(n, edges):
    a = np.zeros((n, n))
    for u, v, w in edges:
        a[v, u] = w
    return _mat(wl.csr_from_dense(a))


def test_sssp_path_star_and_orientation():
    n = 30
    w = [(i % 5) + 0.5 for i in range(n - 1)]
    g = _weighted(n, [(i, i + 1, w[i]) for i in range(n - 1)])          # directed path 0 -> 1 -> ...
    want = np.concatenate([[0.0], np.cumsum(w)])
    assert np.array_equal(oracle.ref_sssp(g, 0), want)
    d5 = oracle.ref_sssp(g, 5)
    assert np.all(np.isinf(d5[:5])) and np.array_equal(d5[5:], want[5:] - want[5])   # nothing upstream is reached
    # a shortcut that is longer in hops but shorter in weight wins: 0 -> 1 (10), 0 -> 2 (1), 2 -> 3 (1), 3 -> 1 (1)
    g = _weighted(4, [(0, 1, 10.0), (0, 2, 1.0), (2, 3, 1.0), (3, 1, 1.0)])
    assert oracle.ref_sssp(g, 0).tolist() == [0.0, 3.0, 1.0, 2.0]
    assert oracle.ref_sssp_frontier(g, 0).tolist() == [0.0, 3.0, 1.0, 2.0]


def test_sssp_unit_weights_equal_bfs_levels():
    csr = wl.random_sparse(300, 300, 800, 77, values=False)
    g = _mat(csr)
    for src in (0, 150):
        lv = oracle.ref_bfs(g, src).astype(np.float64)
        lv[lv < 0] = np.inf
        assert np.array_equal(oracle.ref_sssp(g, src), lv)
        assert np.array_equal(oracle.ref_sssp_frontier(g, src), lv)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_sssp_equals_library_dijkstra_and_frontier_form(seed):
    """Bellman-Ford sweeps vs scipy's Dijkstra on positive weights that are exact in binary
    (multiples of 1/8: every path sum is exact, so the comparison is for equality), and vs the
    frontier-driven iteration of (min, +) products."""
    import scipy.sparse as sp
    from scipy.sparse.csgraph import dijkstra
    n = 500
    csr = wl.random_sparse(n, n, 3000, 300 + seed)
    rng = np.random.default_rng(seed)
    val = (rng.integers(1, 64, size=csr.nnz) / 8.0).astype(np.float32)
    g = oracle.RefMatrix(n, n, csr.row_ptr, csr.col_idx, val)
    # scipy: entry [u, v] = edge u -> v; the stored A[i][j] is the edge j -> i, so pass the transpose
    m_lib = sp.csr_matrix((val.astype(np.float64), csr.col_idx, csr.row_ptr), shape=(n, n)).T.tocsr()
    for src in (0, 123):
        want = dijkstra(m_lib, directed=True, indices=src)
        assert np.array_equal(oracle.ref_sssp(g, src), want)
        assert np.array_equal(oracle.ref_sssp_frontier(g, src), want)
