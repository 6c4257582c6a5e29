"""Pins for the seeded input generators (shapes, counts and structure of the synthetic
stand-ins for the paper's workloads)."""
import numpy as np

from paper_2608_16308_b200 import workloads as wl


def test_counter_based_streams_are_reproducible_and_independent():
    a = wl.rand_u64(3, 1, np.arange(1000, dtype=np.uint64))
    b = wl.rand_u64(3, 1, np.arange(500, 1000, dtype=np.uint64))
    assert np.array_equal(a[500:], b)
    assert not np.array_equal(a, wl.rand_u64(3, 2, np.arange(1000, dtype=np.uint64)))
    u = wl.rand_f32(0, 0, np.arange(200000, dtype=np.uint64))
    assert 0.0 <= u.min() and u.max() < 1.0 and abs(u.mean() - 0.5) < 0.005


def test_distinct_indices():
    idx = wl.distinct_indices(1, 0, 1000, 1000)
    assert np.array_equal(np.sort(idx), np.arange(1000))
    idx = wl.distinct_indices(1, 0, 1 << 20, 5000)
    assert np.unique(idx).size == 5000 and idx.min() >= 0 and idx.max() < (1 << 20)


def test_uniform_rows_config():
    a = wl.uniform_rows()
    assert (a.m, a.n, a.nnz) == (16384, 16384, 131072)
    cols = a.col_idx.reshape(16384, 8)
    assert (np.diff(cols, axis=1) > 0).all()          # 8 distinct sorted columns per row
    assert a.val.min() >= -1.0 and a.val.max() < 1.0
    x = wl.sparse_x(0, 1, a.n, 164)
    assert np.unique(x.idx).size == 164


def test_rmat_small_properties():
    g = wl.rmat(12, 16, seed=3, values=False, symmetrise=True)
    r = g.rows().astype(np.int64)
    c = g.col_idx.astype(np.int64)
    assert (r != c).all()                              # no self loops
    k = r * g.n + c
    assert (np.diff(k) > 0).all()                      # sorted, no duplicates
    assert np.array_equal(np.sort(c * g.n + r), k)     # symmetric
    a = wl.rmat(12, 16, seed=1)
    assert a.val.dtype == np.float32 and a.nnz <= 16 << 12
    # skew: the top-left quadrant holds about 57 % of the raw draws
    keys = wl.rmat_keys(12, 16, 1)
    rr, cc = keys // 4096, keys % 4096
    frac = ((rr < 2048) & (cc < 2048)).mean()
    assert abs(frac - 0.57) < 0.01
    assert abs(((rr < 2048) & (cc >= 2048)).mean() - 0.19) < 0.01
    assert abs(((rr >= 2048) & (cc < 2048)).mean() - 0.19) < 0.01


def test_rmat_sweep_sizes():
    n = 1 << 20
    sizes = [int(np.floor(n * f + 0.5)) for f in wl.RMAT_SWEEP]
    assert sizes == [10, 105, 1049, 10486, 104858, 524288]


def test_stencil_counts_and_row_sums():
    d = 32
    a = wl.stencil27(d, values=False)
    assert a.nnz == (3 * d - 2) ** 3
    # row length = number of in-grid neighbours (self included)
    ar = np.arange(d)
    per_axis = 3 - (ar == 0) - (ar == d - 1)
    want = (per_axis[:, None, None] * per_axis[None, :, None] * per_axis[None, None, :]).reshape(-1)
    assert np.array_equal(np.diff(a.row_ptr), want)
    # block census at 16 x 16: with d a multiple of 16, the blocks are the tridiagonal ones
    # (same x-line segment or x-neighbouring lines) and corner singletons
    r = a.rows().astype(np.int64)
    bk = (r >> 4) * (a.n >> 4) + (a.col_idx >> 4)
    _, cnt = np.unique(bk, return_counts=True)
    segs = d // 16
    lines = (3 * d - 2) ** 2                           # (y,z) line pairs within distance 1
    assert (cnt == 46).sum() == lines * segs
    assert (cnt == 1).sum() == lines * 2 * (segs - 1)
    assert cnt.size == lines * (segs + 2 * (segs - 1))
    v = wl.stencil27(8).val
    a8 = wl.stencil27(8, values=False)
    diag = a8.rows() == a8.col_idx
    assert (v[diag] == 27.0).all() and v[~diag].min() >= 0.5 and v[~diag].max() < 1.5


def test_clustered_x_runs():
    n = 4096000
    x = wl.clustered_x(n, 64)
    assert x.idx.size == 4096 and np.unique(x.idx).size == 4096
    runs = x.idx.reshape(64, 64)
    assert (np.diff(runs, axis=1) == 1).all()
    assert runs[:, 0].min() >= 0 and runs[:, -1].max() < n


def test_pruned_weight_and_activation():
    m, n = 256, 512
    for rho in (0.5, 0.7):
        w = wl.pruned_weight(m, n, rho)
        assert w.nnz == m * n - int(np.floor(rho * m * n))
        bits = w.val.view(np.uint32)
        assert (bits & 0xFFFF == 0).all()              # exactly representable in bf16
        assert abs(w.val.std() - 0.02 * (1.45 if rho == 0.5 else 1.8)) < 0.01
    x = wl.relu_activation(1 << 16, 0.9)
    assert abs((x == 0).mean() - 0.9) < 4 * np.sqrt(0.9 * 0.1 / (1 << 16))
    x = wl.relu_activation(1 << 16, 0.7)
    assert abs((x == 0).mean() - 0.7) < 4 * np.sqrt(0.7 * 0.3 / (1 << 16))
    assert (x >= 0).all() and (x.view(np.uint32) & 0xFFFF == 0).all()


def test_bf16_rounding_is_nearest_even():
    a = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.140625], dtype=np.float32)
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7 -> even mantissa (1.0); 1 + 3*2^-8 -> 1 + 2^-6
    got = wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(a))
    assert got.tolist() == [1.0, 1.0, 1.015625, -2.5, 3.140625]


def test_rmat_relabelled_is_the_same_graph_under_a_permutation():
    a = wl.rmat(10, 8, seed=7)
    b = wl.rmat(10, 8, seed=7, relabel=True)
    perm = wl.vertex_permutation(1 << 10, 7)
    assert sorted(perm.tolist()) == list(range(1 << 10))
    assert a.nnz == b.nnz
    ka = np.sort(perm[a.rows().astype(np.int64)] * (1 << 10) + perm[a.col_idx.astype(np.int64)])
    kb = np.sort(b.rows().astype(np.int64) * (1 << 10) + b.col_idx.astype(np.int64))
    assert np.array_equal(ka, kb)
    # the degree multiset survives, the hubs move away from the low indices
    assert np.array_equal(np.sort(np.diff(a.row_ptr)), np.sort(np.diff(b.row_ptr)))
    assert np.argmax(np.diff(a.row_ptr)) == 0 and np.argmax(np.diff(b.row_ptr)) == perm[0]
