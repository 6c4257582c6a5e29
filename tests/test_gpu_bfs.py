"""GPU parity of db_bfs: levels bit-identical to the queue BFS of the oracle, for forced push,
forced pull and the per-level automatic switch."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_16308_b200 import binding as B
from paper_2608_16308_b200 import workloads as wl
from gpu_util import Handle, ref_matrix, DEV

pytestmark = pytest.mark.gpu
PATHS = [B.PATH_AUTO, B.PATH_PUSH, B.PATH_PULL]


def bfs(h, src):
    levels = torch.full((h.csr.n,), -5, dtype=torch.int32, device=DEV)
    B.db_bfs(h.h, int(src), levels)
    torch.cuda.synchronize()
    return levels.cpu().numpy()


def graph_from_edges(n, edges):
    a = np.zeros((n, n), dtype=np.float32)
    for u, v in edges:
        a[v, u] = 1.0                      # stored A[v][u] is the edge u -> v
    return wl.csr_from_dense(a)


GRAPHS = [
    ("rmat12", lambda: wl.rmat(12, 16, seed=3, values=False, symmetrise=True)),
    ("rmat14", lambda: wl.rmat(14, 16, seed=4, values=False, symmetrise=True)),
    ("grid20", lambda: wl.stencil27(20, values=False)),
    ("directed_random", lambda: wl.random_sparse(3000, 3000, 9000, 5, values=False)),
    ("ragged_directed", lambda: wl.random_sparse(1000 + 7, 1000 + 7, 4000, 6, values=False)),
]


@pytest.mark.parametrize("name,make", GRAPHS, ids=[g[0] for g in GRAPHS])
@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("inline_max,no_index", [(31, 0), (3, 0), (31, 1)], ids=["inline", "coo_lists", "no_row_index"])
def test_levels_bit_exact(name, make, path, inline_max, no_index):
    g = make()
    o = B.default_create_opts()
    o.inline_max = inline_max            # 3: blocks of 4..31 entries become packed coordinate lists
    o.no_bfs_index = no_index            # 1: pull levels walk the row-block segments
    h = Handle(g, B.PATTERN, opts=o)
    h.set_opts(force_path=path)
    A = ref_matrix(g)
    deg = np.diff(g.row_ptr)
    srcs = [0, int(np.argmax(deg)), g.n - 1] + [int(s) for s in wl.bfs_sources(g, 3, seed=9)]
    for s in srcs:
        want = oracle.ref_bfs(A, s)
        got = bfs(h, s)
        assert np.array_equal(got, want), f"source {s}"
        st = h.get_stats()
        assert st.bfs_reached == int((want >= 0).sum())
        assert st.bfs_levels == int(want.max()) + 1     # the last expansion finds nothing new
    h.close()


def test_small_graphs_with_known_levels():
    n = 50
    path = graph_from_edges(n, [(i, i + 1) for i in range(n - 1)] + [(i + 1, i) for i in range(n - 1)])
    h = Handle(path, B.PATTERN)
    for p in PATHS:
        h.set_opts(force_path=p)
        assert bfs(h, 0).tolist() == list(range(n))
        assert bfs(h, 20).tolist() == [abs(i - 20) for i in range(n)]
    h.close()
    cyc = graph_from_edges(3, [(0, 1), (1, 2), (2, 0)])     # pins the edge orientation
    h = Handle(cyc, B.PATTERN)
    for p in PATHS:
        h.set_opts(force_path=p)
        assert bfs(h, 0).tolist() == [0, 1, 2]
    h.close()
    two = graph_from_edges(7, [(0, i) for i in range(1, 5)] + [(i, 0) for i in range(1, 5)] + [(5, 6), (6, 5)])
    h = Handle(two, B.PATTERN)
    for p in PATHS:
        h.set_opts(force_path=p)
        assert bfs(h, 0).tolist() == [0, 1, 1, 1, 1, -1, -1]
        assert bfs(h, 5).tolist() == [-1, -1, -1, -1, -1, 0, 1]
    h.close()


def test_isolated_source_and_bad_arguments():
    g = graph_from_edges(40, [(1, 2), (2, 1)])
    h = Handle(g, B.PATTERN)
    lv = bfs(h, 0)
    assert lv[0] == 0 and (lv[1:] == -1).all()
    assert h.get_stats().bfs_levels == 1 and h.get_stats().bfs_reached == 1
    levels = torch.empty(40, dtype=torch.int32, device=DEV)
    for bad in (-1, 40):
        with pytest.raises(B.DbSpmspvError) as e:
            B.db_bfs(h.h, bad, levels)
        assert e.value.status == B.ERR_INVALID_ARG
    h.close()
    rect = Handle(wl.random_sparse(30, 40, 100, 1, values=False), B.PATTERN)
    with pytest.raises(B.DbSpmspvError) as e:
        B.db_bfs(rect.h, 0, levels)
    assert e.value.status == B.ERR_UNSUPPORTED
    rect.close()


def test_chebyshev_closed_form_and_valued_handle():
    """On the 27-point grid graph level(v) = max(|dx|,|dy|,|dz|); a valued (fp32) handle gives
    the same levels as the pattern one; an SpMSpV call after a BFS on the same handle is clean."""
    d = 32
    g = wl.stencil27(d, seed=2)
    h = Handle(g, B.F32)
    ar = np.arange(d)
    z, y, x = np.meshgrid(ar, ar, ar, indexing="ij")
    sx, sy, sz = 3, 30, 17
    want = np.maximum(np.maximum(abs(x - sx), abs(y - sy)), abs(z - sz)).reshape(-1).astype(np.int32)
    for p in PATHS:
        h.set_opts(force_path=p)
        assert np.array_equal(bfs(h, sx + d * (sy + d * sz)), want)
    st = h.get_stats()
    assert st.bfs_levels == want.max() + 1        # the last expansion finds nothing new
    from gpu_util import check_against_oracle
    xs = wl.clustered_x(g.n, 8)
    h.set_opts()
    check_against_oracle(h.run(xs), oracle.ref_pull(ref_matrix(g), xs.idx, xs.val))
    h.close()


def test_auto_switches_direction_across_levels():
    g = wl.rmat(14, 16, seed=4, values=False, symmetrise=True)
    h = Handle(g, B.PATTERN)
    h.set_opts(th3_bfs=0.01)
    src = int(wl.bfs_sources(g, 1, seed=9)[0])
    bfs(h, src)
    st = h.get_stats()
    paths = list(st.bfs_level_path[:st.bfs_levels])
    nz = list(st.bfs_level_nzblk[:st.bfs_levels])
    nblk = (g.n + 15) // 16
    for p, k in zip(paths, nz):
        assert p == (B.PATH_PUSH if np.float32(k) / np.float32(nblk) < np.float32(0.01) else B.PATH_PULL)
    assert B.PATH_PUSH in paths and B.PATH_PULL in paths
    h.close()


def test_hub_column_goes_through_the_hub_list():
    """A star with 12,000 leaves: the centre's column holds more INLINE elements than the hub
    threshold, so its push is not cut into tasks but strided over by all warps."""
    n = 12001
    rows = np.r_[np.zeros(n - 1, np.int64), np.arange(1, n)]
    cols = np.r_[np.arange(1, n), np.zeros(n - 1, np.int64)]
    order = np.lexsort((cols, rows))
    rows, cols = rows[order], cols[order]
    row_ptr = np.r_[0, np.cumsum(np.bincount(rows, minlength=n))].astype(np.int64)
    g = wl.CSR(n, n, row_ptr, cols.astype(np.int32), None)
    A = ref_matrix(g)
    for path in (B.PATH_PUSH, B.PATH_AUTO):
        h = Handle(g, B.PATTERN)
        h.set_opts(force_path=path)
        for s in (5, 0, n - 1):
            assert np.array_equal(bfs(h, s), oracle.ref_bfs(A, s)), f"source {s}"
        h.close()
