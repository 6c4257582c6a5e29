"""GPU parity of dbspmspv_run against the CPU oracle: structural index set identical, values
within 2e-5 * sum|a x|, for forced push, forced pull and the automatic selector, every block
format variant and every value type, including empty and ragged inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_16308_b200 import binding as B
from paper_2608_16308_b200 import workloads as wl
from gpu_util import Handle, check_against_oracle, ref_matrix
from test_gpu_format import mixed_matrix

pytestmark = pytest.mark.gpu

PATHS = [B.PATH_AUTO, B.PATH_PUSH, B.PATH_PULL]


def dense_x(n, seed, frac):
    k = max(1, int(n * frac))
    return wl.sparse_x(seed, 0, n, k)


MATS = [
    ("uniform300x200", lambda: wl.random_sparse(300, 200, 4000, 1)),
    ("ragged77x131", lambda: wl.random_sparse(77, 131, 900, 2)),
    ("mixed", lambda: mixed_matrix(96, 112, 3)),
    ("rmat12", lambda: wl.rmat(12, 16, seed=1)),
    ("stencil16", lambda: wl.stencil27(16, seed=2)),
    ("wide", lambda: wl.random_sparse(40, 5000, 6000, 5)),
    ("tall", lambda: wl.random_sparse(5000, 40, 6000, 6)),
]


@pytest.mark.parametrize("name,make", MATS, ids=[m[0] for m in MATS])
@pytest.mark.parametrize("dtype,inline_max", [(B.F32, 31), (B.BF16, 31), (B.F32, 4), (B.BF16, 2)])
def test_parity_all_paths(name, make, dtype, inline_max):
    csr = make()
    o = B.default_create_opts()
    o.inline_max = inline_max          # below th0 - 1 the packed-COO class comes into play
    h = Handle(csr, dtype, opts=o)
    A = ref_matrix(csr, bf16=dtype == B.BF16)
    for frac in (0.002, 0.05, 0.5, 1.0):
        x = dense_x(csr.n, 7, frac)
        if dtype == B.BF16:
            x.val = wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(x.val))
        want = oracle.ref_pull(A, x.idx, x.val)
        for path in PATHS:
            for thr in (1, 8, 17):
                # (a short x may take the one-kernel form of the call: both forms are checked)
                for no_small in ((0, 1) if path != B.PATH_PULL and thr == 8 else (0,)):
                    h.set_opts(force_path=path, popc_threshold=thr, no_small_call=no_small)
                    check_against_oracle(h.run(x), want)
                    st = h.get_stats()
                    if path != B.PATH_AUTO:
                        assert st.last_path == path
                    assert st.last_n_nzblk == np.unique(x.idx >> 4).size
                    assert st.last_y_nnz == want[0].size
    h.close()


@pytest.mark.parametrize("fmt", [B.FORMAT_COO, B.FORMAT_CSR])
def test_forced_single_format_equals_auto(fmt):
    csr = mixed_matrix(96, 112, 3)
    o = B.default_create_opts()
    o.force_format = fmt
    h = Handle(csr, B.F32, opts=o)
    A = ref_matrix(csr)
    for frac in (0.05, 0.6):
        x = dense_x(csr.n, 11, frac)
        want = oracle.ref_pull(A, x.idx, x.val)
        for path in (B.PATH_PUSH, B.PATH_PULL):
            h.set_opts(force_path=path)
            check_against_oracle(h.run(x), want)
    h.close()


def test_selector_follows_the_block_ratio_rule():
    """push iff N_nzblk / N_blk < th3, evaluated in fp32 from the same integers."""
    csr = wl.random_sparse(4096, 4096, 30000, 3)
    h = Handle(csr, B.F32)
    nblk = (csr.n + 15) // 16
    for k in (1, 2, 3, 5, 40, 400):
        x = wl.sparse_x(50 + k, 0, csr.n, k)
        nz = np.unique(x.idx >> 4).size
        for th3 in (0.01, 0.005, 0.5):
            h.set_opts(th3=th3)
            h.run(x)
            st = h.get_stats()
            assert st.last_n_nzblk == nz
            want = B.PATH_PUSH if np.float32(nz) / np.float32(nblk) < np.float32(th3) else B.PATH_PULL
            assert st.last_path == want
    h.close()


def test_boolean_semiring_on_pattern_and_valued_handles():
    csr = wl.rmat(11, 8, seed=5)
    A = ref_matrix(csr)
    x = dense_x(csr.n, 3, 0.03)
    want = oracle.ref_pull(A, x.idx, None)
    for dtype in (B.PATTERN, B.F32):
        h = Handle(csr, dtype)
        for path in PATHS:
            h.set_opts(force_path=path)
            check_against_oracle(h.run(x, semiring=B.OR_AND), want, boolean=True)
        h.close()
    h = Handle(csr, B.PATTERN)
    xi = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(B.DbSpmspvError) as e:
        B.dbspmspv_run(h.h, xi, xi.float(), 4, B.PLUS_TIMES, h.y_idx, h.y_val, 10, h.y_nnz)
    assert e.value.status == B.ERR_UNSUPPORTED
    h.close()


def test_empty_x_and_empty_matrix_and_isolated_columns():
    csr = wl.random_sparse(100, 100, 300, 8)
    h = Handle(csr, B.F32)
    yi, yv, k = h.run(wl.SparseVec(100, np.zeros(0, np.int32), np.zeros(0, np.float32)))
    assert k == 0 and yi.size == 0
    # x listed only on columns that hold no entry
    empty_cols = np.setdiff1d(np.arange(100), csr.col_idx)[:5].astype(np.int32)
    assert empty_cols.size > 0
    for path in PATHS:
        h.set_opts(force_path=path)
        yi, yv, k = h.run(wl.SparseVec(100, empty_cols, np.ones(empty_cols.size, np.float32)))
        assert k == 0
    h.close()
    e = wl.CSR(50, 60, np.zeros(51, np.int64), np.zeros(0, np.int32), np.zeros(0, np.float32))
    h = Handle(e, B.F32)
    assert h.stats.n_blocks == 0
    yi, yv, k = h.run(wl.sparse_x(1, 0, 60, 10))
    assert k == 0
    h.close()


def test_state_is_clean_between_calls():
    """Back-to-back calls with different x on one handle: nothing leaks from the previous call
    (accumulator, hit masks, vector-block masks, worklist)."""
    csr = wl.rmat(12, 16, seed=2)
    h = Handle(csr, B.F32)
    A = ref_matrix(csr)
    for rep, (frac, path) in enumerate([(0.3, B.PATH_PUSH), (0.001, B.PATH_PULL), (0.02, B.PATH_PUSH),
                                        (0.5, B.PATH_PULL), (0.0005, B.PATH_PUSH)]):
        x = dense_x(csr.n, 20 + rep, frac)
        h.set_opts(force_path=path)
        check_against_oracle(h.run(x), oracle.ref_pull(A, x.idx, x.val))
    h.close()


def test_capacity_overflow_is_reported_not_written():
    csr = wl.random_sparse(500, 500, 5000, 4)
    h = Handle(csr, B.F32)
    x = dense_x(csr.n, 5, 0.2)
    want = oracle.ref_pull(ref_matrix(csr), x.idx, x.val)
    cap = want[0].size // 2
    h.y_idx.fill_(-1)
    yi, yv, k = h.run(x, capacity=cap)
    assert k == want[0].size                                  # full count is still reported
    assert np.array_equal(yi, want[0][:cap])
    assert (h.y_idx[cap:].cpu().numpy() == -1).all()          # nothing beyond capacity
    st = h.get_stats(raise_on_device_status=False)
    assert st.device_status == B.ERR_CAPACITY
    assert h.get_stats().device_status == B.OK                # reported once, then cleared
    check_against_oracle(h.run(x), want)                      # the handle stays usable
    h.close()


def test_out_of_range_index_is_skipped_and_reported():
    """With the default options too: the bad entry is never written through, the call reports
    ERR_BOUNDS once, the other entries give their result, and the handle stays usable."""
    csr = wl.random_sparse(100, 100, 300, 8)
    A = ref_matrix(csr)
    good = wl.SparseVec(100, np.array([1, 7], np.int32), np.ones(2, np.float32))
    want = oracle.ref_pull(A, good.idx, good.val)
    for validate in (0, 1):
        h = Handle(csr, B.F32)
        h.set_opts(validate=validate)
        for bad in (5000, -3, 100):
            x = wl.SparseVec(100, np.array([1, bad, 7], np.int32), np.ones(3, np.float32))
            check_against_oracle(h.run(x), want)
            assert h.get_stats(raise_on_device_status=False).device_status == B.ERR_BOUNDS
            assert h.get_stats().device_status == B.OK
        check_against_oracle(h.run(good), want)
        h.close()


def test_validate_reports_a_duplicate_index():
    csr = wl.random_sparse(100, 100, 300, 8)
    h = Handle(csr, B.F32)
    x = wl.SparseVec(100, np.array([4, 9, 4], np.int32), np.ones(3, np.float32))
    h.run(x)
    assert h.get_stats().device_status == B.OK               # not checked by default
    h.set_opts(validate=1)
    h.run(x)
    assert h.get_stats(raise_on_device_status=False).device_status == B.ERR_INVALID_ARG
    h.close()


def test_identity_permutation_and_block_diagonal_dense():
    n = 333
    eye = wl.CSR(n, n, np.arange(n + 1, dtype=np.int64), np.arange(n, dtype=np.int32), np.ones(n, np.float32))
    h = Handle(eye, B.F32)
    x = wl.sparse_x(3, 0, n, 50)
    order = np.argsort(x.idx)
    for path in PATHS:
        h.set_opts(force_path=path)
        yi, yv, k = h.run(x)
        assert np.array_equal(yi, x.idx[order]) and np.array_equal(yv, x.val[order])   # bit exact
    h.close()
    # block-diagonal matrix of dense 16 x 16 blocks == a small dense GEMV per block
    nb = 6
    a = np.zeros((16 * nb, 16 * nb), dtype=np.float32)
    for b in range(nb):
        a[16 * b:16 * b + 16, 16 * b:16 * b + 16] = wl.rand_f32(5, b, np.arange(256, dtype=np.uint64)).reshape(16, 16) + 0.1
    csr = wl.csr_from_dense(a)
    h = Handle(csr, B.F32)
    assert h.stats.class_blocks[B.BLK_DENSE] == nb
    x = wl.sparse_x(8, 0, 16 * nb, 40)
    xd = np.zeros(16 * nb)
    xd[x.idx] = x.val
    want = a.astype(np.float64) @ xd
    for path in PATHS:
        h.set_opts(force_path=path)
        yi, yv, k = h.run(x)
        assert k == 16 * len(np.unique(x.idx >> 4))
        scale = np.abs(a).astype(np.float64) @ np.abs(xd)                   # per row: sum |a x|
        assert (np.abs(yv.astype(np.float64) - want[yi]) <= 2e-5 * scale[yi]).all()
    h.close()


def test_stencil_unit_values_give_integer_neighbour_counts():
    """0/1-valued stencil with x = ones on a full grid line: y counts neighbours on the line
    (exact in fp32)."""
    d = 16
    csr = wl.stencil27(d, values=False)
    csr.val = np.ones(csr.nnz, dtype=np.float32)
    h = Handle(csr, B.F32)
    line = (np.arange(d) + d * (5 + d * 7)).astype(np.int32)        # y = 5, z = 7
    x = wl.SparseVec(csr.n, line, np.ones(d, np.float32))
    for path in PATHS:
        h.set_opts(force_path=path)
        yi, yv, k = h.run(x)
        assert k == 9 * d                                           # the 3 x 3 tube around the line
        xs = yi % d
        want = 3 - (xs == 0) - (xs == d - 1)
        assert np.array_equal(yv, want.astype(np.float32))
    h.close()


@pytest.mark.parametrize("frac", [0.002, 0.3], ids=["sparse_x", "dense_x"])
def test_page_locked_host_buffers_are_read_and_written_in_place(frac):
    """x and y in page-locked host memory: the kernels read x and write y (and the count)
    across the bus themselves; same result as with device buffers, and the state is clean for
    the next call (sparse x: entry-by-entry clean-up re-reads x_idx; dense x: wholesale)."""
    csr = wl.rmat(12, 16, seed=7)
    h = Handle(csr, B.F32)
    A = ref_matrix(csr)
    for path in PATHS:
        h.set_opts(force_path=path)
        for rep in range(2):
            x = dense_x(csr.n, 40 + rep, frac)
            xi = torch.from_numpy(np.ascontiguousarray(x.idx, dtype=np.int32)).pin_memory()
            xv = torch.from_numpy(np.ascontiguousarray(x.val, dtype=np.float32)).pin_memory()
            yi = torch.empty(csr.m, dtype=torch.int32).pin_memory()
            yv = torch.empty(csr.m, dtype=torch.float32).pin_memory()
            yn = torch.full((1,), -7, dtype=torch.int32).pin_memory()
            B.dbspmspv_run(h.h, xi, xv, int(x.idx.size), B.PLUS_TIMES, yi, yv, csr.m, yn)
            torch.cuda.synchronize()
            k = int(yn.item())
            check_against_oracle((yi[:k].numpy(), yv[:k].numpy(), k), oracle.ref_pull(A, x.idx, x.val))
            check_against_oracle(h.run(x), oracle.ref_pull(A, x.idx, x.val))      # device buffers, same handle
    h.close()


def test_hub_column_goes_through_the_hub_list():
    """One column with 9,000 stored elements (more than the hub threshold) among sparse ones:
    its push run is listed once and strided over by all warps instead of being cut into tasks."""
    m, n = 9000, 64
    bg = wl.random_sparse(m, n, 3000, 11)
    dense = np.zeros((m, n), dtype=np.float32)
    dense[bg.rows(), bg.col_idx] = bg.val
    dense[:, 7] = np.linspace(0.5, 1.5, m, dtype=np.float32)
    csr = wl.csr_from_dense(dense)
    h = Handle(csr, B.F32)
    A = ref_matrix(csr)
    for path in PATHS:
        h.set_opts(force_path=path)
        for idx in ([7], [3, 7, 40], list(range(0, 64, 3))):
            x = wl.SparseVec(n, np.array(idx, dtype=np.int32), np.linspace(1.0, 2.0, len(idx), dtype=np.float32))
            check_against_oracle(h.run(x), oracle.ref_pull(A, x.idx, x.val))
    h.close()


def test_dense_but_clustered_x_takes_the_push_with_a_late_worklist():
    """x lists more than a quarter of the columns, so the worklist is not built while x is
    blocked -- but the listed columns fill only 40 % of the vector blocks, so the selector still
    chooses the push and the worklist is built from the finished masks."""
    csr = wl.rmat(12, 16, seed=5)
    h = Handle(csr, B.F32)
    A = ref_matrix(csr)
    k = int(0.4 * csr.n) // 16 * 16
    idx = np.arange(k, dtype=np.int32)
    x = wl.SparseVec(csr.n, idx, np.linspace(-1.0, 1.0, k, dtype=np.float32) + 0.25)
    want = oracle.ref_pull(A, x.idx, x.val)
    check_against_oracle(h.run(x), want)
    st = h.get_stats()
    assert st.last_path == B.PATH_PUSH and st.last_n_nzblk == k // 16 and st.last_n_tasks > 0
    h.set_opts(force_path=B.PATH_PULL)
    check_against_oracle(h.run(x), want)
    h.set_opts()
    check_against_oracle(h.run(dense_x(csr.n, 3, 0.01)), oracle.ref_pull(A, dense_x(csr.n, 3, 0.01).idx, dense_x(csr.n, 3, 0.01).val))
    h.close()


def test_rows_that_sum_to_zero_or_hold_stored_zeros_are_still_reported():
    """The push flags a row when its accumulator was zero before the product arrived.  Rows whose
    products are zeros (stored zero values), cancel exactly, or arrive by the thousand (a hub
    row) must all come out as structural hits, on every path."""
    m, n = 600, 4000
    rng = np.random.default_rng(7)
    dense = np.zeros((m, n), dtype=np.float32)
    bg = wl.random_sparse(m, n, 3000, 9)
    dense[bg.rows(), bg.col_idx] = bg.val
    dense[5, :] = 1.0                                  # hub row: every listed column reaches it
    dense[17, :] = 0.0                                 # row 17: stored zeros only
    dense[33, :] = 0.0                                 # row 33: +v and -v under two listed columns
    dense[33, 100], dense[33, 101] = 2.5, -2.5
    mask = dense != 0
    cols = rng.choice(n, 40, replace=False)
    mask[17, cols] = True
    a = wl.csr_from_dense(dense, keep_zeros_mask=mask)
    x_idx = np.unique(np.concatenate([cols[:20], [100, 101], rng.choice(n, 300, replace=False)])).astype(np.int32)
    x = wl.SparseVec(n, x_idx, np.ones(x_idx.size, dtype=np.float32))
    h = Handle(a, B.F32)
    want = oracle.ref_pull(ref_matrix(a), x.idx, x.val)
    assert 17 in want[0] and 33 in want[0] and 5 in want[0]
    for p in (B.PATH_AUTO, B.PATH_PUSH, B.PATH_PULL):
        h.set_opts(force_path=p)
        check_against_oracle(h.run(x), want)
    h.close()


def test_hub_row_blocks_add_into_private_accumulators_and_fold_exactly():
    """Two row blocks hold 10,000 INLINE elements each, so the handle gives them private push
    accumulators (an untouched one holds -0.0).  Rows whose products are stored zeros, partly
    subnormal, or cancel exactly must still come out as structural hits with the oracle's values, and the
    result must not depend on whether the private accumulators are used."""
    m, n = 640, 10000
    rng = np.random.default_rng(3)
    dense = np.zeros((m, n), dtype=np.float32)
    bg = wl.random_sparse(m, n, 6000, 13)
    dense[bg.rows(), bg.col_idx] = bg.val
    mask = dense != 0
    for r in range(32):                                # one element per 16 x 16 block: INLINE class
        cols = np.arange(r % 16, n, 16)
        dense[r, :] = 0.0
        mask[r, :] = False
        dense[r, cols] = rng.uniform(0.5, 1.5, cols.size).astype(np.float32) * rng.choice([-1.0, 1.0], cols.size)
        mask[r, cols] = True
    dense[3, :] = 0.0                                  # row 3: stored zeros only
    c9 = np.arange(9, n, 16)
    dense[9, c9] = np.where(np.arange(c9.size) % 2 == 0, 2.5, -2.5)   # row 9: cancels under x = 1
    c20 = np.arange(4, n, 16)
    dense[20, c20] = np.where(np.arange(c20.size) % 2 == 0, 1e-41, 1.0)   # row 20: every other product subnormal
    a = wl.csr_from_dense(dense, keep_zeros_mask=mask)
    x_idx = np.arange(0, 8000, dtype=np.int32)
    x = wl.SparseVec(n, x_idx, np.ones(x_idx.size, dtype=np.float32))
    h = Handle(a, B.F32)
    assert h.stats.n_hub_row_blocks == 2
    want = oracle.ref_pull(ref_matrix(a), x.idx, x.val)
    assert {3, 9, 20} <= set(want[0].tolist())
    got = {}
    for hub_min in (1, -1):
        h.set_opts(force_path=B.PATH_PUSH, hub_min_nnz_x=hub_min)
        got[hub_min] = h.run(x)
        check_against_oracle(got[hub_min], want)
        assert h.get_stats().last_path == B.PATH_PUSH
    assert np.array_equal(got[1][0], got[-1][0])
    i9 = int(np.searchsorted(got[1][0], 9))
    assert got[1][1][i9] == 0.0
    # the private accumulators are clean again: a second, different call
    x2 = wl.SparseVec(n, np.arange(5, 9000, 3, dtype=np.int32), np.linspace(-1.0, 1.0, len(range(5, 9000, 3)), dtype=np.float32))
    h.set_opts(force_path=B.PATH_PUSH, hub_min_nnz_x=1)
    check_against_oracle(h.run(x2), oracle.ref_pull(ref_matrix(a), x2.idx, x2.val))
    h.set_opts(hub_min_nnz_x=1)
    check_against_oracle(h.run(x2), oracle.ref_pull(ref_matrix(a), x2.idx, x2.val))
    # pattern handle: the products are counts
    hp = Handle(wl.CSR(a.m, a.n, a.row_ptr, a.col_idx, None), B.PATTERN)
    hp.set_opts(force_path=B.PATH_PUSH, hub_min_nnz_x=1)
    wp = oracle.ref_pull(oracle.RefMatrix(a.m, a.n, a.row_ptr, a.col_idx, None), x.idx, None)
    check_against_oracle(hp.run(x, semiring=B.OR_AND), wp, boolean=True)
    h.close(); hp.close()


def test_masked_output_keeps_exactly_the_rows_the_mask_names():
    """dbspmspv_run_masked: y<mask> and y<not mask> are the oracle's y restricted to the rows
    whose bit is set / clear, on every path, and the handle is clean afterwards (the dropped
    rows' sums must not leak into the next call).  As a BFS step: one OR-AND product of the
    frontier masked by the complement of the visited set is the oracle's next level."""
    csr = wl.rmat(12, 16, seed=5)
    A = ref_matrix(csr)
    h = Handle(csr, B.F32)
    rng = np.random.default_rng(11)
    bits = rng.random(csr.m) < 0.4
    n_words = ((csr.m + 15) // 16 + 1) // 2
    words = np.zeros(n_words, dtype=np.uint32)
    rows = np.flatnonzero(bits)
    np.bitwise_or.at(words, rows >> 5, np.uint32(1) << (rows & 31).astype(np.uint32))
    maskd = torch.from_numpy(words.view(np.int32)).to("cuda")
    x = dense_x(csr.n, 3, 0.05)
    xi = torch.from_numpy(x.idx).to("cuda"); xv = torch.from_numpy(x.val).to("cuda")
    ri, rv, rs = oracle.ref_pull(A, x.idx, x.val)
    for path in PATHS:
        h.set_opts(force_path=path)
        for complement in (0, 1):
            keep = bits[ri] if complement == 0 else ~bits[ri]
            h.y_nnz.fill_(-7)
            B.dbspmspv_run_masked(h.h, xi, xv, int(x.idx.size), B.PLUS_TIMES, maskd, complement, h.y_idx, h.y_val, csr.m, h.y_nnz)
            torch.cuda.synchronize()
            k = int(h.y_nnz.item())
            got = (h.y_idx[:k].cpu().numpy(), h.y_val[:k].cpu().numpy(), k)
            check_against_oracle(got, (ri[keep], rv[keep], rs[keep]))
            check_against_oracle(h.run(x), (ri, rv, rs))          # nothing left behind
    # one BFS level from the oracle's levels
    g = wl.rmat(11, 8, seed=5, values=False, symmetrise=True)
    hg = Handle(g, B.PATTERN)
    src = int(wl.bfs_sources(g, 1)[0])
    levels = oracle.ref_bfs(oracle.RefMatrix(g.m, g.n, g.row_ptr, g.col_idx, None), src)
    frontier = np.flatnonzero(levels == 1).astype(np.int32)
    visited = np.flatnonzero((levels >= 0) & (levels <= 1))
    vw = np.zeros(((g.m + 15) // 16 + 1) // 2, dtype=np.uint32)
    np.bitwise_or.at(vw, visited >> 5, np.uint32(1) << (visited & 31).astype(np.uint32))
    B.dbspmspv_run_masked(hg.h, torch.from_numpy(frontier).to("cuda"), None, int(frontier.size), B.OR_AND,
                          torch.from_numpy(vw.view(np.int32)).to("cuda"), 1, hg.y_idx, None, g.m, hg.y_nnz)
    torch.cuda.synchronize()
    k = int(hg.y_nnz.item())
    assert np.array_equal(hg.y_idx[:k].cpu().numpy(), np.flatnonzero(levels == 2))
    h.close(); hg.close()


def test_bounded_wait_runs_out_and_reports_timeout():
    """The staging waits are bounded: a wait on a barrier that nothing arrives on (no copy in
    flight) gives up, the kernel records ERR_TIMEOUT, get_stats returns it once, and the handle
    and the context stay usable."""
    csr = wl.random_sparse(200, 200, 1500, 12)
    h = Handle(csr, B.F32)
    B.dbspmspv_test_bounded_wait(h.h, 64)
    assert h.get_stats(raise_on_device_status=False).device_status == B.ERR_TIMEOUT
    assert h.get_stats().device_status == B.OK
    x = dense_x(csr.n, 5, 0.1)
    for path in PATHS:
        h.set_opts(force_path=path)
        check_against_oracle(h.run(x), oracle.ref_pull(ref_matrix(csr), x.idx, x.val))
    with pytest.raises(B.DbSpmspvError) as e:
        B.dbspmspv_test_bounded_wait(h.h, 0)
    assert e.value.status == B.ERR_INVALID_ARG
    h.close()


def test_one_kernel_form_of_a_short_call():
    """A short x on a hypersparse handle runs as one kernel of one thread block: one launch
    instead of four, same result as the general chain; Boolean and masked output, capacity
    overflow (full count reported, nothing written beyond, the handle clean afterwards), a hub
    column shared out over the warp, a column block with payload entries, and the switch back
    to the chain when x is long or an option asks for it."""
    csr = wl.rmat(14, 16, seed=4)
    A = ref_matrix(csr)
    h = Handle(csr, B.F32)
    rng = np.random.default_rng(3)
    hub = int(np.argmax(np.bincount(csr.col_idx, minlength=csr.n)))
    for k in (1, 17, 256, 257, 5000):
        idx = rng.choice(csr.n, size=k, replace=False).astype(np.int32)
        if hub not in idx:
            idx[0] = hub
        x = wl.SparseVec(csr.n, idx, rng.standard_normal(k).astype(np.float32))
        want = oracle.ref_pull(A, x.idx, x.val)
        launches = []
        for no_small in (0, 1):
            h.set_opts(no_small_call=no_small)
            before = h.get_stats().kernel_launches
            check_against_oracle(h.run(x), want)
            launches.append(h.get_stats().kernel_launches - before)
            check_against_oracle(h.run(x, semiring=B.OR_AND), want, boolean=True)
        assert launches[0] == (1 if k <= 256 else launches[1]) and launches[1] >= 3
    # capacity
    h.set_opts()
    x = wl.SparseVec(csr.n, np.asarray([hub, 5, 77], np.int32), np.ones(3, np.float32))
    want = oracle.ref_pull(A, x.idx, x.val)
    cap = want[0].size // 2
    h.y_idx.fill_(-1)
    yi, yv, k = h.run(x, capacity=cap)
    assert k == want[0].size and np.array_equal(yi, want[0][:cap])
    assert (h.y_idx[cap:].cpu().numpy() == -1).all()
    assert h.get_stats(raise_on_device_status=False).device_status == B.ERR_CAPACITY
    check_against_oracle(h.run(x), want)
    # output mask and its complement
    bits = rng.random(csr.m) < 0.5
    words = np.zeros(((csr.m + 15) // 16 + 1) // 2, dtype=np.uint32)
    r = np.flatnonzero(bits)
    np.bitwise_or.at(words, r >> 5, np.uint32(1) << (r & 31).astype(np.uint32))
    maskd = torch.from_numpy(words.view(np.int32)).to("cuda")
    xi = torch.from_numpy(x.idx).to("cuda"); xv = torch.from_numpy(x.val).to("cuda")
    for complement in (0, 1):
        keep = bits[want[0]] if complement == 0 else ~bits[want[0]]
        B.dbspmspv_run_masked(h.h, xi, xv, 3, B.PLUS_TIMES, maskd, complement, h.y_idx, h.y_val, csr.m, h.y_nnz)
        torch.cuda.synchronize()
        kk = int(h.y_nnz.item())
        check_against_oracle((h.y_idx[:kk].cpu().numpy(), h.y_val[:kk].cpu().numpy(), kk), tuple(a[keep] for a in want))
        check_against_oracle(h.run(x), want)                  # the dropped rows left nothing behind
    h.close()
