"""GPU tests of the blocked preprocessing (Section 3.2.1): nothing is lost, the two views
describe the same blocks, and every block lands in the class the paper's thresholds give."""
import numpy as np
import pytest
import torch

from paper_2608_16308_b200 import binding as B
from paper_2608_16308_b200 import workloads as wl
from gpu_util import Handle, to_bf16_bits

pytestmark = pytest.mark.gpu


def cpu_classify(rows, cols, dtype, th0=32, th1=128, th2=2.0):
    """Block census on the host: strict thresholds (fewer than th0 -> COO, more than th1 ->
    Dense), else ForceCSC iff max column count > th2 * max row count, ForceCSR iff the
    converse, else CSR.  INLINE = COO blocks small enough to live in the view entry."""
    key = (rows.astype(np.int64) >> 4) << 32 | (cols.astype(np.int64) >> 4)
    order = np.argsort(key, kind="stable")
    key, rows, cols = key[order], rows[order], cols[order]
    ub, start, cnt = np.unique(key, return_index=True, return_counts=True)
    cls = np.empty(ub.size, dtype=np.int32)
    cap = 31                               # inline_max: one view entry per stored element
    for b in range(ub.size):
        n = cnt[b]
        if n < th0:
            cls[b] = B.BLK_INLINE if n <= cap else B.BLK_COO
        elif n > th1:
            cls[b] = B.BLK_DENSE
        else:
            r = rows[start[b]:start[b] + n] & 15
            c = cols[start[b]:start[b] + n] & 15
            maxr, maxc = np.bincount(r).max(), np.bincount(c).max()
            if np.float32(maxc) > np.float32(th2) * np.float32(maxr):
                cls[b] = B.BLK_FCSC
            elif np.float32(maxr) > np.float32(th2) * np.float32(maxc):
                cls[b] = B.BLK_FCSR
            else:
                cls[b] = B.BLK_CSR
    return (ub >> 32).astype(np.int32), (ub & 0xFFFFFFFF).astype(np.int32), cls, cnt.astype(np.int32)


def mixed_matrix(m, n, seed):
    """Random background plus planted dense, row-skewed, column-skewed and banded blocks so
    that every class occurs."""
    a = np.zeros((m, n), dtype=np.float32)
    bg = wl.random_sparse(m, n, (m * n) // 40, seed)
    a[bg.rows(), bg.col_idx] = bg.val
    u = lambda k, shape: (wl.rand_f32(seed, 90 + k, np.arange(int(np.prod(shape)), dtype=np.uint64))
                          .reshape(shape) + 0.25).astype(np.float32)
    a[0:16, 0:16] = u(0, (16, 16))                                   # full dense
    a[16:32, 16:32] = u(1, (16, 16)) * (u(2, (16, 16)) > 0.6)        # ~65 % -> dense
    a[32:48, 0:16] = 0
    a[32:35, 0:16] = u(3, (3, 16))                                   # 3 full rows: row skew
    a[0:16, 32:48] = 0
    a[0:16, 33:36] = u(4, (16, 3))                                   # 3 full columns: col skew
    a[48:64, 48:64] = 0
    for r in range(16):
        for c in (r - 1, r, r + 1):
            if 0 <= c < 16:
                a[48 + r, 48 + c] = 1.0 + r + 0.01 * c               # tridiagonal: balanced
    a[80:96, 96:112] = 0
    a[85, 100] = 2.5                                                 # singleton: inline
    return wl.csr_from_dense(a)


CASES = [
    ("uniform", lambda: wl.random_sparse(300, 200, 4000, 1)),
    ("ragged", lambda: wl.random_sparse(77, 131, 900, 2)),
    ("mixed", lambda: mixed_matrix(96, 112, 3)),
    ("tiny", lambda: wl.random_sparse(1, 1, 1, 4)),
    ("rmat12", lambda: wl.rmat(12, 16, seed=1)),
    ("stencil", lambda: wl.stencil27(16, seed=2)),
]


@pytest.mark.parametrize("name,make", CASES, ids=[c[0] for c in CASES])
@pytest.mark.parametrize("dtype", [B.F32, B.BF16, B.PATTERN])
def test_export_equals_input_and_census(name, make, dtype):
    csr = make()
    h = Handle(csr, dtype)
    s = h.stats
    assert (s.m, s.n, s.nnz) == (csr.m, csr.n, csr.nnz)
    r, c, v = h.export_coo()
    assert np.array_equal(r, csr.rows()) and np.array_equal(c, csr.col_idx)
    if dtype == B.F32:
        assert np.array_equal(v.view(np.uint32), csr.val.view(np.uint32))      # bit exact
    elif dtype == B.BF16:
        assert np.array_equal(v.view(np.uint16), to_bf16_bits(csr.val))
    er, ec, ecls, en = h.export_blocks()                 # per view entry, block-CSR view order
    wr, wc, wcls, wn = cpu_classify(csr.rows(), csr.col_idx, dtype)
    # entries -> blocks: group the entries by (row block, column block)
    ekey = er.astype(np.int64) << 32 | ec
    assert (np.diff(er) >= 0).all()                                             # row-block major
    by_block = np.argsort(ekey, kind="stable")
    skey = ekey[by_block]
    first = np.r_[True, np.diff(skey) != 0]
    br, bc, cls = er[by_block][first], ec[by_block][first], ecls[by_block][first]
    bn = np.add.reduceat(en[by_block], np.flatnonzero(first)) if en.size else en
    assert np.array_equal(br, wr) and np.array_equal(bc, wc)
    assert np.array_equal(bn, wn) and int(bn.sum()) == csr.nnz
    assert np.array_equal(cls, wcls)
    assert np.array_equal(ecls[by_block], np.repeat(cls, np.diff(np.r_[np.flatnonzero(first), skey.size])))  # one class per block
    inl = ecls == B.BLK_INLINE
    assert (en[inl] == 1).all() and first[~inl[by_block]].all()                 # a payload block is one entry
    assert s.n_blocks == wr.size and s.n_view_entries == er.size
    for k in range(6):
        assert s.class_blocks[k] == int((wcls == k).sum())
        assert s.class_nnz[k] == int(wn[wcls == k].sum())
    # dual view: same entry set and consistent pointers
    rp, cp, crow, c2r = h.export_views()
    ne = er.size
    assert rp[0] == 0 and rp[-1] == ne and cp[0] == 0 and cp[-1] == ne
    assert np.array_equal(np.diff(rp), np.bincount(er, minlength=s.n_row_blocks))
    assert np.array_equal(np.diff(cp), np.bincount(ec, minlength=s.n_col_blocks))
    assert np.array_equal(np.sort(c2r), np.arange(ne))                          # a permutation
    assert np.array_equal(crow, er[c2r])
    # The two orders mirror each other.  Block-CSR: by row block; inside it the entries with a
    # payload first (by column block), then the INLINE elements row by row (by column), so that
    # a pull sums each row from adjacent entries.  Block-CSC: by column block; inside it the
    # entries with a payload (by row block), then the INLINE elements column by column (by row),
    # so that a push can visit single columns.
    ur, uc, _ = h.export_coo(sort=False)                 # elements in the order of their entries
    elem0 = np.r_[0, np.cumsum(en)[:-1]].astype(np.int64) if ne else np.zeros(0, np.int64)
    lr = np.where(inl, ur[elem0] & 15, 0) if ne else elem0
    lc = np.where(inl, uc[elem0] & 15, 0) if ne else elem0
    if ne:
        assert np.array_equal(ur[elem0] >> 4, er) and np.array_equal(uc[elem0] >> 4, ec)
    e64, c64 = er.astype(np.int64), ec.astype(np.int64)
    key_csr = (e64 << 36) | (np.where(inl, 16 + lr, 0).astype(np.int64) << 31) | (c64 << 4) | lc
    assert (np.diff(key_csr) > 0).all()
    key_csc = ((c64 << 36) | (np.where(inl, 16 + lc, 0).astype(np.int64) << 31) | (e64 << 4) | lr)[c2r]
    assert (np.diff(key_csc) > 0).all()
    h.close()


def test_every_class_occurs_in_mixed():
    """With the packed-COO class enabled for small blocks (inline_max below th0) the planted
    matrix exercises all six classes; with the default (every block under th0 inline) all but COO."""
    o = B.default_create_opts()
    o.inline_max = 4
    h = Handle(mixed_matrix(96, 112, 3), B.F32, opts=o)
    assert all(h.stats.class_blocks[k] > 0 for k in range(6))
    h.close()
    h = Handle(mixed_matrix(96, 112, 3), B.F32)
    assert h.stats.class_blocks[B.BLK_COO] == 0
    assert all(h.stats.class_blocks[k] > 0 for k in range(6) if k != B.BLK_COO)
    h.close()


def _block(entries):
    a = np.zeros((16, 16), dtype=np.float32)
    for r, c in entries:
        a[r, c] = 1.0 + r + c / 16.0
    return wl.csr_from_dense(a)


def test_threshold_edges():
    """31 / 32 entries (COO vs mid), 128 / 129 (mid vs Dense), skew exactly 2.0 vs above."""
    def cls_of(entries):
        h = Handle(_block(entries), B.F32)
        c = h.export_blocks()[2][0]                    # (a single block: every entry has its class)
        h.close()
        return c
    full = [(r, c) for r in range(16) for c in range(16)]
    assert cls_of(full[:32]) in (B.BLK_FCSR, B.BLK_CSR, B.BLK_FCSC)
    assert cls_of(full[:128]) != B.BLK_DENSE
    assert cls_of(full[:129]) == B.BLK_DENSE
    assert cls_of(full[:1]) == B.BLK_INLINE
    assert cls_of(full[:31]) == B.BLK_INLINE          # default inline_max = 31 = th0 - 1
    o = B.default_create_opts()
    o.inline_max = 8
    h = Handle(_block(full[:9]), B.F32, opts=o)       # above inline_max, below th0 -> packed COO
    assert h.export_blocks()[2][0] == B.BLK_COO
    h.close()
    # 32 entries as two full rows: max row 16, max col 2 -> ForceCSR
    assert cls_of(full[:32]) == B.BLK_FCSR
    assert cls_of([(c, r) for r, c in full[:32]]) == B.BLK_FCSC
    # rows of 8 in 4 rows (cols 0-7) + extra: max row = 8, max col = 4 -> ratio exactly 2: CSR
    e = [(r, c) for r in range(4) for c in range(8)]
    assert cls_of(e) == B.BLK_CSR
    # one more entry in row 0 -> max row 9 > 2 * 4
    assert cls_of(e + [(0, 8)]) == B.BLK_FCSR
    assert cls_of([(c, r) for r, c in e + [(0, 8)]]) == B.BLK_FCSC


def test_duplicates_are_merged_and_coo_input_matches():
    rows = np.array([3, 3, 3, 40, 40, 0], dtype=np.int32)
    cols = np.array([5, 5, 6, 1, 1, 0], dtype=np.int32)
    vals = np.array([1.0, 2.0, 4.0, 0.5, 0.25, 0.0], dtype=np.float32)
    h = B.dbspmspv_create_coo(48, 16, 6, torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda(),
                              torch.from_numpy(vals).cuda(), B.F32)
    s = B.dbspmspv_get_stats(h)
    assert s.nnz == 4
    r = torch.empty(4, dtype=torch.int32, device="cuda")
    c = torch.empty(4, dtype=torch.int32, device="cuda")
    v = torch.empty(4, dtype=torch.float32, device="cuda")
    B.dbspmspv_export_coo(h, r, c, v)
    got = sorted(zip(r.tolist(), c.tolist(), v.tolist()))
    assert got == [(0, 0, 0.0), (3, 5, 3.0), (3, 6, 4.0), (40, 1, 0.75)]      # explicit zero kept
    B.dbspmspv_destroy(h)
    csr = wl.random_sparse(200, 150, 2000, 9)
    a, b = Handle(csr, B.F32), Handle(csr, B.F32, from_coo=True)
    for x, y in zip(a.export_coo(), b.export_coo()):
        assert np.array_equal(x, y)
    c = Handle(csr, B.F32, host_input=True)
    for x, y in zip(a.export_coo(), c.export_coo()):
        assert np.array_equal(x, y)
    a.close(); b.close(); c.close()


@pytest.mark.parametrize("fmt", [B.FORMAT_COO, B.FORMAT_CSR])
def test_forced_formats_round_trip(fmt):
    csr = mixed_matrix(96, 112, 3)
    o = B.default_create_opts()
    o.force_format = fmt
    h = Handle(csr, B.F32, opts=o)
    want = B.BLK_COO if fmt == B.FORMAT_COO else B.BLK_CSR
    assert (h.export_blocks()[2] == want).all() and h.stats.n_view_entries == h.stats.n_blocks
    r, c, v = h.export_coo()
    assert np.array_equal(r, csr.rows()) and np.array_equal(c, csr.col_idx)
    assert np.array_equal(v.view(np.uint32), csr.val.view(np.uint32))
    h.close()


def test_bad_arguments_are_rejected_synchronously():
    csr = wl.random_sparse(64, 64, 100, 1)
    rp = torch.from_numpy(csr.row_ptr).cuda()
    ci = torch.from_numpy(csr.col_idx).cuda()
    v = torch.from_numpy(csr.val).cuda()
    with pytest.raises(B.DbSpmspvError) as e:
        B.dbspmspv_create_csr(64, 64, csr.nnz, rp, ci, v, B.F32, 32)
    assert e.value.status == B.ERR_UNSUPPORTED
    with pytest.raises(B.DbSpmspvError) as e:
        B.dbspmspv_create_csr(64, 64, csr.nnz, None, ci, v, B.F32)
    assert e.value.status == B.ERR_INVALID_ARG
    with pytest.raises(B.DbSpmspvError) as e:
        B.dbspmspv_create_csr(64, 32, csr.nnz, rp, ci, v, B.F32)      # columns out of range
    assert e.value.status == B.ERR_INVALID_ARG
    with pytest.raises(B.DbSpmspvError) as e:
        B.dbspmspv_create_csr(0, 64, 0, rp, ci, v, B.F32)
    assert e.value.status == B.ERR_INVALID_ARG
