"""GPU parity of the (min, +) semiring of dbspmspv_run against the CPU oracle.  The kernel
forms fl32(a + x) for every (stored element, listed entry) pair and takes the exact minimum;
rounding to fp32 is monotone, so the result must equal the oracle's fp64 minimum rounded to
fp32 -- bit for bit -- and the index set must be identical."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_16308_b200 import binding as B
from paper_2608_16308_b200 import workloads as wl
from gpu_util import Handle, ref_matrix
from test_gpu_format import mixed_matrix
from test_gpu_spmspv import MATS, dense_x

pytestmark = pytest.mark.gpu


def check_exact(got, want):
    gi, gv, k = got
    wi, wv = want
    assert k == wi.size
    assert np.array_equal(gi, wi)
    assert np.array_equal(gv.view(np.uint32), wv.astype(np.float32).view(np.uint32))


@pytest.mark.parametrize("name,make", MATS, ids=[m[0] for m in MATS])
@pytest.mark.parametrize("dtype,inline_max", [(B.F32, 31), (B.BF16, 31), (B.F32, 4), (B.BF16, 2), (B.PATTERN, 31)])
def test_minplus_parity(name, make, dtype, inline_max):
    csr = make()
    o = B.default_create_opts()
    o.inline_max = inline_max
    h = Handle(csr, dtype, opts=o)
    A = ref_matrix(csr, bf16=dtype == B.BF16)
    if dtype == B.PATTERN:
        A = oracle.RefMatrix(csr.m, csr.n, csr.row_ptr, csr.col_idx, None)
    for frac in (0.002, 0.05, 0.5, 1.0):
        x = dense_x(csr.n, 7, frac)
        if dtype == B.BF16:
            x.val = wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(x.val))
        want = oracle.ref_minplus(A, x.idx, x.val)
        for path in (B.PATH_AUTO, B.PATH_PUSH, B.PATH_PULL, -1):
            # (-1: the push once more with the one-kernel form of a short call switched off)
            h.set_opts(force_path=B.PATH_PUSH if path < 0 else path, no_small_call=int(path < 0))
            path = B.PATH_PUSH if path < 0 else path
            check_exact(h.run(x, semiring=B.MIN_PLUS), want)
            st = h.get_stats()
            assert st.last_y_nnz == want[0].size
            # the pull is the streaming kernel of hypersparse valued handles; everything else pushes
            if name == "rmat12" and dtype != B.PATTERN and path == B.PATH_PULL:
                assert st.last_path == B.PATH_PULL
            if path == B.PATH_PUSH or dtype == B.PATTERN:
                assert st.last_path == B.PATH_PUSH
    h.close()


def test_minplus_listed_zero_negative_weights_and_clean_state():
    """A listed 0 takes part (it is not "absent"); negative sums order correctly; and the
    accumulator a (min, +) call leaves behind serves a (+, *) call and the other way round."""
    csr = wl.rmat(12, 16, seed=3)
    csr.val = (csr.val - 0.5).astype(np.float32)              # weights of both signs
    h = Handle(csr, B.F32)
    A = ref_matrix(csr)
    x = dense_x(csr.n, 5, 0.03)
    x.val[::3] = 0.0
    x.val[1::3] *= -1.0
    want_mp = oracle.ref_minplus(A, x.idx, x.val)
    want_pt = oracle.ref_pull(A, x.idx, x.val)
    from gpu_util import check_against_oracle
    for _ in range(2):
        check_exact(h.run(x, semiring=B.MIN_PLUS), want_mp)
        check_against_oracle(h.run(x), want_pt)
    # x = {j: 0} returns column j of A
    j = int(np.argmax(np.bincount(csr.col_idx, minlength=csr.n)))
    one = wl.SparseVec(csr.n, np.asarray([j], np.int32), np.asarray([0.0], np.float32))
    gi, gv, k = h.run(one, semiring=B.MIN_PLUS)
    rows = csr.rows()[csr.col_idx == j]
    assert np.array_equal(gi, np.sort(rows))
    dense_col = np.zeros(csr.m, np.float32)
    dense_col[csr.rows()[csr.col_idx == j]] = csr.val[csr.col_idx == j]
    assert np.array_equal(gv, dense_col[gi])
    h.close()


def test_minplus_masked_and_hub_column():
    """Output mask and its complement under (min, +); a column long enough to go through the
    hub list of the worklist."""
    m, n = 9000, 64
    rng = np.random.default_rng(4)
    bg = wl.random_sparse(m, n, 3000, 11)
    dense = np.zeros((m, n), dtype=np.float32)
    dense[bg.rows(), bg.col_idx] = bg.val
    dense[:, 7] = np.linspace(0.5, 1.5, m, dtype=np.float32)
    csr = wl.csr_from_dense(dense)
    h = Handle(csr, B.F32)
    A = ref_matrix(csr)
    x = wl.SparseVec(n, np.array([3, 7, 40], dtype=np.int32), np.array([1.0, 0.25, -2.0], dtype=np.float32))
    wi, wv = oracle.ref_minplus(A, x.idx, x.val)
    check_exact(h.run(x, semiring=B.MIN_PLUS), (wi, wv))
    bits = rng.random(m) < 0.5
    words = np.zeros(((m + 15) // 16 + 1) // 2, dtype=np.uint32)
    r = np.flatnonzero(bits)
    np.bitwise_or.at(words, r >> 5, np.uint32(1) << (r & 31).astype(np.uint32))
    maskd = torch.from_numpy(words.view(np.int32)).to("cuda")
    xi = torch.from_numpy(x.idx).to("cuda"); xv = torch.from_numpy(x.val).to("cuda")
    for complement in (0, 1):
        keep = bits[wi] if complement == 0 else ~bits[wi]
        B.dbspmspv_run_masked(h.h, xi, xv, int(x.idx.size), B.MIN_PLUS, maskd, complement, h.y_idx, h.y_val, m, h.y_nnz)
        torch.cuda.synchronize()
        k = int(h.y_nnz.item())
        check_exact((h.y_idx[:k].cpu().numpy(), h.y_val[:k].cpu().numpy(), k), (wi[keep], wv[keep]))
    check_exact(h.run(x, semiring=B.MIN_PLUS), (wi, wv))
    h.close()


def test_minplus_argument_errors():
    csr = wl.random_sparse(64, 64, 200, 1)
    h = Handle(csr, B.F32)
    xi = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(B.DbSpmspvError):
        B.dbspmspv_run(h.h, xi, None, 1, B.MIN_PLUS, h.y_idx, h.y_val, 64, h.y_nnz)      # values are required
    with pytest.raises(B.DbSpmspvError):
        B.dbspmspv_run(h.h, xi, xi.float(), 1, 3, h.y_idx, h.y_val, 64, h.y_nnz)          # unknown semiring
    h.close()


# ---- db_sssp ------------------------------------------------------------------------------

def _sssp(h, src):
    dist = torch.empty(h.csr.n, dtype=torch.float32, device="cuda")
    steps = B.db_sssp(h.h, int(src), dist)
    torch.cuda.synchronize()
    return dist.cpu().numpy(), steps


@pytest.mark.parametrize("make", [lambda: wl.rmat(12, 16, seed=2, symmetrise=True), lambda: wl.rmat(14, 8, seed=3),
                                  lambda: wl.stencil27(12, seed=1), lambda: wl.random_sparse(3000, 3000, 9000, 8)],
                         ids=["rmat12_sym", "rmat14_directed", "stencil12", "uniform3000"])
def test_sssp_exact_on_dyadic_weights(make):
    """Weights that are multiples of 1/8 below 8: every path sum is exact in fp32 and in the
    oracle's fp64, so the distances must be identical, unreachable vertices +inf."""
    csr = make()
    csr.val = (1 + (wl.rand_u64(11, 3, np.arange(csr.nnz)) % 63)).astype(np.float32) / 8.0
    h = Handle(csr, B.F32)
    A = ref_matrix(csr)
    deg = np.bincount(csr.col_idx, minlength=csr.n)
    srcs = [int(np.argmax(deg)), int(np.flatnonzero(deg > 0)[0]), int(np.flatnonzero(deg > 0)[-1])]
    for src in srcs:
        got, steps = _sssp(h, src)
        want = oracle.ref_sssp(A, src)
        assert np.array_equal(got.astype(np.float64), want)
        assert steps >= 1
    h.close()


def test_sssp_general_weights_within_rounding():
    """Arbitrary fp32 weights: a path of k edges accumulates k roundings of 2^-24 relative."""
    csr = wl.rmat(13, 16, seed=5, symmetrise=True)
    csr.val = (0.05 + wl.rand_f32(7, 1, np.arange(csr.nnz))).astype(np.float32)
    h = Handle(csr, B.F32)
    A = ref_matrix(csr)
    for src in wl.bfs_sources(csr, 3):
        got, steps = _sssp(h, src)
        want = oracle.ref_sssp(A, int(src))
        assert np.array_equal(np.isinf(got), np.isinf(want))
        fin = np.isfinite(want)
        assert np.all(np.abs(got[fin] - want[fin]) <= 64 * 2.0 ** -24 * want[fin] + 1e-30)
    h.close()


def test_sssp_pattern_handle_gives_bfs_levels_and_negative_edges():
    g = wl.rmat(12, 8, seed=9, values=False, symmetrise=True)
    h = Handle(g, B.PATTERN)
    src = int(wl.bfs_sources(g, 1)[0])
    lv = oracle.ref_bfs(oracle.RefMatrix(g.m, g.n, g.row_ptr, g.col_idx, None), src).astype(np.float64)
    lv[lv < 0] = np.inf
    got, _ = _sssp(h, src)
    assert np.array_equal(got.astype(np.float64), lv)
    h.close()
    # negative edges without a negative cycle; then one with: 0 -> 1 -> 2 -> 0 of total weight -1
    a = np.zeros((5, 5), dtype=np.float32)
    a[1, 0], a[2, 1], a[3, 2], a[3, 0], a[4, 3] = 4.0, -2.0, 1.0, 5.0, -1.0
    csr = wl.csr_from_dense(a)
    h = Handle(csr, B.F32)
    got, steps = _sssp(h, 0)
    assert got.tolist() == [0.0, 4.0, 2.0, 3.0, 2.0]
    assert np.array_equal(got.astype(np.float64), oracle.ref_sssp(ref_matrix(csr), 0))
    got, steps = _sssp(h, 4)                                  # no out-edges: one product, nothing reached
    assert got.tolist() == [np.inf] * 4 + [0.0] and steps == 1
    h.close()
    a = np.zeros((3, 3), dtype=np.float32)
    a[1, 0], a[2, 1], a[0, 2] = 1.0, 1.0, -3.0
    h = Handle(wl.csr_from_dense(a), B.F32)
    with pytest.raises(B.DbSpmspvError):
        _sssp(h, 0)
    torch.cuda.synchronize()
    h.close()
