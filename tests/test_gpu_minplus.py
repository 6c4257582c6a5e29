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
        check_exact(h.run(x, semiring=B.MIN_PLUS), want)
        st = h.get_stats()
        assert st.last_path == B.PATH_PUSH and st.last_y_nnz == want[0].size
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
