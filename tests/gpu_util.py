"""Helpers shared by the GPU parity tests: upload a generated matrix, call the C ABI through
the binding, fetch results, and compare against the CPU oracle."""
import os

import numpy as np
import torch

import oracle
from paper_2608_16308_b200 import binding as B
from paper_2608_16308_b200 import workloads as wl

DEV = "cuda:0"
TOL = 2e-5          # |y - y_ref| <= TOL * sum_k |a_ik x_k|  (fp32 and bf16-in / fp32-accumulate)


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    return wl.f32_to_bf16_bits(a)


class Handle:
    """Owns a library handle built from a workloads.CSR."""

    def __init__(self, csr: wl.CSR, dtype=B.F32, opts=None, from_coo=False, host_input=False):
        self.csr, self.dtype = csr, dtype
        val = None
        if dtype == B.F32:
            val = np.ascontiguousarray(csr.val, dtype=np.float32)
        elif dtype == B.BF16:
            val = to_bf16_bits(csr.val).view(np.int16)
        if opts is None:
            opts = B.default_create_opts()
        opts.input_on_host = 1 if host_input else 0
        up = (lambda a: None if a is None else np.ascontiguousarray(a)) if host_input else \
            (lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(DEV))
        self._keep = []
        if from_coo:
            args = (up(csr.rows()), up(csr.col_idx), up(val))
            self.h = B.dbspmspv_create_coo(csr.m, csr.n, csr.nnz, *args, dtype, 16, opts)
        else:
            args = (up(csr.row_ptr), up(csr.col_idx), up(val))
            self.h = B.dbspmspv_create_csr(csr.m, csr.n, csr.nnz, *args, dtype, 16, opts)
        self.stats = B.dbspmspv_get_stats(self.h)
        self.y_idx = torch.empty(csr.m, dtype=torch.int32, device=DEV)
        self.y_val = torch.empty(csr.m, dtype=torch.float32, device=DEV)
        self.y_nnz = torch.zeros(1, dtype=torch.int32, device=DEV)

    def set_opts(self, **kw):
        o = B.default_run_opts()
        for k, v in kw.items():
            setattr(o, k, v)
        B.dbspmspv_set_run_opts(self.h, o)

    def run(self, x: wl.SparseVec, semiring=B.PLUS_TIMES, capacity=None):
        xi = torch.from_numpy(np.ascontiguousarray(x.idx, dtype=np.int32)).to(DEV)
        xv = None
        if x.val is not None and semiring != B.OR_AND:
            if self.dtype == B.BF16:
                xv = torch.from_numpy(to_bf16_bits(x.val).view(np.int16)).to(DEV)
            else:
                xv = torch.from_numpy(np.ascontiguousarray(x.val, dtype=np.float32)).to(DEV)
        cap = self.csr.m if capacity is None else capacity
        self.y_nnz.fill_(-7)
        B.dbspmspv_run(self.h, xi, xv, int(x.idx.size), semiring, self.y_idx, self.y_val, cap, self.y_nnz)
        torch.cuda.synchronize()
        k = int(self.y_nnz.item())
        kk = min(k, cap)
        return self.y_idx[:kk].cpu().numpy(), self.y_val[:kk].cpu().numpy(), k

    def export_coo(self, sort=True):
        """Stored elements as (row, col, value); sorted by (row, col), or -- sort=False -- in the
        order of the block-CSR view entries that hold them."""
        nnz = int(self.stats.nnz)
        r = torch.empty(max(nnz, 1), dtype=torch.int32, device=DEV)
        c = torch.empty(max(nnz, 1), dtype=torch.int32, device=DEV)
        v = None
        if self.dtype == B.F32:
            v = torch.empty(max(nnz, 1), dtype=torch.float32, device=DEV)
        elif self.dtype == B.BF16:
            v = torch.empty(max(nnz, 1), dtype=torch.int16, device=DEV)
        B.dbspmspv_export_coo(self.h, r, c, v)
        r, c = r[:nnz].cpu().numpy(), c[:nnz].cpu().numpy()
        v = None if v is None else v[:nnz].cpu().numpy()
        if not sort:
            return r, c, v
        order = np.lexsort((c, r))
        return r[order], c[order], (None if v is None else v[order])

    def export_blocks(self):
        nb = int(self.stats.n_view_entries)
        out = [torch.empty(max(nb, 1), dtype=torch.int32, device=DEV) for _ in range(4)]
        B.dbspmspv_export_blocks(self.h, *out)
        return [t[:nb].cpu().numpy() for t in out]

    def export_views(self):
        s = self.stats
        a = torch.empty(s.n_row_blocks + 1, dtype=torch.int32, device=DEV)
        b = torch.empty(s.n_col_blocks + 1, dtype=torch.int32, device=DEV)
        c = torch.empty(max(s.n_view_entries, 1), dtype=torch.int32, device=DEV)
        d = torch.empty(max(s.n_view_entries, 1), dtype=torch.int32, device=DEV)
        B.dbspmspv_export_views(self.h, a, b, c, d)
        nb = int(s.n_view_entries)
        return a.cpu().numpy(), b.cpu().numpy(), c[:nb].cpu().numpy(), d[:nb].cpu().numpy()

    def get_stats(self, **kw):
        return B.dbspmspv_get_stats(self.h, **kw)

    def close(self):
        if self.h:
            if os.environ.get("DBSPMSPV_LIBRARY"):
                # a run with the range-checked library: no kernel may have met a bad index
                st = B.dbspmspv_get_stats(self.h, raise_on_device_status=False)
                assert st.device_status != B.ERR_INTERNAL, "range check failed inside a kernel"
            B.dbspmspv_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def ref_matrix(csr: wl.CSR, bf16=False) -> oracle.RefMatrix:
    val = csr.val
    if bf16 and val is not None:
        val = wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(val))
    return oracle.RefMatrix(csr.m, csr.n, csr.row_ptr, csr.col_idx, val)


def check_against_oracle(got, want, boolean=False, tol=TOL):
    """Index set identical (structural); values within tol * sum |a x|."""
    yi, yv, k = got
    ri, rv, rs = want
    assert k == ri.size, f"y_nnz {k} != oracle {ri.size}"
    assert np.array_equal(yi, ri), "output index set differs from the oracle"
    if boolean:
        assert (yv == 1.0).all()
        return 0.0
    err = np.abs(yv.astype(np.float64) - rv)
    bound = tol * rs
    bad = err > bound
    assert not bad.any(), f"{bad.sum()} values out of tolerance; worst ratio {(err[bad] / rs[bad]).max():.3e}"
    with np.errstate(divide="ignore", invalid="ignore"):
        ratio = np.where(rs > 0, err / rs, 0.0)
    return float(ratio.max()) if ratio.size else 0.0
