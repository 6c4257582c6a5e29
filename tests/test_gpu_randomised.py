"""Seeded random sweep over shapes, densities, value types, semirings, forced paths, the
one-kernel form of short calls and output masks: every case against the CPU oracle.  Shapes
are ragged on purpose (m, n not multiples of 16 or 32), x runs from one entry to every column."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2608_16308_b200 import binding as B
from paper_2608_16308_b200 import workloads as wl
from gpu_util import Handle, check_against_oracle, ref_matrix
from test_gpu_format import mixed_matrix

pytestmark = pytest.mark.gpu


def _case(rng):
    kind = rng.integers(0, 4)
    m, n = int(rng.integers(1, 3000)), int(rng.integers(1, 3000))
    if kind == 0:
        csr = wl.random_sparse(m, n, min(m * n, int(rng.integers(0, 6 * max(m, n)) + 1)), int(rng.integers(1 << 30)))
    elif kind == 1:
        csr = mixed_matrix(16 * int(rng.integers(6, 14)), 16 * int(rng.integers(7, 14)), int(rng.integers(1 << 30)))
    elif kind == 2:
        csr = wl.rmat(int(rng.integers(6, 12)), int(rng.integers(2, 20)), seed=int(rng.integers(1 << 30)))
    else:
        csr = wl.stencil27(int(rng.integers(3, 14)), seed=int(rng.integers(1 << 30)))
    return csr


@pytest.mark.parametrize("seed", range(int(os.environ.get("DBS_RANDOM_CASES", "24"))))     # (more for a soak run)
def test_random_cases(seed):
    rng = np.random.default_rng(1000 + seed)
    csr = _case(rng)
    dtype = [B.F32, B.BF16, B.PATTERN][int(rng.integers(0, 3))]
    o = B.default_create_opts()
    o.inline_max = int(rng.choice([31, 31, 8, 2]))
    h = Handle(csr, dtype, opts=o)
    A = ref_matrix(csr, bf16=dtype == B.BF16)
    if dtype == B.PATTERN:
        A = oracle.RefMatrix(csr.m, csr.n, csr.row_ptr, csr.col_idx, None)
    n_words = ((csr.m + 15) // 16 + 1) // 2
    for rep in range(6):
        k = int(rng.choice([1, min(csr.n, 7), max(1, csr.n // 50), max(1, csr.n // 3), csr.n]))
        x = wl.sparse_x(int(rng.integers(1 << 30)), 0, csr.n, k)
        if dtype == B.BF16:
            x.val = wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(x.val))
        semiring = [B.PLUS_TIMES, B.OR_AND, B.MIN_PLUS][int(rng.integers(0, 3))]
        if dtype == B.PATTERN and semiring == B.PLUS_TIMES:
            semiring = B.OR_AND
        h.set_opts(force_path=int(rng.choice([B.PATH_AUTO, B.PATH_PUSH, B.PATH_PULL])), no_small_call=int(rng.integers(0, 2)),
                   popc_threshold=int(rng.choice([1, 8, 17])))
        masked = bool(rng.integers(0, 2))
        bits = rng.random(csr.m) < 0.5
        complement = int(rng.integers(0, 2))
        if semiring == B.MIN_PLUS:
            wi, wv = oracle.ref_minplus(A, x.idx, x.val)
            ws = None
        else:
            wi, wv, ws = oracle.ref_pull(A, x.idx, x.val)
        if masked:
            words = np.zeros(n_words, dtype=np.uint32)
            r = np.flatnonzero(bits)
            np.bitwise_or.at(words, r >> 5, np.uint32(1) << (r & 31).astype(np.uint32))
            keep = bits[wi] if complement == 0 else ~bits[wi]
            wi, wv = wi[keep], wv[keep]
            ws = None if ws is None else ws[keep]
            xi = torch.from_numpy(x.idx).to("cuda")
            xv = None
            if semiring != B.OR_AND:
                xv = torch.from_numpy(wl.f32_to_bf16_bits(x.val).view(np.int16) if dtype == B.BF16 else x.val).to("cuda")
            B.dbspmspv_run_masked(h.h, xi, xv, k, semiring, torch.from_numpy(words.view(np.int32)).to("cuda"), complement,
                                  h.y_idx, h.y_val, csr.m, h.y_nnz)
            torch.cuda.synchronize()
            kk = int(h.y_nnz.item())
            got = (h.y_idx[:kk].cpu().numpy(), h.y_val[:kk].cpu().numpy(), kk)
        else:
            got = h.run(x, semiring=semiring)
        if semiring == B.MIN_PLUS:
            assert got[2] == wi.size and np.array_equal(got[0], wi)
            assert np.array_equal(got[1].view(np.uint32), wv.astype(np.float32).view(np.uint32))
        else:
            check_against_oracle(got, (wi, wv, ws), boolean=semiring == B.OR_AND)
    h.close()


@pytest.mark.parametrize("seed", range(int(os.environ.get("DBS_RANDOM_CASES", "24")) // 2))
def test_random_graph_drivers(seed):
    """db_bfs (levels bit-exact) and db_sssp (dyadic weights: distances exact) on random square
    graphs, directed and symmetrised, from random sources including isolated ones."""
    rng = np.random.default_rng(5000 + seed)
    kind = int(rng.integers(0, 3))
    if kind == 0:
        n = int(rng.integers(2, 4000))
        g = wl.random_sparse(n, n, min(n * n, int(rng.integers(1, 5 * n))), int(rng.integers(1 << 30)))
    elif kind == 1:
        g = wl.rmat(int(rng.integers(6, 13)), int(rng.integers(2, 16)), seed=int(rng.integers(1 << 30)), symmetrise=bool(rng.integers(0, 2)))
    else:
        g = wl.stencil27(int(rng.integers(3, 12)), seed=int(rng.integers(1 << 30)))
    g.val = (1 + (wl.rand_u64(seed, 3, np.arange(g.nnz)) % 63)).astype(np.float32) / 8.0
    hv = Handle(g, B.F32)
    hp = Handle(wl.CSR(g.m, g.n, g.row_ptr, g.col_idx, None), B.PATTERN)
    A = ref_matrix(g)
    P = oracle.RefMatrix(g.m, g.n, g.row_ptr, g.col_idx, None)
    levels = torch.empty(g.n, dtype=torch.int32, device="cuda")
    dist = torch.empty(g.n, dtype=torch.float32, device="cuda")
    for src in rng.integers(0, g.n, size=3):
        B.db_bfs(hp.h, int(src), levels)
        B.db_sssp(hv.h, int(src), dist)
        torch.cuda.synchronize()
        assert np.array_equal(levels.cpu().numpy(), oracle.ref_bfs(P, int(src)))
        assert np.array_equal(dist.cpu().numpy().astype(np.float64), oracle.ref_sssp(A, int(src)))
    hv.close(); hp.close()
