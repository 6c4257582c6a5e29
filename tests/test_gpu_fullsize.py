"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration
bench.py times (automatic path selection, default options), against the CPU oracle: the whole
result for SpMSpV and BFS (the C oracle is fast enough), all rows for decode."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_16308_b200 import binding as B
from paper_2608_16308_b200 import workloads as wl
from gpu_util import Handle, check_against_oracle, ref_matrix, DEV, TOL

pytestmark = pytest.mark.gpu


def test_c1_uniform_16384():
    a = wl.uniform_rows()
    x = wl.sparse_x(0, 1, a.n, 164)
    h = Handle(a, B.F32)
    want = oracle.ref_pull(ref_matrix(a), x.idx, x.val)
    for path in (B.PATH_AUTO, B.PATH_PUSH, B.PATH_PULL):
        h.set_opts(force_path=path)
        check_against_oracle(h.run(x), want)
    h.close()


def test_c2_rmat20_sweep():
    a = wl.rmat(20, 16, seed=1)
    h = Handle(a, B.F32)
    A = ref_matrix(a)
    for k, f in enumerate(wl.RMAT_SWEEP):
        x = wl.rmat_x(a.n, f, k)
        want = oracle.ref_push(A, x.idx, x.val) if f < 0.05 else oracle.ref_pull(A, x.idx, x.val)
        h.set_opts()
        check_against_oracle(h.run(x), want)
        if f in (1e-3, 0.5):                      # both forced paths at a sparse and a dense point
            for path in (B.PATH_PUSH, B.PATH_PULL):
                h.set_opts(force_path=path)
                check_against_oracle(h.run(x), want)
        if x.idx.size <= 256:                     # the short points once more as the general chain of kernels
            h.set_opts(no_small_call=1)
            check_against_oracle(h.run(x), want)
        if f in (1e-5, 1e-2, 0.5):                # (min, +) on the same x: one-kernel form, push, streaming pull
            h.set_opts()
            wi, wv = oracle.ref_minplus(A, x.idx, x.val)
            gi, gv, kk = h.run(x, semiring=B.MIN_PLUS)
            assert kk == wi.size and np.array_equal(gi, wi)
            assert np.array_equal(gv.view(np.uint32), wv.astype(np.float32).view(np.uint32))
    h.close()


def test_sssp_rmat20_symmetric_weighted():
    """db_sssp at the size the benchmark times: distances against the Bellman-Ford oracle."""
    import torch
    g = wl.rmat(20, 16, seed=3, symmetrise=True)
    g.val = (0.05 + wl.rand_f32(7, 1, np.arange(g.nnz))).astype(np.float32)
    h = Handle(g, B.F32)
    A = ref_matrix(g)
    for src in wl.bfs_sources(g, 2):
        dist = torch.empty(g.n, dtype=torch.float32, device="cuda")
        steps = B.db_sssp(h.h, int(src), dist)
        torch.cuda.synchronize()
        got = dist.cpu().numpy()
        want = oracle.ref_sssp(A, int(src))
        fin = np.isfinite(want)
        assert np.array_equal(np.isfinite(got), fin) and steps >= 2
        assert np.all(np.abs(got[fin] - want[fin]) <= 64 * 2.0 ** -24 * want[fin] + 1e-30)
    h.close()


def test_c3_stencil160_clustered_x():
    a = wl.stencil27(160, seed=2)
    h = Handle(a, B.F32)
    A = ref_matrix(a)
    for runs in (64, 3200):
        x = wl.clustered_x(a.n, runs)
        want = oracle.ref_push(A, x.idx, x.val)
        for path in (B.PATH_AUTO, B.PATH_PUSH, B.PATH_PULL):
            h.set_opts(force_path=path)
            check_against_oracle(h.run(x), want)
    # BFS on the grid graph: closed form level(v) = Chebyshev distance from the source
    d = 160
    src = 7 + d * (150 + d * 80)
    levels = torch.empty(a.n, dtype=torch.int32, device=DEV)
    h.set_opts()
    B.db_bfs(h.h, src, levels)
    torch.cuda.synchronize()
    ar = np.arange(d)
    z, y, xx = np.meshgrid(ar, ar, ar, indexing="ij")
    want = np.maximum(np.maximum(abs(xx - 7), abs(y - 150)), abs(z - 80)).reshape(-1).astype(np.int32)
    assert np.array_equal(levels.cpu().numpy(), want)
    h.close()


def test_c4_bfs_rmat22_symmetric():
    g = wl.rmat(22, 16, seed=3, values=False, symmetrise=True)
    h = Handle(g, B.PATTERN)
    A = ref_matrix(g)
    levels = torch.empty(g.n, dtype=torch.int32, device=DEV)
    for s in wl.bfs_sources(g, 16):                      # every source the configuration names
        B.db_bfs(h.h, int(s), levels)
        torch.cuda.synchronize()
        assert np.array_equal(levels.cpu().numpy(), oracle.ref_bfs(A, int(s))), f"source {s}"
    # an isolated vertex as the source
    iso = int(np.flatnonzero(np.diff(g.row_ptr) == 0)[0])
    B.db_bfs(h.h, iso, levels)
    torch.cuda.synchronize()
    lv = levels.cpu().numpy()
    assert lv[iso] == 0 and (np.delete(lv, iso) == -1).all()
    h.close()


@pytest.mark.parametrize("shape", wl.DECODE_SHAPES, ids=[f"{m}x{n}" for m, n in wl.DECODE_SHAPES])
def test_c5_decode_layers(shape):
    m, n = shape
    for prune in (0.5, 0.7):
        w = wl.pruned_weight(m, n, prune)
        h = Handle(w, B.BF16)
        A = ref_matrix(w)
        for zf in (0.7, 0.9):
            x = wl.relu_activation(n, zf)
            xd = torch.from_numpy(wl.f32_to_bf16_bits(x).view(np.int16)).to(DEV)
            y = torch.empty(m, dtype=torch.float32, device=DEV)
            want, scale = oracle.ref_decode(A, x)
            for legacy in (0, 1):          # the single-kernel form, and the general kernels
                h.set_opts(no_fused_decode=legacy)
                y.fill_(7.0)
                B.dbspmspv_decode(h.h, xd, y)
                torch.cuda.synchronize()
                err = np.abs(y.cpu().numpy().astype(np.float64) - want)
                assert (err <= TOL * scale).all(), f"prune {prune} zeros {zf} legacy {legacy}: worst {np.max(err / np.maximum(scale, 1e-300)):.2e}"
        h.close()
