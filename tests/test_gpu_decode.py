"""GPU parity of dbspmspv_decode (dense bf16/fp32 x in, dense fp32 y out) against the oracle's
dense-output loop on the bf16-rounded operands."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_16308_b200 import binding as B
from paper_2608_16308_b200 import workloads as wl
from gpu_util import Handle, ref_matrix, DEV, TOL

pytestmark = pytest.mark.gpu
PATHS = [B.PATH_AUTO, B.PATH_PUSH, B.PATH_PULL]


def decode(h, x_f32):
    if h.dtype == B.BF16:
        xd = torch.from_numpy(wl.f32_to_bf16_bits(x_f32).view(np.int16)).to(DEV)
    else:
        xd = torch.from_numpy(np.ascontiguousarray(x_f32, dtype=np.float32)).to(DEV)
    y = torch.full((h.csr.m,), 123.0, dtype=torch.float32, device=DEV)
    B.dbspmspv_decode(h.h, xd, y)
    torch.cuda.synchronize()
    return y.cpu().numpy()


def check(y, want, scale):
    err = np.abs(y.astype(np.float64) - want)
    assert (err <= TOL * scale).all(), f"worst {np.max(err / np.maximum(scale, 1e-300)):.3e}"
    assert (y[scale == 0] == 0.0).all()            # rows without a structural hit are exactly 0


@pytest.mark.parametrize("shape", [(192, 256), (1000, 333), (333, 1000)])
@pytest.mark.parametrize("prune,zf", [(0.5, 0.7), (0.5, 0.9), (0.7, 0.9), (0.95, 0.7)])
def test_decode_parity_bf16(shape, prune, zf):
    m, n = shape
    w = wl.pruned_weight(m, n, prune, seed=5, stream=m)
    x = wl.relu_activation(n, zf, seed=5, stream=60)
    h = Handle(w, B.BF16)
    want, scale = oracle.ref_decode(ref_matrix(w), x)
    for p in PATHS:
        for thr in (1, 8):
            for legacy in (0, 3, 2, 1):  # auto / streaming / selective one-kernel forms (where the handle qualifies), general kernels
                h.set_opts(force_path=p, popc_threshold=thr, no_fused_decode=legacy)
                check(decode(h, x), want, scale)
                if p != B.PATH_AUTO:
                    assert h.get_stats().last_path == p
    assert h.get_stats().last_n_nzblk == int((x.reshape(-1)[: (n // 16) * 16].reshape(-1, 16) != 0).any(axis=1).sum()
                                             + (1 if n % 16 and (x[(n // 16) * 16:] != 0).any() else 0))
    h.close()


@pytest.mark.parametrize("dtype", [B.BF16, B.F32])
def test_decode_non_finite_activations_reach_only_stored_elements(dtype):
    # Dense blocks keep explicit zeros for absent elements: an infinite or NaN activation must
    # not leak through them (0 * inf), only through the stored elements of its column
    m, n = 192, 256
    w = wl.pruned_weight(m, n, 0.5, seed=5, stream=11)
    x = wl.relu_activation(n, 0.8, seed=5, stream=61)
    act = np.flatnonzero(x)
    x[act[0]] = np.inf
    x[act[3]] = np.nan
    h = Handle(w, dtype)
    assert h.get_stats().class_blocks[B.BLK_DENSE] > 0
    want, scale = oracle.ref_decode(ref_matrix(w), x)
    nan, inf = np.isnan(want), np.isinf(want)
    assert nan.any() and inf.any() and (~nan & ~inf).any()
    for p, legacy in [(p, l) for p in PATHS for l in (0, 3, 2, 1)]:
        h.set_opts(force_path=p, no_fused_decode=legacy)
        y = decode(h, x)
        assert (np.isnan(y) == nan).all()
        assert (y[inf] == want[inf]).all()
        fin = ~nan & ~inf
        check(y[fin], want[fin], scale[fin])
    h.close()


def test_decode_wide_layer_many_entries_per_row_block():
    # more than 1024 view entries per row block: the single-kernel form runs 16 warps per row
    # block and keeps 80 KB of x in shared memory
    m, n = 48, 20000
    w = wl.pruned_weight(m, n, 0.5, seed=5, stream=21)
    x = wl.relu_activation(n, 0.9, seed=5, stream=62)
    h = Handle(w, B.BF16)
    want, scale = oracle.ref_decode(ref_matrix(w), x)
    for p in PATHS:
        for legacy in (0, 3, 2, 1):
            h.set_opts(force_path=p, no_fused_decode=legacy)
            check(decode(h, x), want, scale)
    h.close()


def test_decode_fp32_handle_small_integers_exact_and_negative_zero():
    a = (wl.rand_below(3, 0, np.arange(64 * 48, dtype=np.uint64), 7).reshape(64, 48) - 3).astype(np.float32)
    w = wl.csr_from_dense(a)
    x = (wl.rand_below(3, 1, np.arange(48, dtype=np.uint64), 5) - 2).astype(np.float32)
    x[5] = -0.0
    for dtype in (B.F32, B.BF16):
        h = Handle(w, dtype)
        want, _ = oracle.ref_decode(ref_matrix(w), x)
        for p in PATHS:
            for legacy in (0, 3, 2, 1):
                h.set_opts(force_path=p, no_fused_decode=legacy)
                assert np.array_equal(decode(h, x).astype(np.float64), want)
        h.close()


def test_decode_all_zero_x_and_interleaving_with_run():
    w = wl.pruned_weight(128, 160, 0.5, seed=5, stream=7)
    h = Handle(w, B.BF16)
    y = decode(h, np.zeros(160, dtype=np.float32))
    assert (y == 0).all()
    x = wl.relu_activation(160, 0.7, seed=5, stream=61)
    want, scale = oracle.ref_decode(ref_matrix(w), x)
    check(decode(h, x), want, scale)
    # a sparse-output call on the same handle right after a decode call, and back
    from gpu_util import check_against_oracle
    xs = wl.sparse_x(4, 0, 160, 12)
    xs.val = wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(xs.val))
    check_against_oracle(h.run(xs), oracle.ref_pull(ref_matrix(w), xs.idx, xs.val))
    check(decode(h, x), want, scale)
    h.close()


def test_decode_choice_follows_the_previous_x_and_every_form_agrees():
    """Automatic mode streams the payload unless the x of the handle's previous decode call had
    fewer than 15 % nonzero elements; whichever form runs, the result is the oracle's -- for a
    dense x after a sparse one and the other way round."""
    m, n = 512, 2048
    w = wl.pruned_weight(m, n, 0.5, seed=5, stream=31)
    h = Handle(w, B.BF16)
    assert h.get_stats().class_blocks[B.BLK_DENSE] + h.get_stats().class_blocks[B.BLK_FCSC] > 0
    xs = {zf: wl.relu_activation(n, zf, seed=5, stream=70 + i) for i, zf in enumerate((0.5, 0.95, 0.99, 0.7))}
    refs = {zf: oracle.ref_decode(ref_matrix(w), x) for zf, x in xs.items()}
    launches = []
    for zf in (0.5, 0.95, 0.95, 0.99, 0.7, 0.7, 0.5):
        before = h.get_stats().kernel_launches
        check(decode(h, xs[zf]), *refs[zf])
        launches.append(h.get_stats().kernel_launches - before)
    # streaming = zero kernel + stream kernel; selective = one kernel.  The call after a sparse x is selective.
    assert launches == [2, 2, 1, 1, 1, 2, 2]
    h.close()


@pytest.mark.parametrize("dtype", [B.BF16, B.F32])
def test_decode_magnitude_threshold_is_fused_into_the_blocking(dtype):
    """decode_threshold = tau: x_j takes part iff |x_j| > tau (Section 5.3's activation sparsity
    by magnitude thresholding), on a dense activation vector without a single zero; every form
    and path must equal the oracle run on the thresholded vector."""
    m, n = 512, 1024
    w = wl.pruned_weight(m, n, 0.5, seed=5, stream=41)
    x = wl.rand_normal_f32(5, 77, np.arange(n, dtype=np.uint64))
    assert (x != 0).all()
    xr = wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(x)) if dtype == B.BF16 else x
    h = Handle(w, dtype)
    for keep in (0.1, 0.6):
        tau = float(np.quantile(np.abs(xr), 1.0 - keep))
        xt = np.where(np.abs(xr) > np.float32(tau), xr, 0.0).astype(np.float32)
        want, scale = oracle.ref_decode(ref_matrix(w, bf16=dtype == B.BF16), xt)
        for p in PATHS:
            for legacy in (0, 3, 2, 1):
                h.set_opts(force_path=p, no_fused_decode=legacy, decode_threshold=tau)
                check(decode(h, x), want, scale)
        assert h.get_stats().last_n_nzblk == int((xt.reshape(-1, 16) != 0).any(axis=1).sum())
    with pytest.raises(B.DbSpmspvError):
        h.set_opts(decode_threshold=-1.0)
    h.close()


def test_decode_chain_up_relu_cut_down_without_leaving_the_device():
    """Two bf16 layers chained on the device: the fp32 output of the first decode call is the x
    of the second (decode_x_f32), with the ReLU and the magnitude cut fused into its blocking
    (decode_relu, decode_threshold) -- no kernel in between.  Each layer is checked against the
    oracle on the operands it was given: the second one on the bf16-rounded, rectified and cut
    output of the first as the GPU produced it."""
    n0, n1, n2 = 512, 1408, 512
    w_up = wl.pruned_weight(n1, n0, 0.5, seed=5, stream=51)
    w_down = wl.pruned_weight(n2, n1, 0.5, seed=5, stream=52)
    h_up, h_down = Handle(w_up, B.BF16), Handle(w_down, B.BF16)
    x0 = wl.relu_activation(n0, 0.7, seed=5, stream=63)
    want1, scale1 = oracle.ref_decode(ref_matrix(w_up, bf16=True), wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(x0)))
    x0d = torch.from_numpy(wl.f32_to_bf16_bits(x0).view(np.int16)).to(DEV)
    y1 = torch.empty(n1, dtype=torch.float32, device=DEV)
    y2 = torch.full((n2,), 7.0, dtype=torch.float32, device=DEV)
    for legacy in (0, 3, 2, 1):
        h_up.set_opts(no_fused_decode=legacy)
        B.dbspmspv_decode(h_up.h, x0d, y1)
        torch.cuda.synchronize()
        y1h = y1.cpu().numpy()
        check(y1h, want1, scale1)
        x1 = wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(y1h))
        for tau in (0.0, float(np.quantile(x1[x1 > 0], 0.5))):
            x1t = np.where(x1 > np.float32(tau), x1, 0.0).astype(np.float32)
            want2, scale2 = oracle.ref_decode(ref_matrix(w_down, bf16=True), x1t)
            h_down.set_opts(no_fused_decode=legacy, decode_x_f32=1, decode_relu=1, decode_threshold=tau)
            B.dbspmspv_decode(h_down.h, y1, y2)          # y1 never left the device
            torch.cuda.synchronize()
            check(y2.cpu().numpy(), want2, scale2)
            assert h_down.get_stats().last_n_nzblk == int((x1t.reshape(-1, 16) != 0).any(axis=1).sum())
    h_up.close(); h_down.close()


@pytest.mark.parametrize("shape,dtype", [((512, 1024), B.BF16), ((333, 1000), B.BF16), ((512, 1024), B.F32), ((48, 20000), B.BF16)])
def test_decode_batch_equals_the_oracle_vector_by_vector(shape, dtype):
    """dbspmspv_decode_batch: 1 to 9 vectors of different activation densities (one all zero),
    leading dimensions larger than n and m, with and without the fused ReLU cut; groups of
    vectors share one pass over the payload (bf16: up to eight, on the tensor cores), the rest
    goes through the single-vector forms.  Every y vector is checked against the oracle for its
    own x vector.  Then one vector gets an infinite and a NaN entry: the tensor-core kernel hands
    the group over to the per-column kernel, and non-finite values reach only stored elements."""
    m, n = shape
    w = wl.pruned_weight(m, n, 0.5, seed=5, stream=71)
    h = Handle(w, dtype)
    ldx, ldy = n + 24, m + 8
    zfs = [0.7, 0.9, 0.5, 1.0, 0.99, 0.3, 0.8, 0.6, 0.95]
    nv = len(zfs)
    xs = np.zeros((nv, ldx), dtype=np.float32)
    for b, zf in enumerate(zfs):
        if zf < 1.0:
            xs[b, :n] = wl.relu_activation(n, zf, seed=5, stream=80 + b)
    xs[2, :n] *= np.where(np.arange(n) % 3 == 0, -1.0, 1.0)        # negative entries for the ReLU case
    A = ref_matrix(w, bf16=dtype == B.BF16)

    def upload(a):
        return torch.from_numpy(wl.f32_to_bf16_bits(a).view(np.int16)).to(DEV) if dtype == B.BF16 else torch.from_numpy(a).to(DEV)

    def rounded(a):
        return wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(a)) if dtype == B.BF16 else a

    xr, xd = rounded(xs), upload(xs)
    for relu, tau in ((0, 0.0), (1, 0.3)):
        refs = []
        for b in range(nv):
            xt = xr[b, :n]
            xt = np.where(xt > np.float32(tau), xt, 0.0).astype(np.float32) if relu else xt
            refs.append(oracle.ref_decode(A, xt))
        for legacy in (0, 1):
            for batch in (1, 2, 3, 4, 5, 8, 9):
                h.set_opts(no_fused_decode=legacy, decode_relu=relu, decode_threshold=tau)
                y = torch.full((batch, ldy), 55.0, dtype=torch.float32, device=DEV)
                B.dbspmspv_decode_batch(h.h, xd, ldx, y, ldy, batch)
                torch.cuda.synchronize()
                yh = y.cpu().numpy()
                for b in range(batch):
                    check(yh[b, :m], *refs[b])
                assert (yh[:, m:] == 55.0).all()                 # nothing is written past m
    # non-finite activations in one vector of the group
    act = np.flatnonzero(xs[1, :n])
    xs[1, act[0]], xs[1, act[2]] = np.inf, np.nan
    xr, xd = rounded(xs), upload(xs)
    h.set_opts()
    for batch in (4, 8):
        y = torch.full((batch, ldy), 55.0, dtype=torch.float32, device=DEV)
        B.dbspmspv_decode_batch(h.h, xd, ldx, y, ldy, batch)
        torch.cuda.synchronize()
        yh = y.cpu().numpy()
        for b in range(batch):
            want, scale = oracle.ref_decode(A, xr[b, :n])
            nan, inf = np.isnan(want), np.isinf(want)
            assert (np.isnan(yh[b, :m]) == nan).all() and (yh[b, :m][inf] == want[inf]).all()
            fin = ~nan & ~inf
            check(yh[b, :m][fin], want[fin], scale[fin])
        assert np.isnan(yh[1, :m]).any()
    with pytest.raises(B.DbSpmspvError):
        B.dbspmspv_decode_batch(h.h, xd, n - 1, y, ldy, 2)
    h.close()


def test_decode_rejects_pattern_handles():
    h = Handle(wl.random_sparse(32, 32, 50, 1, values=False), B.PATTERN)
    t = torch.zeros(32, device=DEV)
    with pytest.raises(B.DbSpmspvError) as e:
        B.dbspmspv_decode(h.h, t, t)
    assert e.value.status == B.ERR_UNSUPPORTED
    h.close()


@pytest.mark.parametrize("inline_max", [31, 3])
def test_decode_on_a_matrix_with_every_block_class(inline_max):
    """Planted dense, row-skewed, column-skewed and banded blocks over a sparse background
    (with inline_max = 3 also packed-COO blocks): the decode entry's own kernels meet every
    class, row-major and column-major, on both paths."""
    from test_gpu_format import mixed_matrix
    a = mixed_matrix(160, 176, 9)
    o = B.default_create_opts()
    o.inline_max = inline_max
    x = wl.relu_activation(a.n, 0.6, seed=3, stream=61)
    for dtype in (B.F32, B.BF16):
        h = Handle(a, dtype, opts=o)
        want, scale = oracle.ref_decode(ref_matrix(a, bf16=dtype == B.BF16), x if dtype == B.F32 else wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(x)))
        for p in PATHS:
            for legacy in (0, 3, 2, 1):
                h.set_opts(force_path=p, no_fused_decode=legacy)
                check(decode(h, x), want, scale)
        h.close()
