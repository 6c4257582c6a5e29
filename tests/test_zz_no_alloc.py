"""dbspmspv_compact_noalloc, the entry point for callers that cannot allocate device memory
when they call (allocator-free real-time loops, hosts that own the whole device heap): it must
produce exactly what the library's ordinary path produces.  The ordinary path here is
dbspmspv_run, whose last step is the same compaction; its sparse result is scattered back into
a dense vector plus a row-hit bitmap, handed to the no-allocation entry point, and the two
sparse vectors are compared -- twice in a row, the second time on a smaller problem, so stale
contents of the shared fixed scratch from the first call are in play.  Collected last on
purpose (file name), and self-contained so that it also passes alone in a fresh process."""
import numpy as np
import pytest
import torch

from paper_2608_16308_b200 import binding as B
from paper_2608_16308_b200 import workloads as wl
from gpu_util import Handle, DEV

pytestmark = pytest.mark.gpu


def reference_sparse_result(csr, x):
    h = Handle(csr, B.F32)
    yi, yv, k = h.run(x)
    h.close()
    return yi, yv, k


def dense_and_bitmap(m, yi, yv):
    acc = np.zeros(m, dtype=np.float32)
    acc[yi] = yv
    words = np.zeros((m + 31) // 32, dtype=np.uint32)
    np.bitwise_or.at(words, yi >> 5, np.uint32(1) << (yi & 31).astype(np.uint32))
    return acc, words


def compact(m, acc, words, capacity=None):
    cap = m if capacity is None else capacity
    d_acc = torch.from_numpy(acc).to(DEV)
    d_words = torch.from_numpy(words.view(np.int32)).to(DEV)
    y_idx = torch.full((max(cap, 1),), -1, dtype=torch.int32, device=DEV)
    y_val = torch.full((max(cap, 1),), -1.0, dtype=torch.float32, device=DEV)
    y_nnz = torch.full((1,), -1, dtype=torch.int32, device=DEV)
    B.dbspmspv_compact_noalloc(d_acc, d_words, m, y_idx, y_val, cap, y_nnz)
    torch.cuda.synchronize()
    k = int(y_nnz.item())
    kk = min(k, cap)
    return y_idx[:kk].cpu().numpy(), y_val[:kk].cpu().numpy(), k, y_idx.cpu().numpy()


def test_matches_the_ordinary_path_on_two_calls_in_a_row():
    # first call: large enough for many tiles of the fixed scratch (300,000 rows -> 37 tiles)
    a = wl.random_sparse(300000, 4096, 900000, 31)
    x = wl.sparse_x(32, 0, a.n, 1500)
    yi, yv, k = reference_sparse_result(a, x)
    assert k > 1000
    acc, words = dense_and_bitmap(a.m, yi, yv)
    gi, gv, gk, _ = compact(a.m, acc, words)
    assert gk == k and np.array_equal(gi, yi)
    assert np.array_equal(gv, yv)          # compaction moves values, it does no arithmetic
    # second call right after it: a smaller, ragged problem; the scratch still holds call one
    b = wl.random_sparse(20011, 777, 60000, 33)
    x2 = wl.sparse_x(34, 0, b.n, 90)
    yi2, yv2, k2 = reference_sparse_result(b, x2)
    acc2, words2 = dense_and_bitmap(b.m, yi2, yv2)
    gi2, gv2, gk2, _ = compact(b.m, acc2, words2)
    assert gk2 == k2 and np.array_equal(gi2, yi2) and np.array_equal(gv2, yv2)
    # and the first problem once more
    gi, gv, gk, _ = compact(a.m, acc, words)
    assert gk == k and np.array_equal(gi, yi) and np.array_equal(gv, yv)


def test_capacity_empty_and_size_limit():
    m = 10000
    yi = np.arange(0, m, 7, dtype=np.int64)
    yv = (yi % 13).astype(np.float32) - 6.0
    acc, words = dense_and_bitmap(m, yi, yv)
    cap = yi.size // 3
    gi, gv, gk, raw = compact(m, acc, words, capacity=cap)
    assert gk == yi.size and np.array_equal(gi, yi[:cap]) and np.array_equal(gv, yv[:cap])
    assert (raw[cap:] == -1).all()                      # nothing beyond the capacity
    gi, gv, gk, _ = compact(m, np.zeros(m, np.float32), np.zeros((m + 31) // 32, np.uint32))
    assert gk == 0 and gi.size == 0
    # more rows than the fixed scratch covers: refused with its own status, nothing launched
    t = torch.zeros(8, dtype=torch.int32, device=DEV)
    with pytest.raises(B.DbSpmspvError) as e:
        B.dbspmspv_compact_noalloc(t, t, 33554432 + 1, t, None, 8, t)
    assert e.value.status == B.ERR_TOO_LARGE
    assert "scratch" in B.dbspmspv_strerror(B.ERR_TOO_LARGE)


def test_garbage_bits_beyond_the_last_row_are_ignored():
    """m not a multiple of 32 and the unused high bits of the last bitmap word set: neither the
    count nor the placement may see them."""
    m = 1003                                             # last word holds rows 992..1002
    yi = np.array([0, 5, 991, 992, 1002], dtype=np.int64)
    yv = np.array([1.0, -2.0, 3.0, 4.5, -0.25], dtype=np.float32)
    acc, words = dense_and_bitmap(m, yi, yv)
    words[-1] |= np.uint32(0xFFFFF800)                   # bits for rows 1003..1023
    gi, gv, gk, raw = compact(m, acc, words)
    assert gk == yi.size and np.array_equal(gi, yi) and np.array_equal(gv, yv)
    assert (raw[yi.size:] == -1).all()
    with pytest.raises(B.DbSpmspvError) as e:            # m = 0 is rejected, as documented
        t = torch.zeros(8, dtype=torch.int32, device=DEV)
        B.dbspmspv_compact_noalloc(t, t, 0, t, None, 8, t)
    assert e.value.status == B.ERR_INVALID_ARG
