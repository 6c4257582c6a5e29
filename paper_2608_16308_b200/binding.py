"""Thin ctypes binding over libdbspmspv.so: argument marshalling only -- every step of the hot
path runs in the library's CUDA kernels.  PyTorch supplies device memory and streams.

The names mirror the C ABI in include/dbspmspv.h (dbspmspv_create_csr, dbspmspv_run, db_bfs,
dbspmspv_decode, ...).  There is no CPU fallback: if the shared library is missing or cannot
be loaded, importing a symbol raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

HERE = os.path.dirname(os.path.abspath(__file__))
# DBSPMSPV_LIBRARY: another build of the same library (the range-checked one, for the tests)
LIB_PATH = os.environ.get("DBSPMSPV_LIBRARY") or os.path.join(HERE, "libdbspmspv.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALLOC, ERR_CUDA, ERR_CAPACITY, ERR_TIMEOUT, ERR_BOUNDS, ERR_TOO_LARGE, ERR_INTERNAL = range(10)
F32, BF16, PATTERN = 0, 1, 2
PLUS_TIMES, OR_AND, MIN_PLUS = 0, 1, 2
PATH_AUTO, PATH_PUSH, PATH_PULL = 0, 1, 2
FORMAT_AUTO, FORMAT_COO, FORMAT_CSR = 0, 1, 2
BLK_INLINE, BLK_COO, BLK_FCSR, BLK_FCSC, BLK_CSR, BLK_DENSE = range(6)
BLK_NAMES = ("inline", "coo", "fcsr", "fcsc", "csr", "dense")
MAX_BFS_LEVELS_RECORDED = 64

EXPORTED_SYMBOLS = (
    "dbspmspv_default_create_opts", "dbspmspv_default_run_opts", "dbspmspv_create_csr",
    "dbspmspv_create_coo", "dbspmspv_run", "db_bfs", "db_sssp", "dbspmspv_decode", "dbspmspv_get_stats",
    "dbspmspv_export_coo", "dbspmspv_export_blocks", "dbspmspv_export_views",
    "dbspmspv_set_run_opts", "dbspmspv_destroy", "dbspmspv_strerror", "dbspmspv_compact_noalloc",
    "dbspmspv_test_bounded_wait", "dbspmspv_test_corrupt_entry", "dbspmspv_decode_batch", "dbspmspv_run_masked", "dbspmspv_count_call_bytes", "dbspmspv_probe_floor",
)


class CreateOpts(ctypes.Structure):
    _fields_ = [("th0", ctypes.c_int32), ("th1", ctypes.c_int32), ("th2", ctypes.c_float),
                ("seg_cut", ctypes.c_int32), ("w_dense", ctypes.c_int32), ("w_mid", ctypes.c_int32),
                ("w_coo", ctypes.c_int32), ("force_format", ctypes.c_int32),
                ("input_on_host", ctypes.c_int32), ("inline_max", ctypes.c_int32),
                ("w_inline", ctypes.c_int32), ("w_dense_sparse", ctypes.c_int32),
                ("w_mid_sparse", ctypes.c_int32), ("no_bfs_index", ctypes.c_int32),
                ("reserved", ctypes.c_int32 * 2)]


class RunOpts(ctypes.Structure):
    _fields_ = [("th3", ctypes.c_float), ("force_path", ctypes.c_int32),
                ("popc_threshold", ctypes.c_int32), ("validate", ctypes.c_int32),
                ("timing", ctypes.c_int32), ("th3_bfs", ctypes.c_float),
                ("th3_decode", ctypes.c_float), ("no_fused_decode", ctypes.c_int32),
                ("bfs_push_max_edge_frac", ctypes.c_float), ("hub_min_nnz_x", ctypes.c_int32),
                ("decode_threshold", ctypes.c_float), ("decode_relu", ctypes.c_int32),
                ("decode_x_f32", ctypes.c_int32), ("no_small_call", ctypes.c_int32),
                ("reserved", ctypes.c_int32 * 2)]


class Stats(ctypes.Structure):
    _fields_ = [("m", ctypes.c_int64), ("n", ctypes.c_int64), ("nnz", ctypes.c_int64),
                ("n_blocks", ctypes.c_int64), ("n_view_entries", ctypes.c_int64), ("class_blocks", ctypes.c_int64 * 6),
                ("class_nnz", ctypes.c_int64 * 6), ("n_row_blocks", ctypes.c_int64),
                ("n_col_blocks", ctypes.c_int64), ("n_segments", ctypes.c_int64),
                ("payload_bytes", ctypes.c_int64), ("csr_view_bytes", ctypes.c_int64),
                ("csc_view_bytes", ctypes.c_int64), ("segment_bytes", ctypes.c_int64),
                ("workspace_bytes", ctypes.c_int64), ("last_path", ctypes.c_int32),
                ("last_n_nzblk", ctypes.c_int32), ("last_n_tasks", ctypes.c_int32),
                ("last_y_nnz", ctypes.c_int32), ("bfs_levels", ctypes.c_int32),
                ("bfs_reached", ctypes.c_int32),
                ("bfs_level_path", ctypes.c_int32 * MAX_BFS_LEVELS_RECORDED),
                ("bfs_level_nzblk", ctypes.c_int32 * MAX_BFS_LEVELS_RECORDED),
                ("device_status", ctypes.c_int32), ("last_compute_ms", ctypes.c_float),
                ("kernel_launches", ctypes.c_int64), ("bfs_index_bytes", ctypes.c_int64),
                ("lean_index_bytes", ctypes.c_int64), ("bfs_setup_us", ctypes.c_float),
                ("bfs_level_us", ctypes.c_float * MAX_BFS_LEVELS_RECORDED), ("n_hub_row_blocks", ctypes.c_int32)]


class CallBytes(ctypes.Structure):
    _fields_ = [("view_entries", ctypes.c_int64), ("view_bytes", ctypes.c_int64),
                ("payload_blocks", ctypes.c_int64), ("payload_bytes", ctypes.c_int64),
                ("pointer_bytes", ctypes.c_int64), ("active_vector_blocks", ctypes.c_int64),
                ("reserved", ctypes.c_int64 * 2)]


_lib = None


def lib() -> ctypes.CDLL:
    """Load the CUDA library (no fallback: a missing library is an error)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2608_16308_b200.build` "
                "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
        L.dbspmspv_default_create_opts.argtypes = [ctypes.POINTER(CreateOpts)]
        L.dbspmspv_default_create_opts.restype = None
        L.dbspmspv_default_run_opts.argtypes = [ctypes.POINTER(RunOpts)]
        L.dbspmspv_default_run_opts.restype = None
        L.dbspmspv_create_csr.argtypes = [ctypes.POINTER(vp), i64, i64, i64, vp, vp, vp, ctypes.c_int,
                                          ctypes.c_int, ctypes.POINTER(CreateOpts), vp]
        L.dbspmspv_create_coo.argtypes = L.dbspmspv_create_csr.argtypes
        L.dbspmspv_run.argtypes = [vp, vp, vp, i32, ctypes.c_int, vp, vp, i64, vp, vp]
        L.dbspmspv_run_masked.argtypes = [vp, vp, vp, i32, ctypes.c_int, vp, ctypes.c_int, vp, vp, i64, vp, vp]
        L.db_bfs.argtypes = [vp, i32, vp, vp]
        L.db_sssp.argtypes = [vp, i32, vp, ctypes.POINTER(ctypes.c_int32), vp]
        L.dbspmspv_decode.argtypes = [vp, vp, vp, vp]
        L.dbspmspv_decode_batch.argtypes = [vp, vp, i64, vp, i64, i32, vp]
        L.dbspmspv_get_stats.argtypes = [vp, ctypes.POINTER(Stats)]
        L.dbspmspv_export_coo.argtypes = [vp, vp, vp, vp]
        L.dbspmspv_export_blocks.argtypes = [vp, vp, vp, vp, vp]
        L.dbspmspv_export_views.argtypes = [vp, vp, vp, vp, vp]
        L.dbspmspv_compact_noalloc.argtypes = [vp, vp, i64, vp, vp, i64, vp, vp]
        L.dbspmspv_test_bounded_wait.argtypes = [vp, i32, vp]
        L.dbspmspv_test_corrupt_entry.argtypes = [vp, i32, ctypes.c_uint32]
        L.dbspmspv_count_call_bytes.argtypes = [vp, vp, i32, ctypes.c_int, ctypes.POINTER(CallBytes)]
        L.dbspmspv_probe_floor.argtypes = [ctypes.c_int, vp, i32, i32, vp, vp]
        L.dbspmspv_set_run_opts.argtypes = [vp, ctypes.POINTER(RunOpts)]
        L.dbspmspv_destroy.argtypes = [vp]
        L.dbspmspv_strerror.argtypes = [ctypes.c_int]
        L.dbspmspv_strerror.restype = ctypes.c_char_p
        for name in EXPORTED_SYMBOLS:
            f = getattr(L, name)
            if f.restype is ctypes.c_int and name not in ("dbspmspv_strerror",):
                f.restype = ctypes.c_int
        _lib = L
    return _lib


class DbSpmspvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib().dbspmspv_strerror(status).decode()} (status {status})")


def _check(status: int, where: str) -> None:
    if status != OK:
        raise DbSpmspvError(status, where)


def _ptr(t) -> Optional[int]:
    """Device (or host) address of a torch tensor / numpy array; None passes NULL."""
    if t is None:
        return None
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    return t.ctypes.data


def _stream() -> int:
    import torch
    return torch.cuda.current_stream().cuda_stream


def default_create_opts() -> CreateOpts:
    o = CreateOpts()
    lib().dbspmspv_default_create_opts(ctypes.byref(o))
    return o


def default_run_opts() -> RunOpts:
    o = RunOpts()
    lib().dbspmspv_default_run_opts(ctypes.byref(o))
    return o


def dbspmspv_create_csr(m, n, nnz, row_ptr, col_idx, val, dtype, block_size=16,
                        opts: Optional[CreateOpts] = None, stream: Optional[int] = None) -> int:
    """Marshals to dbspmspv_create_csr; returns the opaque handle as an integer."""
    h = ctypes.c_void_p()
    st = lib().dbspmspv_create_csr(ctypes.byref(h), m, n, nnz, _ptr(row_ptr), _ptr(col_idx), _ptr(val),
                                   dtype, block_size, ctypes.byref(opts) if opts is not None else None,
                                   _stream() if stream is None else stream)
    _check(st, "dbspmspv_create_csr")
    return h.value


def dbspmspv_create_coo(m, n, nnz, row, col, val, dtype, block_size=16,
                        opts: Optional[CreateOpts] = None, stream: Optional[int] = None) -> int:
    h = ctypes.c_void_p()
    st = lib().dbspmspv_create_coo(ctypes.byref(h), m, n, nnz, _ptr(row), _ptr(col), _ptr(val), dtype,
                                   block_size, ctypes.byref(opts) if opts is not None else None,
                                   _stream() if stream is None else stream)
    _check(st, "dbspmspv_create_coo")
    return h.value


def dbspmspv_run(h, x_idx, x_val, nnz_x, semiring, y_idx, y_val, y_capacity, y_nnz,
                 stream: Optional[int] = None) -> None:
    _check(lib().dbspmspv_run(h, _ptr(x_idx), _ptr(x_val), nnz_x, semiring, _ptr(y_idx), _ptr(y_val),
                              y_capacity, _ptr(y_nnz), _stream() if stream is None else stream),
           "dbspmspv_run")


def db_bfs(h, src, levels, stream: Optional[int] = None) -> None:
    _check(lib().db_bfs(h, src, _ptr(levels), _stream() if stream is None else stream), "db_bfs")


def db_sssp(h, src, dist, stream: Optional[int] = None) -> int:
    """Returns the number of (min, +) products the search made."""
    steps = ctypes.c_int32(0)
    _check(lib().db_sssp(h, src, _ptr(dist), ctypes.byref(steps), _stream() if stream is None else stream), "db_sssp")
    return int(steps.value)


def dbspmspv_decode(h, x, y, stream: Optional[int] = None) -> None:
    _check(lib().dbspmspv_decode(h, _ptr(x), _ptr(y), _stream() if stream is None else stream),
           "dbspmspv_decode")


def dbspmspv_get_stats(h, raise_on_device_status: bool = True) -> Stats:
    s = Stats()
    st = lib().dbspmspv_get_stats(h, ctypes.byref(s))
    if raise_on_device_status:
        _check(st, "dbspmspv_get_stats")
    return s


def dbspmspv_export_coo(h, row, col, val) -> None:
    _check(lib().dbspmspv_export_coo(h, _ptr(row), _ptr(col), _ptr(val)), "dbspmspv_export_coo")


def dbspmspv_export_blocks(h, block_row, block_col, block_class, block_nnz) -> None:
    _check(lib().dbspmspv_export_blocks(h, _ptr(block_row), _ptr(block_col), _ptr(block_class),
                                        _ptr(block_nnz)), "dbspmspv_export_blocks")


def dbspmspv_export_views(h, csr_row_ptr, csc_col_ptr, csc_row, csc2csr) -> None:
    _check(lib().dbspmspv_export_views(h, _ptr(csr_row_ptr), _ptr(csc_col_ptr), _ptr(csc_row),
                                       _ptr(csc2csr)), "dbspmspv_export_views")


def dbspmspv_compact_noalloc(acc, hit_bitmap, m, y_idx, y_val, y_capacity, y_nnz,
                             stream: Optional[int] = None) -> None:
    """Marshals to dbspmspv_compact_noalloc: compaction of (dense values, row-hit bitmap) into a
    sorted sparse vector for callers that may not allocate device memory (the library keeps the
    16 KB of scratch it needs in a fixed device array; at most 33,554,432 rows per call)."""
    _check(lib().dbspmspv_compact_noalloc(_ptr(acc), _ptr(hit_bitmap), m, _ptr(y_idx), _ptr(y_val),
                                          y_capacity, _ptr(y_nnz), _stream() if stream is None else stream),
           "dbspmspv_compact_noalloc")


def dbspmspv_test_bounded_wait(h, max_tries: int, stream: Optional[int] = None) -> None:
    _check(lib().dbspmspv_test_bounded_wait(h, max_tries, _stream() if stream is None else stream),
           "dbspmspv_test_bounded_wait")


def dbspmspv_run_masked(h, x_idx, x_val, nnz_x: int, semiring: int, row_mask, complement: int, y_idx, y_val,
                        y_capacity: int, y_nnz, stream: Optional[int] = None) -> None:
    _check(lib().dbspmspv_run_masked(h, _ptr(x_idx), _ptr(x_val), nnz_x, semiring, _ptr(row_mask), complement, _ptr(y_idx),
                                     _ptr(y_val), y_capacity, _ptr(y_nnz), _stream() if stream is None else stream),
           "dbspmspv_run_masked")


def dbspmspv_decode_batch(h, x, ldx: int, y, ldy: int, batch: int, stream: Optional[int] = None) -> None:
    _check(lib().dbspmspv_decode_batch(h, _ptr(x), ldx, _ptr(y), ldy, batch, _stream() if stream is None else stream),
           "dbspmspv_decode_batch")


def dbspmspv_test_corrupt_entry(h, position: int, block_index: int) -> None:
    _check(lib().dbspmspv_test_corrupt_entry(h, position, block_index), "dbspmspv_test_corrupt_entry")


def dbspmspv_count_call_bytes(h, x_idx, nnz_x: int, path: int) -> CallBytes:
    out = CallBytes()
    _check(lib().dbspmspv_count_call_bytes(h, _ptr(x_idx), nnz_x, path, ctypes.byref(out)), "dbspmspv_count_call_bytes")
    return out


def dbspmspv_probe_floor(kind: int, chain=None, start: int = 0, steps: int = 1, out=None, stream: Optional[int] = None) -> None:
    _check(lib().dbspmspv_probe_floor(kind, _ptr(chain), start, steps, _ptr(out), _stream() if stream is None else stream),
           "dbspmspv_probe_floor")


def dbspmspv_set_run_opts(h, opts: RunOpts) -> None:
    _check(lib().dbspmspv_set_run_opts(h, ctypes.byref(opts)), "dbspmspv_set_run_opts")


def dbspmspv_destroy(h) -> None:
    _check(lib().dbspmspv_destroy(h), "dbspmspv_destroy")


def dbspmspv_strerror(status: int) -> str:
    return lib().dbspmspv_strerror(status).decode()
