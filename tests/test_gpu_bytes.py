"""The benchmark's host-side byte model against the library's counting pass: the format bytes
one call reads on a path (view entries, payloads, pointer words) are derived twice -- by
bench.ByteModel from the matrix structure and the documented sizes alone, and by
dbspmspv_count_call_bytes walking the format as built -- and must agree exactly."""
import os
import sys

import numpy as np
import pytest
import torch

from paper_2608_16308_b200 import binding as B
from paper_2608_16308_b200 import workloads as wl
from gpu_util import Handle, DEV
from test_gpu_format import mixed_matrix

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench  # noqa: E402

pytestmark = pytest.mark.gpu

FIELDS = ("view_entries", "view_bytes", "payload_blocks", "payload_bytes", "pointer_bytes", "active_vector_blocks")


def counted(h, x, path):
    xi = torch.from_numpy(np.ascontiguousarray(x.idx, dtype=np.int32)).to(DEV)
    c = B.dbspmspv_count_call_bytes(h.h, xi, int(x.idx.size), path)
    return {f: int(getattr(c, f)) for f in FIELDS}


@pytest.mark.parametrize("name,make,vs,dtype", [
    ("rmat13", lambda: wl.rmat(13, 16, seed=1), 4, B.F32),
    ("uniform", lambda: wl.random_sparse(3000, 2000, 40000, 1), 4, B.F32),
    ("mixed", lambda: mixed_matrix(96, 112, 3), 4, B.F32),
    ("rmat12_pattern", lambda: wl.rmat(12, 16, seed=3, values=False, symmetrise=True), 0, B.PATTERN),
])
def test_model_equals_counting_pass(name, make, vs, dtype):
    csr = make()
    h = Handle(csr, dtype)
    model = bench.ByteModel(csr, vs)
    for frac in (0.002, 0.05, 0.6):
        x = wl.sparse_x(9, 0, csr.n, max(1, int(csr.n * frac)))
        for path in (B.PATH_PUSH, B.PATH_PULL):
            if path == B.PATH_PULL and model.heavy:
                continue                      # (its pull tables are a property of the handle, not of the matrix)
            assert model.format_bytes(x.idx, path) == counted(h, x, path), (name, frac, path)
        # the counting pass leaves the workspace clean: a real call still gives the right answer
        yi, yv, k = h.run(x, semiring=B.OR_AND)
        assert k == np.unique(csr.rows()[np.isin(csr.col_idx, x.idx)]).size
    h.close()


def test_stencil_push_counts_whole_column_blocks():
    """A handle whose elements sit mostly in blocks with a payload pushes whole column blocks."""
    csr = wl.stencil27(16, seed=2)
    h = Handle(csr, B.F32)
    model = bench.ByteModel(csr, 4)
    assert model.heavy
    x = wl.clustered_x(csr.n, 6)
    assert model.format_bytes(x.idx, B.PATH_PUSH) == counted(h, x, B.PATH_PUSH)
    c = counted(h, x, B.PATH_PULL)
    assert c["view_entries"] == h.stats.n_view_entries and c["payload_blocks"] > 0
    h.close()
