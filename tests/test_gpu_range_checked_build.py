"""The range-checked build of the library (-DDBS_BOUNDS_CHECK: every index a kernel reads from
the handle's arrays is tested, a violation records ERR_INTERNAL and skips the access) runs the
small parity cases of run (all semirings), decode, BFS and shortest paths in a child process; every handle's status must stay
clean and every parity check must hold.  It stands in for a memory checker."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_small_parity_cases_pass_under_the_range_checked_library():
    from paper_2608_16308_b200 import build
    lib = build.build_library(checked=True)
    env = dict(os.environ, DBSPMSPV_LIBRARY=lib)
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
           "tests/test_gpu_spmspv.py", "tests/test_gpu_decode.py", "tests/test_gpu_bfs.py", "tests/test_gpu_format.py",
           "tests/test_gpu_minplus.py", "tests/test_gpu_randomised.py"]
    r = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-4000:] + r.stderr[-2000:]


def test_a_corrupted_view_entry_is_caught_not_followed():
    """An entry whose column block index was overwritten with a value past the last column block:
    the checked library reports ERR_INTERNAL and the call still returns; the context stays usable."""
    code = r"""
import sys, os
sys.path.insert(0, os.getcwd()); sys.path.insert(0, os.path.join(os.getcwd(), "tests"))
import numpy as np, torch
from paper_2608_16308_b200 import binding as B, workloads as wl
from gpu_util import Handle, DEV
a = wl.random_sparse(300, 200, 4000, 1)
h = Handle(a, B.F32)
B.dbspmspv_test_corrupt_entry(h.h, 5, 0x07FFFFF0)
x = wl.sparse_x(3, 0, a.n, 150)
h.set_opts(force_path=B.PATH_PULL)
h.run(x)
st = B.dbspmspv_get_stats(h.h, raise_on_device_status=False)
assert st.device_status == B.ERR_INTERNAL, st.device_status
h2 = Handle(a, B.F32); h2.run(x); h2.close()
print("caught")
"""
    from paper_2608_16308_b200 import build
    lib = build.build_library(checked=True)
    env = dict(os.environ, DBSPMSPV_LIBRARY=lib)
    r = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "caught" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]
