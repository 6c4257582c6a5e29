"""The C-ABI library loads and exports every symbol that include/dbspmspv.h declares (no
compute call is made, so this runs without a GPU)."""
import ctypes
import os
import re

from paper_2608_16308_b200 import binding as B
from paper_2608_16308_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "dbspmspv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(dbspmspv_[a-z_]+|db_bfs|db_sssp)\s*\(", text)
    return sorted(set(names))


def test_library_builds_loads_and_exports_every_declared_symbol():
    build_mod.build_library()
    lib = ctypes.CDLL(B.LIB_PATH)
    names = declared_functions()
    assert "dbspmspv_run" in names and "db_bfs" in names and "dbspmspv_decode" in names
    for name in names:
        assert hasattr(lib, name), f"{name} declared in the header but not exported"
    assert sorted(B.EXPORTED_SYMBOLS) == names


def test_host_only_entry_points():
    o = B.default_create_opts()
    assert (o.th0, o.th1, o.th2) == (32, 128, 2.0)          # Section 3.2.1 thresholds
    assert o.w_dense > o.w_mid > o.w_coo >= o.w_inline >= 1   # Section 3.3.2 ordering of segment weights
    r = B.default_run_opts()
    assert r.force_path == B.PATH_AUTO and r.th3 > 0
    assert B.dbspmspv_strerror(B.OK) == "ok"
    assert "capacity" in B.dbspmspv_strerror(B.ERR_CAPACITY)
    assert ctypes.sizeof(B.Stats) % 8 == 0


def test_struct_layouts_match_the_header():
    """Field order of the ctypes mirrors = field order in the header."""
    text = open(os.path.join(ROOT, "include", "dbspmspv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    for cname, cls in (("dbspmspv_create_opts", B.CreateOpts), ("dbspmspv_run_opts", B.RunOpts),
                       ("dbspmspv_stats", B.Stats), ("dbspmspv_call_bytes", B.CallBytes)):
        body = re.search(r"typedef struct \{([^}]*)\}\s*" + cname + ";", text).group(1)
        fields = []
        for decl in body.split(";"):
            decl = decl.strip()
            if not decl:
                continue
            names = decl.split(None, 1)[1]
            for nm in names.split(","):
                fields.append(re.sub(r"\[.*\]", "", nm).strip())
        assert fields == [f[0] for f in cls._fields_], cname
