"""The C-ABI library builds, loads and exports every symbol include/sfb.h declares (no GPU needed)."""
import ctypes
import os
import re

from paper_1511_08486_b200 import binding as B
from paper_1511_08486_b200.build import build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "sfb.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sfb_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    path = build_library()
    lib = ctypes.CDLL(path)
    names = declared_symbols()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), f"{n} declared in sfb.h but not exported"
    assert set(B.EXPORTS) <= set(names)


def test_host_only_calls():
    build_library()
    d = B.make_desc("mlr", "f32", 10, 64, 4, 8)
    assert B.sfb_ld(d) == (12, 64)
    assert B.sfb_sf_buffer_bytes(d) == 256 + 4 * (384 + 2048)
    dbf = B.make_desc("mlr", "bf16", 10, 64, 4, 8)
    assert B.sfb_ld(dbf) == (16, 64)
    assert B.sfb_sf_buffer_bytes(B.make_desc("mlr", "f32", 0, 64, 4, 8)) == 0
    assert B.strerror(0) == "ok" and "CUDA" in B.strerror(-4)
    # the layout the library reports equals the oracle packer's, field by field
    from oracle import sfb_oracle as orc
    for (m, p, J, D, P, Bs, sp, cap) in [("mlr", "f32", 1000, 20000, 8, 128, 0, 0), ("mlr", "bf16", 32768, 8192, 16, 256, 0, 0),
                                         ("dml", "f32", 600, 10000, 8, 256, 0, 0), ("sc", "f32", 4096, 10000, 16, 64, 1, 16 * 32992),
                                         ("mlr", "f32", 37, 203, 3, 7, 0, 0)]:
        desc = B.make_desc(m, p, J, D, P, Bs, v_sparse=sp, nnz_capacity=cap)
        lay = orc.sf_layout(B.MODELS[m], 1 if p == "bf16" else 0, J, D, P, Bs, bool(sp), cap)
        assert B.sfb_sf_buffer_bytes(desc) == lay["total_bytes"]
        assert B.sfb_ld(desc) == (lay["ldu"], lay["ldv"])
