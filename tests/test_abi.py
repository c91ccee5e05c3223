"""The C-ABI library builds, loads without a GPU and exports every declared symbol."""
import ctypes
import os
import re

import pytest

from paper_2602_08329_b200 import binding as P
from paper_2602_08329_b200 import build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    B.build()
    return P.load()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "prhs.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(prhs_[a-z_]+)\s*\(", text)))


def test_header_and_binding_agree():
    assert declared_symbols() == sorted(P.EXPORTS)


def test_header_constants_and_binding_agree(lib):
    # every PRHS_* integer constant the header defines has the same value in the binding, and a
    # configuration flag the header does not define is rejected at creation
    text = open(os.path.join(ROOT, "include", "prhs.h")).read()
    defs = dict(re.findall(r"#define\s+(PRHS_(?:CFG|FLAG)_[A-Z0-9_]+)\s+(\d+)u?", text))
    assert {"PRHS_CFG_NO_TMA", "PRHS_CFG_TMA_GATHER", "PRHS_CFG_MMA_SYNC_SCORE", "PRHS_CFG_GROUP_TCGEN05"} <= set(defs)
    for name, value in defs.items():
        assert getattr(P, name) == int(value), name
    known = 0
    for name, value in defs.items():
        if name.startswith("PRHS_CFG_"):
            known |= int(value)
    h = ctypes.c_void_p()
    bad = P.Config(1, 1, 4, 2, 128, 1000, 0, 16, 16, 4, 1, -1, 1, 1, (known + 1) & ~known)
    assert lib.prhs_create(ctypes.byref(bad), ctypes.byref(h)) == 1 and not h.value


def test_library_exports_every_declared_symbol(lib):
    for name in declared_symbols():
        assert hasattr(lib, name), name


def test_version_and_struct_layout(lib):
    assert P.version().startswith("prhs-b200")
    # the ctypes mirrors must have the C layout the header implies (LP64)
    assert ctypes.sizeof(P.Config) == 15 * 4
    assert ctypes.sizeof(P.KvView) == 64
    assert ctypes.sizeof(P.Schedule) == 64
    assert P.KvView.seq_lens.offset == 48 and P.Schedule.top_k_per_seq.offset == 16
    assert P.Schedule.psaw_phi.offset == 44 and P.Schedule.psaw_layer_start.offset == 52


def test_create_validates_before_touching_the_device(lib):
    h = ctypes.c_void_p()
    bad = P.Config(1, 1, 4, 2, 64, 1000, 0, 16, 16, 4, 1, -1, 1, 1, 0)          # head_dim 64
    assert lib.prhs_create(ctypes.byref(bad), ctypes.byref(h)) == 2 and not h.value
    bad = P.Config(1, 1, 4, 3, 128, 1000, 0, 16, 16, 4, 1, -1, 1, 1, 0)         # Hkv does not divide Hq
    assert lib.prhs_create(ctypes.byref(bad), ctypes.byref(h)) == 1
    bad = P.Config(1, 1, 4, 2, 128, 1000, 8, 16, 16, 4, 1, -1, 1, 1, 0)         # page size 8
    assert lib.prhs_create(ctypes.byref(bad), ctypes.byref(h)) == 2
    assert b"page_size" in lib.prhs_last_error(None)
    assert lib.prhs_create(None, ctypes.byref(h)) == 1
    assert lib.prhs_destroy(None) == 0
    assert lib.prhs_launch_count(None) == 0 and lib.prhs_index_capacity(None) == 0


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(P, "_lib", None)
    monkeypatch.setattr(P, "LIB_PATH", str(tmp_path / "libprhs.so"))
    with pytest.raises(ImportError):
        P.load()
