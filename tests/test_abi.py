"""The C-ABI library loads without a GPU and exports every symbol include/oilbird.h
declares; host-only entry points behave.  No compute calls."""
import ctypes
import os
import re

import pytest

from paper_2608_03839_b200 import binding as B
from paper_2608_03839_b200 import build as libbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    libbuild.build()
    return B.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "oilbird.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(oilbird_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(L):
    names = declared_symbols()
    assert "oilbird_pool_create" in names and "oilbird_pool_query" in names
    assert "oilbird_pool_append" in names and "oilbird_pool_reset" in names
    for n in names:
        assert hasattr(L, n), f"{n} declared in oilbird.h but not exported"
    assert sorted(B.SYMBOLS) == names, "binding and header disagree on the symbol list"


def test_defaults_are_the_papers_constants(L):
    p = B.CQueryParams()
    L.oilbird_query_params_default(ctypes.byref(p))
    assert (p.k, p.offset, p.depth_mode, p.n_tiers) == (8, 2, B.DEPTH_TIERED, 2)
    assert abs(p.theta - 0.8) < 1e-7
    assert [round(p.tier_thr[i], 4) for i in range(2)] == [0.90, 0.82]
    assert [p.tier_depth[i] for i in range(2)] == [48, 8]
    py = B.QueryParams()
    assert (py.k, py.theta, py.offset, py.tier_thr, py.tier_depth) == (8, 0.8, 2, (0.90, 0.82), (48, 8))


def test_struct_layout_constants_match_header():
    text = open(os.path.join(ROOT, "include", "oilbird.h")).read()
    for name, val in [("OILBIRD_MAX_NQ", B.MAX_NQ), ("OILBIRD_MAX_K", B.MAX_K),
                      ("OILBIRD_MAX_CONT_LEN", B.MAX_CONT_LEN), ("OILBIRD_MAX_TIERS", B.MAX_TIERS)]:
        m = re.search(rf"#define\s+{name}\s+(\d+)", text)
        assert m and int(m.group(1)) == val
    for name, val in [("EINVAL", B.EINVAL), ("ECAPACITY", B.ECAPACITY), ("ENOMEM", B.ENOMEM),
                      ("ECUDA", B.ECUDA), ("ESTALL", B.ESTALL), ("EGUARD", B.EGUARD)]:
        m = re.search(rf"#define\s+OILBIRD_{name}\s+\((-\d+)\)", text)
        assert m and int(m.group(1)) == val


def test_arena_size_and_strerror(L):
    cfg = B.PoolConfig(d=4096, capacity_rows=65536)
    n = L.oilbird_pool_arena_bytes(ctypes.byref(cfg))
    assert n > 65536 * 4096 * 2 and n < 65536 * 4096 * 2 + (1 << 30)
    bad = B.PoolConfig(d=12, capacity_rows=10)
    assert L.oilbird_pool_arena_bytes(ctypes.byref(bad)) == 0
    assert L.oilbird_strerror(0) == b"ok"
    assert b"capacity" in L.oilbird_strerror(B.ECAPACITY)
    assert L.oilbird_pool_size(None) == 0


def test_product_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2608_03839_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in src and "from oracle" not in src, f
                assert "oilbird_oracle" not in src, f


def test_missing_library_fails_loudly(monkeypatch):
    """No CPU or PyTorch fallback: without liboilbird.so the binding refuses to work."""
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", "/nonexistent/liboilbird.so")
    with pytest.raises(ImportError, match="no CPU or PyTorch fallback"):
        B.lib()


def test_pool_needs_a_cuda_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("this check is for the CPU-only box")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        B.Pool(64, 16)
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        B.Ring(64, 16)


def test_merge_defaults_are_the_papers_constants(L):
    p = B.MergeParams()
    L.oilbird_merge_params_default(ctypes.byref(p))
    assert (p.budget, p.max_nodes, p.min_len, p.root_attached) == (16, 60, 2, 0)
