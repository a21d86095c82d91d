"""The C-ABI library loads on a machine without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

from paper_2609_33570_b200 import api, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return api.lib()


def declared_functions():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(hilore_[a-z0-9_]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported(lib):
    decl = declared_functions()
    assert {"hilore_grpo_coeffs", "hilore_unit_exposure", "hilore_compress", "hilore_recover",
            "hilore_plan_apply"} <= decl
    for name in decl:
        assert hasattr(lib, name), name
    assert decl == set(api.EXPORTS) | {n for n in decl if n not in api.EXPORTS}
    assert set(api.EXPORTS) <= decl


def test_status_strings_and_version(lib):
    assert api.status_string(api.OK) == "ok"
    assert len({api.status_string(s) for s in range(7)}) == 7
    assert lib.hilore_abi_version() >= 1000


def test_unit_struct_layout_matches_header():
    assert ctypes.sizeof(api.HiloreUnit) == 5 * 8 + 3 * 8 + 2 * 4
    assert api.HiloreUnit.rows.offset == 40 and api.HiloreUnit.fmt.offset == 64


def test_workspace_bytes_formula(lib):
    assert api.hilore_workspace_bytes(84, 8192) == 85 * 8 * 16
    assert api.hilore_workspace_bytes(1, 1) == 2 * 16
    assert api.hilore_workspace_bytes(3, 0) == 4 * 16


def test_argument_validation_needs_no_gpu(lib):
    """Status codes that are decided on the host before anything is launched."""
    A = 0x1000  # a fake, suitably aligned device address: never dereferenced on these paths
    c = lambda *a, **k: api.hilore_compress(*a, stream=0, check=False, **k)
    assert c(None, 8, 64, 64, api.FMT_E4M3FN_RAW, 0, A, None, None) == api.INVALID_ARG
    assert c(A, 8, 64, 64, 7, 0, A, None, None) == api.INVALID_ARG
    assert c(A, 8, 64, 64, api.FMT_E4M3FN_BLK, 32, A, A, None) == api.INVALID_ARG
    assert c(A, 8, 96, 96, api.FMT_E4M3FN_RAW, 0, A, None, None) == api.SHAPE
    assert c(A, 8, 128, 64, api.FMT_E4M3FN_RAW, 0, A, None, None) == api.SHAPE
    assert c(A, 8, 64, 72, api.FMT_E4M3FN_RAW, 0, A, None, None) == api.ALIGN
    assert c(A + 2, 8, 64, 64, api.FMT_E4M3FN_RAW, 0, A, None, None) == api.ALIGN
    assert c(A, 8, 64, 64, api.FMT_E4M3FN_BLK, 64, A, None, None) == api.INVALID_ARG
    assert c(A, 8, 64, 64, api.FMT_E4M3FN_RAW, 0, None, None, None) == api.INVALID_ARG
    assert c(A, 0, 64, 64, api.FMT_E4M3FN_RAW, 0, A, None, None) == api.OK          # empty unit: nothing to do
    r = lambda *a: api.hilore_recover(*a, stream=0, check=False)
    assert r(A, None, 8, 64, api.FMT_E4M3FN_BLK, 64, A, 64) == api.INVALID_ARG
    assert r(A, A, 8, 64, api.FMT_E4M3FN_BLK, 64, A + 16, 64) == api.ALIGN
    g = lambda **k: api.hilore_grpo_coeffs(k.get("rewards", A), k.get("n", 16), k.get("G", 8), k.get("off", 0),
                                           k.get("rows", 8), k.get("T", 64), A, A, k.get("ref"), A, k.get("N", 10),
                                           None, 0.2, k.get("beta", 0.0), 1e-6, None, A, None, None, stream=0,
                                           check=False)
    assert g(n=15) == api.SHAPE
    assert g(T=66) == api.SHAPE
    assert g(off=12) == api.SHAPE
    assert g(N=0) == api.ZERO_NORM
    assert g(beta=1e-3) == api.INVALID_ARG
    assert g(G=0) == api.INVALID_ARG
    assert g(rows=0) == api.OK
    e = lambda **k: api.hilore_unit_exposure(A, A, 2, 64, A, k.get("U", 3), k.get("ld", 128), k.get("shift", 0), 1e-8,
                                             A, None, A, k.get("ws", 1 << 20), stream=0, check=False)
    assert e(ld=100) == api.SHAPE
    assert e(ws=8) == api.WORKSPACE
    assert e(shift=2) == api.INVALID_ARG
    assert e(U=0) == api.OK
