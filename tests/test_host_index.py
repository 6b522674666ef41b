"""CPU tests of the library's host logic: closed-form index arithmetic against the oracle's
running-counter walk, the exported symbols, and host-side argument validation."""
import ctypes
import os
import re
import subprocess
import tempfile

import numpy as np
import pytest

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CSRC = os.path.join(ROOT, "paper_2211_10482_b200", "csrc")


@pytest.fixture(scope="module")
def shim():
    out = os.path.join(tempfile.mkdtemp(prefix="st_shim_"), "shim.so")
    subprocess.check_call(["g++", "-O2", "-shared", "-fPIC", "-std=c++17", "-x", "c++", "-I", CSRC,
                           os.path.join(ROOT, "tests", "index_host_shim.cpp"), "-o", out])
    L = ctypes.CDLL(out)
    ll = ctypes.c_longlong
    for name in ("shim_tri_rows", "shim_tet_rows", "shim_check_all_tri", "shim_check_all_tet", "shim_simp4_rows",
                 "shim_check_all_simp4"):
        getattr(L, name).argtypes = [ll]
        getattr(L, name).restype = ll
    L.shim_tri_encode.argtypes = [ll, ll, ll]
    L.shim_tri_encode.restype = ll
    L.shim_tet_encode.argtypes = [ll, ll, ll, ll]
    L.shim_tet_encode.restype = ll
    L.shim_tri_decode.argtypes = [ll, ll, ctypes.POINTER(ll), ctypes.POINTER(ll)]
    L.shim_tet_decode.argtypes = [ll, ll, ctypes.POINTER(ll), ctypes.POINTER(ll), ctypes.POINTER(ll)]
    return L


def test_closed_forms_match_the_oracle_walk(shim):
    for d in list(range(1, 13)) + [17, 31]:
        assert shim.shim_tri_rows(d) == oracle.packed_rows(oracle.KIND_TRI, d)
        assert shim.shim_tet_rows(d) == oracle.packed_rows(oracle.KIND_TET, d)
    for d in (1, 2, 5, 9):
        for i in range(d):
            for j in range(i, d):
                assert shim.shim_tri_encode(d, i, j) == oracle.locate(oracle.KIND_TRI, d, i, j)
                for k in range(j, d):
                    assert shim.shim_tet_encode(d, i, j, k) == oracle.locate(oracle.KIND_TET, d, i, j, k)


def test_decode_is_exact_for_every_position(shim):
    for d in range(1, 49):
        assert shim.shim_check_all_tri(d) == 0
        assert shim.shim_check_all_tet(d) == 0
    for d in (64, 100, 257):
        assert shim.shim_check_all_tet(d) == 0
    for d in (1000, 1024, 4097):
        assert shim.shim_check_all_tri(d) == 0


def test_four_simplex_positions_and_the_count_the_paper_gives(shim):
    # Section 2, "Intricate Structures": the degree-2 polynomial-regression covariance on 4 features has
    # 65 distinct elements = 10 (pairs) + 20 (triples) + 35 (4-tuples with repetition)
    assert shim.shim_tri_rows(4) + shim.shim_tet_rows(4) + shim.shim_simp4_rows(4) == 65
    assert shim.shim_simp4_rows(4) == 35
    for d in list(range(1, 20)) + [33, 64]:
        assert shim.shim_check_all_simp4(d) == 0


def test_decode_at_boundaries_of_large_extents(shim):
    ll = ctypes.c_longlong
    rng = np.random.default_rng(5)
    for d in (1 << 16, (1 << 20) - 3, 1 << 20, (1 << 31) - 1):
        rows = [0, 1, d // 2, d - 2, d - 1] + [int(x) for x in rng.integers(0, d, 20)]
        for i in rows:
            for j in (i, min(i + 1, d - 1), d - 1):
                p = shim.shim_tri_encode(d, i, j)
                a, b = ll(), ll()
                shim.shim_tri_decode(d, p, ctypes.byref(a), ctypes.byref(b))
                assert (a.value, b.value) == (i, j)
        assert shim.shim_tri_encode(d, d - 1, d - 1) == shim.shim_tri_rows(d) - 1
    for d in (1 << 10, 50000, 1 << 20):
        rows = [0, 1, d // 3, d - 2, d - 1] + [int(x) for x in rng.integers(0, d, 10)]
        for i in rows:
            for j in (i, (i + d) // 2, d - 1):
                for k in (j, d - 1):
                    q = shim.shim_tet_encode(d, i, j, k)
                    a, b, c = ll(), ll(), ll()
                    shim.shim_tet_decode(d, q, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c))
                    assert (a.value, b.value, c.value) == (i, j, k)
        assert shim.shim_tet_encode(d, d - 1, d - 1, d - 1) == shim.shim_tet_rows(d) - 1


# ---------------------------------------------------------------- the C ABI library itself

def _declared():
    text = open(os.path.join(ROOT, "include", "structtensor.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(st_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    import paper_2211_10482_b200 as st
    from paper_2211_10482_b200 import _build
    _build.build()
    L = ctypes.CDLL(st.LIB_PATH)
    names = _declared()
    assert len(names) >= 12
    for n in names:
        assert hasattr(L, n), n
    assert sorted(st.EXPORTS) == names
    assert st.lib().st_abi_version() == 1
    assert st.status_string(st.ST_ERR_WORKSPACE) == "workspace missing or too small"


def test_layout_sizes_and_host_side_validation():
    import paper_2211_10482_b200 as st
    L = st.lib()
    assert st.st_packed_elems(st.Layout(st.ST_TRI_UPPER, 64)) == 2080
    assert st.st_packed_elems(st.Layout(st.ST_TET, 64)) == 45760
    assert st.st_packed_elems(st.Layout(st.ST_TRI_UPPER, 512, inner=512)) == 67239936
    assert st.st_packed_elems(st.Layout(st.ST_BLOCKDIAG, 4096, inner=256, nblocks=64, bs=64)) == 67108864
    assert st.st_packed_elems(st.Layout(st.ST_BAND, 10, kl=2, ku=1)) == 40
    assert st.st_packed_elems(st.Layout(st.ST_BLOCKDIAG, 10, nblocks=3, bs=3)) == -1
    assert st.st_packed_elems(st.Layout(st.ST_TRI_UPPER, 0)) == -1
    assert st.st_packed_elems(st.Layout(7, 4)) == -1
    assert st.st_dense_elems(st.Layout(st.ST_TET, 5, inner=2)) == 250
    for kind, kw in ((st.ST_TRI_UPPER, {}), (st.ST_TET, {}), (st.ST_BAND, dict(kl=1, ku=2)),
                     (st.ST_BLOCKDIAG, dict(nblocks=2, bs=3))):
        lay = st.Layout(kind, 6, inner=3, **kw)
        okw = {("nb" if k == "nblocks" else k): v for k, v in kw.items()}
        assert st.st_packed_elems(lay) == 3 * oracle.packed_rows(kind, 6, **okw)
    # argument errors are reported before anything touches a device
    lay = st.Layout(st.ST_TRI_UPPER, 4).c()
    assert L.st_pack(ctypes.byref(lay), st.ST_F32, None, None, None) == st.ST_ERR_NULL
    assert L.st_pack(ctypes.byref(lay), st.ST_F32, 256, 8, None) == st.ST_ERR_ALIGN
    assert L.st_pack(ctypes.byref(lay), 9, 256, 512, None) == st.ST_ERR_DTYPE
    bad = st.Layout(st.ST_BLOCKDIAG, 7, nblocks=2, bs=3).c()
    assert L.st_unpack(ctypes.byref(bad), st.ST_F32, 256, 512, 0, None) == st.ST_ERR_SHAPE
    band = st.Layout(st.ST_BAND, 7, kl=1, ku=1).c()
    assert L.st_unpack(ctypes.byref(band), st.ST_F32, 256, 512, st.ST_FILL_SYMMETRIC, None) == st.ST_ERR_UNSUPPORTED
    assert L.st_sym_moment2(None, st.ST_F32, 4, 4, 4, 256, None, 0, 0, None) == st.ST_ERR_NULL
    assert L.st_sym_moment2(256, st.ST_F32, 4, 4, 3, 512, None, 0, 0, None) == st.ST_ERR_SHAPE
    assert L.st_sym_moment2(256, st.ST_F64, 4, 4, 4, 512, None, 0, 0, None) == st.ST_ERR_DTYPE
    assert L.st_sym_moment2(256, st.ST_F32, 4, 4, 4, 512, None, 0, 0, None) == st.ST_ERR_WORKSPACE
    assert L.st_sym_moment3(256, 4, 257, 257, 512, None, 0, 0, None) == st.ST_ERR_UNSUPPORTED
    assert L.st_sym_moment3(264, 4, 16, 16, 512, None, 0, 0, None) == st.ST_ERR_ALIGN
    assert L.st_sym_moment3(256, 4, 16, 16, 512, None, 0, 0, None) == st.ST_ERR_WORKSPACE
    assert L.st_sym_moment3(256, 4, 12, 18, 512, None, 0, 0, None) == st.ST_ERR_WORKSPACE     # any d, any pitch
    assert L.st_sym_moment3(256, 4, 72, 72, 512, None, 0, st.ST_FLAG_TC_TF32, None) == st.ST_ERR_UNSUPPORTED
    assert L.st_sym_moment3(256, 4, 13, 13, 512, None, 0, st.ST_FLAG_TC_BF16, None) == st.ST_ERR_WORKSPACE
    assert L.st_sym_moment4(256, 4, 129, 129, 512, None, 0, 0, None) == st.ST_ERR_UNSUPPORTED
    assert L.st_sym_moment4(256, 4, 8, 8, 512, None, 0, 0, None) == st.ST_ERR_WORKSPACE
    assert L.st_mttkrp_tri(256, 4, 8, 512, 768, 12, 1024, None, 0, 0, None) == st.ST_ERR_UNSUPPORTED
    assert L.st_mttkrp_tri(256, 4, 8, 512, 768, 0, 1024, None, 0, 0, None) == st.ST_ERR_SHAPE
    assert L.st_ttm_blockdiag(256, 2, 2, 8, 512, 24, 1024, None, 0, 0, None) == st.ST_ERR_UNSUPPORTED
    assert L.st_ttm_blockdiag(256, 2, 2, 8, 520, 32, 1024, None, 0, 0, None) == st.ST_ERR_ALIGN
    assert st.st_workspace_bytes(st.ST_OP_SYM_MOMENT3, 65536, 64) > 45760 * 4
    assert st.st_workspace_bytes(st.ST_OP_SYM_MOMENT3, 65536, 63) > 41664 * 4
    assert st.st_workspace_bytes(st.ST_OP_SYM_MOMENT3, 65536, 257) == 0
    # beyond 64 features the tile table of the call lives in the workspace too
    assert st.st_workspace_bytes(st.ST_OP_SYM_MOMENT3, 100, 128) > 128 * 129 * 130 // 6 * 4 + 6528 * 4
    assert st.st_workspace_bytes(st.ST_OP_SYM_MOMENT2, 4096, 64, st.ST_F32) >= 256
