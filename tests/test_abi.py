"""Host-side checks that need no GPU: the C-ABI library loads and exports what the header declares,
and the size queries and status strings behave."""
import ctypes
import os
import re

import pytest

from paper_2507_19906_b200 import binding as cd
from paper_2507_19906_b200 import build as cdbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    cdbuild.build()          # nvcc cross-compiles for sm_100a without a GPU
    return cd.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "calidrop.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(calidrop_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = declared_functions()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in calidrop.h but not exported"
    assert sorted(cd.EXPORTS) == names


def test_binding_has_the_same_names():
    for n in declared_functions():
        if n == "calidrop_status_string":
            assert hasattr(cd, "status_string")
        else:
            assert hasattr(cd, n), n


def test_size_queries_and_status_strings(lib):
    p = cd.make_params(B=4, Hq=32, Hkv=8, L=32768, window=64, pool=7, budget=2048, n_cal=64, cap=2176)
    ws = cd.calidrop_compress_workspace_bytes(p)
    assert ws >= 2 * 4 * 8 * (32768 - 64) * 4          # votes and pooled votes at least
    assert ws % 256 == 0
    assert cd.calidrop_decode_workspace_bytes(p, 2176) > 0
    off = cd.calidrop_decode_workspace_status_offset(p)
    assert off % 256 == 0 and off + 4 <= cd.calidrop_decode_workspace_bytes(p, 2176)
    lay = cd.calidrop_compress_workspace_layout(p)
    assert lay.vote_offset % 256 == 0 and lay.pooled_offset > lay.vote_offset
    bad = cd.make_params(B=4, Hq=32, Hkv=8, L=32768, window=64, pool=6, budget=2048, n_cal=64, cap=2176)
    assert cd.calidrop_compress_workspace_bytes(bad) == 0
    assert cd.status_string(cd.OK) == "ok"
    assert "workspace" in cd.status_string(cd.WORKSPACE_TOO_SMALL)
    assert cd.calidrop_version() >= 100
    assert ctypes.sizeof(cd.Params) == 14 * 4


def test_null_arguments_are_rejected_before_any_cuda_call(lib):
    """Validation is host-side and precedes every CUDA call, so it works without a device."""
    p = cd.make_params(B=1, Hq=4, Hkv=2, L=300, window=8, pool=5, budget=40, n_cal=1, cap=40)
    rc = lib.calidrop_compress(ctypes.byref(p), None, None, None, None, None, None, None, None, None, None,
                               None, 0, None)
    assert rc == cd.INVALID_ARG
    rc = lib.calidrop_decode(ctypes.byref(p), None, None, None, None, None, 1, None, None, None, None, None,
                             None, None, 0, None)
    assert rc == cd.INVALID_ARG
    rc = lib.calidrop_calibrate(ctypes.byref(p), None, None, None, None, None, None, None, None, None, None,
                                None, 0, None)
    assert rc == cd.INVALID_ARG
    rc = lib.calidrop_gather_evicted(ctypes.byref(p), None, None, None, None, None, None, None, 0, None)
    assert rc == cd.INVALID_ARG
    buf = (ctypes.c_char * 4096)()
    a = ctypes.addressof(buf)
    a = (a + 255) & ~255                                   # an aligned host address: never dereferenced
    ptr = ctypes.c_void_p(a)
    # slot outside [0, n_cal) and an empty evicted set are refused before any CUDA call
    assert lib.calidrop_recalibrate(ctypes.byref(p), ptr, ptr, ptr, 10, 1, ptr, ptr, ptr, ptr, 1 << 20, None) == cd.INVALID_ARG
    assert lib.calidrop_recalibrate(ctypes.byref(p), ptr, ptr, ptr, 0, 0, ptr, ptr, ptr, ptr, 1 << 20, None) == cd.INVALID_ARG
    assert lib.calidrop_recalibrate(ctypes.byref(p), None, ptr, ptr, 10, 0, ptr, ptr, ptr, ptr, 1 << 20, None) == cd.INVALID_ARG


def test_entry_points_of_the_other_eviction_rules_and_the_offload_validate_on_the_host(lib):
    """The kept-list, accumulated-score and offload entry points refuse bad arguments before any CUDA call."""
    p = cd.make_params(B=1, Hq=4, Hkv=2, L=300, window=8, pool=1, budget=40, n_cal=1, cap=40)
    buf = (ctypes.c_char * 8192)()
    ptr = ctypes.c_void_p((ctypes.addressof(buf) + 255) & ~255)     # an aligned host address: never dereferenced
    pp = ctypes.byref(p)
    # StreamingLLM's list: sinks must leave room for the window rows
    assert lib.calidrop_select_streaming(pp, 40, ptr, None) == cd.INVALID_ARG
    assert lib.calidrop_select_streaming(pp, -1, ptr, None) == cd.INVALID_ARG
    assert lib.calidrop_select_streaming(pp, 4, None, None) == cd.INVALID_ARG
    # H2O's list: window <= tail < budget
    assert lib.calidrop_select_from_scores(pp, ptr, 7, ptr, ptr, 1 << 30, None) == cd.INVALID_ARG
    assert lib.calidrop_select_from_scores(pp, ptr, 40, ptr, ptr, 1 << 30, None) == cd.INVALID_ARG
    assert lib.calidrop_select_from_scores(pp, None, 20, ptr, ptr, 1 << 30, None) == cd.INVALID_ARG
    assert lib.calidrop_select_from_scores(pp, ptr, 20, ptr, ptr, 16, None) == cd.WORKSPACE_TOO_SMALL
    # accumulated scores: workspace = 4 B Hq L bytes, rounded up to 256
    need = cd.calidrop_accumulated_scores_workspace_bytes(p)
    assert need >= 4 * 1 * 4 * 300 and need % 256 == 0
    assert lib.calidrop_accumulated_scores(pp, None, ptr, ptr, ptr, need, None) == cd.INVALID_ARG
    assert lib.calidrop_accumulated_scores(pp, ptr, ptr, ptr, ptr, need - 256, None) == cd.WORKSPACE_TOO_SMALL
    # calibration size below -1 is no setting
    bad = cd.make_params(B=1, Hq=4, Hkv=2, L=300, window=8, pool=1, budget=40, n_cal=1, cap=40, calib_size=-2)
    assert cd.calidrop_compress_workspace_bytes(bad) == 0
