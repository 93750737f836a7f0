"""The C-ABI library builds, loads without a GPU, exports what the header declares and
rejects bad arguments on the host (no device work happens in any of these calls)."""
import ctypes as C
import os
import re

import pytest

from paper_2504_00030_b200 import binding as sv
from paper_2504_00030_b200 import build as svbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    svbuild.build()
    return sv.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "specverify.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"^\s*(?:const\s+char\s*\*|sv_status|size_t|uint64_t)\s*\**\s*(\w+)\s*\(", text, flags=re.M)
    return sorted(set(names))


def test_header_and_binding_agree(lib):
    declared = declared_functions()
    assert len(declared) >= 11
    assert sorted(sv.EXPORTS) == declared
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in the header but not exported"


def test_status_strings(lib):
    assert sv.status_str(sv.SV_OK) == "ok"
    for code in (sv.SV_EINVAL, sv.SV_EUNSUPPORTED, sv.SV_EALIGN, sv.SV_ECUDA, sv.SV_EWORKSPACE):
        assert sv.status_str(code) not in ("ok", "unknown status")
    assert sv.status_str(-99) == "unknown status"


def test_workspace_queries_are_host_only(lib):
    assert sv.spec_accept_sample_workspace_bytes(128, 16, 128256) > 0
    assert sv.spec_accept_sample_workspace_bytes(0, 16, 128256) == 0
    assert sv.spec_verify_attn_workspace_bytes(128, 16, 64, 8, 128, 16384) > 0
    assert sv.spec_verify_attn_workspace_bytes(128, 16, 64, 8, 128, 0) == 0


def test_null_and_bad_arguments_are_rejected_before_any_launch(lib):
    assert lib.gamma_tune_update(None, None) == sv.SV_EINVAL
    assert lib.spec_accept_sample(None, None, 0, None) == sv.SV_EINVAL
    assert lib.spec_verify_attn(None, None, 0, None) == sv.SV_EINVAL
    assert lib.spec_verify_step_host(None, None, None, 0, None, None, 0, None, None) == sv.SV_EINVAL
    handle = C.c_void_p()
    st = (C.c_int64 * 4)(8 * 16 * 128, 16 * 128, 128, 1)
    assert lib.spec_kv_pool_register(None, None, 4, 16, 8, 128, st, C.byref(handle)) == sv.SV_EINVAL
    assert lib.spec_kv_pool_register(4096, 8192, 4, 32, 8, 128, st, C.byref(handle)) == sv.SV_EUNSUPPORTED
    assert lib.spec_kv_pool_register(4096 + 2, 8192, 4, 16, 8, 128, st, C.byref(handle)) == sv.SV_EALIGN
    g = sv.GammaParams()
    g.batch = 4
    assert lib.gamma_tune_update(C.byref(g), None) == sv.SV_EINVAL        # null state pointers
    a = sv.AcceptParams()
    a.batch, a.vocab, a.gamma_max = 4, 100, 80
    assert lib.spec_accept_sample(C.byref(a), None, 0, None) == sv.SV_EUNSUPPORTED


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(sv, "_lib", None)
    monkeypatch.setattr(sv, "LIB_PATH", "/nonexistent/libspecverify.so")
    with pytest.raises(RuntimeError, match="no fallback"):
        sv.load()
