"""The C-ABI library loads without a GPU and exports every function include/cosa.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2607_25291_b200 import build
    return ctypes.CDLL(build.build())


def declared_functions():
    text = open(os.path.join(ROOT, "include", "cosa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cosa_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert "cosa_kap_select" in names and "cosa_osk_attention" in names and len(names) >= 12
    for name in names:
        assert hasattr(lib, name), name


def test_binding_covers_the_header():
    from paper_2607_25291_b200 import binding
    assert sorted(binding.EXPORTS) == declared_functions()


def test_host_only_entry_points(lib):
    from paper_2607_25291_b200 import binding
    from oracle.cosa_oracle import budget_count
    for b in (0.04, 0.08, 0.1, 0.2, 0.25, 0.5, 1.0):
        for J in (1, 2, 7, 103, 512, 1024):
            assert binding.cosa_budget_count(b, J) == budget_count(b, J)
    assert binding.cosa_version() >= 100
    assert binding.library().cosa_status_string(-6).decode().startswith("order list")


def test_argument_checks_need_no_gpu(lib):
    from paper_2607_25291_b200 import binding as B
    L = B.library()
    shape = B.CosaShape(1, 4, 1, 4096, 128, 128, 128, 1)
    one = ctypes.c_void_p(256)            # never dereferenced: the checks fail first
    assert L.cosa_kap_select(None, one, ctypes.byref(shape), 0.5, one, one, None) == B.COSA_ERR_INVALID_ARG
    assert L.cosa_kap_select(one, one, ctypes.byref(shape), 0.0, one, one, None) == B.COSA_ERR_INVALID_ARG
    assert L.cosa_kap_select(one, one, ctypes.byref(shape), 1.5, one, one, None) == B.COSA_ERR_INVALID_ARG
    bad = B.CosaShape(1, 4, 1, 4096, 64, 128, 128, 1)
    assert L.cosa_kap_select(one, one, ctypes.byref(bad), 0.5, one, one, None) == B.COSA_ERR_UNSUPPORTED
    bad = B.CosaShape(1, 4, 1, 4100, 128, 128, 128, 1)
    assert L.cosa_osk_attention(one, one, one, ctypes.byref(bad), one, one, 0.5, one, None, None, None) == B.COSA_ERR_UNSUPPORTED
    bad = B.CosaShape(1, 4, 3, 4096, 128, 128, 128, 1)
    assert L.cosa_osk_attention(one, one, one, ctypes.byref(bad), one, one, 0.5, one, None, None, None) == B.COSA_ERR_INVALID_ARG
    opt = B.default_options(skip_scale=4096.0)     # Delta >= N would skip the first block
    assert L.cosa_osk_attention_ex(one, one, one, ctypes.byref(shape), one, one, 0.5, one, None, None, None,
                                   ctypes.byref(opt)) == B.COSA_ERR_INVALID_ARG
    opt = B.default_options(stride=3)
    assert L.cosa_kap_select_ex(one, one, ctypes.byref(shape), 0.5, one, one, None, ctypes.byref(opt)) == B.COSA_ERR_UNSUPPORTED
    assert B.cosa_host_call_workspace_bytes(shape) > 4 * 4096 * 128 * 2
