"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, its workspace query has no N^2 term, and argument errors are caught before
any CUDA call."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def fd():
    import __graft_entry__ as g
    g.build()
    import paper_2609_38198_b200 as fd
    return fd


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "fd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fd_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(fd):
    names = _declared_functions()
    assert len(names) >= 15
    lib = ctypes.CDLL(fd.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in fd.h but not exported"
    assert sorted(fd.EXPORTS) == names


def test_workspace_has_no_quadratic_term(fd):
    w1 = fd.fd_workspace_bytes(1 << 16, 12, 64, 384)
    w2 = fd.fd_workspace_bytes(1 << 20, 12, 64, 384)
    assert 0 < w1 < w2
    assert w2 < 16.5 * w1                      # linear in N (16x), nowhere near 256x
    assert w2 < 8 * (1 << 30)                  # a few GB at N = 2^20, vs 4 TiB for a dense fp32 K
    assert fd.fd_workspace_bytes(0, 12, 64, 0) == 0
    assert fd.fd_workspace_bytes(100, 12, 0, 0) == 0
    assert fd.fd_workspace_bytes(100, 12, 257, 0) == 0


def test_argument_errors_before_any_launch(fd):
    h = ctypes.c_void_p()
    st = fd.lib.fd_create(ctypes.byref(h), None, 10, 2, 2, 1, 8, 0, None, 0, None)
    assert st == fd.FD_ERR_INVALID and not h.value
    assert fd.lib.fd_create(None, None, 10, 2, 2, 1, 8, 0, None, 0, None) == fd.FD_ERR_INVALID
    assert fd.lib.fd_beta0(None, None) == fd.FD_ERR_INVALID
    assert fd.lib.fd_apply(None, None, 0, 1, None, 0, 0) == fd.FD_ERR_INVALID
    assert fd.lib.fd_degree(None, 1.0, 1.0, 0, None, None, None, None, None) == fd.FD_ERR_INVALID
    assert fd.lib.fd_status_string(0) == b"ok"
    assert b"workspace" in fd.lib.fd_status_string(2)
    assert fd.fd_version() >= 100
    assert fd.fd_launch_count() == 0           # nothing ran on this CPU-only path
