"""Host-side checks of the C ABI that need no GPU: the library loads, exports
every symbol include/tk.h declares, and rejects bad arguments before any
launch."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2302_01425_b200 import build, binding
    build.build()
    return binding.load()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "tk.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tk_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_boundary():
    names = declared_symbols()
    for must in ("tk_fwd", "tk_fwd_ex", "tk_vjp", "tk_argsort", "tk_workspace_bytes",
                 "tk_status_string", "tk_version"):
        assert must in names


def test_library_exports_every_declared_symbol(lib):
    for name in declared_symbols():
        assert hasattr(lib, name), name


def test_binding_lists_the_same_symbols():
    from paper_2302_01425_b200 import binding
    assert sorted(binding.EXPORTS) == declared_symbols()


def test_rowstate_layout_matches_header():
    from paper_2302_01425_b200 import binding
    text = open(os.path.join(ROOT, "include", "tk.h")).read()
    body = re.search(r"typedef struct \{([^}]*)\} tk_rowstate;", text).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = [f.strip() for f in body.split(";") if f.strip()]
    assert fields == ["float pivot", "float offset", "int32_t a", "int32_t b"]
    assert binding.ROWSTATE_BYTES == 16


def test_version_and_status_strings(lib):
    assert b"sm_100a" in lib.tk_version()
    seen = {lib.tk_status_string(i) for i in range(6)}
    assert len(seen) == 6 and lib.tk_status_string(99) == b"unknown status"


def test_bad_arguments_are_rejected_on_the_host(lib):
    from paper_2302_01425_b200 import binding as b
    fake = ctypes.c_void_p(256)   # never dereferenced: every call below fails validation first
    P43 = 4.0 / 3.0
    fwd = lambda rows, n, k, p, lam, mode, theta=fake, out=fake: lib.tk_fwd(
        theta, rows, n, k, p, lam, mode, out, None)
    assert fwd(4, 8, 0, 2.0, 1.0, 0) == b.TK_ERR_INVALID_ARG        # k = 0
    assert fwd(4, 8, 9, 2.0, 1.0, 0) == b.TK_ERR_INVALID_ARG        # k > n
    assert fwd(4, 0, 1, 2.0, 1.0, 0) == b.TK_ERR_INVALID_ARG        # n = 0
    assert fwd(-1, 8, 2, 2.0, 1.0, 0) == b.TK_ERR_INVALID_ARG       # rows < 0
    assert fwd(4, 8, 2, 1.0, 1.0, 0) == b.TK_ERR_INVALID_ARG        # p <= 1
    assert fwd(4, 8, 2, 2.0, 0.0, 0) == b.TK_ERR_INVALID_ARG        # lambda <= 0
    assert fwd(4, 8, 2, 2.0, float("nan"), 0) == b.TK_ERR_INVALID_ARG
    assert fwd(4, 8, 2, 2.0, 1.0, 3) == b.TK_ERR_INVALID_ARG        # mode
    assert fwd(4, 8, 2, 3.0, 1.0, 0) == b.TK_ERR_UNSUPPORTED        # q = 1.5 < 2
    assert fwd(4, 8, 2, 1.8, 1.0, 0) == b.TK_ERR_UNSUPPORTED        # 2 < q < 3
    assert fwd(4, 8, 2, 1.5, 1.0, 2) == b.TK_ERR_UNSUPPORTED        # q = 3 with the magnitude mode
    assert fwd(1, 20000, 2, 1.5, 1.0, 0) == b.TK_ERR_UNSUPPORTED    # q = 3 on a row held in global memory
    assert lib.tk_vjp(fake, fake, 4, 200, 2, 1.5, 1.0, 0, fake, None, None) == b.TK_ERR_UNSUPPORTED  # q = 3, n > 128, no saved state
    assert fwd(4, 8, 2, 2.0, 1.0, 0, theta=None) == b.TK_ERR_INVALID_ARG
    assert fwd(4, 8, 2, P43, 1.0, 0, out=None) == b.TK_ERR_INVALID_ARG
    assert fwd(0, 8, 2, 2.0, 1.0, 0) == b.TK_OK                     # rows = 0: nothing to do
    assert lib.tk_vjp(fake, None, 4, 8, 2, 2.0, 1.0, 0, fake, None, None) == b.TK_ERR_INVALID_ARG
    assert lib.tk_vjp(fake, fake, 0, 8, 2, 2.0, 1.0, 0, fake, None, None) == b.TK_OK
    assert lib.tk_argsort(fake, 4, 8, 0, None, None, None, None) == b.TK_ERR_INVALID_ARG
    assert lib.tk_argsort(fake, 0, 8, 0, fake, None, None, None) == b.TK_OK
    o = b.TkOpts()
    o.solver = 7
    assert lib.tk_fwd_ex(fake, 4, 8, 2, 2.0, 1.0, 0, fake, ctypes.byref(o), None) == b.TK_ERR_INVALID_ARG


def test_product_path_does_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_2302_01425_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"import\s+oracle|from\s+oracle|oracle[/.]|libtko|tko_", text), f
