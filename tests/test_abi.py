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
    assert fwd(4, 8, 2, 1.01, 1.0, 0) == b.TK_ERR_UNSUPPORTED       # q = 101 > 64
    assert lib.tk_vjp(fake, fake, 4, 8, 2, 1.8, 1.0, 0, fake, None, None) == b.TK_ERR_UNSUPPORTED   # 2 < q < 3: forward pass only
    assert lib.tk_jvp(fake, fake, 4, 8, 2, 1.8, 1.0, 0, fake, None, None) in (b.TK_ERR_UNSUPPORTED, b.TK_ERR_INVALID_ARG)
    assert fwd(1, 20000, 2, 1.5, 1.0, 0) == b.TK_ERR_UNSUPPORTED    # q = 3 on a row held in global memory
    assert lib.tk_vjp(fake, fake, 4, 200, 2, 1.5, 1.0, 0, fake, None, None) == b.TK_ERR_WORKSPACE  # q = 3, n > 128, no saved state: the forward pass is run again and needs room for its row state
    assert lib.tk_workspace_bytes(4, 200, 2, 1.5, 0, 0) == 256 and lib.tk_workspace_bytes(4, 200, 2, 2.0, 0, 0) == 0
    assert lib.tk_workspace_bytes(40, 100, 2, 1.5, 2, 0) == 768 and lib.tk_workspace_bytes(40, 100, 2, 1.5, 0, 0) == 0
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
    o = b.TkOpts()
    o.solver, o.tol = b.TK_SOLVER_DYKSTRA, -1.0
    assert lib.tk_fwd_ex(fake, 4, 8, 2, 2.0, 1.0, 0, fake, ctypes.byref(o), None) == b.TK_ERR_INVALID_ARG
    o.tol = float("nan")
    assert lib.tk_fwd_ex(fake, 4, 8, 2, 2.0, 1.0, 0, fake, ctypes.byref(o), None) == b.TK_ERR_INVALID_ARG
    o.tol = 1e-6                                                     # run to tolerance: rows of one thread block only
    assert lib.tk_fwd_ex(fake, 4, 20000, 2, 2.0, 1.0, 0, fake, ctypes.byref(o), None) == b.TK_ERR_UNSUPPORTED


def test_opts_layout_matches_header():
    from paper_2302_01425_b200 import binding as b
    text = open(os.path.join(ROOT, "include", "tk.h")).read()
    body = re.search(r"typedef struct \{([^}]*)\} tk_opts;", text).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    names = [f.strip().split()[-1].lstrip("*") for f in body.split(";") if f.strip()]
    assert names == [f[0] for f in b.TkOpts._fields_]


def test_general_w_arguments_are_rejected_on_the_host(lib):
    from paper_2302_01425_b200 import binding as b
    fake = ctypes.c_void_p(256)
    fw = lambda rows, n, w_rows, p, lam, theta=fake, w=fake, out=fake: lib.tk_fwd_w(
        theta, w, rows, n, w_rows, p, lam, out, None, None)
    assert fw(4, 0, 1, 2.0, 1.0) == b.TK_ERR_INVALID_ARG
    assert fw(-1, 8, 1, 2.0, 1.0) == b.TK_ERR_INVALID_ARG
    assert fw(4, 8, 3, 2.0, 1.0) == b.TK_ERR_INVALID_ARG            # w_rows is 1 or rows
    assert fw(4, 8, 1, 2.0, 0.0) == b.TK_ERR_INVALID_ARG
    assert fw(4, 8, 1, 2.0, 1.0, w=None) == b.TK_ERR_INVALID_ARG
    assert fw(4, 8, 1, 2.0, 1.0, out=None) == b.TK_ERR_INVALID_ARG
    assert fw(4, 8, 1, 1.5, 1.0) == b.TK_ERR_UNSUPPORTED            # p = 2 and p = 4/3 only
    assert fw(4, 4096, 1, 2.0, 1.0) == b.TK_ERR_UNSUPPORTED         # rows of up to 2048 elements
    assert fw(0, 8, 1, 2.0, 1.0) == b.TK_OK
    assert lib.tk_vjp_w(fake, fake, None, 4, 8, 1, 2.0, 1.0, fake, None, None, None) == b.TK_ERR_INVALID_ARG
    assert lib.tk_vjp_w(fake, fake, fake, 0, 8, 1, 2.0, 1.0, fake, fake, None, None) == b.TK_OK


class FakeDeviceTensor:
    """Stands in for a CUDA tensor in the binding's checks (which run before any call into the library)."""

    def __init__(self, numel, dtype, contiguous=True, cuda=True):
        import torch
        self._numel, self.dtype, self._c, self.is_cuda = numel, getattr(torch, dtype), contiguous, cuda

    def numel(self):
        return self._numel

    def is_contiguous(self):
        return self._c

    def data_ptr(self):
        return 256


def test_binding_refuses_buffers_shorter_than_the_call_needs(lib, monkeypatch):
    from paper_2302_01425_b200 import binding as b

    class Unreachable:
        def __getattr__(self, name):
            def call(*args):
                raise AssertionError(f"{name}: the library must not be called with a short buffer")
            return call

    monkeypatch.setattr(b, "load", lambda: Unreachable())
    monkeypatch.setattr(b, "_stream", lambda: None)
    T = FakeDeviceTensor
    ok = lambda m: T(m, "float32")
    with pytest.raises(ValueError, match="theta: 31 elements, the call needs 32"):
        b.tk_fwd(ok(31), 4, 8, 2, 2.0, 1.0, 0, ok(32))
    with pytest.raises(ValueError, match="out: 16 elements"):
        b.tk_fwd_noalloc(T(10 ** 6, "float32"), 2, 40000, 2, 2.0, 1.0, 0, ok(16))
    with pytest.raises(ValueError, match="perm_out"):
        b.tk_fwd_ex(ok(32), 4, 8, 2, 2.0, 1.0, 0, ok(32), perm_out=T(8, "int32"))
    with pytest.raises(ValueError, match="state"):
        b.tk_fwd_ex(ok(32), 4, 8, 2, 2.0, 1.0, 0, ok(32), state_out=T(63, "uint8"))
    with pytest.raises(ValueError, match="status_out"):
        b.tk_fwd_ex(ok(32), 4, 8, 2, 2.0, 1.0, 0, ok(32), status_out=T(0, "int32"))
    with pytest.raises(ValueError, match="grad_out"):
        b.tk_vjp(ok(32), ok(8), 4, 8, 2, 2.0, 1.0, 0, ok(32))
    with pytest.raises(ValueError, match="grad_theta"):
        b.tk_vjp(ok(32), ok(32), 4, 8, 2, 2.0, 1.0, 0, ok(31))
    with pytest.raises(ValueError, match="out_tangent"):
        b.tk_jvp(ok(32), ok(32), 4, 8, 2, 2.0, 1.0, 0, ok(3), state=T(64, "uint8"))
    with pytest.raises(ValueError, match="target"):
        b.tk_topk_loss(ok(32), T(3, "int32"), 4, 8, 2, 2.0, 1.0, ok(4), ok(32))
    with pytest.raises(ValueError, match="loss"):
        b.tk_topk_loss(ok(32), T(4, "int32"), 4, 8, 2, 2.0, 1.0, ok(3), ok(32))
    with pytest.raises(ValueError, match="theta"):       # [n, cols] with a leading dimension: (n - 1) * ld + cols
        b.tk_fwd_cols(ok(7 * 10 + 6 - 1), 8, 6, 10, 2, 2.0, 1.0, 0, ok(100), workspace=T(1 << 20, "uint8"))
    with pytest.raises(ValueError, match="sorted_out"):
        b.tk_argsort(ok(32), 4, 8, 0, T(32, "int32"), ok(31))
    with pytest.raises(ValueError, match="w: 8 elements, the call needs 32"):
        b.tk_fwd_w(ok(32), ok(8), 1, 32, 2.0, 1.0, ok(32))
    with pytest.raises(ValueError, match="grad_theta"):
        b.tk_vjp_w(ok(32), ok(8), ok(32), 4, 8, 2.0, 1.0, ok(31))
    with pytest.raises(ValueError, match="grad_w"):
        b.tk_vjp_w(ok(32), ok(8), ok(32), 4, 8, 2.0, 1.0, ok(32), grad_w=ok(31))
    # wrong dtype, host memory and strided views are refused too
    with pytest.raises(ValueError, match="contiguous CUDA tensor"):
        b.tk_fwd(T(32, "float64"), 4, 8, 2, 2.0, 1.0, 0, ok(32))
    with pytest.raises(ValueError, match="contiguous CUDA tensor"):
        b.tk_fwd(T(32, "float32", cuda=False), 4, 8, 2, 2.0, 1.0, 0, ok(32))
    with pytest.raises(ValueError, match="contiguous CUDA tensor"):
        b.tk_fwd(T(32, "float32", contiguous=False), 4, 8, 2, 2.0, 1.0, 0, ok(32))


def test_product_path_does_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_2302_01425_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"import\s+oracle|from\s+oracle|oracle[/.]|libtko|tko_", text), f
