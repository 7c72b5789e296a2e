"""The range-checked build of the library (libtk_bounds.so, -DTK_DEBUG_BOUNDS): the kernels of the
default path test every index they form and report a violation in the status word instead of
touching memory.  No memory checker can be run on the GPUs these tests use, so this build is the
stand-in: a seeded sweep over row lengths around every layout boundary must leave TK_FLAG_BOUNDS
clear, and the checked kernels must return exactly what the regular ones return."""
import numpy as np
import pytest
import torch

from paper_2302_01425_b200 import binding as tk, build, workloads as wl

P43 = 4.0 / 3.0
pytestmark = pytest.mark.gpu


@pytest.fixture()
def bounds_library():
    regular = build.build()
    checked = build.build(bounds=True)
    tk.use_library(checked)
    tk.load()
    try:
        yield regular
    finally:
        tk.use_library(regular)
        tk.load()


def run_default_path(x, g, k, p, lam, mode, workspace=None):
    rows, n = x.shape
    th, gt = torch.from_numpy(x).cuda(), torch.from_numpy(g).cuda()
    out, grad = torch.full_like(th, float("nan")), torch.full_like(th, float("nan"))
    st = tk.new_state(rows)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tk.tk_fwd_ex(th, rows, n, k, p, lam, mode, out, state_out=st, status_out=status, workspace=workspace)
    tk.tk_vjp(th, gt, rows, n, k, p, lam, mode, grad, state=st, status_out=status, workspace=workspace)
    torch.cuda.synchronize()
    return out.cpu().numpy(), grad.cpu().numpy(), st.cpu().numpy().copy(), int(status.item())


def cases():
    rng = np.random.Generator(np.random.PCG64(77))
    lengths = [17, 31, 32, 33, 63, 64, 65, 100, 127, 128, 129, 255, 256, 257, 500, 512, 513, 1000, 1024, 1025,
               2047, 2048, 2049, 4096, 5000, 8192, 8193, 16384, 16385, 20000, 32768]
    for it in range(60):
        n = int(rng.choice(lengths))
        k = int(rng.integers(1, n + 1)) if rng.random() < 0.5 else int(rng.choice([1, 2, max(1, n // 8)]))
        lam = float(rng.choice([0.05, 0.3, 1.0, 10.0]))
        p = float(rng.choice([2.0, P43]))
        mode = int(rng.integers(0, 3))
        rows = int(rng.choice([1, 3, 7])) if n > 2048 else int(rng.choice([1, 5, 37, 130, 1000]))
        yield it, rows, n, k, p, lam, mode


def test_seeded_sweep_leaves_the_bounds_flag_clear(bounds_library):
    got = {}
    for it, rows, n, k, p, lam, mode in cases():
        x = wl.normal_rows(rows, n, 4000 + it)
        g = wl.cotangent_like(x, 4000 + it)
        out, grad, st, status = run_default_path(x, g, k, p, lam, mode)
        assert status & tk.TK_FLAG_BOUNDS == 0, f"it={it} rows={rows} n={n} k={k} p={p} mode={mode}"
        assert np.isfinite(out).all() and np.isfinite(grad).all()
        got[it] = (out, grad, st)
    # the same calls through the regular build: bit-identical results
    tk.use_library(bounds_library)
    tk.load()
    for it, rows, n, k, p, lam, mode in cases():
        x = wl.normal_rows(rows, n, 4000 + it)
        g = wl.cotangent_like(x, 4000 + it)
        out, grad, st, status = run_default_path(x, g, k, p, lam, mode)
        assert np.array_equal(out, got[it][0]) and np.array_equal(grad, got[it][1]), f"it={it} n={n}"
        assert np.array_equal(st, got[it][2])


def test_long_row_and_general_w_leave_the_bounds_flag_clear(bounds_library):
    # a few very long rows: the cooperative kernel
    rows, n, k = 2, 300001, 30000
    x = wl.normal_rows(rows, n, 51, 0.02)
    need = tk.tk_workspace_bytes(rows, n, k, 2.0, tk.TK_TOPKMAG)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    th = torch.from_numpy(x).cuda()
    out = torch.full_like(th, float("nan"))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tk.tk_fwd_ex(th, rows, n, k, 2.0, 1e-3, tk.TK_TOPKMAG, out, workspace=ws, status_out=status)
    torch.cuda.synchronize()
    assert int(status.item()) & tk.TK_FLAG_BOUNDS == 0
    assert torch.isfinite(out).all()
    # any sorted w: parallel pool-adjacent-violators, rows of every padded size
    for n in (5, 33, 64, 100, 1000, 2048):
        rows = 9
        x = wl.normal_rows(rows, n, 60 + n)
        w = (np.arange(n, 0, -1, dtype=np.float32) / n)
        th, wt = torch.from_numpy(x).cuda(), torch.from_numpy(w).cuda()
        gt = torch.from_numpy(wl.cotangent_like(x, 61)).cuda()
        out, grad = torch.full_like(th, float("nan")), torch.full_like(th, float("nan"))
        status.zero_()
        for p in (2.0, P43):
            tk.tk_fwd_w(th, wt, rows, n, p, 0.7, out, status_out=status)
            tk.tk_vjp_w(th, wt, gt, rows, n, p, 0.7, grad, status_out=status)
            torch.cuda.synchronize()
            assert int(status.item()) & tk.TK_FLAG_BOUNDS == 0, (n, p)
            assert torch.isfinite(out).all() and torch.isfinite(grad).all()
