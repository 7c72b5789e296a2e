"""tk_fwd_noalloc: the forward pass for callers that cannot allocate device memory
(plugins under a foreign allocator, real-time loops, fully committed pools).

For long rows it runs on a scratch array compiled into the library.  The check
is that it returns what tk_fwd_ex returns with a caller-supplied workspace and
what the CPU oracle computes -- on calls in a row with different shapes, so
that whatever one call left in the shared scratch is shown not to matter.
This file sorts last so that a run stopping at the first failure has already
been through every other test."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2302_01425_b200 import binding as tk, build, workloads as wl

P43 = 4.0 / 3.0


@pytest.fixture(scope="module", autouse=True)
def built():
    build.build()
    tk.load()


def reference_output(th, rows, n, k, p, lam, mode):
    out = torch.empty_like(th)
    need = tk.tk_workspace_bytes(rows, n, k, p, mode)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda") if need else None
    tk.tk_fwd_ex(th, rows, n, k, p, lam, mode, out, workspace=ws)
    torch.cuda.synchronize()
    return out


@pytest.mark.gpu
def test_two_calls_in_a_row_match_the_workspace_entry_point():
    calls = [
        (3, 50000, 5000, P43, 0.5, tk.TK_TOPKMAG, 91),
        (5, 20011, 77, 2.0, 1.0, tk.TK_MASK, 92),      # other shape: reuses the scratch as it was left
        (2, 1000, 5, P43, 0.5, tk.TK_TOPK, 93),        # short rows: handed to tk_fwd
        (12, 30000, 3000, 2.0, 1.0, tk.TK_MASK, 94),   # needs no scratch although rows * n is above its limit
        (2, 131072, 1000, 2.0, 0.05, tk.TK_TOPKMAG, 95),  # the largest problem the scratch holds
    ]
    from oracle import tko
    for rows, n, k, p, lam, mode, seed in calls:
        x = wl.normal_rows(rows, n, seed)
        th = torch.from_numpy(x).cuda()
        ref = reference_output(th, rows, n, k, p, lam, mode)
        out = torch.full_like(th, float("nan"))
        tk.tk_fwd_noalloc(th, rows, n, k, p, lam, mode, out)
        torch.cuda.synchronize()
        a, b = out.cpu().numpy().astype(np.float64), ref.cpu().numpy().astype(np.float64)
        assert np.isfinite(a).all()
        assert np.max(np.abs(a - b) / np.maximum(1.0, np.abs(b))) <= 1e-5
        want = tko.fwd(x, k, p, lam, mode)
        assert np.max(np.abs(a - want) / np.maximum(1.0, np.abs(want))) <= 1e-5, (rows, n)


def test_sizes_beyond_the_built_in_scratch_are_refused():
    lib = tk.load()
    fake = ctypes.c_void_p(256)      # never dereferenced: the size check comes first
    too_many = tk.TK_NOALLOC_MAX_ELEMENTS + 1
    assert lib.tk_fwd_noalloc(fake, 1, too_many, 10, 2.0, 1.0, 0, fake, None) == tk.TK_ERR_WORKSPACE
    assert lib.tk_fwd_noalloc(fake, 8, 40000, 10, 2.0, 1.0, 0, fake, None) == tk.TK_ERR_WORKSPACE
    assert lib.tk_fwd_noalloc(fake, 1, 40000, 0, 2.0, 1.0, 0, fake, None) == tk.TK_ERR_INVALID_ARG
    assert lib.tk_fwd_noalloc(fake, 0, 40000, 5, 2.0, 1.0, 0, fake, None) == tk.TK_OK
    assert lib.tk_fwd_noalloc(fake, 1, 40000, 5, 1.5, 1.0, 0, fake, None) == tk.TK_ERR_UNSUPPORTED
