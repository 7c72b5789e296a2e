"""Element-by-element comparison of the CUDA library with the CPU oracle.

Tolerances (written here once, used by every GPU test):
  * permutations: bit-exact;
  * forward values: |gpu - ref| <= 1e-5 * max(1, |ref|);
  * VJP: |gpu - ref| <= 1e-5 * max(1, |ref|) on rows where the fp32 path and
    the fp64 oracle found the same pooled block.  The VJP is discontinuous
    where an element enters or leaves the pooled block, so a row where the two
    disagree is accepted only when every disputed rank sits within
    1e-5 * max(1, |s_j|) of the block's edge in the oracle; such rows are
    counted, reported and left out of the VJP maximum.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import tko
from paper_2302_01425_b200 import binding as tk

TOL = 1e-5


def rel_err(gpu: np.ndarray, ref: np.ndarray) -> np.ndarray:
    return np.abs(gpu.astype(np.float64) - ref) / np.maximum(1.0, np.abs(ref))


def oracle_blocks(det, k):
    """[rows, 2] pooled block [a, b) per row from the oracle's partition (a = b = k if none)."""
    lo = det["block_lo"][:, k - 1].astype(np.int64)
    hi = det["block_hi"][:, k - 1].astype(np.int64)
    none = (hi - lo) <= 1
    lo = np.where(none, k, lo)
    hi = np.where(none, k, hi)
    return np.stack([lo, hi], axis=1)


def read_state(state: torch.Tensor, rows: int):
    raw = state.cpu().numpy().view(np.dtype([("pivot", "<f4"), ("offset", "<f4"), ("a", "<i4"), ("b", "<i4")]))
    return raw[:rows]


def disputed_rows_ok(theta, k, p, lam, mode, det, gpu_ab, ref_ab):
    """Rows whose block bounds differ; each must be a near-tie at the block edge in the oracle."""
    bad_rows = np.nonzero((gpu_ab != ref_ab).any(axis=1))[0]
    q = p / (p - 1.0)
    mag = mode == tko.TOPKMAG
    _, s_all = tko.argsort(theta[bad_rows], mode) if len(bad_rows) else (None, None)
    for n_i, r in enumerate(bad_rows):
        s = s_all[n_i]
        v = det["v"][r]
        ga, gb = gpu_ab[r]
        ra, rb = ref_ab[r]
        ranks = set(range(min(ga, ra), max(ga, ra))) | set(range(min(gb, rb), max(gb, rb)))
        # gamma the oracle would pool at: the value of the pooled block, or of rank k-1 / k
        for j in ranks:
            if rb > ra:
                gamma = v[ra]
            else:
                gamma = v[min(j, len(v) - 1)]
            width = lam * (gamma ** (1.0 / (q - 1.0)) if mag else 1.0)
            margin = min(abs(s[j] - gamma), abs(s[j] - (gamma + width)))
            # also accept a near-violation between rank k-1 and k when one side sees no block
            if rb == ra or gb == ga:
                top = det["v"][r][k - 1]
                margin = min(margin, abs(top - s[k]) if k < len(s) else margin)
            assert margin <= TOL * max(1.0, abs(s[j])), (
                f"row {r}: block gpu [{ga},{gb}) vs oracle [{ra},{rb}), rank {j} margin {margin}")
    return bad_rows


def run_case(theta: np.ndarray, k: int, p: float, lam: float, mode: int, g: np.ndarray | None = None,
             check_perm: bool = True, label: str = "", solver: int = 0):
    """Runs forward (+ argsort, + both VJP paths) on the GPU and compares with the oracle.
    Returns a dict of measured errors."""
    theta = np.ascontiguousarray(theta, np.float32)
    rows, n = theta.shape
    dev = torch.device("cuda")
    th = torch.from_numpy(theta).to(dev)
    out = torch.full((rows, n), float("nan"), device=dev)
    perm = torch.full((rows, n), -1, dtype=torch.int32, device=dev)
    state = tk.new_state(rows)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    ws_bytes = tk.tk_workspace_bytes(rows, n, k, p, mode)
    ws = torch.empty(max(ws_bytes, 1), dtype=torch.uint8, device=dev) if ws_bytes else None
    q = p / (p - 1.0)
    general = min(abs(q - 2.0), abs(q - 4.0)) > 1e-6  # no closed-form block solve: no permutation output either
    sorts = solver != tk.TK_SOLVER_THRESHOLD and not general   # the sort-free solver has no permutation to give
    tk.tk_fwd_ex(th, rows, n, k, p, lam, mode, out, perm_out=perm if sorts else None, state_out=state,
                 workspace=ws, status_out=status, solver=solver)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, f"{label}: status {int(status.item())}"
    ref, det = tko.fwd(theta, k, p, lam, mode, details=True)
    res = {}
    if check_perm and sorts:
        assert np.array_equal(perm.cpu().numpy(), det["perm"]), f"{label}: permutation differs"
    gout = out.cpu().numpy()
    assert np.isfinite(gout).all(), f"{label}: non-finite output"
    res["fwd_max_rel"] = float(rel_err(gout, ref).max())
    res["fwd_max_abs"] = float(np.abs(gout - ref).max())
    assert res["fwd_max_rel"] <= TOL, f"{label}: forward error {res}"
    bad_noperm = np.zeros(0, np.int64)
    # the call without a permutation output takes its own path for short rows (keys sorted alone,
    # results placed by value): same tolerance against the oracle, same pooled blocks
    if sorts:
        out2 = torch.full_like(out, float("nan"))
        state2 = tk.new_state(rows)
        tk.tk_fwd_ex(th, rows, n, k, p, lam, mode, out2, state_out=state2, status_out=status, workspace=ws)
        out3 = out2
        if ws_bytes == 0 or n <= 32768:       # no scratch needed: the plain entry point must agree
            out3 = torch.full_like(out, float("nan"))
            tk.tk_fwd(th, rows, n, k, p, lam, mode, out3)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        g2 = out2.cpu().numpy()
        assert np.isfinite(g2).all(), f"{label}: non-finite output (no permutation)"
        res["fwd_noperm_max_rel"] = float(rel_err(g2, ref).max())
        assert res["fwd_noperm_max_rel"] <= TOL, f"{label}: forward error without permutation {res}"
        assert torch.equal(out2, out3), f"{label}: tk_fwd differs from tk_fwd_ex"
        st2 = read_state(state2, rows)
        ab2 = np.stack([st2["a"], st2["b"]], axis=1).astype(np.int64)
        bad_noperm = disputed_rows_ok(theta, k, p, lam, mode, det, ab2, oracle_blocks(det, k))
        res["rows_block_disputed_noperm"] = int(len(bad_noperm))
    st = read_state(state, rows)
    gpu_ab = np.stack([st["a"], st["b"]], axis=1).astype(np.int64)
    ref_ab = oracle_blocks(det, k)
    bad = disputed_rows_ok(theta, k, p, lam, mode, det, gpu_ab, ref_ab)
    res["rows_block_disputed"] = int(len(bad))
    if g is not None:
        g = np.ascontiguousarray(g, np.float32)
        gt = torch.from_numpy(g).to(dev)
        gref = tko.vjp(theta, g, k, p, lam, mode)
        # Magnitude mode, exact zeros tied across rank k (the k-th largest |theta| is 0): the output
        # is 0 for all of them, but which of them count as selected is the sort's tie-break, and the
        # derivative follows it.  The oracle gives the top-singleton slope to the first of them in
        # index order; the by-value kernels give it to every one (which is each element's own partial
        # derivative: moved off zero alone, it outranks the other zeros).  Compared: everything else;
        # checked there: the entry is 0 or the slope times the cotangent.
        free = np.zeros(theta.shape, bool)
        if mode == tko.TOPKMAG:
            kth = np.sort(np.abs(theta), axis=1)[:, ::-1][:, k - 1]
            free = (theta == 0.0) & (kth == 0.0)[:, None]
        for name, kwargs in (("vjp_state", {"state": state}), ("vjp_recompute", {})):
            recomputes = sorts or (general and solver == tk.TK_SOLVER_AUTO and n <= 128)
            if name == "vjp_recompute" and (ws_bytes or not recomputes):
                continue
            # rows left out: near-ties at a block edge in the solve this VJP rests on (the saved
            # state of the first call; its own solve, the one of the second call, when it recomputes)
            keep = np.ones(rows, bool)
            keep[bad if (name == "vjp_state" or not sorts) else bad_noperm] = False
            grad = torch.full((rows, n), float("nan"), device=dev)
            tk.tk_vjp(th, gt, rows, n, k, p, lam, mode, grad, workspace=ws, **kwargs)
            torch.cuda.synchronize()
            gg = grad.cpu().numpy()
            assert np.isfinite(gg).all(), f"{label}: non-finite {name}"
            e = rel_err(gg, gref)
            e[free] = 0.0
            if free.any():
                slope = np.abs(gg[free]) / np.maximum(np.abs(g[free]), 1e-30)
                assert np.all((gg[free] == 0.0) | (slope <= 1.0 + 1e-5)), f"{label}: {name} at tied zeros"
            res[name + "_max_rel"] = float(e[keep].max()) if keep.any() else 0.0
            res[name + "_max_abs"] = float((np.abs(gg - gref) * ~free)[keep].max()) if keep.any() else 0.0
            assert res[name + "_max_rel"] <= TOL, f"{label}: {name} error {res}"
    return res


def run_sampled(theta: np.ndarray, k: int, p: float, lam: float, mode: int, g: np.ndarray,
                sample: np.ndarray, label: str = ""):
    """Full-size launch as the benchmark times it (default path: no permutation, row state saved,
    VJP from state); the oracle checks the sampled rows only, element by element."""
    theta = np.ascontiguousarray(theta, np.float32)
    g = np.ascontiguousarray(g, np.float32)
    rows, n = theta.shape
    dev = torch.device("cuda")
    th = torch.from_numpy(theta).to(dev)
    gt = torch.from_numpy(g).to(dev)
    out = torch.full((rows, n), float("nan"), device=dev)
    grad = torch.full((rows, n), float("nan"), device=dev)
    state = tk.new_state(rows)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    ws_bytes = tk.tk_workspace_bytes(rows, n, k, p, mode)
    ws = torch.empty(max(ws_bytes, 1), dtype=torch.uint8, device=dev) if ws_bytes else None
    tk.tk_fwd_ex(th, rows, n, k, p, lam, mode, out, state_out=state, workspace=ws, status_out=status)
    tk.tk_vjp(th, gt, rows, n, k, p, lam, mode, grad, state=state, workspace=ws)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, f"{label}: status {int(status.item())}"
    assert bool(torch.isfinite(out).all()) and bool(torch.isfinite(grad).all()), f"{label}: non-finite result"
    sample = np.asarray(sample, np.int64)
    idx = torch.from_numpy(sample).to(dev)
    sub = theta[sample]
    ref, det = tko.fwd(sub, k, p, lam, mode, details=True)
    res = {"fwd_max_rel": float(rel_err(out[idx].cpu().numpy(), ref).max())}
    assert res["fwd_max_rel"] <= TOL, f"{label}: forward error {res}"
    st = read_state(state, rows)[sample]
    gpu_ab = np.stack([st["a"], st["b"]], axis=1).astype(np.int64)
    bad = disputed_rows_ok(sub, k, p, lam, mode, det, gpu_ab, oracle_blocks(det, k))
    keep = np.ones(len(sample), bool)
    keep[bad] = False
    gref = tko.vjp(sub, g[sample], k, p, lam, mode)
    e = rel_err(grad[idx].cpu().numpy(), gref)
    res["vjp_max_rel"] = float(e[keep].max()) if keep.any() else 0.0
    res["rows_block_disputed"] = int(len(bad))
    assert res["vjp_max_rel"] <= TOL, f"{label}: VJP error {res}"
    return res
