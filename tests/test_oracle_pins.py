"""Pins for the CPU oracle: every check here compares the oracle with something
that is not the oracle -- a closed form, a textbook special case, brute force
over the permutahedron's vertices, an optimality condition of the defining
problem, a limit the paper states, or finite differences.

None of these tests needs a GPU.
"""
import itertools
import os

import numpy as np
import pytest
from scipy.optimize import minimize

from oracle import tko

P43 = 4.0 / 3.0
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# --------------------------------------------------------------------------
# independent helpers (none of them sorts-then-pools)
# --------------------------------------------------------------------------
def q_of(p):
    return p / (p - 1.0)


def rho_np(t, p, lam):
    q = q_of(p)
    return np.sign(t) * (np.abs(t) / lam) ** (q - 1.0)


def mask_by_threshold(x, k, p, lam):
    """KKT form of max_{y in [0,1]^n, sum y = k} <y,x> - (lam/p) sum y^p
    (Sec. 3, P(1_k) is the capped simplex scaled by k): stationarity gives
    y_i = clip(((x_i - tau)_+/lam)^(q-1), 0, 1) and tau is fixed by sum y = k.
    For p = 2 this is the Euclidean projection of x/lam onto that polytope."""
    x = np.asarray(x, np.float64)
    q = q_of(p)

    def total(tau):
        return np.clip((np.maximum(x - tau, 0.0) / lam) ** (q - 1.0), 0.0, 1.0).sum()

    lo, hi = x.min() - lam - 1.0, x.max()
    for _ in range(300):
        mid = 0.5 * (lo + hi)
        if total(mid) > k:
            lo = mid
        else:
            hi = mid
    tau = 0.5 * (lo + hi)
    return np.clip((np.maximum(x - tau, 0.0) / lam) ** (q - 1.0), 0.0, 1.0)


def vertices(n, k):
    out = []
    for idx in itertools.combinations(range(n), k):
        v = np.zeros(n)
        v[list(idx)] = 1.0
        out.append(v)
    return np.array(out)


def mask_by_vertex_hull(x, k, p, lam):
    """max over the convex hull of all permutations of 1_k of <y,x> - R(y),
    y = V^T a, a in the simplex (Sec. 3, definition of the permutahedron)."""
    x = np.asarray(x, np.float64)
    V = vertices(len(x), k)
    m = len(V)

    def neg(a):
        y = a @ V
        return -(y @ x) + lam / p * np.sum(np.abs(y) ** p)

    def grad(a):
        y = a @ V
        gy = -x + lam * np.sign(y) * np.abs(y) ** (p - 1.0)
        return V @ gy

    best = None
    for start in range(3):
        rng = np.random.default_rng(start)
        a0 = rng.dirichlet(np.ones(m))
        res = minimize(neg, a0, jac=grad, method="SLSQP", bounds=[(0, 1)] * m,
                       constraints=[{"type": "eq", "fun": lambda a: a.sum() - 1.0,
                                     "jac": lambda a: np.ones(m)}],
                       options={"ftol": 1e-15, "maxiter": 500})
        if best is None or res.fun < best.fun:
            best = res
    return best.x @ V


def primal_objective(x, u, k, p, lam, mag):
    """R*(x - u) + f_phi(u, 1_k) of Prop. 2: sum of the k largest phi(u_i)."""
    q = q_of(p)
    rstar = np.sum(np.abs(x - u) ** q) / (q * lam ** (q - 1.0))
    phi = 0.5 * u * u if mag else u
    return rstar + np.sort(phi)[::-1][:k].sum()


def mag_by_epigraph(x, k, p, lam):
    """Prop. 2 for phi = x^2/2 solved with no sorting: min_u max_S of
    R*(x-u) + 1/2 sum_{i in S} u_i^2 over all k-subsets S, as an epigraph
    programme; then y = grad R*(x - u)."""
    x = np.asarray(x, np.float64)
    n = len(x)
    q = q_of(p)
    subsets = [list(s) for s in itertools.combinations(range(n), k)]

    def rstar(u):
        return np.sum(np.abs(x - u) ** q) / (q * lam ** (q - 1.0))

    def drstar(u):
        return -np.sign(x - u) * np.abs(x - u) ** (q - 1.0) / lam ** (q - 1.0)

    cons = []
    for S in subsets:
        def fun(z, S=S):
            u, t = z[:n], z[n]
            return t - rstar(u) - 0.5 * np.sum(u[S] ** 2)

        def jac(z, S=S):
            u = z[:n]
            g = -drstar(u)
            g[S] -= u[S]
            return np.concatenate([g, [1.0]])
        cons.append({"type": "ineq", "fun": fun, "jac": jac})
    u0 = x / (1.0 + lam)
    z0 = np.concatenate([u0, [primal_objective(x, u0, k, p, lam, True) + 1.0]])
    res = minimize(lambda z: z[n], z0, jac=lambda z: np.concatenate([np.zeros(n), [1.0]]),
                   method="SLSQP", constraints=cons, options={"ftol": 1e-16, "maxiter": 1000})
    u = res.x[:n]
    return rho_np(x - u, p, lam), u


def random_rows(rows, n, seed, scale=1.0):
    return (np.random.default_rng(seed).standard_normal((rows, n)) * scale).astype(np.float32)


# --------------------------------------------------------------------------
# hard operators and the sort
# --------------------------------------------------------------------------
def test_hard_operator_example_from_paper():
    spec = {}
    with open(os.path.join(GOLDEN, "hard_operators_example.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            key, *vals = line.split()
            spec[key] = [int(v) for v in vals]
    x = np.array([1.0, -3.0, 2.0], np.float32)   # x3 >= x1 >= x2 and |x2| >= |x3| >= |x1|
    k = spec["k"][0]
    perm, s = tko.argsort(x, tko.MASK)
    assert (perm[0] + 1).tolist() == spec["argsort"]
    assert s[0].tolist() == [2.0, 1.0, -3.0]
    rank = np.empty(3, int)
    rank[perm[0]] = np.arange(1, 4)
    assert rank.tolist() == spec["rank"]
    tiny = 1e-9   # lambda -> 0: the relaxed operators are the hard ones
    assert np.allclose(tko.fwd(x, k, 2.0, tiny, tko.MASK)[0], spec["topkmask"], atol=1e-12)
    assert np.allclose(tko.fwd(x, k, 2.0, tiny, tko.TOPK)[0], x * np.array(spec["topk_keep"]),
                       atol=1e-8)
    assert np.allclose(tko.fwd(x, k, 2.0, tiny, tko.TOPKMAG)[0], x * np.array(spec["topkmag_keep"]),
                       atol=1e-8)


@pytest.mark.parametrize("mode", [tko.MASK, tko.TOPKMAG])
def test_argsort_against_rank_count(mode):
    rng = np.random.default_rng(5)
    x = rng.standard_normal((40, 37)).astype(np.float32)
    x[:, 5] = x[:, 20]            # exact ties
    x[:, 7] = -x[:, 9]            # |.| ties in magnitude mode
    x[3, 2], x[3, 30] = 0.0, -0.0  # signed zeros compare equal
    perm, s = tko.argsort(x, mode)
    key = np.abs(x) if mode == tko.TOPKMAG else x
    for r in range(x.shape[0]):
        kr = key[r].astype(np.float64)
        # position of element i = #{j: key_j > key_i} + #{j < i: key_j == key_i}
        pos = [(np.sum(kr > kr[i]) + np.sum(kr[:i] == kr[i])) for i in range(len(kr))]
        expect = np.empty(len(kr), np.int32)
        expect[pos] = np.arange(len(kr))
        assert np.array_equal(perm[r], expect)
        assert np.array_equal(s[r], kr[expect])
        assert np.all(np.diff(s[r]) <= 0)


# --------------------------------------------------------------------------
# the mask: closed form, brute force, polytope, limits, invariances
# --------------------------------------------------------------------------
@pytest.mark.parametrize("p", [2.0, P43, 1.5])
@pytest.mark.parametrize("lam", [0.1, 1.0, 3.0])
def test_mask_equals_threshold_form(p, lam):
    for seed, (n, k) in enumerate([(5, 2), (17, 4), (64, 2), (64, 8), (200, 20), (33, 33), (9, 1)]):
        x = random_rows(6, n, 100 + seed)
        y = tko.fwd(x, k, p, lam, tko.MASK)
        for r in range(x.shape[0]):
            ref = mask_by_threshold(x[r], k, p, lam)
            assert np.max(np.abs(y[r] - ref)) < 1e-9


@pytest.mark.parametrize("p", [2.0, P43])
def test_mask_equals_projection_on_vertex_hull(p):
    rng = np.random.default_rng(11)
    for n, k in [(3, 1), (4, 2), (5, 2), (6, 3), (6, 2)]:
        for lam in (0.5, 1.5):
            x = rng.standard_normal(n).astype(np.float32)
            ref = mask_by_vertex_hull(x, k, p, lam)
            y = tko.fwd(x, k, p, lam, tko.MASK)[0]
            assert np.max(np.abs(y - ref)) < 2e-5, (n, k, lam)


@pytest.mark.parametrize("p", [2.0, P43])
def test_mask_lies_in_the_polytope(p):
    for lam in (0.01, 0.3, 1.0, 10.0):
        x = random_rows(50, 40, 7, scale=2.0)
        for k in (1, 5, 39, 40):
            y = tko.fwd(x, k, p, lam, tko.MASK)
            assert y.min() >= 0.0 and y.max() <= 1.0 + 1e-12   # rounding of rho(s - (s - lam))
            assert np.max(np.abs(y.sum(axis=1) - k)) < 1e-11


@pytest.mark.parametrize("p", [2.0, P43])
@pytest.mark.parametrize("mode", [tko.MASK, tko.TOPK, tko.TOPKMAG])
def test_small_lambda_gives_hard_operator(p, mode):
    x = random_rows(20, 30, 3)
    k = 6
    key = np.abs(x) if mode == tko.TOPKMAG else x
    order = np.argsort(-key, axis=1, kind="stable")
    hard_mask = np.zeros_like(x, dtype=np.float64)
    np.put_along_axis(hard_mask, order[:, :k], 1.0, axis=1)
    gap = np.min(np.abs(np.diff(np.sort(key.astype(np.float64), axis=1), axis=1)))
    lam = 0.05 * gap
    y = tko.fwd(x, k, p, lam, mode)
    # a top singleton's output is rho(s - (s - lam)): 1 up to the rounding of s - lam
    slack = 8 * np.finfo(np.float64).eps * np.max(np.abs(x)) / lam
    if mode == tko.MASK:
        assert np.array_equal(y == 0.0, hard_mask == 0.0)
        assert np.max(np.abs(y - hard_mask)) <= slack
    elif mode == tko.TOPK:
        assert np.array_equal(y == 0.0, hard_mask == 0.0)
        assert np.max(np.abs(y - hard_mask * x)) <= slack * np.max(np.abs(x))
    else:
        hard = hard_mask * x
        # error bound of Sec. 5 / App. A.6: ||topkmag_R - topkmag||_inf <= lam ||x||_inf
        assert np.max(np.abs(y - hard)) <= lam * np.max(np.abs(x)) + slack * np.max(np.abs(x))
        if p == 2.0:   # App. A.6, remark: y = w x / (lam w + 1)
            assert np.allclose(y, hard / (1.0 + lam), rtol=0, atol=slack * np.max(np.abs(x)))
        assert np.array_equal(y == 0.0, hard_mask == 0.0)


@pytest.mark.parametrize("p", [2.0, P43])
def test_large_lambda_mask_goes_to_k_over_n(p):
    x = random_rows(5, 12, 4)
    y = tko.fwd(x, 3, p, 1e7, tko.MASK)
    assert np.max(np.abs(y - 3.0 / 12.0)) < 1e-5      # Sec. 7, limit lambda -> infinity


@pytest.mark.parametrize("p", [2.0, P43])
def test_mask_invariances(p):
    rng = np.random.default_rng(9)
    x = random_rows(8, 21, 9)
    k, lam = 4, 0.7
    y = tko.fwd(x, k, p, lam, tko.MASK)
    # permutation equivariance
    perm = rng.permutation(21)
    assert np.max(np.abs(tko.fwd(x[:, perm], k, p, lam, tko.MASK) - y[:, perm])) < 1e-12
    # shift invariance (exactly representable shift)
    assert np.max(np.abs(tko.fwd(x + np.float32(2.0), k, p, lam, tko.MASK) - y)) < 1e-6
    # mask_lam(x) = mask_1(x / lam): use a power of two so x/lam is exact in fp32
    y2 = tko.fwd(x * np.float32(4.0), k, p, 4.0 * lam, tko.MASK)
    assert np.max(np.abs(y2 - y)) < 1e-12
    # topkmag with p = 2 is positively homogeneous of degree 1
    z = tko.fwd(x, k, 2.0, lam, tko.TOPKMAG)
    z2 = tko.fwd(x * np.float32(8.0), k, 2.0, lam, tko.TOPKMAG)
    assert np.max(np.abs(z2 - 8.0 * z)) < 1e-12


# --------------------------------------------------------------------------
# Figure 1 (k = 2, theta(s) = (3, 1, -1+s, s), lambda = 1)
# --------------------------------------------------------------------------
def figure1_rows(points=101):
    """points=101: the grid s = -3 + 0.06 j; points=97: step 1/16, on which s and
    s - 1 are exact in fp32 so that the tie v_2 = v_3 at s >= 2 is exact too."""
    s = np.linspace(-3.0, 3.0, points)
    x = np.stack([np.full_like(s, 3.0), np.full_like(s, 1.0), s - 1.0, s], axis=1)
    return s, x.astype(np.float32)


def test_figure1_p2_closed_form():
    # With y_1 = 1 and y_3 = 0 on this range, y_2 + y_4 = 1 with y_2 = 1 - tau,
    # y_4 = s - tau  =>  tau = s/2 and y_2 = clamp(1 - s/2, 0, 1).
    s, x = figure1_rows()
    y = tko.fwd(x, 2, 2.0, 1.0, tko.MASK)
    f = y[:, 1] + y[:, 2]
    sf = x[:, 3].astype(np.float64)
    assert np.max(np.abs(f - np.clip(1.0 - sf / 2.0, 0.0, 1.0))) < 1e-6
    assert np.allclose(y[:, 0], 1.0)
    s, x = figure1_rows(97)
    y = tko.fwd(x, 2, 2.0, 1.0, tko.MASK)
    f = y[:, 1] + y[:, 2]
    assert np.array_equal(f, np.clip(1.0 - s / 2.0, 0.0, 1.0))   # exact on the dyadic grid
    assert np.all(f[s >= 2.0] == 0.0)             # sparse: exactly zero


def test_figure1_p43_closed_form():
    # p = 4/3: y_2 = a^3, y_4 = (a + s - 1)^3 with a = 1 - tau and a^3 + (a+s-1)^3 = 1.
    for points in (101, 97):
        check_figure1_p43(points)


def check_figure1_p43(points):
    s, x = figure1_rows(points)
    y = tko.fwd(x, 2, P43, 1.0, tko.MASK)
    f = y[:, 1] + y[:, 2]
    sf = x[:, 3].astype(np.float64)
    for fi, si in zip(f, sf):
        if si <= 0.0:
            assert abs(fi - 1.0) < 1e-12
        elif si >= 2.0:
            # on the 101-point grid fl(s - 1) and fl(s) - 1 differ in the last bit
            assert fi == 0.0 if points == 97 else abs(fi) < 1e-12
        else:
            lo, hi = 0.0, 1.0
            for _ in range(200):
                a = 0.5 * (lo + hi)
                if a ** 3 + max(a + si - 1.0, 0.0) ** 3 > 1.0:
                    hi = a
                else:
                    lo = a
            assert abs(fi - (0.5 * (lo + hi)) ** 3) < 1e-9
    if points == 97:
        mid = np.argmin(np.abs(sf - 1.0))
        assert sf[mid] == 1.0 and abs(f[mid] - 0.5) < 1e-12     # 2 a^3 = 1 at s = 1
        # f(1 + d) + f(1 - d) = 1: the equation for a is symmetric under s -> 2 - s, a <-> a + s - 1
        for j, sj in enumerate(sf):
            if -1.0 <= sj <= 3.0:
                jj = int(np.argmin(np.abs(sf - (2.0 - sj))))
                assert sf[jj] == 2.0 - sj and abs(f[j] + f[jj] - 1.0) < 1e-12


def test_figure3_is_sparse_and_continuous():
    # x = (x1, x2, 1/2, 1), phi = x^2/2, k = 2, lambda = 0.3: output_1 + output_2 is
    # exactly 0 around the origin and continuous (Figure 3 caption).
    grid = np.linspace(-2.0, 2.0, 81)
    for p in (2.0, P43):
        rows = np.array([[a, b, 0.5, 1.0] for a in grid for b in grid], np.float32)
        y = tko.fwd(rows, 2, p, 0.3, tko.TOPKMAG)
        tot = (y[:, 0] + y[:, 1]).reshape(81, 81)
        inner = (np.abs(grid)[:, None] < 0.25) & (np.abs(grid)[None, :] < 0.25)
        assert np.all(tot[inner] == 0.0)
        # continuity along a line: |d out_i / d x_j| <= rho' <= (q-1)/lam on [0,1]-valued
        # pieces, so a step of 1e-3 moves the sum of two outputs by < 2 * 1e-3 * 3 / lam + slack;
        # the unregularised operator jumps by about 0.5 on the same line.
        line = np.linspace(-2.0, 2.0, 4001)
        rows = np.array([[a, 0.7, 0.5, 1.0] for a in line], np.float32)
        y = tko.fwd(rows, 2, p, 0.3, tko.TOPKMAG)
        assert np.max(np.abs(np.diff(y[:, 0] + y[:, 1]))) < 0.025


# --------------------------------------------------------------------------
# magnitude operator: brute force and optimality of u*
# --------------------------------------------------------------------------
@pytest.mark.parametrize("p", [2.0, P43, 1.5])
def test_topkmag_equals_epigraph_solution(p):
    rng = np.random.default_rng(21)
    for n, k in [(3, 1), (4, 2), (5, 2), (5, 3)]:
        for lam in (0.3, 1.0):
            x = rng.standard_normal(n).astype(np.float32)
            ref, _ = mag_by_epigraph(x, k, p, lam)
            y = tko.fwd(x, k, p, lam, tko.TOPKMAG)[0]
            assert np.max(np.abs(y - ref)) < 5e-5, (n, k, lam, y, ref)


@pytest.mark.parametrize("p", [2.0, P43, 1.5])
@pytest.mark.parametrize("mode", [tko.MASK, tko.TOPKMAG])
def test_u_star_minimises_the_primal(p, mode):
    rng = np.random.default_rng(31)
    mag = mode == tko.TOPKMAG
    for n, k, lam in [(6, 2, 0.5), (12, 3, 1.0), (30, 7, 0.2), (30, 29, 2.0)]:
        x = rng.standard_normal((3, n)).astype(np.float32)
        _, det = tko.fwd(x, k, p, lam, mode, details=True)
        for r in range(3):
            v = det["v"][r]
            u = np.empty(n)
            u[det["perm"][r]] = v
            xr = x[r].astype(np.float64)
            if mag:
                u *= np.where(np.signbit(xr) & (xr != 0), -1.0, 1.0)
            f0 = primal_objective(xr, u, k, p, lam, mag)
            for scale in (1e-1, 1e-2, 1e-3, 1e-4, 1e-5):
                for _ in range(200):
                    d = rng.standard_normal(n) * scale
                    if rng.random() < 0.5:       # sparse directions probe single coordinates
                        d *= rng.random(n) < 0.2
                    assert primal_objective(xr, u + d, k, p, lam, mag) >= f0 - 1e-13


# --------------------------------------------------------------------------
# internals of the isotonic solution
# --------------------------------------------------------------------------
@pytest.mark.parametrize("p", [2.0, P43, 1.5])
@pytest.mark.parametrize("mode", [tko.MASK, tko.TOPKMAG])
def test_isotonic_solution_structure(p, mode):
    mag = mode == tko.TOPKMAG
    for n, k, lam, seed in [(50, 5, 1.0, 1), (50, 25, 0.3, 2), (128, 16, 1.0, 3), (10, 10, 1.0, 4)]:
        x = random_rows(10, n, seed)
        if seed == 2:
            x[:, 3] = x[:, 11]
        _, det = tko.fwd(x, k, p, lam, mode, details=True)
        perm, s = tko.argsort(x, mode)
        for r in range(x.shape[0]):
            v, lo, hi = det["v"][r], det["block_lo"][r], det["block_hi"][r]
            assert np.all(np.diff(v) <= 1e-15)                      # v in the monotone cone
            if mag:
                assert v.min() >= 0.0
            pooled = 0
            i = 0
            while i < n:
                a, b = lo[i], hi[i]
                assert a == i and b > a
                g = v[a]
                assert np.all(v[a:b] == g)
                w = (np.arange(a, b) < k).astype(float)
                resid = np.sum(-rho_np(s[r][a:b] - g, p, lam) + w * (g if mag else 1.0))
                assert abs(resid) < 1e-9 * max(1.0, b - a)           # block stationarity
                pooled += (b - a) > 1
                if b - a > 1:
                    assert a < k < b                                  # the pooled block straddles rank k
                i = b
            assert pooled <= 1                                        # w = 1_k: at most one pooled block


@pytest.mark.parametrize("p", [2.0, P43])
@pytest.mark.parametrize("mode", [tko.MASK, tko.TOPK, tko.TOPKMAG])
def test_member_resolve_matches_closed_form_solves(p, mode):
    x = random_rows(12, 300, 8)
    g = random_rows(12, 300, 9)
    a = tko.fwd(x, 30, p, 1.0, mode)
    b = tko.fwd(x, 30, p, 1.0, mode, flags=tko.FLAG_RESUM)
    assert np.max(np.abs(a - b)) < 1e-11
    ga = tko.vjp(x, g, 30, p, 1.0, mode)
    gb = tko.vjp(x, g, 30, p, 1.0, mode, flags=tko.FLAG_RESUM)
    assert np.max(np.abs(ga - gb)) < 1e-8


# --------------------------------------------------------------------------
# alternating projections
# --------------------------------------------------------------------------
@pytest.mark.parametrize("p", [2.0, P43])
@pytest.mark.parametrize("mode", [tko.MASK, tko.TOPKMAG])
def test_dykstra_converges_to_pav(p, mode):
    x = random_rows(8, 24, 13)
    for k, lam in [(3, 1.0), (12, 0.4)]:
        exact, det = tko.fwd(x, k, p, lam, mode, details=True)
        out, v = tko.dykstra(x, k, p, lam, mode, sweeps=6000, return_v=True)
        assert np.max(np.abs(v - det["v"])) < 1e-9
        assert np.max(np.abs(out - exact)) < 1e-8


def test_dykstra_single_element_is_s_minus_lambda_w():
    # n = 1: no constraint, so the iteration must return the unconstrained
    # minimiser s - lambda w (phi = x) after any number of sweeps.
    x = np.array([[0.75]], np.float32)
    for sweeps in (0, 1, 5):
        _, v = tko.dykstra(x, 1, 2.0, 0.5, tko.MASK, sweeps=sweeps, return_v=True)
        assert v[0, 0] == 0.75 - 0.5


def test_dykstra_hundred_sweeps_small_block():
    # Sec. 5: 100 iterations reproduce PAV (small pooled blocks)
    x = random_rows(64, 16, 17)
    exact = tko.fwd(x, 2, 2.0, 0.3, tko.MASK)
    out = tko.dykstra(x, 2, 2.0, 0.3, tko.MASK, sweeps=100)
    assert np.max(np.abs(out - exact)) < 1e-6


def test_dykstra_iterates_after_one_and_two_sweeps_by_hand():
    """Algorithm 1 at a finite sweep count, worked by hand (fractions, no oracle value involved).

    phi(x) = x, k = 1, lambda = 4, s = (4, 3, 2): z = s - lambda w = (0, 3, 2), p = q = 0.
      sweep 1, C1 (pair 1,2): (0, 3) -> 3/2 each, p = (-3/2, 3/2, 0);
               C2 (pair 2,3): (3/2, 2) -> 7/4 each, q = (0, -1/4, 1/4);      v = (3/2, 7/4, 7/4)
      sweep 2, C1: v + p = (0, 13/4, 7/4) -> (13/8, 13/8, 7/4), p = (-13/8, 13/8, 0);
               C2: y + q = (13/8, 11/8, 2) -> (13/8, 27/16, 27/16);          v = (13/8, 27/16, 27/16)
    (C2 before C1, or a correction dropped on the pair that does not violate, gives other numbers;
    the limit is the mean 5/3.)  Output y = (s - v)/lambda.
    phi(x) = x^2/2, k = 1, lambda = 1, s = (4, 3, 5/2): metric c = (2, 1, 1), z = s/c = (2, 3, 5/2).
      sweep 1, C1: (2, 3) -> (2*2 + 3)/3 = 7/3, p = (-1/3, 2/3, 0);
               C2: (7/3, 5/2) -> 29/12, q = (0, -1/12, 1/12);                v = (7/3, 29/12, 29/12)
      sweep 2, C1: v + p = (2, 37/12, 29/12) -> 85/36, p = (-13/36, 26/36, 0);
               C2: y + q = (85/36, 82/36, 90/36) -> 43/18;                   v = (85/36, 43/18, 43/18)
    """
    from fractions import Fraction as Fr
    theta = np.array([[3.0, 2.0, 4.0]], np.float32)            # unsorted on purpose: s = (4, 3, 2)
    expect_v = {0: [Fr(0), Fr(3), Fr(2)], 1: [Fr(3, 2), Fr(7, 4), Fr(7, 4)], 2: [Fr(13, 8), Fr(27, 16), Fr(27, 16)]}
    s = [Fr(4), Fr(3), Fr(2)]
    for sweeps, ev in expect_v.items():
        out, v = tko.dykstra(theta, 1, 2.0, 4.0, tko.MASK, sweeps=sweeps, return_v=True)
        assert np.max(np.abs(v[0] - np.array([float(a) for a in ev]))) < 1e-14
        y_sorted = [float((si - vi) / 4) for si, vi in zip(s, ev)]
        assert np.max(np.abs(out[0] - np.array([y_sorted[1], y_sorted[2], y_sorted[0]]))) < 1e-14
    theta = np.array([[-3.0, 2.5, 4.0]], np.float32)           # |theta| sorted: (4, 3, 5/2), signs (+, -, +)
    expect_v = {1: [Fr(7, 3), Fr(29, 12), Fr(29, 12)], 2: [Fr(85, 36), Fr(43, 18), Fr(43, 18)]}
    s = [Fr(4), Fr(3), Fr(5, 2)]
    for sweeps, ev in expect_v.items():
        out, v = tko.dykstra(theta, 1, 2.0, 1.0, tko.TOPKMAG, sweeps=sweeps, return_v=True)
        assert np.max(np.abs(v[0] - np.array([float(a) for a in ev]))) < 1e-14
        y_sorted = [float(si - vi) for si, vi in zip(s, ev)]    # rho(t) = t / lambda, lambda = 1
        assert np.max(np.abs(out[0] - np.array([-y_sorted[1], y_sorted[2], y_sorted[0]]))) < 1e-14


def test_dual_coordinate_ascent_first_updates_by_hand():
    """App. A.8 for p = 4/3 (rho(t) = (t/lambda)^3), phi(x) = x, k = 1, lambda = 1, three equal keys s.

    Sweep 1, odd coordinate alpha_1 (pair 1,2; alpha_0 = alpha_2 = 0): separate minimisers s - 1 < s,
    so both take the common gamma with 2 (s - gamma)^3 = 1, and alpha_1 = 1 - (s - gamma)^3 = 1/2.
    Even coordinate alpha_2 (pair 2,3; alpha_1 = 1/2, alpha_3 = 0): s - cbrt(1/2) < s, common gamma
    with 2 (s - gamma)^3 = 1/2, alpha_2 = 1/2 - 1/4 = 1/4.  Primal iterate v_i = s - cbrt(w_i + alpha_{i-1}
    - alpha_i): outputs y = (1/2, 1/4, 1/4).
    Sweep 2: alpha_1 solves 2 a^3 = 1 - 1/4 -> alpha_1 = 1 - 3/8 = 5/8; alpha_2 solves 2 a^3 = 5/8 ->
    alpha_2 = 5/8 - 5/16 = 5/16: y = (3/8, 5/16, 5/16).  (Even before odd would give (1/2, 1/2, 0) after
    the first sweep; the limit is (1/3, 1/3, 1/3).)
    """
    theta = np.full((1, 3), 0.625, np.float32)
    for sweeps, y in ((1, [0.5, 0.25, 0.25]), (2, [0.375, 0.3125, 0.3125])):
        out, v = tko.dykstra(theta, 1, P43, 1.0, tko.MASK, sweeps=sweeps, return_v=True)
        assert np.max(np.abs(out[0] - np.array(y))) < 1e-13
        assert np.max(np.abs(v[0] - (0.625 - np.cbrt(np.array(y))))) < 1e-13


# --------------------------------------------------------------------------
# general sorted w: relaxed linear maximisation over the permutahedron P(w)
# --------------------------------------------------------------------------
def lmo_by_vertex_hull(x, w, p, lam):
    """max over the convex hull of all permutations of w of <y, x> - R(y), y = a^T V with a in the simplex
    (Sec. 3, definition of the permutahedron); no sort, no isotonic solve."""
    import itertools
    x = np.asarray(x, np.float64)
    V = np.array(sorted(set(itertools.permutations([float(a) for a in w]))))
    m = len(V)

    def neg(a):
        y = a @ V
        return -(y @ x) + lam / p * np.sum(np.abs(y) ** p)

    def grad(a):
        y = a @ V
        return V @ (-x + lam * np.sign(y) * np.abs(y) ** (p - 1.0))

    best = None
    for start in range(3):
        a0 = np.random.default_rng(start).dirichlet(np.ones(m))
        res = minimize(neg, a0, jac=grad, method="SLSQP", bounds=[(0, 1)] * m,
                       constraints=[{"type": "eq", "fun": lambda a: a.sum() - 1.0, "jac": lambda a: np.ones(m)}],
                       options={"ftol": 1e-15, "maxiter": 800})
        if best is None or res.fun < best.fun:
            best = res
    return best.x @ V


@pytest.mark.parametrize("p", [2.0, P43])
def test_general_w_equals_maximiser_over_vertex_hull(p):
    rng = np.random.default_rng(23)
    for w in ([3.0, 2.0, 1.0], [4.0, 3.0, 2.0, 1.0], [2.0 / 3, 1.0 / 3, 0.0], [1.0, 1.0, 0.5, 0.0],
              [5.0, 4.0, 3.0, 2.0, 1.0], [2.0, 0.5, 0.5, -1.0]):
        for lam in (0.4, 1.5):
            x = (rng.standard_normal(len(w)) * 1.5).astype(np.float32)
            ref = lmo_by_vertex_hull(x, w, p, lam)
            y = tko.fwd_w(x, w, p, lam)[0]
            assert np.max(np.abs(y - ref)) < 5e-5, (w, lam, y, ref)


@pytest.mark.parametrize("p", [2.0, P43])
def test_general_w_reduces_to_the_mask_and_to_the_hard_operators(p):
    x = random_rows(20, 12, 29, scale=2.0)
    for k in (1, 4, 11):
        w = np.r_[np.ones(k), np.zeros(12 - k)]
        assert np.max(np.abs(tko.fwd_w(x, w, p, 0.7) - tko.fwd(x, k, p, 0.7, tko.MASK))) < 1e-10
    # lambda -> 0: the linear maximisation oracle y(x, w) = w_rank(x) (Prop. 1), hence sort and rank (Sec. 3)
    w = np.linspace(3.0, -1.0, 12)
    perm, _ = tko.argsort(x, tko.MASK)
    y = tko.fwd_w(x, w, p, 1e-7)
    for r in range(x.shape[0]):
        want = np.empty(12); want[perm[r]] = w
        assert np.max(np.abs(y[r] - want)) < 1e-5
    ranks = tko.soft_rank(x, p, 1e-7)
    srt = tko.soft_sort(x, p, 1e-7)
    for r in range(x.shape[0]):
        hard_rank = np.empty(12); hard_rank[perm[r]] = np.arange(1, 13)
        assert np.max(np.abs(ranks[r] - hard_rank)) < 1e-5
        assert np.max(np.abs(srt[r] - np.sort(x[r].astype(np.float64))[::-1])) < 1e-5


@pytest.mark.parametrize("p", [2.0, P43])
def test_general_w_output_lies_in_the_permutahedron_and_is_optimal(p):
    """y in P(w): same total, and the l largest entries of y sum to at most w_1 + .. + w_l (majorisation);
    no point of P(w) (random convex combinations of permutations of w) does better in <x, y> - R(y)."""
    rng = np.random.default_rng(31)
    n = 9
    x = random_rows(12, n, 33, scale=1.5)
    w = np.array([4.0, 3.5, 3.5, 2.0, 1.0, 1.0, 0.5, 0.0, -1.0])
    for lam in (0.2, 1.0, 5.0):
        y = tko.fwd_w(x, w, p, lam)
        assert np.max(np.abs(y.sum(axis=1) - w.sum())) < 1e-9
        ys = -np.sort(-y, axis=1)
        assert np.all(np.cumsum(ys, axis=1) <= np.cumsum(w)[None, :] + 1e-9)
        for r in range(x.shape[0]):
            xr = x[r].astype(np.float64)
            best = y[r] @ xr - lam / p * np.sum(np.abs(y[r]) ** p)
            for _ in range(200):
                a = rng.dirichlet(np.ones(6) * 0.5)
                z = sum(ai * w[rng.permutation(n)] for ai in a)
                assert z @ xr - lam / p * np.sum(np.abs(z) ** p) <= best + 1e-10
            # and towards y itself from those points the objective increases (concavity: a local check)
            z = 0.9 * y[r] + 0.1 * w[rng.permutation(n)]
            assert z @ xr - lam / p * np.sum(np.abs(z) ** p) <= best + 1e-10


@pytest.mark.parametrize("p", [2.0, P43])
def test_general_w_vjp_matches_finite_differences(p):
    rng = np.random.default_rng(37)
    n = 7
    w = np.array([3.0, 2.5, 2.0, 2.0, 1.0, 0.2, 0.0])
    for lam in (0.5, 2.0):
        x = (rng.standard_normal(n) * 1.2).astype(np.float32)
        J = np.empty((n, n))
        h = 1e-3
        for j in range(n):
            xp = x.copy(); xm = x.copy()
            xp[j] = np.float32(x[j] + h); xm[j] = np.float32(x[j] - h)
            J[:, j] = (tko.fwd_w(xp, w, p, lam)[0] - tko.fwd_w(xm, w, p, lam)[0]) / (float(xp[j]) - float(xm[j]))
        Jv = np.empty((n, n))
        for i in range(n):
            e = np.zeros(n, np.float32); e[i] = 1.0
            Jv[i, :] = tko.vjp_w(x, w, e, p, lam)[0]
        # away from the kinks where a block forms or splits (a perturbation of 1e-3 must not change the partition)
        _, d0 = tko.fwd_w(x, w, p, lam, details=True)
        same = True
        for j in range(n):
            for sgn in (-1, 1):
                xq = x.copy(); xq[j] = np.float32(x[j] + sgn * h)
                _, d1 = tko.fwd_w(xq, w, p, lam, details=True)
                same &= np.array_equal(d0["block_lo"], d1["block_lo"]) and np.array_equal(d0["perm"], d1["perm"])
        if same:
            assert np.max(np.abs(J - Jv)) < 2e-5, (lam, J, Jv)
    # w sorted is required
    with pytest.raises(ValueError):
        tko.fwd_w(np.zeros((1, 3), np.float32), [1.0, 2.0, 0.0], 2.0, 1.0)


@pytest.mark.parametrize("p", [2.0, P43])
def test_general_w_cotangent_pulled_back_to_w(p):
    """The gradient in w (what makes the relaxed sort of Sec. 3 differentiable in its input, which enters as
    w).  Pins: (1) every point of P(w) has sum y = sum w, so the cotangent g = 1 must pull back to 1 for every
    w_j; (2) central differences of the forward pass in w (w is a float64 input: small steps that keep it
    sorted), away from the kinks where the partition changes; (3) a singleton has y_j = w_j."""
    rng = np.random.default_rng(41)
    n = 7
    for lam in (0.5, 2.0):
        x = (rng.standard_normal((1, n)) * 1.2).astype(np.float32)
        w = np.array([3.0, 2.6, 2.1, 1.9, 1.0, 0.2, 0.0])
        _, gw1 = tko.vjp_w(x, w, np.ones((1, n), np.float32), p, lam, with_w=True)
        assert np.max(np.abs(gw1 - 1.0)) < 1e-12
        g = rng.standard_normal((1, n)).astype(np.float32)
        _, gw = tko.vjp_w(x, w, g, p, lam, with_w=True)
        _, d0 = tko.fwd_w(x, w, p, lam, details=True)
        h = 1e-6
        fd = np.empty(n)
        same = True
        for j in range(n):
            wp = w.copy(); wm = w.copy()
            wp[j] += h; wm[j] -= h
            yp, dp = tko.fwd_w(x, wp, p, lam, details=True)
            ym, dm = tko.fwd_w(x, wm, p, lam, details=True)
            same &= np.array_equal(d0["block_lo"], dp["block_lo"]) and np.array_equal(d0["block_lo"], dm["block_lo"])
            fd[j] = float(np.dot(g[0].astype(np.float64), (yp[0] - ym[0]))) / (2 * h)
        if same:
            assert np.max(np.abs(fd - gw[0])) < 1e-6, (lam, fd, gw)
    # lambda -> 0: nothing pools, y = w through the permutation, so the pull-back is g in sorted order
    x = np.array([[0.3, -1.0, 2.0, 0.9]], np.float32)
    w = np.array([4.0, 3.0, 2.0, 1.0])
    g = np.array([[1.0, 2.0, 3.0, 4.0]], np.float32)
    _, gw = tko.vjp_w(x, w, g, p, 1e-3, with_w=True)
    order = np.argsort(-x[0], kind="stable")
    assert np.allclose(gw[0], g[0][order], atol=1e-9)


# --------------------------------------------------------------------------
# VJP
# --------------------------------------------------------------------------
def jacobian_fd(x, k, p, lam, mode, h=1e-3):
    """central differences in fp32-representable steps (inputs are fp32)."""
    n = len(x)
    J = np.empty((n, n))
    for j in range(n):
        xp = x.copy(); xm = x.copy()
        xp[j] = np.float32(x[j] + h); xm[j] = np.float32(x[j] - h)
        step = float(xp[j]) - float(xm[j])
        J[:, j] = (tko.fwd(xp, k, p, lam, mode)[0] - tko.fwd(xm, k, p, lam, mode)[0]) / step
    return J


def jacobian_vjp(x, k, p, lam, mode):
    n = len(x)
    J = np.empty((n, n))
    for i in range(n):
        e = np.zeros(n, np.float32); e[i] = 1.0
        J[i, :] = tko.vjp(x, e, k, p, lam, mode)[0]
    return J


@pytest.mark.parametrize("p", [2.0, P43])
@pytest.mark.parametrize("mode", [tko.MASK, tko.TOPK, tko.TOPKMAG])
def test_vjp_matches_finite_differences(p, mode):
    rng = np.random.default_rng(41)
    checked = 0
    for trial in range(12):
        n, k, lam = 9, 3, 0.8
        x = (rng.standard_normal(n) * 1.0).astype(np.float32)
        # keep away from kinks: block membership must not change within +-h
        _, d0 = tko.fwd(x, k, p, lam, mode, details=True)
        stable = True
        for j in range(n):
            for sgn in (-1, 1):
                xx = x.copy(); xx[j] = np.float32(xx[j] + sgn * 2e-3)
                _, d1 = tko.fwd(xx, k, p, lam, mode, details=True)
                if not (np.array_equal(d0["perm"], d1["perm"]) and
                        np.array_equal(d0["block_lo"], d1["block_lo"]) and
                        np.array_equal(d0["block_hi"], d1["block_hi"])):
                    stable = False
        if not stable:
            continue
        J = jacobian_vjp(x, k, p, lam, mode)
        Jfd = jacobian_fd(x, k, p, lam, mode)
        tol = 1e-8 if p == 2.0 else 2e-5      # p = 2 is piecewise linear: differences are exact
        assert np.max(np.abs(J - Jfd)) < tol * max(1.0, np.max(np.abs(J)))
        checked += 1
    assert checked >= 4


@pytest.mark.parametrize("mode", [tko.MASK, tko.TOPK, tko.TOPKMAG])
def test_jvp_is_the_finite_difference_jacobian_applied_to_the_tangent(mode):
    """p = 2: the operator is piecewise linear, central differences are exact away from kinks."""
    rng = np.random.default_rng(43)
    checked = 0
    for trial in range(10):
        n, k, lam = 8, 3, 0.7
        x = rng.standard_normal(n).astype(np.float32)
        _, d0 = tko.fwd(x, k, 2.0, lam, mode, details=True)
        stable = True
        for j in range(n):
            for sgn in (-1, 1):
                xx = x.copy(); xx[j] = np.float32(xx[j] + sgn * 2e-3)
                _, d1 = tko.fwd(xx, k, 2.0, lam, mode, details=True)
                stable &= (np.array_equal(d0["perm"], d1["perm"]) and np.array_equal(d0["block_lo"], d1["block_lo"])
                           and np.array_equal(d0["block_hi"], d1["block_hi"]))
        if not stable:
            continue
        v = rng.standard_normal(n)
        Jfd = jacobian_fd(x, k, 2.0, lam, mode)
        got = tko.jvp(x[None, :], v[None, :], k, 2.0, lam, mode)[0]
        assert np.max(np.abs(got - Jfd @ v)) < 1e-7 * max(1.0, np.max(np.abs(Jfd)))
        checked += 1
    assert checked >= 3


@pytest.mark.parametrize("p", [2.0, P43])
def test_mask_jacobian_is_symmetric_with_zero_row_sums(p):
    x = random_rows(1, 14, 51)[0]
    J = jacobian_vjp(x, 4, p, 1.0, tko.MASK)
    assert np.max(np.abs(J - J.T)) < 1e-12
    assert np.max(np.abs(J.sum(axis=0))) < 1e-12 and np.max(np.abs(J.sum(axis=1))) < 1e-12
    assert np.max(np.abs(J)) > 0.01


def test_topkmag_p2_top_singletons_have_slope_one_over_one_plus_lambda():
    x = np.array([[5.0, -4.0, 0.1, 0.05, -0.02]], np.float32)
    lam = 0.25
    g = np.ones((1, 5), np.float32)
    grad = tko.vjp(x, g, 2, 2.0, lam, tko.TOPKMAG)[0]
    assert np.allclose(grad[:2], 1.0 / (1.0 + lam)) and np.all(grad[2:] == 0.0)


# ---------------------------------------------------------------- smooth top-k loss
def sum_of_k_largest(u, k):
    return np.sort(u)[::-1][:k].sum()


def conj_R(t, p, lam):
    """R*(t) = sum |t_i|^q / (q lambda^(q-1)) for R(y) = (lambda/p) sum |y_i|^p."""
    q = q_of(p)
    return np.sum(np.abs(t) ** q) / (q * lam ** (q - 1.0))


@pytest.mark.parametrize("p", [2.0, P43, 1.5])
def test_topk_loss_value_sits_between_primal_and_dual_bounds(p):
    """f(x, 1_k) = max_{y in P(1_k)} <y,x> - R(y) = min_u R*(x - u) + (sum of the k largest u):
    every feasible y bounds it from below, every u from above, and the two bounds meet at the
    oracle's value (checked with y, u that the oracle did not produce)."""
    rng = np.random.default_rng(5)
    for n, k, lam in [(6, 2, 1.0), (9, 3, 0.3), (17, 5, 2.0)]:
        x = random_rows(1, n, 40 + n)[0]
        x64 = x.astype(np.float64)
        loss, _ = tko.topk_loss(x, [-1], k, p, lam)
        f = loss[0]
        best_lo, best_hi = -np.inf, np.inf
        ystar = mask_by_threshold(x64, k, p, lam)          # KKT form, shares nothing with sort + PAV
        q = q_of(p)
        for trial in range(400):
            if trial == 0:
                y = ystar
            elif trial == 1:
                y = np.zeros(n); y[np.argsort(-x64)[:k]] = 1.0      # a vertex: the hard mask
            else:
                y = np.clip(ystar + rng.normal(size=n) * 10.0 ** rng.integers(-6, 0), 0, 1)
                y = np.clip(y * (k / y.sum()), 0, 1)
                if abs(y.sum() - k) > 1e-12:
                    continue
            lo = y @ x64 - (lam / p) * np.sum(np.abs(y) ** p)
            assert lo <= f + 1e-10
            best_lo = max(best_lo, lo)
            u = x64 - lam * ystar ** (1.0 / (q - 1.0)) if trial == 0 else x64 * rng.uniform(0, 1) + rng.normal(size=n) * 0.3
            hi = conj_R(x64 - u, p, lam) + sum_of_k_largest(u, k)
            assert hi >= f - 1e-10
            best_hi = min(best_hi, hi)
        assert abs(best_lo - f) <= 1e-10 and abs(best_hi - f) <= 1e-9


@pytest.mark.parametrize("p", [2.0, P43])
def test_topk_loss_gradient_is_the_finite_difference_of_its_value(p):
    x = random_rows(3, 12, 91)
    tgt = np.array([0, 7, 11])
    loss, grad = tko.topk_loss(x, tgt, 4, p, 0.7)
    h = 1e-3                                            # inputs are float32: a step it represents
    for r in range(3):
        for i in range(12):
            xp, xm = x.copy(), x.copy()
            xp[r, i] += np.float32(h); xm[r, i] -= np.float32(h)
            d = float(xp[r, i]) - float(xm[r, i])
            fd = (tko.topk_loss(xp, tgt, 4, p, 0.7)[0][r] - tko.topk_loss(xm, tgt, 4, p, 0.7)[0][r]) / d
            assert abs(fd - grad[r, i]) <= 5e-3, (r, i, fd, grad[r, i])
    assert np.allclose(grad.sum(axis=1), 4 - 1, atol=1e-12)   # <y*, 1> = k, <t, 1> = 1


def test_topk_loss_limits_and_two_element_closed_form():
    x = random_rows(5, 20, 17, scale=3.0)
    tgt = np.array([3, 3, -1, 20, 0])                      # rows 2 and 3: no target, loss = f
    lam0 = 1e-6
    loss, grad = tko.topk_loss(x, tgt, 3, 2.0, lam0)
    for r in range(5):
        hard = sum_of_k_largest(x[r].astype(np.float64), 3)
        t = float(x[r, tgt[r]]) if 0 <= tgt[r] < 20 else 0.0
        # lambda -> 0: f -> sum of the k largest, from below and by no more than R's largest value on P(1_k)
        assert hard - t - lam0 * 3 / 2.0 - 1e-8 <= loss[r] <= hard - t + 1e-8
    # n = 2, k = 1, p = 2: y1 = clip(1/2 + (x1 - x2)/(2 lam), 0, 1), y2 = 1 - y1
    for x1, x2, lam in [(0.3, 0.1, 1.0), (2.0, -1.0, 0.5), (-0.2, 0.4, 3.0)]:
        y1 = min(1.0, max(0.0, 0.5 + (np.float32(x1).astype(float) - np.float32(x2).astype(float)) / (2 * lam)))
        y = np.array([y1, 1 - y1])
        xv = np.array([np.float32(x1), np.float32(x2)], dtype=np.float64)
        want = y @ xv - 0.5 * lam * (y ** 2).sum() - xv[1]
        got, g = tko.topk_loss(np.array([[x1, x2]], np.float32), [1], 1, 2.0, lam)
        assert abs(got[0] - want) <= 1e-12
        assert np.allclose(g[0], y - np.array([0.0, 1.0]), atol=1e-12)


def test_hard_operators_match_the_paper_example_and_the_small_lambda_limit():
    """tko.hard against the worked example of Sec. 3 (golden file) and against the relaxed
    operators as lambda -> 0 (no ties: the limit is unique)."""
    gold = {}
    with open(os.path.join(GOLDEN, "hard_operators_example.txt")) as fh:
        for line in fh:
            if line.strip() and not line.startswith("#"):
                key, *vals = line.split()
                gold[key] = [int(v) for v in vals]
    x = np.array([[0.5, -3.0, 2.0]], np.float32)       # x3 >= x1 >= x2 and |x2| >= |x3| >= |x1|
    k = gold["k"][0]
    assert tko.hard(x, k, tko.MASK)[0].tolist() == gold["topkmask"]
    assert tko.hard(x, k, tko.TOPK)[0].tolist() == (np.array(gold["topk_keep"]) * x[0].astype(float)).tolist()
    assert tko.hard(x, k, tko.TOPKMAG)[0].tolist() == (np.array(gold["topkmag_keep"]) * x[0].astype(float)).tolist()
    xs = random_rows(6, 40, 3)
    for mode in (tko.MASK, tko.TOPK, tko.TOPKMAG):
        soft = tko.fwd(xs, 7, 2.0, 1e-7, mode)
        assert np.max(np.abs(soft - tko.hard(xs, 7, mode))) <= 1e-5
    tied = np.array([[1.0, 2.0, 2.0, 2.0, 0.0]], np.float32)     # ties: the earlier index wins
    assert tko.hard(tied, 2, tko.MASK)[0].tolist() == [0, 1, 1, 0, 0]


def test_invalid_arguments_are_rejected():
    x = np.zeros((1, 4), np.float32)
    for k, p, lam in [(0, 2.0, 1.0), (5, 2.0, 1.0), (2, 1.0, 1.0), (2, 2.0, 0.0)]:
        with pytest.raises(ValueError):
            tko.fwd(x, k, p, lam, tko.MASK)
