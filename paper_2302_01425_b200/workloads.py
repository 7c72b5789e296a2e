"""Seeded synthetic inputs for the smoothed top-k operators.

This module only draws numbers.  It contains none of the method's arithmetic
(no sorting for the operator, no isotonic solve, no dual map) so that the CPU
oracle and the CUDA library can both be fed from it without sharing any code
of the method itself.

Every generator is a pure function of its arguments: numpy's PCG64 bit
generator with the given seed, float32 results, C-contiguous (rows, n).
Cotangents for the VJP use seed + 1_000_003.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List

import numpy as np

MODE_MASK = 0      # topkmask: phi(x) = x
MODE_TOPK = 1      # topk: theta * topkmask(theta)
MODE_TOPKMAG = 2   # topkmag: phi(x) = x^2 / 2, sorted by |theta|

COTANGENT_SEED_OFFSET = 1_000_003


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def normal_rows(rows: int, n: int, seed: int, scale: float = 1.0) -> np.ndarray:
    """rows x n float32 drawn from N(0, scale^2)."""
    x = _rng(seed).standard_normal((rows, n), dtype=np.float32)
    if scale != 1.0:
        x *= np.float32(scale)
    return np.ascontiguousarray(x)


def cotangent_like(theta: np.ndarray, seed: int) -> np.ndarray:
    """N(0,1) cotangent with the shape of theta; seed is the data seed."""
    g = _rng(seed + COTANGENT_SEED_OFFSET).standard_normal(theta.shape, dtype=np.float32)
    return np.ascontiguousarray(g)


def figure1_rows(points: int = 101, lo: float = -3.0, hi: float = 3.0) -> np.ndarray:
    """The rows theta(s) = (3, 1, -1 + s, s) of the paper's Figure 1 on a grid of s."""
    s = np.linspace(lo, hi, points, dtype=np.float64)
    x = np.stack([np.full_like(s, 3.0), np.full_like(s, 1.0), s - 1.0, s], axis=1)
    return np.ascontiguousarray(x.astype(np.float32))


def class_logit_rows(rows: int, n: int, seed: int, scale: float = 3.0,
                     dup_fraction: float = 0.10) -> np.ndarray:
    """Classifier-logit stand-in: N(0, scale^2) with forced exact ties.

    Per row a seeded permutation of the positions is drawn; the first
    d = floor(dup_fraction * n) positions are targets, the next d are sources,
    and theta[target] <- theta[source], so that dup_fraction of the entries are
    exact duplicates of other entries.
    """
    g = _rng(seed)
    x = g.standard_normal((rows, n), dtype=np.float32) * np.float32(scale)
    d = int(dup_fraction * n)
    if d > 0 and 2 * d <= n:
        for r in range(rows):
            perm = g.permutation(n)
            x[r, perm[:d]] = x[r, perm[d:2 * d]]
    return np.ascontiguousarray(x)


@dataclass
class Case:
    """One operator call: shape, hyper-parameters and how to draw its input."""
    name: str
    rows: int
    n: int
    k: int
    p: float
    lam: float
    mode: int
    seed: int
    kind: str = "normal"          # normal | class_logit | figure1
    scale: float = 1.0
    extra: Dict[str, float] = field(default_factory=dict)

    @property
    def elements(self) -> int:
        return self.rows * self.n

    def theta(self, rows: int | None = None) -> np.ndarray:
        """Draw the input.  rows < self.rows draws only a leading sample of the
        rows (same stream, so the sample equals the first rows of the full
        draw for the 'normal' kind)."""
        r = self.rows if rows is None else min(rows, self.rows)
        if self.kind == "normal":
            return normal_rows(r, self.n, self.seed, self.scale)
        if self.kind == "class_logit":
            return class_logit_rows(r, self.n, self.seed, self.scale)
        if self.kind == "figure1":
            return figure1_rows(self.rows)
        raise ValueError(self.kind)

    def cotangent(self, theta: np.ndarray) -> np.ndarray:
        return cotangent_like(theta, self.seed)


P43 = 4.0 / 3.0


def tiny_cases() -> List[Case]:
    out = [Case("tiny", 64, 32, 4, 2.0, 1.0, MODE_MASK, seed=0)]
    for p in (2.0, P43):
        out.append(Case(f"figure1_p{'2' if p == 2.0 else '43'}", 101, 4, 2, p, 1.0,
                        MODE_MASK, seed=0, kind="figure1"))
    return out


def moe_router_cases() -> List[Case]:
    """Token-choice router logits: 16384 tokens x 64 experts, k = 2."""
    out = []
    for p in (2.0, P43):
        for lam in (0.1, 1.0):
            out.append(Case(f"moe_p{'2' if p == 2.0 else '43'}_lam{lam:g}", 16384, 64, 2, p, lam,
                            MODE_MASK, seed=1))
    return out


def class_logit_case() -> Case:
    return Case("class_logit", 8192, 1000, 5, P43, 0.5, MODE_TOPK, seed=2,
                kind="class_logit", scale=3.0)


def expert_choice_case() -> Case:
    """Expert-choice routing: every expert picks k = 28 of n = 400 tokens (32 experts x 1024 groups
    of tokens = 32768 rows), p = 2.  The regularisation strength of that experiment is not stated;
    lambda = 1 here."""
    return Case("expert_choice", 32 * 1024, 400, 28, 2.0, 1.0, MODE_MASK, seed=4)


def pruning_case() -> Case:
    n = 2048 * 2048
    return Case("pruning", 1, n, n // 10, 2.0, 1e-3, MODE_TOPKMAG, seed=3, scale=0.02)


def shape_sweep_cases(total_log2: int = 26) -> List[Case]:
    out = []
    for n in (8, 64, 512, 4096, 32768):
        lg = n.bit_length() - 1
        rows = (1 << total_log2) // n
        for p in (2.0, P43):
            out.append(Case(f"sweep_n{n}_p{'2' if p == 2.0 else '43'}", rows, n, n // 8, p, 1.0,
                            MODE_MASK, seed=1000 + lg))
    return out


def all_cases() -> List[Case]:
    return (tiny_cases() + moe_router_cases() + [class_logit_case(), expert_choice_case(), pruning_case()]
            + shape_sweep_cases())
