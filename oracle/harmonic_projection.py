"""Oracle (test infrastructure only): the irreducible harmonic projection Q_l.

Follows Section 3.3.1 ("Irreducible Harmonic Projection"): for each angular
order l the degree-l Cartesian monomials of the unit vector are left-multiplied
by a (2l+1) x C(l+2,2) matrix Q_l fixed by the two constraints

    L_l Q_l^T = 0            (rows are harmonic: the Laplacian annihilates them)
    Q_l D_l^{-1} Q_l^T = I   (rows are orthonormal under the multinomial metric)

where L_l is the Laplacian from degree-l to degree-(l-2) homogeneous
polynomials and D_l = diag(l! / (ax! ay! az!)).  D_l has one entry per monomial
(the paper's "l x l" is read as C(l+2,2) x C(l+2,2)).

Monomials are ordered as in the paper's examples below Eq. 11:
[x, y, z] and [x^2, xy, xz, y^2, yz, z^2] - descending power of x, then of y.

Q_l is unique only up to an orthogonal mixing of its rows; every quantity the
method exposes (the invariants of Eq. 5 and everything after) is independent of
that choice.  `q_matrix` makes one deterministic choice.
"""
from __future__ import annotations

from math import factorial

import numpy as np
import scipy.linalg


def monomial_exponents(l: int) -> list[tuple[int, int, int]]:
    return [(ax, ay, l - ax - ay) for ax in range(l, -1, -1) for ay in range(l - ax, -1, -1)]


def n_monomials(l: int) -> int:
    return (l + 1) * (l + 2) // 2


def reducible_dim(l_max: int) -> int:
    """Eq. 11: cumulative number of Cartesian monomials up to l_max."""
    return sum(n_monomials(l) for l in range(l_max + 1))


def reduced_dim(l_max: int) -> int:
    return sum(2 * l + 1 for l in range(l_max + 1))


def laplacian_matrix(l: int) -> np.ndarray:
    """L_l: coefficients of a degree-l polynomial -> coefficients of its Laplacian."""
    src = monomial_exponents(l)
    if l < 2:
        return np.zeros((0, len(src)))
    dst = {e: i for i, e in enumerate(monomial_exponents(l - 2))}
    L = np.zeros((len(dst), len(src)))
    for col, e in enumerate(src):
        for axis in range(3):
            if e[axis] >= 2:
                t = list(e)
                t[axis] -= 2
                L[dst[tuple(t)], col] += e[axis] * (e[axis] - 1)
    return L


def multinomial_metric(l: int) -> np.ndarray:
    return np.array([factorial(l) / (factorial(ax) * factorial(ay) * factorial(az))
                     for ax, ay, az in monomial_exponents(l)], dtype=np.float64)


def q_matrix(l: int) -> np.ndarray:
    """One solution of the two constraints, shape (2l+1, C(l+2,2))."""
    L = laplacian_matrix(l)
    n = n_monomials(l)
    basis = scipy.linalg.null_space(L).T if L.shape[0] else np.eye(n)   # step 1: harmonic rows
    assert basis.shape == (2 * l + 1, n)
    d_inv = 1.0 / multinomial_metric(l)
    gram = (basis * d_inv) @ basis.T                                      # step 2: orthonormalise
    chol = np.linalg.cholesky(gram)
    return np.linalg.solve(chol, basis)


def q_table(l_max: int) -> np.ndarray:
    """Q_0 .. Q_lmax flattened row-major and concatenated (the C core's input)."""
    return np.concatenate([q_matrix(l).ravel() for l in range(l_max + 1)])


def canonical_table(l_max: int) -> np.ndarray:
    """Identity blocks in place of Q_l: the canonical (reducible) basis keeps every degree-l monomial (Section 3.3)."""
    return np.concatenate([np.eye(n_monomials(l)).ravel() for l in range(l_max + 1)])


def metric_diagonal(l_max: int, basis: int) -> np.ndarray:
    """Diagonal of C_0 .. C_lmax of Eq. 5: ones for the irreducible basis, the multinomial multiplicities
    l! / (ax! ay! az!) for the canonical one."""
    if basis == 0:
        return np.ones(reduced_dim(l_max))
    return np.concatenate([multinomial_metric(l) for l in range(l_max + 1)])
