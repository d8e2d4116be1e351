"""Pins for the oracle's angular basis (Eq. 3, Eq. 11, Section 3.3.1)."""
from math import factorial

import numpy as np
import pytest
from scipy.special import eval_legendre
from scipy.stats import ortho_group, special_ortho_group

import oracle
from oracle import harmonic_projection as hp
from conftest import golden_lines


def _model(l_max, q=None):
    return oracle.Model(1, 6.0, np.zeros(4), np.zeros(4), k=1, l_max=l_max, enc_hidden=1, enc_layers=1,
                        head_hidden=1, head_layers=1, q=q)


def _unit(rng, n):
    v = rng.standard_normal((n, 3))
    return v / np.linalg.norm(v, axis=1, keepdims=True)


def test_dimension_table_matches_paper():
    for line in golden_lines("angular_dims.txt"):
        l_max, original, reduced = map(int, line.split())
        assert hp.reducible_dim(l_max) == original
        assert hp.reducible_dim(l_max) == (l_max + 1) * (l_max + 2) * (l_max + 3) // 6   # Eq. 11 closed form
        assert hp.reduced_dim(l_max) == reduced
        assert _model(l_max).d == reduced


def test_monomial_order_matches_paper_examples():
    for line in golden_lines("monomial_order.txt"):
        l, triples = line.split(":")
        want = [tuple(int(ch) for ch in t) for t in triples.split()]
        assert hp.monomial_exponents(int(l)) == want


@pytest.mark.parametrize("l", range(6))
def test_q_satisfies_both_constraints(l):
    q = hp.q_matrix(l)
    assert q.shape == (2 * l + 1, (l + 1) * (l + 2) // 2)
    L = hp.laplacian_matrix(l)
    if L.size:
        assert np.abs(L @ q.T).max() < 1e-12
    d = hp.multinomial_metric(l)
    assert d[0] == 1 and d.sum() == 3 ** l            # multinomial theorem: (1+1+1)^l
    assert np.abs((q / d) @ q.T - np.eye(2 * l + 1)).max() < 1e-12


def test_laplacian_matrix_on_known_polynomials():
    # x^2 + y^2 + z^2 has Laplacian 6; x^2 - y^2 and xy are harmonic.
    e = hp.monomial_exponents(2)
    coef = lambda terms: np.array([terms.get(t, 0.0) for t in e])
    L = hp.laplacian_matrix(2)
    assert np.allclose(L @ coef({(2, 0, 0): 1, (0, 2, 0): 1, (0, 0, 2): 1}), [6.0])
    assert np.allclose(L @ coef({(2, 0, 0): 1, (0, 2, 0): -1}), [0.0])
    assert np.allclose(L @ coef({(1, 1, 0): 1}), [0.0])
    # x^3: Laplacian 6x (degree-1 order is x, y, z)
    e3 = hp.monomial_exponents(3)
    c3 = np.array([1.0 if t == (3, 0, 0) else 0.0 for t in e3])
    assert np.allclose(hp.laplacian_matrix(3) @ c3, [6.0, 0.0, 0.0])


@pytest.mark.parametrize("l_max", [3, 5])
def test_addition_theorem(l_max):
    """h_l(a) . h_l(b) = l!/(2l-1)!! P_l(a.b): fixes span, scale and harmonicity of every block."""
    rng = np.random.default_rng(1)
    m = _model(l_max)
    a, b = _unit(rng, 20), _unit(rng, 20)
    for ua, ub in zip(a, b):
        ha, _ = oracle.angular(m, ua)
        hb, _ = oracle.angular(m, ub)
        row = 0
        for l in range(l_max + 1):
            dfact = np.prod(np.arange(2 * l - 1, 0, -2)) if l else 1.0
            want = factorial(l) / dfact * eval_legendre(l, float(ua @ ub))
            got = ha[row:row + 2 * l + 1] @ hb[row:row + 2 * l + 1]
            assert abs(got - want) < 1e-12
            row += 2 * l + 1


def test_low_orders_closed_form():
    rng = np.random.default_rng(2)
    m = _model(3)
    for u in _unit(rng, 5):
        h, _ = oracle.angular(m, u)
        assert abs(h[0] - 1.0) < 1e-14                       # l = 0 is the constant 1
        assert abs(h[1:4] @ h[1:4] - 1.0) < 1e-13            # l = 1 is a rotation of (x, y, z)
        assert abs(h[4:9] @ h[4:9] - 2.0 / 3.0) < 1e-13      # l = 2: trace removed
        assert abs(h[9:16] @ h[9:16] - 2.0 / 5.0) < 1e-13


def test_blocks_transform_equivariantly():
    """Rotating the direction mixes each block by an orthogonal matrix (Section 3.1.1)."""
    rng = np.random.default_rng(3)
    m = _model(3)
    R = special_ortho_group.rvs(3, random_state=4)
    U = _unit(rng, 40)
    H = np.array([oracle.angular(m, u)[0] for u in U])
    HR = np.array([oracle.angular(m, R @ u)[0] for u in U])
    row = 0
    for l in range(4):
        blk = slice(row, row + 2 * l + 1)
        M, res, *_ = np.linalg.lstsq(H[:, blk], HR[:, blk], rcond=None)
        assert np.abs(H[:, blk] @ M - HR[:, blk]).max() < 1e-12
        assert np.abs(M @ M.T - np.eye(2 * l + 1)).max() < 1e-12
        row += 2 * l + 1


def test_derivative_matches_finite_difference():
    rng = np.random.default_rng(5)
    m = _model(3)
    for u in rng.standard_normal((5, 3)):       # u free (not normalised): dh is the plain polynomial gradient
        _, dh = oracle.angular(m, u)
        for b in range(3):
            e = np.zeros(3); e[b] = 1e-6
            fd = (oracle.angular(m, u + e)[0] - oracle.angular(m, u - e)[0]) / 2e-6
            assert np.abs(fd - dh[:, b]).max() < 1e-8


def test_invariants_do_not_depend_on_the_choice_of_q():
    """Q_l is fixed only up to an orthogonal mixing of rows; energies must not notice."""
    import workloads as wl
    w = wl.make_workload(1, n_cells=4)
    enc, head = wl.workload_weights(1, 6)
    base = oracle.Model(6, 6.0, enc, head)
    q_mixed = np.concatenate([((ortho_group.rvs(2 * l + 1, random_state=10 + l) if l else np.eye(1))
                               @ hp.q_matrix(l)).ravel() for l in range(4)])
    mixed = oracle.Model(6, 6.0, enc, head, q=q_mixed)
    rows = np.arange(8)
    nl = oracle.neighbors(w.pos, w.species, 6, w.box, 6.0, rows=rows)
    a = oracle.compute(base, w.pos, w.species, w.box, nl, want_G=True)
    b = oracle.compute(mixed, w.pos, w.species, w.box, nl, want_G=True)
    assert np.abs(a["G"] - b["G"]).max() < 1e-11
    assert np.abs(a["forces"] - b["forces"]).max() < 1e-11
