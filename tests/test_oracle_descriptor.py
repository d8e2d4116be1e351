"""Pins for moments, invariants, energies, forces and virial (Eq. 4-10)."""
from math import factorial

import numpy as np
from scipy.special import eval_legendre
from scipy.stats import special_ortho_group

import oracle
import workloads as wl

BIG = np.array([60.0, 60.0, 60.0])


def _c(l):
    return factorial(l) / (np.prod(np.arange(2 * l - 1, 0, -2)) if l else 1.0)


def _cluster(rng, n, n_species, spread=3.0):
    """n atoms around the box centre, no periodic image within reach."""
    while True:
        pos = 30.0 + rng.uniform(-spread, spread, size=(n, 3))
        d = np.linalg.norm(pos[:, None] - pos[None], axis=-1) + 10 * np.eye(n)
        if d.min() > 1.2:
            return pos, rng.integers(0, n_species, n).astype(np.int32)


def _all(model, pos, species, box=BIG):
    return oracle.compute(model, pos, species, box,
                          oracle.neighbors(pos, species, model.n_species, box, model.r_cut), want_G=True)


def test_invariants_equal_three_body_legendre_sums():
    """G_lk = sum_jj' g_jk g_j'k c_l P_l(cos theta_jj'), independent of any basis choice."""
    rng = np.random.default_rng(0)
    enc, head = wl.make_weights(3, seed=3)
    m = oracle.Model(3, 6.0, enc, head)
    pos, sp = _cluster(rng, 9, 3)
    out = _all(m, pos, sp)
    for i in range(9):
        others = [j for j in range(9) if j != i and np.linalg.norm(pos[j] - pos[i]) < 6.0]
        assert len(others) >= 4
        g = np.array([oracle.radial(m, sp[i], sp[j], np.linalg.norm(pos[j] - pos[i]))[0] for j in others])
        u = np.array([(pos[j] - pos[i]) / np.linalg.norm(pos[j] - pos[i]) for j in others])
        cos = np.clip(u @ u.T, -1, 1)
        for l in range(4):
            want = np.einsum("jk,jm,mk->k", g, _c(l) * eval_legendre(l, cos), g) if l else g.sum(0)
            got = out["G"][i, l * 32:(l + 1) * 32]
            assert np.abs(got - want).max() < 1e-11 * max(1.0, np.abs(want).max())


def test_dimer():
    enc, head = wl.make_weights(2, seed=4)
    m = oracle.Model(2, 6.0, enc, head)
    pos = np.array([[30.0, 30.0, 30.0], [31.1, 32.3, 28.9]])
    sp = np.array([0, 1], dtype=np.int32)
    out = _all(m, pos, sp)
    r = np.linalg.norm(pos[1] - pos[0])
    g01, g10 = oracle.radial(m, 0, 1, r)[0], oracle.radial(m, 1, 0, r)[0]
    for l in range(4):
        assert np.abs(out["G"][0, l * 32:(l + 1) * 32] - (_c(l) * g01 ** 2 if l else g01)).max() < 1e-12
        assert np.abs(out["G"][1, l * 32:(l + 1) * 32] - (_c(l) * g10 ** 2 if l else g10)).max() < 1e-12
    F = out["forces"]
    assert np.abs(F[0] + F[1]).max() < 1e-12                       # equal and opposite
    axis = (pos[1] - pos[0]) / r
    assert np.abs(F[0] - (F[0] @ axis) * axis).max() < 1e-12       # central
    # magnitude: -dE/dr by finite difference along the bond
    def e_at(rr):
        p = np.array([pos[0], pos[0] + axis * rr])
        return _all(m, p, sp)["energy"]
    fd = -(e_at(r + 1e-5) - e_at(r - 1e-5)) / 2e-5
    assert abs(F[1] @ axis - fd) < 1e-7 * max(1.0, abs(fd))


def test_lmax0_is_a_pair_functional():
    """With l_max = 0: E_i = R(sum_j g(r_ij)) and forces follow the embedded-atom formula."""
    rng = np.random.default_rng(5)
    enc, head = wl.make_weights(2, seed=6, l_max=0)
    m = oracle.Model(2, 6.0, enc, head, l_max=0)
    pos, sp = _cluster(rng, 7, 2)
    out = _all(m, pos, sp)
    n = len(pos)
    rho = np.zeros((n, 32)); dE = np.zeros((n, 32))
    for i in range(n):
        for j in range(n):
            if j != i:
                rho[i] += oracle.radial(m, sp[i], sp[j], np.linalg.norm(pos[j] - pos[i]))[0]
        e, dE[i] = oracle.head(m, sp[i], rho[i], want_grad=True)
        assert abs(e - out["e_atom"][i]) < 1e-12
    F = np.zeros((n, 3))
    for a in range(n):
        for b in range(n):
            if a == b:
                continue
            d = pos[b] - pos[a]; r = np.linalg.norm(d)
            slope = dE[a] @ oracle.radial(m, sp[a], sp[b], r)[1] + dE[b] @ oracle.radial(m, sp[b], sp[a], r)[1]
            F[a] += slope * d / r
    assert np.abs(F - out["forces"]).max() < 1e-11


def test_forces_match_central_differences_of_the_energy():
    w = wl.make_workload(1)
    enc, head = wl.workload_weights(1, 6)
    m = oracle.Model(6, 6.0, enc, head)
    base = oracle.evaluate(m, w.pos, w.species, w.box)
    assert np.abs(base["forces"].sum(0)).max() < 1e-10                       # Newton's third law
    h = 1e-5
    for a, b in [(0, 0), (3, 1), (101, 2), (255, 0)]:
        p = w.pos.copy(); p[a, b] += h
        ep = oracle.evaluate(m, p, w.species, w.box)["energy"]
        p[a, b] -= 2 * h
        em = oracle.evaluate(m, p, w.species, w.box)["energy"]
        assert abs(-(ep - em) / (2 * h) - base["forces"][a, b]) < 2e-7


def test_virial_matches_strain_derivative_periodic():
    """Xi_ab = -dE/d eps_ab under x -> (I + eps) x of atoms and box (diagonal strains, periodic)."""
    w = wl.make_workload(1)
    enc, head = wl.workload_weights(1, 6)
    m = oracle.Model(6, 6.0, enc, head)
    xi = oracle.evaluate(m, w.pos, w.species, w.box)["virial"]
    assert np.abs(xi - xi.T).max() < 1e-9
    h = 1e-6
    for a in range(3):
        es = []
        for sgn in (+1, -1):
            s = np.ones(3); s[a] += sgn * h
            es.append(oracle.evaluate(m, w.pos * s, w.species, w.box * s)["energy"])
        assert abs(-(es[0] - es[1]) / (2 * h) - xi[a, a]) < 1e-5 * abs(xi[a, a])


def test_virial_matches_strain_derivative_with_shear():
    rng = np.random.default_rng(8)
    enc, head = wl.make_weights(2, seed=9)
    m = oracle.Model(2, 6.0, enc, head)
    pos, sp = _cluster(rng, 8, 2)
    xi = _all(m, pos, sp)["virial"]
    c = pos.mean(0)
    h = 1e-6
    for a in range(3):
        for b in range(3):
            es = []
            for sgn in (+1, -1):
                eps = np.zeros((3, 3)); eps[a, b] = sgn * h
                es.append(_all(m, c + (pos - c) @ (np.eye(3) + eps).T, sp)["energy"])
            assert abs(-(es[0] - es[1]) / (2 * h) - xi[a, b]) < 1e-6 * max(1.0, np.abs(xi).max())


def test_translation_rotation_permutation_invariance():
    w = wl.make_workload(1)
    enc, head = wl.workload_weights(1, 6)
    m = oracle.Model(6, 6.0, enc, head)
    base = oracle.evaluate(m, w.pos, w.species, w.box)
    e0 = base["energy"]
    # rigid translation with periodic wrap
    p = w.pos + np.array([1.234, -7.7, 20.01]); p -= np.floor(p / w.box) * w.box
    t = oracle.evaluate(m, p, w.species, w.box)
    assert abs(t["energy"] - e0) < 1e-9 and np.abs(t["forces"] - base["forces"]).max() < 1e-9
    # 90 degree rotation about z maps the cubic periodic box onto itself
    p = np.stack([-w.pos[:, 1], w.pos[:, 0], w.pos[:, 2]], axis=1); p -= np.floor(p / w.box) * w.box
    r = oracle.evaluate(m, p, w.species, w.box)
    assert abs(r["energy"] - e0) < 1e-9
    assert np.abs(r["forces"] - np.stack([-base["forces"][:, 1], base["forces"][:, 0], base["forces"][:, 2]], 1)).max() < 1e-9
    # relabelling atoms (a permutation of the storage order) changes nothing
    perm = np.random.default_rng(0).permutation(w.n_atoms)
    q = oracle.evaluate(m, w.pos[perm], w.species[perm], w.box)
    assert abs(q["energy"] - e0) < 1e-9 and np.abs(q["forces"] - base["forces"][perm]).max() < 1e-9
    # exchanging the positions of two atoms of one species is such a relabelling; of two species it is not
    same = np.flatnonzero(w.species == w.species[0])[:2]
    diff = np.array([0, np.flatnonzero(w.species != w.species[0])[0]])
    for pair, invariant in ((same, True), (diff, False)):
        p = w.pos.copy(); p[pair] = p[pair[::-1]]
        e = oracle.evaluate(m, p, w.species, w.box)["energy"]
        assert (abs(e - e0) < 1e-9) == invariant


def test_arbitrary_rotation_of_an_isolated_cluster():
    rng = np.random.default_rng(11)
    enc, head = wl.make_weights(3, seed=12)
    m = oracle.Model(3, 6.0, enc, head)
    pos, sp = _cluster(rng, 10, 3)
    a = _all(m, pos, sp)
    R = special_ortho_group.rvs(3, random_state=13)
    c = pos.mean(0)
    b = _all(m, c + (pos - c) @ R.T, sp)
    assert abs(a["energy"] - b["energy"]) < 1e-10
    assert np.abs(a["G"] - b["G"]).max() < 1e-10
    assert np.abs(a["forces"] @ R.T - b["forces"]).max() < 1e-10
    assert np.abs(R @ a["virial"] @ R.T - b["virial"]).max() < 1e-9


def test_skin_shell_contributes_nothing():
    w = wl.make_workload(1)
    enc, head = wl.workload_weights(1, 6)
    m = oracle.Model(6, 6.0, enc, head)
    a = oracle.evaluate(m, w.pos, w.species, w.box)
    b = oracle.evaluate(m, w.pos, w.species, w.box, r_list=7.1)
    assert abs(a["energy"] - b["energy"]) < 1e-10 and np.abs(a["forces"] - b["forces"]).max() < 1e-11


def test_sampled_evaluation_equals_full_evaluation():
    w = wl.make_workload(5, n_cells=5)
    enc, head = wl.workload_weights(5, 6)
    m = oracle.Model(6, 6.0, enc, head)
    full = oracle.evaluate(m, w.pos, w.species, w.box)
    atoms = np.array([0, 77, 499])
    s = oracle.sampled(m, w.pos, w.species, w.box, atoms)
    assert np.abs(s["e_atom"] - full["e_atom"][atoms]).max() < 1e-12
    assert np.abs(s["forces"] - full["forces"][atoms]).max() < 1e-11


# ---- canonical (reducible) angular basis: all monomials of each degree, C_l = multinomial multiplicities (Section 3.3, Eq. 5)

def test_canonical_basis_has_the_dimensions_of_eq_11_and_its_metric_is_the_multinomial_count():
    from oracle import harmonic_projection as hp
    enc, head = wl.make_weights(1, seed=2)
    for l_max, d in [(0, 1), (1, 4), (2, 10), (3, 20), (4, 35), (5, 56)]:
        assert hp.reducible_dim(l_max) == d
        assert hp.metric_diagonal(l_max, 1).size == d
    # (x + y + z)^l expands with exactly these multiplicities
    for l in range(6):
        assert hp.multinomial_metric(l).sum() == 3 ** l
    m = oracle.Model(1, 6.0, enc, head, basis=1)
    assert m.d == 20
    h, dh = oracle.angular(m, np.array([0.6, 0.0, 0.8]))
    # degree-2 block in the order x^2, xy, xz, y^2, yz, z^2 (the paper's example)
    assert np.allclose(h[4:10], [0.36, 0.0, 0.48, 0.0, 0.0, 0.64])


def test_canonical_invariants_are_sums_of_powers_of_the_cosine():
    """With C_l = multiplicities, p^T C_l p = sum_jj' g_jk g_j'k (u_j . u_j')^l by the multinomial theorem."""
    rng = np.random.default_rng(10)
    enc, head = wl.make_weights(3, seed=3)
    m = oracle.Model(3, 6.0, enc, head, basis=1)
    pos, sp = _cluster(rng, 9, 3)
    out = _all(m, pos, sp)
    for i in range(9):
        others = [j for j in range(9) if j != i and np.linalg.norm(pos[j] - pos[i]) < 6.0]
        g = np.array([oracle.radial(m, sp[i], sp[j], np.linalg.norm(pos[j] - pos[i]))[0] for j in others])
        u = np.array([(pos[j] - pos[i]) / np.linalg.norm(pos[j] - pos[i]) for j in others])
        cos = u @ u.T
        for l in range(4):
            want = np.einsum("jk,jm,mk->k", g, cos ** l, g) if l else g.sum(0)
            got = out["G"][i, l * 32:(l + 1) * 32]
            assert np.abs(got - want).max() < 1e-11 * max(1.0, np.abs(want).max())


def test_canonical_and_irreducible_invariants_differ_by_lower_orders():
    """cos^2 = (cos^2 - 1/3) + 1/3 and cos^3 = (cos^3 - 3/5 cos) + 3/5 cos: the canonical order-2 invariant repeats the
    scalar one (squared), the order-3 invariant repeats order 1 -- the redundancy the irreducible projection removes."""
    rng = np.random.default_rng(11)
    enc, head = wl.make_weights(2, seed=8)
    pos, sp = _cluster(rng, 10, 2)
    irr = _all(oracle.Model(2, 6.0, enc, head), pos, sp)["G"]
    can = _all(oracle.Model(2, 6.0, enc, head, basis=1), pos, sp)["G"]
    k = 32
    assert np.allclose(can[:, :2 * k], irr[:, :2 * k], rtol=1e-12, atol=1e-12)
    assert np.allclose(can[:, 2 * k:3 * k], irr[:, 2 * k:3 * k] + irr[:, :k] ** 2 / 3.0, rtol=1e-11, atol=1e-11)
    assert np.allclose(can[:, 3 * k:], irr[:, 3 * k:] + 0.6 * irr[:, k:2 * k], rtol=1e-11, atol=1e-11)
    assert np.abs(can[:, 2 * k:] - irr[:, 2 * k:]).max() > 1e-3          # the two descriptors really differ


def test_canonical_forces_match_central_differences_and_energy_is_rotation_invariant():
    rng = np.random.default_rng(12)
    enc, head = wl.make_weights(2, seed=9, enc_out_scale=0.3)
    m = oracle.Model(2, 6.0, enc, head, basis=1)
    pos, sp = _cluster(rng, 7, 2)
    out = _all(m, pos, sp)
    eps = 1e-5
    for a in (0, 3, 6):
        for b in range(3):
            p1, p2 = pos.copy(), pos.copy()
            p1[a, b] += eps
            p2[a, b] -= eps
            fd = -(_all(m, p1, sp)["energy"] - _all(m, p2, sp)["energy"]) / (2 * eps)
            assert abs(fd - out["forces"][a, b]) < 1e-7 * max(1.0, np.abs(out["forces"]).max())
    assert np.abs(out["forces"].sum(0)).max() < 1e-10 * max(1.0, np.abs(out["forces"]).max())
    rot = special_ortho_group.rvs(3, random_state=5)
    turned = 30.0 + (pos - 30.0) @ rot.T
    assert abs(_all(m, turned, sp)["energy"] - out["energy"]) < 1e-10 * abs(out["energy"])
