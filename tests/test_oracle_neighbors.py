"""Pins for the oracle's neighbor lists (Section 3.1.1: atoms within a cutoff)."""
import numpy as np
import pytest

import oracle
import workloads as wl

# textbook coordination shells: (squared distance in units of a^2, multiplicity)
FCC_SHELLS = [(0.5, 12), (1.0, 6), (1.5, 24), (2.0, 12), (2.5, 24), (3.0, 8), (3.5, 48), (4.0, 6)]
BCC_SHELLS = [(0.75, 8), (1.0, 6), (2.0, 12), (2.75, 24), (3.0, 8), (4.0, 6), (4.75, 24), (5.0, 24)]
SC_SHELLS = [(1, 6), (2, 12), (3, 8), (4, 6), (5, 24), (6, 24), (8, 12), (9, 30)]


def _shell_sum(shells, a, r):
    return sum(mult for d2, mult in shells if d2 * a * a < r * r)


@pytest.mark.parametrize("basis,a,n,shells", [
    (wl._FCC_BASIS, 3.6, 4, FCC_SHELLS), (wl._BCC_BASIS, 3.3, 5, BCC_SHELLS),
    (wl._FCC_BASIS, 4.05, 4, FCC_SHELLS), (wl._SC_BASIS, 20.0 ** (1 / 3), 6, SC_SHELLS)])
def test_perfect_lattice_shell_counts(basis, a, n, shells):
    pos = wl.lattice_sites((n, n, n), a, basis)
    box = np.full(3, n * a)
    species = np.zeros(len(pos), dtype=np.int32)
    for r in (6.0, 7.0):
        if box[0] < 2 * r:
            continue
        for method in ("brute", "cell"):
            nl = oracle.neighbors(pos, species, 1, box, r, method=method)
            counts = np.diff(nl.seg_ptr)
            assert counts.min() == counts.max() == _shell_sum(shells, a, r)


def test_expected_counts_of_the_workload_lattices():
    assert _shell_sum(FCC_SHELLS, 3.6, 6.0) == 78 and _shell_sum(FCC_SHELLS, 3.6, 7.0) == 134
    assert _shell_sum(BCC_SHELLS, 3.3, 6.0) == 58 and _shell_sum(BCC_SHELLS, 3.3, 7.0) == 64
    assert _shell_sum(FCC_SHELLS, 4.05, 6.0) == 54 and _shell_sum(FCC_SHELLS, 4.05, 7.0) == 78


def _check_canonical(nl, pos, species, n_species, box, r):
    n = len(pos)
    d = pos[None, :, :] - pos[:, None, :]
    d -= box * np.round(d / box)
    d2 = (d ** 2).sum(-1)
    for i in range(n):
        for s in range(n_species):
            seg = nl.nbr[nl.seg_ptr[i * n_species + s]:nl.seg_ptr[i * n_species + s + 1]]
            want = np.flatnonzero((d2[i] < r * r) & (species == s) & (np.arange(n) != i))
            assert np.array_equal(seg, want)


@pytest.mark.parametrize("cfg,n_cells,r", [(1, 4, 6.0), (1, 4, 7.2), (3, 4, 7.0), (4, 6, 7.0)])
def test_brute_force_equals_cell_list_and_numpy_definition(cfg, n_cells, r):
    w = wl.make_workload(cfg, n_cells=n_cells)
    b = oracle.neighbors(w.pos, w.species, w.n_species, w.box, r, method="brute")
    c = oracle.neighbors(w.pos, w.species, w.n_species, w.box, r, method="cell")
    assert np.array_equal(b.seg_ptr, c.seg_ptr) and np.array_equal(b.nbr, c.nbr)
    _check_canonical(b, w.pos, w.species, w.n_species, w.box, r)


def test_random_gas_with_non_cubic_box():
    rng = np.random.default_rng(3)
    box = np.array([15.0, 21.5, 29.0])
    pos = rng.uniform(0, 1, (700, 3)) * box
    species = rng.integers(0, 4, 700).astype(np.int32)
    b = oracle.neighbors(pos, species, 4, box, 7.0, method="brute")
    c = oracle.neighbors(pos, species, 4, box, 7.0, method="cell")
    assert np.array_equal(b.seg_ptr, c.seg_ptr) and np.array_equal(b.nbr, c.nbr)
    _check_canonical(c, pos, species, 4, box, 7.0)
    # symmetry: j lists i whenever i lists j
    pairs = set()
    for i in range(700):
        for j in c.nbr[c.seg_ptr[i * 4]:c.seg_ptr[i * 4 + 4]]:
            pairs.add((i, int(j)))
    assert all((j, i) in pairs for i, j in pairs)


def test_row_subset_matches_full_lists():
    w = wl.make_workload(5, n_cells=5)
    full = oracle.neighbors(w.pos, w.species, 6, w.box, 7.0)
    rows = np.array([3, 250, 499])
    sub = oracle.neighbors(w.pos, w.species, 6, w.box, 7.0, rows=rows)
    for q, i in enumerate(rows):
        for s in range(6):
            a = sub.nbr[sub.seg_ptr[q * 6 + s]:sub.seg_ptr[q * 6 + s + 1]]
            b = full.nbr[full.seg_ptr[i * 6 + s]:full.seg_ptr[i * 6 + s + 1]]
            assert np.array_equal(a, b)
