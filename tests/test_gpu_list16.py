"""The compact list format (mlip_config.list_format = 1: 16-bit cell-relative codes, half the bytes of the int32 lists):
same lists, same results, smaller footprint."""
import numpy as np
import pytest

import oracle
import workloads as wl
from helpers import canonical_equal, make_pair

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cfg,n_cells,skin", [(1, 6, 1.0), (2, 8, 1.0), (3, 6, 1.0), (4, 10, 1.0), (5, 7, 1.0)])
def test_compact_lists_export_the_same_canonical_lists(cfg, n_cells, skin):
    w, model, pot = make_pair(cfg, n_cells, skin, list_format=1)
    pot.build_neighbors(w.pos, w.species, w.box)
    seg, nbr = pot.neighbors()
    pot.sync_status()
    nl = oracle.neighbors(w.pos, w.species, w.n_species, w.box, w.r_cut + w.skin)
    assert canonical_equal(nl, seg, nbr)


@pytest.mark.parametrize("precision", [0, 1])
@pytest.mark.parametrize("cfg,n_cells", [(5, 7), (3, 6), (4, 10)])
def test_compact_lists_give_the_oracles_energies_and_forces(cfg, n_cells, precision):
    w, model, pot = make_pair(cfg, n_cells, 1.0, precision=precision, list_format=1)
    pot.build_neighbors(w.pos, w.species, w.box)
    out = pot.compute(want_e_atom=True)
    pot.sync_status()
    ref = oracle.evaluate(model, w.pos, w.species, w.box)
    e_tol, f_tol, ea_tol = (1e-10, 2e-9, 1e-9) if precision == 1 else (1e-6, 1e-4, 2e-5)
    assert abs(float(out["energy"].cpu()) - ref["energy"]) <= e_tol * abs(ref["energy"])
    assert np.abs(out["forces"].cpu().numpy() - ref["forces"]).max() <= f_tol
    assert np.abs(out["e_atom"].cpu().numpy() - ref["e_atom"]).max() <= ea_tol * max(1.0, np.abs(ref["e_atom"]).max())


def test_both_formats_give_bit_identical_results_and_trajectories_in_deterministic_mode():
    """The two formats hold the same entries in the same order, so with the integer scatter everything agrees bit for bit
    -- over 55,296 atoms (every warp group prefetches codes and cell bases for many tiles) and through in-step rebuilds."""
    import paper_2608_16329_b200 as mlip
    w = wl.make_workload(5, n_cells=24)
    enc, head = wl.workload_weights(5, 6)
    runs = []
    for fmt in (0, 1):
        pot = mlip.Potential(6, w.r_cut, 1.0, enc, head, w.masses, force_mode=1, list_format=fmt)
        pot.build_neighbors(w.pos, w.species, w.box)
        pot.set_velocities(w.vel)
        first = pot.compute(want_e_atom=True)
        pot.step(12, 1.0, 5)
        assert pot.sync_status(raise_on_error=False) == 0
        pos, vel, _ = pot.state()
        runs.append((first, pos.cpu().numpy(), vel.cpu().numpy(), mlip.mlip_resident_bytes(pot.ctx), mlip.mlip_get_counters(pot.ctx)))
        pot.close()
    a, b = runs
    for key in ("energy", "forces", "virial", "e_atom"):
        assert a[0][key].cpu().numpy().tobytes() == b[0][key].cpu().numpy().tobytes(), key
    assert a[1].tobytes() == b[1].tobytes() and a[2].tobytes() == b[2].tobytes()
    assert a[4]["list_entries"] == b[4]["list_entries"]
    saved = (a[3] - b[3]) / w.n_atoms
    print(f"resident bytes per atom: {a[3] / w.n_atoms:.0f} (int32 lists) -> {b[3] / w.n_atoms:.0f} (16-bit codes)")
    assert 230 < saved < 300                       # ~134 entries x 2 bytes less 4 bytes per atom for the cell ids (+ spare capacity)
    model = oracle.Model(6, w.r_cut, enc, head)
    rows = np.arange(0, w.n_atoms, 27)
    ref = oracle.sampled(model, w.pos, w.species, w.box, rows)
    assert np.abs(b[0]["forces"].cpu().numpy()[rows] - ref["forces"]).max() <= 1e-4
    assert np.abs(b[0]["e_atom"].cpu().numpy()[rows] - ref["e_atom"]).max() <= 2e-5 * max(1.0, np.abs(ref["e_atom"]).max())


def test_compact_lists_after_in_step_rebuilds_are_the_lists_of_the_current_positions():
    w, model, pot = make_pair(3, 16, 1.0, list_format=1)
    pot.build_neighbors(w.pos, w.species, w.box)
    pot.set_velocities(w.vel)
    pot.step(20, 1.0, 10)
    assert pot.sync_status(raise_on_error=False) == 0 and pot.rebuilds() == 3
    pos, _, _ = pot.state()
    seg, nbr = pot.neighbors()
    nl = oracle.neighbors(pos.cpu().numpy(), w.species, w.n_species, w.box, w.r_cut + w.skin)
    assert canonical_equal(nl, seg, nbr)


def test_grids_with_fewer_than_three_cells_fall_back_to_plain_indices():
    w, model, pot = make_pair(1, 4, 0.0, list_format=1)           # 14.4 Angstrom box, 6 Angstrom list radius: 2 cells per edge
    pot.build_neighbors(w.pos, w.species, w.box)
    out = pot.compute()
    pot.sync_status()
    ref = oracle.evaluate(model, w.pos, w.species, w.box)
    assert np.abs(out["forces"].cpu().numpy() - ref["forces"]).max() <= 1e-4
    seg, nbr = pot.neighbors()
    assert canonical_equal(oracle.neighbors(w.pos, w.species, w.n_species, w.box, w.r_cut), seg, nbr)
    # the same context, a larger system: the format switches to codes
    w2 = wl.make_workload(1, n_cells=7)
    pot.build_neighbors(w2.pos, w2.species, w2.box)
    out2 = pot.compute()
    pot.sync_status()
    ref2 = oracle.evaluate(model, w2.pos, w2.species, w2.box)
    assert np.abs(out2["forces"].cpu().numpy() - ref2["forces"]).max() <= 1e-4


def test_compact_lists_with_ghost_atoms_and_lists_longer_than_the_hit_buffer():
    import paper_2608_16329_b200 as mlip
    w, model, pot = make_pair(1, 8, 2.5, list_format=1)             # ~220 entries per atom
    pot.build_neighbors(w.pos, w.species, w.box)
    pot.set_velocities(w.vel)
    pot.step(4, 1.0, 2)
    assert pot.sync_status(raise_on_error=False) == 0
    pos, _, _ = pot.state()
    seg, nbr = pot.neighbors()
    assert canonical_equal(oracle.neighbors(pos.cpu().numpy(), w.species, w.n_species, w.box, w.r_cut + 2.5), seg, nbr)
    w5 = wl.make_workload(5, n_cells=12)
    enc, head = wl.workload_weights(5, 6)
    dom = mlip.decomposition.slab_domain(w5.pos, w5.species, w5.box, 0, 2, halo=7.0)
    dpot = mlip.Potential(6, 6.0, 1.0, enc, head, w5.masses, list_format=1)
    dpot.build_neighbors(dom.pos, dom.species, dom.box, n_owned=dom.n_owned)
    out = dpot.compute()
    dpot.sync_status()
    m5 = oracle.Model(6, 6.0, enc, head)
    nl = oracle.neighbors(w5.pos, w5.species, 6, w5.box, 6.0, rows=dom.index[:dom.n_owned])
    ref = oracle.compute(m5, w5.pos, w5.species, w5.box, nl)
    assert np.abs(out["forces"].cpu().numpy() - ref["forces"][dom.index]).max() <= 1e-4
