"""Spatial decomposition on one GPU: two slabs with ghost atoms reproduce the undivided evaluation.

Section 4.4 scales the potential by domain decomposition (sub-domains exchange ghost atoms and send the forces on them
back).  The primitive that needs is a context whose central atoms are a subset of the atoms it lists; here a periodic
box is cut into two slabs along x, each slab is evaluated in its own context with its halo of ghosts, the ghosts'
reaction forces are added back where they belong on the host, and the sum is compared with the single-context result
and with the oracle."""
import numpy as np
import pytest

import oracle
import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("precision", [0, 1])
def test_two_slabs_with_ghosts_sum_to_the_undivided_evaluation(precision):
    import paper_2608_16329_b200 as mlip
    w = wl.make_workload(5, n_cells=12)                       # 6,912 atoms, box 43.2 Angstrom
    enc, head = wl.workload_weights(5, w.n_species)
    r_list = w.r_cut + 1.0

    def fresh():
        return mlip.Potential(w.n_species, w.r_cut, 1.0, enc, head, w.masses, precision=precision)

    whole = fresh()
    whole.build_neighbors(w.pos, w.species, w.box)
    ref_gpu = whole.compute(want_e_atom=True)
    whole.sync_status()

    forces = np.zeros((w.n_atoms, 3))
    e_atom = np.zeros(w.n_atoms)
    energy, virial = 0.0, np.zeros(9)
    n_ghosts = 0
    for rank in range(2):
        dom = mlip.decomposition.slab_domain(w.pos, w.species, w.box, rank, 2, halo=r_list)
        idx, n_owned = dom.index, dom.n_owned
        n_ghosts += idx.size - n_owned
        pot = fresh()
        pot.build_neighbors(dom.pos, dom.species, dom.box, n_owned=n_owned)
        out = pot.compute(want_e_atom=True)
        pot.sync_status()
        f = out["forces"].cpu().numpy().astype(np.float64)
        mlip.decomposition.scatter_forces(dom, f, forces)      # owned parts and the ghosts' reaction forces, back home
        ea = out["e_atom"].cpu().numpy().astype(np.float64)
        assert np.all(ea[n_owned:] == 0.0)
        e_atom[idx[:n_owned]] = ea[:n_owned]
        energy += float(out["energy"].cpu())
        virial += out["virial"].cpu().numpy()
        with pytest.raises(mlip.MlipError) as err:            # the owner integrates, not the ghost context
            pot.step(1, 1.0, 0)
        assert err.value.code == mlip.binding.CODES["MLIP_ERR_UNSUPPORTED"]
        pot.close()
    assert n_ghosts > 0.5 * w.n_atoms                          # the halos are a large part of such small slabs

    model = oracle.Model(w.n_species, w.r_cut, enc, head)
    ref = oracle.evaluate(model, w.pos, w.species, w.box)
    e_tol, f_tol, ea_tol, xi_tol = (1e-10, 2e-9, 1e-9, 1e-9) if precision == 1 else (1e-6, 1e-4, 2e-5, 1e-5)
    assert abs(energy - ref["energy"]) <= e_tol * abs(ref["energy"])
    assert np.abs(forces - ref["forces"]).max() <= f_tol
    assert np.abs(e_atom - ref["e_atom"]).max() <= ea_tol * max(1.0, np.abs(ref["e_atom"]).max())
    assert np.abs(virial.reshape(3, 3) - ref["virial"]).max() <= xi_tol * np.abs(ref["virial"]).max()
    # and against the undivided run of the same kernels (same arithmetic per pair: only summation order differs)
    tight = 1e-9 if precision == 1 else 2e-5
    assert np.abs(forces - ref_gpu["forces"].cpu().numpy()).max() <= tight
    assert abs(energy - float(ref_gpu["energy"].cpu())) <= (1e-12 if precision == 1 else 1e-7) * abs(energy)


def test_ghost_positions_are_refreshed_through_set_positions():
    """Between list builds a domain receives new ghost (and owned) coordinates; the lists stay."""
    import paper_2608_16329_b200 as mlip
    w = wl.make_workload(5, n_cells=12)
    enc, head = wl.workload_weights(5, w.n_species)
    r_list = w.r_cut + 1.0
    rng = np.random.default_rng(4)
    moved = w.pos + rng.uniform(-0.15, 0.15, w.pos.shape)
    moved -= np.floor(moved / w.box) * w.box
    dom = mlip.decomposition.slab_domain(w.pos, w.species, w.box, 0, 2, halo=r_list)
    idx, n_owned = dom.index, dom.n_owned
    pot = mlip.Potential(w.n_species, w.r_cut, 1.0, enc, head, w.masses)
    pot.build_neighbors(dom.pos, dom.species, dom.box, n_owned=n_owned)
    # the same atoms at their new places, in the slab's frame (an atom that crossed the periodic boundary of the whole
    # box keeps its place next to the slab)
    pot.set_positions(mlip.decomposition.to_local(dom, moved, w.box))
    out = pot.compute(want_e_atom=True)
    pot.sync_status()
    model = oracle.Model(w.n_species, w.r_cut, enc, head)
    ref = oracle.sampled(model, moved, w.species, w.box, idx[:64])
    assert np.abs(out["e_atom"][:64].cpu().numpy() - ref["e_atom"]).max() <= 2e-5 * max(1.0, np.abs(ref["e_atom"]).max())
    nl = oracle.neighbors(moved, w.species, w.n_species, w.box, w.r_cut, rows=idx[:n_owned])
    ref_dom = oracle.compute(model, moved, w.species, w.box, nl)           # forces exerted by this domain's central atoms
    f = out["forces"].cpu().numpy().astype(np.float64)
    assert np.abs(f - ref_dom["forces"][idx]).max() <= 1e-4
    assert abs(float(out["energy"].cpu()) - ref_dom["energy"]) <= 1e-6 * abs(ref_dom["energy"])
