"""The fp64 evaluation path (precision = 1) against the fp64 oracle, through the C ABI.

Both sides now compute in double precision; what remains is the radial-table interpolation error
(tolerance 1e-10 relative to max|g|) and summation order, so the bars are several orders of
magnitude tighter than those of the fp32 path.
"""
import numpy as np
import pytest

import oracle
from helpers import make_pair

pytestmark = pytest.mark.gpu

E_RTOL_F64 = 1e-10      # relative, total energy
F_ATOL_F64 = 2e-9       # eV/Angstrom, max-abs


@pytest.mark.parametrize("cfg,n_cells,skin", [(1, 4, 0.0), (5, 6, 1.0), (2, 6, 1.0), (3, 5, 1.0), (4, 8, 1.0)])
def test_fp64_energy_forces_virial_match_oracle(cfg, n_cells, skin):
    import paper_2608_16329_b200 as mlip
    w, model, pot = make_pair(cfg, n_cells, skin, precision=1)
    pot.build_neighbors(w.pos, w.species, w.box)
    out = pot.compute(want_e_atom=True)
    pot.sync_status()
    ref = oracle.evaluate(model, w.pos, w.species, w.box)
    e = float(out["energy"].cpu())
    f = out["forces"].cpu().numpy()
    ea = out["e_atom"].cpu().numpy()
    xi = out["virial"].cpu().numpy().reshape(3, 3)
    assert f.dtype == np.float64 and ea.dtype == np.float64
    print(f"cfg {cfg} fp64: N={w.n_atoms} rel dE={abs(e - ref['energy']) / abs(ref['energy']):.2e} "
          f"max|dF|={np.abs(f - ref['forces']).max():.2e} max|dE_i|={np.abs(ea - ref['e_atom']).max():.2e} "
          f"max|dXi|/max|Xi|={np.abs(xi - ref['virial']).max() / np.abs(ref['virial']).max():.2e} "
          f"table err={mlip.mlip_table_error(pot.ctx)}")
    assert abs(e - ref["energy"]) <= E_RTOL_F64 * abs(ref["energy"])
    assert np.abs(f - ref["forces"]).max() <= F_ATOL_F64
    assert np.abs(ea - ref["e_atom"]).max() <= 1e-9 * max(1.0, np.abs(ref["e_atom"]).max())
    assert np.abs(xi - ref["virial"]).max() <= 1e-9 * np.abs(ref["virial"]).max()
    assert abs(f.sum(0)).max() < 1e-9


def test_fp32_entry_point_on_an_fp64_context_rounds_the_same_result():
    import paper_2608_16329_b200 as mlip
    w, model, pot = make_pair(5, 6, 1.0, precision=1)
    pot.build_neighbors(w.pos, w.species, w.box)
    f64 = pot.compute()["forces"]
    t = pot.torch
    f32 = t.empty((w.n_atoms, 3), dtype=t.float32, device=pot.device)
    mlip.mlip_compute(pot.ctx, None, f32, None, None)
    pot.sync_status()
    # the scatter atomics run in a different order between the two launches: agreement to fp32 rounding
    assert np.abs(f32.cpu().numpy() - f64.cpu().numpy()).max() <= 1e-6 * max(1.0, float(f64.abs().max()))


def test_fp64_entry_point_is_refused_on_an_fp32_context():
    import paper_2608_16329_b200 as mlip
    w, model, pot = make_pair(1, 4, 0.0)
    pot.build_neighbors(w.pos, w.species, w.box)
    t = pot.torch
    f = t.empty((w.n_atoms, 3), dtype=t.float64, device=pot.device)
    with pytest.raises(mlip.MlipError) as err:
        mlip.mlip_compute_f64(pot.ctx, None, f, None, None)
    assert err.value.code == mlip.binding.CODES["MLIP_ERR_UNSUPPORTED"]


def test_fp64_nve_follows_the_oracle_trajectory():
    w, model, pot = make_pair(2, 6, 1.0, precision=1)
    pot.build_neighbors(w.pos, w.species, w.box)
    pot.set_velocities(w.vel)
    pot.compute()
    e0 = pot.energies().cpu().numpy()
    ref = oracle.nve(model, w.pos, w.vel, w.species, w.masses, w.box, 10, 1.0, r_list=w.r_cut + w.skin, rebuild_every=5)
    pot.step(10, 1.0, 5)
    pot.sync_status()
    pos, vel, step = pot.state()
    e1 = pot.energies().cpu().numpy()
    d = pos.cpu().numpy() - ref["pos"]
    d -= w.box * np.round(d / w.box)
    print(f"fp64 NVE: max|dx|={np.abs(d).max():.2e} max|dv|={np.abs(vel.cpu().numpy() - ref['vel']).max():.2e} "
          f"dE_tot={e1.sum() - e0.sum():.3e}")
    assert step == 10
    assert np.abs(d).max() < 1e-10
    assert np.abs(vel.cpu().numpy() - ref["vel"]).max() < 1e-11
    assert abs(e1[0] - ref["e_pot"][-1]) <= 1e-10 * abs(ref["e_pot"][-1])


def test_fp64_dense_neighborhood_matches_oracle():
    """More than two 32-pair batches per atom with a ragged tail, and lists far longer than the pair count."""
    w, model, pot = make_pair(1, 5, 2.5, precision=1)
    pos = w.pos.copy()
    rng = np.random.default_rng(5)
    pos += rng.uniform(-0.1, 0.1, pos.shape)
    pos -= np.floor(pos / w.box) * w.box
    pot.build_neighbors(pos, w.species, w.box)
    out = pot.compute()
    pot.sync_status()
    ref = oracle.evaluate(model, pos, w.species, w.box)
    assert abs(float(out["energy"].cpu()) - ref["energy"]) <= E_RTOL_F64 * abs(ref["energy"])
    assert np.abs(out["forces"].cpu().numpy() - ref["forces"]).max() <= F_ATOL_F64


@pytest.mark.parametrize("basis", [0, 1])
def test_fp64_more_pairs_than_the_kept_queue_holds_matches_oracle(basis):
    """A lattice compressed to ~150 pairs per atom: the derivation cannot take the pairs from the encoding's queue
    (128 entries) and scans the list again.  Both the tensor-pipe form (basis 0) and the general form (canonical basis)."""
    import paper_2608_16329_b200 as mlip
    import workloads as wl
    w = wl.make_workload(1, n_cells=5)
    enc, head = wl.workload_weights(1, w.n_species)
    model = oracle.Model(w.n_species, w.r_cut, enc, head, basis=basis)
    pot = mlip.Potential(w.n_species, w.r_cut, 1.0, enc, head, w.masses, precision=1, basis=basis)
    pos, box = 0.8 * w.pos, 0.8 * np.asarray(w.box)
    pot.build_neighbors(pos, w.species, box)
    out = pot.compute(want_e_atom=True)
    pot.sync_status()
    ref = oracle.evaluate(model, pos, w.species, box)
    assert mlip.mlip_get_counters(pot.ctx)["pairs_in_cutoff"] > 140 * w.n_atoms
    f = out["forces"].cpu().numpy()
    assert abs(float(out["energy"].cpu()) - ref["energy"]) <= E_RTOL_F64 * abs(ref["energy"])
    assert np.abs(f - ref["forces"]).max() <= F_ATOL_F64 * max(1.0, np.abs(ref["forces"]).max())
    assert np.abs(out["e_atom"].cpu().numpy() - ref["e_atom"]).max() <= 1e-9 * max(1.0, np.abs(ref["e_atom"]).max())


@pytest.mark.parametrize("k,l_max", [(16, 3), (64, 3), (32, 1), (32, 2), (16, 2), (64, 1)])
def test_fp64_descriptor_shape_variants_match_oracle(k, l_max):
    """Radial width k and angular order l_max of the paper's ablations (Tables 6 and 7, Fig. 4(c)); the fp64 kernel is
    compiled for each shape, the oracle is generic in both."""
    import paper_2608_16329_b200 as mlip
    import workloads as wl
    C = 3
    w = wl.make_workload(3, n_cells=5)
    enc, head = wl.make_weights(C, 77, wl.ENC_OUT_SCALE[3], wl.HEAD_OUT_SCALE[3], k=k, l_max=l_max)
    model = oracle.Model(C, w.r_cut, enc, head, k=k, l_max=l_max)
    pot = mlip.Potential(C, w.r_cut, 1.0, enc, head, w.masses, precision=1, k=k, l_max=l_max)
    pot.build_neighbors(w.pos, w.species, w.box)
    out = pot.compute(want_e_atom=True)
    pot.sync_status()
    ref = oracle.evaluate(model, w.pos, w.species, w.box)
    e = float(out["energy"].cpu())
    f = out["forces"].cpu().numpy()
    print(f"k={k} l_max={l_max}: rel dE={abs(e - ref['energy']) / abs(ref['energy']):.2e} max|dF|={np.abs(f - ref['forces']).max():.2e}")
    assert abs(e - ref["energy"]) <= E_RTOL_F64 * abs(ref["energy"])
    assert np.abs(f - ref["forces"]).max() <= F_ATOL_F64
    assert np.abs(out["e_atom"].cpu().numpy() - ref["e_atom"]).max() <= 1e-9 * max(1.0, np.abs(ref["e_atom"]).max())
    assert np.abs(out["virial"].cpu().numpy().reshape(3, 3) - ref["virial"]).max() <= 1e-9 * np.abs(ref["virial"]).max()


@pytest.mark.parametrize("k,l_max,basis", [(32, 4, 0), (32, 5, 0), (32, 1, 1), (32, 2, 1), (32, 3, 1), (64, 3, 1)])
def test_fp64_higher_orders_and_the_canonical_basis_match_oracle(k, l_max, basis):
    """l_max = 4, 5 (d = 25, 36: Table 4, Fig. 4(c)) through projection matrices built on the host, and the canonical
    monomial basis (d = 4, 10, 20) with the multiplicity metric of Eq. 5 -- the descriptor before the irreducible reduction
    (Table 7).  The library's Q_l differ from the oracle's by a rotation of their rows; the invariants do not."""
    import paper_2608_16329_b200 as mlip
    import workloads as wl
    C = 3
    w = wl.make_workload(3, n_cells=5)
    enc, head = wl.make_weights(C, 78, wl.ENC_OUT_SCALE[3], wl.HEAD_OUT_SCALE[3], k=k, l_max=l_max)
    model = oracle.Model(C, w.r_cut, enc, head, k=k, l_max=l_max, basis=basis)
    pot = mlip.Potential(C, w.r_cut, 1.0, enc, head, w.masses, precision=1, k=k, l_max=l_max, basis=basis)
    pot.build_neighbors(w.pos, w.species, w.box)
    out = pot.compute(want_e_atom=True)
    pot.sync_status()
    ref = oracle.evaluate(model, w.pos, w.species, w.box)
    e = float(out["energy"].cpu())
    f = out["forces"].cpu().numpy()
    print(f"k={k} l_max={l_max} basis={basis}: rel dE={abs(e - ref['energy']) / abs(ref['energy']):.2e} max|dF|={np.abs(f - ref['forces']).max():.2e}")
    scale = max(1.0, float(np.abs(ref["forces"]).max()))
    assert abs(e - ref["energy"]) <= E_RTOL_F64 * abs(ref["energy"])
    assert np.abs(f - ref["forces"]).max() <= F_ATOL_F64 * scale
    assert np.abs(out["e_atom"].cpu().numpy() - ref["e_atom"]).max() <= 1e-9 * max(1.0, np.abs(ref["e_atom"]).max())
    assert np.abs(out["virial"].cpu().numpy().reshape(3, 3) - ref["virial"]).max() <= 1e-9 * np.abs(ref["virial"]).max()


def test_shapes_outside_the_compiled_set_are_refused():
    import paper_2608_16329_b200 as mlip
    import workloads as wl
    for k, l_max, basis, precision in [(32, 3, 1, 0), (16, 3, 1, 1), (64, 5, 0, 1), (32, 4, 1, 1)]:
        enc, head = wl.make_weights(1, 3, k=k, l_max=l_max)
        with pytest.raises(mlip.MlipError) as err:
            mlip.Potential(1, 6.0, 1.0, enc, head, np.array([50.0]), k=k, l_max=l_max, basis=basis, precision=precision)
        assert err.value.code == mlip.binding.CODES["MLIP_ERR_UNSUPPORTED"]


def test_other_shapes_are_refused_by_the_fp32_path():
    import paper_2608_16329_b200 as mlip
    import workloads as wl
    enc, head = wl.make_weights(1, 3, k=64, l_max=3)
    with pytest.raises(mlip.MlipError) as err:
        mlip.Potential(1, 6.0, 1.0, enc, head, np.array([50.0]), k=64, l_max=3)
    assert err.value.code == mlip.binding.CODES["MLIP_ERR_UNSUPPORTED"]
