"""CUDA path vs the CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest

import oracle
from helpers import canonical_equal, make_pair

pytestmark = pytest.mark.gpu

# fp32 kernel: energy to 1e-6 relative, forces to 1e-4 eV/Angstrom max-abs (spec tolerances)
E_RTOL, F_ATOL = 1e-6, 1e-4


@pytest.mark.parametrize("cfg,n_cells,skin", [(1, 4, 0.0), (1, 5, 1.0), (2, 6, 1.0), (3, 5, 1.0), (4, 8, 1.0), (5, 6, 1.0)])
def test_neighbor_lists_bit_exact(cfg, n_cells, skin):
    w, model, pot = make_pair(cfg, n_cells, skin)
    pot.build_neighbors(w.pos, w.species, w.box)
    seg, nbr = pot.neighbors()
    pot.sync_status()
    nl = oracle.neighbors(w.pos, w.species, w.n_species, w.box, w.r_cut + w.skin, method="brute" if w.n_atoms <= 1100 else "cell")
    assert canonical_equal(nl, seg, nbr)


def test_neighbor_lists_non_cubic_random_gas():
    import paper_2608_16329_b200 as mlip
    import workloads as wl
    rng = np.random.default_rng(3)
    box = np.array([15.0, 21.5, 29.0])
    pos = rng.uniform(0, 1, (3000, 3)) * box
    species = rng.integers(0, 4, 3000).astype(np.int32)
    enc, head = wl.make_weights(4, seed=1)
    pot = mlip.Potential(4, 6.0, 1.0, enc, head, np.ones(4), table_tol=1.0)
    pot.build_neighbors(pos, species, box)
    seg, nbr = pot.neighbors()
    nl = oracle.neighbors(pos, species, 4, box, 7.0)
    assert canonical_equal(nl, seg, nbr)


@pytest.mark.parametrize("cfg,n_cells,skin", [(1, 4, 0.0), (5, 6, 1.0), (2, 6, 1.0), (3, 5, 1.0), (4, 8, 1.0)])
def test_energy_forces_virial_match_oracle(cfg, n_cells, skin):
    w, model, pot = make_pair(cfg, n_cells, skin)
    pot.build_neighbors(w.pos, w.species, w.box)
    out = pot.compute(want_e_atom=True)
    pot.sync_status()
    ref = oracle.evaluate(model, w.pos, w.species, w.box)
    e = float(out["energy"].cpu())
    f = out["forces"].cpu().numpy().astype(np.float64)
    ea = out["e_atom"].cpu().numpy().astype(np.float64)
    xi = out["virial"].cpu().numpy().reshape(3, 3)
    print(f"cfg {cfg}: N={w.n_atoms} E={e:.6f} rel dE={abs(e - ref['energy']) / abs(ref['energy']):.2e} "
          f"max|dF|={np.abs(f - ref['forces']).max():.2e} max|dE_i|={np.abs(ea - ref['e_atom']).max():.2e} "
          f"table err={pot_table(pot)}")
    assert abs(e - ref["energy"]) <= E_RTOL * abs(ref["energy"])
    assert np.abs(f - ref["forces"]).max() <= F_ATOL
    assert np.abs(ea - ref["e_atom"]).max() <= 2e-5 * max(1.0, np.abs(ref["e_atom"]).max())
    assert np.abs(xi - ref["virial"]).max() <= 1e-5 * np.abs(ref["virial"]).max()
    assert abs(f.sum(0)).max() < 1e-2


def pot_table(pot):
    import paper_2608_16329_b200 as mlip
    return tuple(f"{x:.1e}" for x in mlip.mlip_table_error(pot.ctx))


def test_results_are_returned_in_the_callers_order():
    w, model, pot = make_pair(1, 4, 0.0)
    perm = np.random.default_rng(0).permutation(w.n_atoms)
    pot.build_neighbors(w.pos, w.species, w.box)
    a = pot.compute()["forces"].cpu().numpy()
    pot.build_neighbors(w.pos[perm], w.species[perm], w.box)
    b = pot.compute()["forces"].cpu().numpy()
    assert np.abs(a[perm] - b).max() < 2e-5


def test_set_positions_keeps_lists_and_matches_oracle():
    w, model, pot = make_pair(5, 6, 1.0)
    pot.build_neighbors(w.pos, w.species, w.box)
    rng = np.random.default_rng(1)
    pos = w.pos + rng.uniform(-0.2, 0.2, w.pos.shape)
    pos -= np.floor(pos / w.box) * w.box
    pot.set_positions(pos)
    out = pot.compute()
    pot.sync_status()
    ref = oracle.evaluate(model, pos, w.species, w.box)
    assert np.abs(out["forces"].cpu().numpy() - ref["forces"]).max() <= F_ATOL
    assert abs(float(out["energy"].cpu()) - ref["energy"]) <= E_RTOL * abs(ref["energy"])


def test_compute_host_matches_device_entry():
    import paper_2608_16329_b200 as mlip
    w, model, pot = make_pair(5, 6, 1.0)
    pot.build_neighbors(w.pos, w.species, w.box)
    dev = pot.compute()
    f = np.zeros((w.n_atoms, 3), dtype=np.float32)
    xi = np.zeros(9)
    e = mlip.mlip_compute_host(pot.ctx, w.pos, w.species, w.box, True, f, xi)
    assert abs(e - float(dev["energy"].cpu())) < 1e-9 * abs(e)
    assert np.abs(f - dev["forces"].cpu().numpy()).max() < 2e-5
    e2 = mlip.mlip_compute_host(pot.ctx, w.pos, None, None, False, f, xi)
    assert abs(e2 - e) < 1e-9 * abs(e)


def test_nve_tracks_the_oracle_and_conserves_energy():
    w, model, pot = make_pair(2, 6, 1.0)
    pot.build_neighbors(w.pos, w.species, w.box)
    pot.set_velocities(w.vel)
    pot.compute()
    e0 = pot.energies().cpu().numpy()
    ref = oracle.nve(model, w.pos, w.vel, w.species, w.masses, w.box, 10, 1.0, r_list=w.r_cut + w.skin, rebuild_every=5)
    assert abs(e0[1] - ref["e_kin"][0]) < 1e-9 * ref["e_kin"][0]
    pot.step(10, 1.0, 5)
    pot.sync_status()
    pos, vel, step = pot.state()
    e1 = pot.energies().cpu().numpy()
    assert step == 10
    d = pos.cpu().numpy() - ref["pos"]
    d -= w.box * np.round(d / w.box)
    assert np.abs(d).max() < 1e-6
    assert np.abs(vel.cpu().numpy() - ref["vel"]).max() < 1e-7
    assert abs(e1.sum() - e0.sum()) < 5e-3 * np.ptp(ref["e_kin"]) + 1e-6 * abs(e0[0])
    # 40 more steps: total energy stays put while kinetic and potential energy exchange
    pot.step(40, 1.0, 10)
    pot.sync_status()
    e2 = pot.energies().cpu().numpy()
    assert abs(e2.sum() - e0.sum()) < 0.02 * abs(e2[1] - e0[1]) + 2e-6 * abs(e0[0])


def test_device_side_problems_become_status_codes():
    import paper_2608_16329_b200 as mlip
    C = mlip.binding.CODES
    w, model, pot = make_pair(5, 6, 1.0)
    with pytest.raises(mlip.MlipError) as err:
        pot.compute()
    assert err.value.code == C["MLIP_ERR_NOT_BUILT"]
    with pytest.raises(mlip.MlipError) as err:
        pot.build_neighbors(w.pos, w.species, np.array([10.0, 30.0, 30.0]))
    assert err.value.code == C["MLIP_ERR_BOX_TOO_SMALL"]
    bad = w.pos.copy(); bad[5, 1] = np.nan
    with pytest.raises(mlip.MlipError) as err:          # a synchronising build reports broken input at once
        pot.build_neighbors(bad, w.species, w.box)
    assert err.value.code == C["MLIP_ERR_NONFINITE"]
    assert pot.sync_status(raise_on_error=False) == C["MLIP_OK"]
    with pytest.raises(mlip.MlipError) as err:
        pot.compute()
    assert err.value.code == C["MLIP_ERR_NOT_BUILT"]
    outside = w.pos.copy(); outside[9, 2] = w.box[2] + 0.5
    with pytest.raises(mlip.MlipError) as err:
        pot.build_neighbors(outside, w.species, w.box)
    assert err.value.code == C["MLIP_ERR_NONFINITE"]
    pot.build_neighbors(w.pos, w.species, w.box)
    assert pot.sync_status(raise_on_error=False) == C["MLIP_OK"]
    moved = w.pos.copy(); moved[7] += 0.9; moved -= np.floor(moved / w.box) * w.box
    pot.set_positions(moved)
    assert pot.sync_status(raise_on_error=False) == C["MLIP_ERR_SKIN_EXCEEDED"]
    close = w.pos.copy(); close[1] = close[0] + np.array([0.3, 0.0, 0.0]); close -= np.floor(close / w.box) * w.box
    pot.build_neighbors(close, w.species, w.box)
    pot.compute()
    assert pot.sync_status(raise_on_error=False) == C["MLIP_ERR_TABLE_RANGE"]


def test_table_tolerance_is_enforced():
    import paper_2608_16329_b200 as mlip
    import workloads as wl
    enc, head = wl.workload_weights(5, 6)
    with pytest.raises(mlip.MlipError) as err:
        mlip.Potential(6, 6.0, 1.0, enc, head, np.ones(6), table_knots=8)
    assert err.value.code == mlip.binding.CODES["MLIP_ERR_TABLE_TOLERANCE"]
    pot = mlip.Potential(6, 6.0, 1.0, enc, head, np.ones(6))
    ev, ed = mlip.mlip_table_error(pot.ctx)
    assert ev < 1e-6


def test_full_size_benchmark_workload_sampled_against_oracle():
    """8,001,504 atoms (the benchmark's launch configuration): sampled E_i and forces, global invariants."""
    w, model, pot = make_pair(5, 126, 1.0)
    pot.build_neighbors(w.pos, w.species, w.box)
    out = pot.compute(want_e_atom=True)
    pot.sync_status()
    atoms = np.array([0, 1, 4_000_751, 8_001_503, 123_456, 6_543_210, 2_718_281, 3_141_592])
    ref = oracle.sampled(model, w.pos, w.species, w.box, atoms)
    f = out["forces"][atoms].cpu().numpy().astype(np.float64)
    ea = out["e_atom"][atoms].cpu().numpy().astype(np.float64)
    assert np.abs(f - ref["forces"]).max() <= F_ATOL
    assert np.abs(ea - ref["e_atom"]).max() <= 2e-5 * max(1.0, np.abs(ref["e_atom"]).max())
    # properties that hold at any size: energy is the sum of the per-atom energies, no net force
    e = float(out["energy"].cpu())
    e_sum = float(out["e_atom"].double().sum().cpu())
    assert abs(e - e_sum) <= 1e-6 * abs(e)
    net = out["forces"].double().sum(0).cpu().numpy()
    assert np.abs(net).max() < 1e-3 * np.sqrt(w.n_atoms)
    import paper_2608_16329_b200 as mlip
    c = mlip.mlip_get_counters(pot.ctx)
    assert 77.5 < c["pairs_in_cutoff"] / w.n_atoms < 78.5 and 133.0 < c["list_entries"] / w.n_atoms < 135.0


# (workload 4 is far from equilibrium under random weights: its kinetic energy grows ~50 % in 8 steps and the light
# species soon outruns skin/2 in a few steps, so it gets a short run with a rebuild every 3 steps)
@pytest.mark.parametrize("cfg,n_cells,steps,every", [(3, 16, 30, 10), (4, 24, 12, 3)])
def test_nve_with_rebuilds_conserves_energy_on_multicomponent_workloads(cfg, n_cells, steps, every):
    w, model, pot = make_pair(cfg, n_cells, 1.0)
    pot.build_neighbors(w.pos, w.species, w.box)
    pot.set_velocities(w.vel)
    pot.compute()
    e0 = pot.energies().cpu().numpy()
    pot.step(steps, 1.0, every)
    assert pot.sync_status(raise_on_error=False) == 0
    e1 = pot.energies().cpu().numpy()
    exchanged = abs(e1[1] - e0[1])
    assert exchanged > 0.05 * e0[1]                       # the system is really moving
    assert abs(e1.sum() - e0.sum()) < 0.02 * exchanged + 2e-6 * abs(e0[0])
    # the lists after in-step rebuilds are the lists of the current positions
    pos, vel, step = pot.state()
    seg, nbr = pot.neighbors()
    p = pos.cpu().numpy()
    nl = oracle.neighbors(p, w.species, w.n_species, w.box, w.r_cut + w.skin)
    assert step == steps and canonical_equal(nl, seg, nbr)


def test_tables_in_global_memory_path_matches_oracle():
    """With 256 knots the six tables of a central species no longer fit in shared memory: the kernel's fallback
    instantiation reads them from global memory."""
    w, model, pot = make_pair(1, 4, 0.0, table_knots=256)
    pot.build_neighbors(w.pos, w.species, w.box)
    out = pot.compute()
    pot.sync_status()
    ref = oracle.evaluate(model, w.pos, w.species, w.box)
    assert abs(float(out["energy"].cpu()) - ref["energy"]) <= E_RTOL * abs(ref["energy"])
    assert np.abs(out["forces"].cpu().numpy() - ref["forces"]).max() <= F_ATOL


def test_dense_system_beyond_the_pair_queue_matches_oracle():
    """A compressed lattice with ~165 neighbors inside the cutoff: more than the 160-entry pair queue, so the
    encoding runs in several rounds and the derivation re-scans the list."""
    import paper_2608_16329_b200 as mlip
    import workloads as wl
    rng = np.random.default_rng(21)
    a, n = 2.8, 6
    box = np.full(3, a * n)
    pos = wl.lattice_sites((n, n, n), a, wl._FCC_BASIS) + rng.normal(0.0, 0.03, (4 * n ** 3, 3))
    pos -= np.floor(pos / box) * box
    species = rng.integers(0, 2, len(pos)).astype(np.int32)
    enc, head = wl.make_weights(2, seed=77, enc_out_scale=0.05, head_out_scale=0.3)
    model = oracle.Model(2, 6.0, enc, head)
    pot = mlip.Potential(2, 6.0, 1.0, enc, head, np.array([50.0, 60.0]))
    pot.build_neighbors(pos, species, box)
    out = pot.compute(want_e_atom=True)
    pot.sync_status()
    c = mlip.mlip_get_counters(pot.ctx)
    assert c["pairs_in_cutoff"] / len(pos) > 160
    ref = oracle.evaluate(model, pos, species, box)
    scale = max(1.0, float(np.sqrt((ref["forces"] ** 2).sum(1).mean())))
    assert abs(float(out["energy"].cpu()) - ref["energy"]) <= E_RTOL * abs(ref["energy"])
    assert np.abs(out["forces"].cpu().numpy() - ref["forces"]).max() <= F_ATOL * scale
    assert np.abs(out["e_atom"].cpu().numpy() - ref["e_atom"]).max() <= 2e-5 * max(1.0, np.abs(ref["e_atom"]).max())


@pytest.mark.parametrize("chi_e,chi_r,precision", [(1, 0, 0), (2, 1, 0), (0, 1, 0), (1, 1, 1)])
def test_species_conditioning_variants_match_oracle(chi_e, chi_r, precision):
    """Section 3.2.2: encoder conditioned on the neighbor species only or on nothing, universal regression network."""
    import paper_2608_16329_b200 as mlip
    import workloads as wl
    C = 3
    w = wl.make_workload(3, n_cells=5)
    enc, head = wl.workload_weights(3, C)
    ne, nh = wl.enc_net_size(), wl.head_net_size(128)
    enc_small = enc.reshape(C * C, ne)[:{0: C * C, 1: C, 2: 1}[chi_e]].ravel()
    head_small = head.reshape(C, nh)[:{0: C, 1: 1}[chi_r]].ravel()
    model = oracle.Model(C, w.r_cut, enc_small, head_small, chi_e=chi_e, chi_r=chi_r)
    pot = mlip.Potential(C, w.r_cut, 1.0, enc_small, head_small, w.masses, precision=precision,
                         enc_conditioning=chi_e, head_conditioning=chi_r)
    pot.build_neighbors(w.pos, w.species, w.box)
    out = pot.compute()
    pot.sync_status()
    ref = oracle.evaluate(model, w.pos, w.species, w.box)
    e_tol, f_tol = (1e-10, 2e-9) if precision == 1 else (E_RTOL, F_ATOL)
    assert abs(float(out["energy"].cpu()) - ref["energy"]) <= e_tol * abs(ref["energy"])
    assert np.abs(out["forces"].cpu().numpy() - ref["forces"]).max() <= f_tol
    # a weight blob of the wrong count for the conditioning is refused
    with pytest.raises(mlip.MlipError) as err:
        mlip.Potential(C, w.r_cut, 1.0, enc, head, w.masses, enc_conditioning=2 if chi_e != 2 else 1, head_conditioning=chi_r)
    assert err.value.code == mlip.binding.CODES["MLIP_ERR_INVALID_ARG"]


def test_displacement_triggered_rebuilds_keep_the_lists_valid():
    """The paper's MD policy (Section 4.2): check the criterion every few steps, rebuild only when an atom has moved far
    enough.  The lists in use must at every moment hold all pairs inside r_cut."""
    w, model, pot = make_pair(3, 8, 1.0)
    pot.build_neighbors(w.pos, w.species, w.box)
    pot.set_velocities(w.vel)
    pot.compute()
    e0 = pot.energies().cpu().numpy()
    assert pot.rebuilds() == 1
    pot.step(60, 1.0, -2)
    assert pot.sync_status(raise_on_error=False) == 0
    n_rebuilds = pot.rebuilds() - 1
    assert 2 <= n_rebuilds < 20                      # triggered, but not at every check
    pos, vel, step = pot.state()
    e1 = pot.energies().cpu().numpy()
    exchanged = abs(e1[1] - e0[1])
    assert abs(e1.sum() - e0.sum()) < 0.02 * exchanged + 2e-6 * abs(e0[0])
    seg, nbr = pot.neighbors()
    seg, nbr = seg.cpu().numpy(), nbr.cpu().numpy().astype(np.int64)
    n, C = w.n_atoms, w.n_species
    have = (np.repeat(np.arange(n * C), np.diff(seg)) // C) * n + nbr
    ref = oracle.neighbors(pos.cpu().numpy(), w.species, C, w.box, w.r_cut)
    want = (np.repeat(np.arange(n * C), np.diff(ref.seg_ptr)) // C) * n + ref.nbr.astype(np.int64)
    assert np.isin(want, have).all()
    assert have.size > want.size                     # the lists carry the skin shell as well


@pytest.mark.parametrize("precision", [0, 1])
def test_dilute_system_with_isolated_atoms_ragged_tiles_and_an_absent_species(precision):
    """Degenerate inputs: atoms with no neighbor inside r_cut (E_i = head(0), no force), lists that hold skin-shell entries
    only, species counts that are not multiples of the tile size, and a declared species that no atom has."""
    import paper_2608_16329_b200 as mlip
    import workloads as wl
    rng = np.random.default_rng(11)
    C, a, m = 4, 5.0, 7
    grid = np.stack(np.meshgrid(*[np.arange(m)] * 3, indexing="ij"), -1).reshape(-1, 3).astype(np.float64)
    keep = rng.random(len(grid)) < 0.3
    pos = (grid[keep] + 0.5) * a + rng.uniform(-0.8, 0.8, (keep.sum(), 3))
    box = np.array([m * a] * 3)
    species = rng.choice([0, 1, 3], size=len(pos)).astype(np.int32)           # species 2 is absent
    enc, head = wl.make_weights(C, 5, wl.ENC_OUT_SCALE[1], wl.HEAD_OUT_SCALE[1])
    masses = np.array([20.0, 30.0, 40.0, 50.0])
    model = oracle.Model(C, 6.0, enc, head)
    pot = mlip.Potential(C, 6.0, 1.0, enc, head, masses, precision=precision)
    pot.build_neighbors(pos, species, box)
    out = pot.compute(want_e_atom=True)
    pot.sync_status()
    ref = oracle.evaluate(model, pos, species, box)
    nl = oracle.neighbors(pos, species, C, box, 6.0)
    counts = np.diff(nl.seg_ptr).reshape(-1, C).sum(1)
    assert (counts == 0).sum() >= 5 and len(pos) % 8 != 0                      # the case really is degenerate
    f = out["forces"].cpu().numpy().astype(np.float64)
    ea = out["e_atom"].cpu().numpy().astype(np.float64)
    e_tol, f_tol, ea_tol = (1e-10, 2e-9, 1e-9) if precision == 1 else (E_RTOL, F_ATOL, 2e-5)
    assert abs(float(out["energy"].cpu()) - ref["energy"]) <= e_tol * abs(ref["energy"])
    assert np.abs(f - ref["forces"]).max() <= f_tol
    assert np.abs(ea - ref["e_atom"]).max() <= ea_tol * max(1.0, np.abs(ref["e_atom"]).max())
    assert np.abs(f[counts == 0]).max() == 0.0                                 # isolated atoms feel nothing


@pytest.mark.parametrize("precision", [0, 1])
def test_single_atom(precision):
    import paper_2608_16329_b200 as mlip
    import workloads as wl
    enc, head = wl.make_weights(2, 9)
    model = oracle.Model(2, 6.0, enc, head)
    pos, species, box = np.array([[3.0, 4.0, 5.0]]), np.array([1], dtype=np.int32), np.array([20.0, 20.0, 20.0])
    pot = mlip.Potential(2, 6.0, 1.0, enc, head, np.array([10.0, 12.0]), precision=precision)
    pot.build_neighbors(pos, species, box)
    out = pot.compute()
    pot.step(2, 1.0, 1)
    pot.sync_status()
    ref = oracle.evaluate(model, pos, species, box)
    assert abs(float(out["energy"].cpu()) - ref["energy"]) <= 1e-6 * abs(ref["energy"])
    assert np.abs(out["forces"].cpu().numpy()).max() == 0.0
    assert np.abs(out["virial"].cpu().numpy()).max() == 0.0


@pytest.mark.parametrize("precision", [0, 1])
def test_quintic_envelope_matches_oracle(precision):
    import paper_2608_16329_b200 as mlip
    import workloads as wl
    w = wl.make_workload(3, n_cells=5)
    enc, head = wl.workload_weights(3, 3)
    model = oracle.Model(3, w.r_cut, enc, head, envelope=1)
    pot = mlip.Potential(3, w.r_cut, 1.0, enc, head, w.masses, precision=precision, envelope=1)
    pot.build_neighbors(w.pos, w.species, w.box)
    out = pot.compute()
    pot.sync_status()
    ref = oracle.evaluate(model, w.pos, w.species, w.box)
    # fp64: the quintic's steeper flank raises the table's derivative error at the same knot count (accepted up to
    # 1e-8 of max|g'|), hence 5e-9 instead of the cosine cases' 2e-9
    e_tol, f_tol = (1e-10, 5e-9) if precision == 1 else (E_RTOL, F_ATOL)
    assert abs(float(out["energy"].cpu()) - ref["energy"]) <= e_tol * abs(ref["energy"])
    assert np.abs(out["forces"].cpu().numpy() - ref["forces"]).max() <= f_tol


def test_timings_cover_the_three_parts_of_a_step():
    import time
    import paper_2608_16329_b200 as mlip
    w, model, pot = make_pair(3, 16, 1.0)
    pot.build_neighbors(w.pos, w.species, w.box)
    pot.set_velocities(w.vel)
    pot.step(2, 1.0, 0)
    pot.sync_status()
    mlip.mlip_get_timings(pot.ctx, reset=True)
    t0 = time.perf_counter()
    pot.step(10, 1.0, 5)
    pot.sync_status()
    wall_ms = (time.perf_counter() - t0) * 1e3
    build, kernel, integrate = mlip.mlip_get_timings(pot.ctx)
    n, k_ms = mlip.mlip_kernel_time(pot.ctx)
    assert n == 10 and abs(k_ms - kernel) < 1e-9
    assert build > 0 and integrate > 0 and kernel > build / 10
    assert build + kernel + integrate <= wall_ms
    assert mlip.mlip_get_timings(pot.ctx, reset=True)[1] == kernel
    assert mlip.mlip_get_timings(pot.ctx) == (0.0, 0.0, 0.0)


def test_deterministic_force_mode_is_bit_reproducible_and_matches_oracle():
    """force_mode = 1 takes every scheduling-dependent sum in integer arithmetic: two contexts fed the same input give
    bit-identical energies, forces, virial and trajectories (the default mode agrees only to rounding)."""
    import paper_2608_16329_b200 as mlip
    import workloads as wl
    w = wl.make_workload(5, n_cells=12)                    # 6,912 atoms: thousands of tiles over all SMs
    enc, head = wl.workload_weights(5, 6)
    runs = []
    for _ in range(2):
        pot = mlip.Potential(6, w.r_cut, 1.0, enc, head, w.masses, force_mode=1)
        pot.build_neighbors(w.pos, w.species, w.box)
        pot.set_velocities(w.vel)
        first = pot.compute(want_e_atom=True)
        again = pot.compute(want_e_atom=True)
        for key in ("energy", "forces", "virial", "e_atom"):
            assert pot.torch.equal(first[key], again[key]), key
        pot.step(12, 1.0, 5)
        pot.sync_status()
        pos, vel, _ = pot.state()
        runs.append((first, pos.cpu().numpy(), vel.cpu().numpy(), pot.energies().cpu().numpy()))
        pot.close()
    a, b = runs
    for key in ("energy", "forces", "virial", "e_atom"):
        assert a[0][key].cpu().numpy().tobytes() == b[0][key].cpu().numpy().tobytes(), key
    assert a[1].tobytes() == b[1].tobytes() and a[2].tobytes() == b[2].tobytes()
    assert a[3][0] == b[3][0]
    model = oracle.Model(6, w.r_cut, enc, head)
    rows = np.arange(0, w.n_atoms, 16)
    ref = oracle.sampled(model, w.pos, w.species, w.box, rows)
    f = a[0]["forces"].cpu().numpy().astype(np.float64)
    assert np.abs(f[rows] - ref["forces"]).max() <= F_ATOL
    assert np.abs(a[0]["e_atom"].cpu().numpy()[rows] - ref["e_atom"]).max() <= 2e-5 * np.abs(ref["e_atom"]).max()
    full = oracle.evaluate(model, w.pos, w.species, w.box)
    assert abs(float(a[0]["energy"].cpu()) - full["energy"]) <= E_RTOL * abs(full["energy"])
    assert np.abs(a[0]["virial"].cpu().numpy().reshape(3, 3) - full["virial"]).max() <= 1e-5 * np.abs(full["virial"]).max()
    with pytest.raises(mlip.MlipError) as err:
        mlip.Potential(6, w.r_cut, 1.0, enc, head, w.masses, force_mode=1, precision=1)
    assert err.value.code == mlip.binding.CODES["MLIP_ERR_UNSUPPORTED"]


def test_in_step_rebuild_with_lists_longer_than_the_hit_buffer():
    """A wide skin gives ~220 entries per atom: the one-pass rebuild then takes its second-traversal path for every atom."""
    w, model, pot = make_pair(1, 8, 2.5)
    pot.build_neighbors(w.pos, w.species, w.box)
    pot.set_velocities(w.vel)
    pot.step(4, 1.0, 2)
    assert pot.sync_status(raise_on_error=False) == 0
    assert pot.rebuilds() == 3
    pos, vel, step = pot.state()
    seg, nbr = pot.neighbors()
    nl = oracle.neighbors(pos.cpu().numpy(), w.species, w.n_species, w.box, w.r_cut + 2.5)
    assert nl.nbr.size / w.n_atoms > 200
    assert canonical_equal(nl, seg, nbr)


def test_saturated_head_activations_match_oracle():
    """First-layer pre-activations of the regression network of order 25 (some beyond 60): SiLU runs on the fast
    exponential, whose error grows with |x| while the sigmoid saturates; E_i and forces must still agree."""
    import paper_2608_16329_b200 as mlip
    import workloads as wl
    w = wl.make_workload(1)
    enc, head = wl.workload_weights(1, w.n_species)
    nets = head.reshape(w.n_species, wl.head_net_size(128)).copy()
    nets[:, :64 * 128 + 64] *= 25.0                                   # W1 and b1 of every species' network
    head_big = nets.ravel()
    model = oracle.Model(w.n_species, w.r_cut, enc, head_big)
    nl = oracle.neighbors(w.pos, w.species, w.n_species, w.box, w.r_cut)
    G = oracle.compute(model, w.pos, w.species, w.box, nl, want_G=True)["G"]
    pre = np.array([nets[s, :64 * 128].reshape(64, 128) @ G[i] + nets[s, 64 * 128:64 * 128 + 64] for i, s in enumerate(w.species)])
    assert 10 < np.abs(pre).mean() < 60 and np.abs(pre).max() > 60
    pot = mlip.Potential(w.n_species, w.r_cut, 0.0, enc, head_big, w.masses)
    pot.build_neighbors(w.pos, w.species, w.box)
    out = pot.compute(want_e_atom=True)
    pot.sync_status()
    ref = oracle.evaluate(model, w.pos, w.species, w.box)
    f_scale = max(1.0, float(np.sqrt((ref["forces"] ** 2).sum(1).mean())))
    e_scale = max(1.0, float(np.abs(ref["e_atom"]).max()))
    print(f"saturated head: mean|pre|={np.abs(pre).mean():.1f} max={np.abs(pre).max():.0f} rms|F|={f_scale:.1f} "
          f"max|dF|={np.abs(out['forces'].cpu().numpy() - ref['forces']).max():.2e} max|dE_i|={np.abs(out['e_atom'].cpu().numpy() - ref['e_atom']).max():.2e}")
    assert abs(float(out["energy"].cpu()) - ref["energy"]) <= E_RTOL * np.abs(ref["e_atom"]).sum()
    assert np.abs(out["e_atom"].cpu().numpy() - ref["e_atom"]).max() <= 2e-5 * e_scale
    assert np.abs(out["forces"].cpu().numpy() - ref["forces"]).max() <= F_ATOL * f_scale


@pytest.mark.parametrize("k,l_max", [(16, 3), (32, 1), (32, 2), (16, 2), (8, 0)])
def test_smaller_descriptor_shapes_run_in_the_fp32_kernel(k, l_max):
    """Models with fewer radial channels or a lower angular order than the compiled shape (k = 32, l_max = 3) are
    zero-filled at create time; the result is that of the smaller model."""
    import paper_2608_16329_b200 as mlip
    import workloads as wl
    C = 3
    w = wl.make_workload(3, n_cells=5)
    enc, head = wl.make_weights(C, 91, wl.ENC_OUT_SCALE[3], wl.HEAD_OUT_SCALE[3], k=k, l_max=l_max)
    model = oracle.Model(C, w.r_cut, enc, head, k=k, l_max=l_max)
    pot = mlip.Potential(C, w.r_cut, 1.0, enc, head, w.masses, k=k, l_max=l_max)
    pot.build_neighbors(w.pos, w.species, w.box)
    out = pot.compute(want_e_atom=True)
    pot.sync_status()
    ref = oracle.evaluate(model, w.pos, w.species, w.box)
    f_scale = max(1.0, float(np.abs(ref["forces"]).max()))
    assert abs(float(out["energy"].cpu()) - ref["energy"]) <= E_RTOL * abs(ref["energy"])
    assert np.abs(out["forces"].cpu().numpy() - ref["forces"]).max() <= F_ATOL * f_scale
    assert np.abs(out["e_atom"].cpu().numpy() - ref["e_atom"]).max() <= 2e-5 * max(1.0, np.abs(ref["e_atom"]).max())


@pytest.mark.parametrize("precision,list_format", [(0, 0), (0, 1), (1, 0)])
def test_eight_species_the_maximum_count_match_oracle(precision, list_format):
    """Eight species: 64 encoders, whose tables no longer fit shared memory, so the fused kernel reads them from global
    memory (its other table path); species drawn at random over the 500-atom lattice."""
    import paper_2608_16329_b200 as mlip
    import workloads as wl
    n_species = 8
    w = wl.make_workload(1, n_cells=5)
    species = np.random.default_rng(3).integers(0, n_species, w.n_atoms).astype(np.int32)
    enc, head = wl.make_weights(n_species, 77, wl.ENC_OUT_SCALE[1], wl.HEAD_OUT_SCALE[1])
    model = oracle.Model(n_species, w.r_cut, enc, head)
    pot = mlip.Potential(n_species, w.r_cut, 1.0, enc, head, np.linspace(20.0, 90.0, n_species), precision=precision, list_format=list_format)
    pot.build_neighbors(w.pos, species, w.box)
    out = pot.compute(want_e_atom=True)
    pot.sync_status()
    ref = oracle.evaluate(model, w.pos, species, w.box)
    e_tol, f_tol = (1e-10, 2e-9) if precision else (1e-6, 1e-4)
    assert abs(float(out["energy"].cpu()) - ref["energy"]) <= e_tol * abs(ref["energy"])
    assert np.abs(out["forces"].cpu().numpy() - ref["forces"]).max() <= f_tol
    assert np.abs(out["e_atom"].cpu().numpy() - ref["e_atom"]).max() <= (1e-9 if precision else 2e-5) * max(1.0, np.abs(ref["e_atom"]).max())


@pytest.mark.parametrize("precision", [0, 1])
def test_absent_species_and_a_species_with_one_atom_match_oracle(precision):
    """Four species declared, two of them without atoms and one with a single atom: empty species ranges and a ragged
    one-atom tile, followed by a few steps with an in-step rebuild."""
    import paper_2608_16329_b200 as mlip
    import workloads as wl
    n_species = 4
    w = wl.make_workload(1, n_cells=4)
    species = np.where(np.arange(w.n_atoms) % 3 == 0, 0, 2).astype(np.int32)
    species[7] = 3
    enc, head = wl.make_weights(n_species, 78, wl.ENC_OUT_SCALE[1], wl.HEAD_OUT_SCALE[1])
    model = oracle.Model(n_species, w.r_cut, enc, head)
    pot = mlip.Potential(n_species, w.r_cut, 1.0, enc, head, np.linspace(20.0, 90.0, n_species), precision=precision)
    pot.build_neighbors(w.pos, species, w.box)
    out = pot.compute()
    pot.sync_status()
    ref = oracle.evaluate(model, w.pos, species, w.box)
    e_tol, f_tol = (1e-10, 2e-9) if precision else (1e-6, 1e-4)
    assert abs(float(out["energy"].cpu()) - ref["energy"]) <= e_tol * abs(ref["energy"])
    assert np.abs(out["forces"].cpu().numpy() - ref["forces"]).max() <= f_tol
    pot.set_velocities(np.zeros_like(w.pos))
    pot.step(12, 0.5, 5)
    pot.sync_status()
