"""Boundary behaviour around the path: cell-vector argument, checkpoint / resume, and the failure paths of in-step
rebuilds (list capacity, a look-back wait that runs out, a diverged configuration) -- all made on the host side; no
kernel faults, traps or hangs."""
import time

import numpy as np
import pytest

import oracle
import workloads as wl
from helpers import canonical_equal, make_pair

pytestmark = pytest.mark.gpu


def test_box_is_given_as_cell_vectors_and_triclinic_cells_are_refused():
    import paper_2608_16329_b200 as mlip
    w, model, pot = make_pair(1, 4, 0.0)
    cell = np.diag(w.box)
    pot.build_neighbors(w.pos, w.species, cell)
    a = pot.compute()
    pot.build_neighbors(w.pos, w.species, w.box)                      # the binding expands three edge lengths
    b = pot.compute()
    assert float(a["energy"].cpu()) == pytest.approx(float(b["energy"].cpu()), rel=1e-12)
    sheared = cell.copy(); sheared[1, 0] = 0.3
    with pytest.raises(mlip.MlipError) as err:
        pot.build_neighbors(w.pos, w.species, sheared)
    assert err.value.code == mlip.binding.CODES["MLIP_ERR_UNSUPPORTED"] and "triclinic" in str(err.value)
    f = np.zeros((w.n_atoms, 3), dtype=np.float32)
    with pytest.raises(mlip.MlipError) as err:
        mlip.mlip_compute_host(pot.ctx, w.pos, w.species, sheared, True, f)
    assert err.value.code == mlip.binding.CODES["MLIP_ERR_UNSUPPORTED"]


@pytest.mark.parametrize("ensemble", ["nve", "nvt"])
def test_checkpoint_and_resume_is_bit_identical_in_deterministic_mode(ensemble):
    """N steps = N/2 steps + save + fresh context + load + N/2 steps, bit for bit, when the save falls on a rebuild step."""
    import paper_2608_16329_b200 as mlip
    w = wl.make_workload(5, n_cells=8)
    enc, head = wl.workload_weights(5, 6)

    def fresh():
        return mlip.Potential(6, w.r_cut, 1.0, enc, head, w.masses, force_mode=1)

    def advance(pot, n):
        if ensemble == "nvt":
            pot.step_nvt(n, 1.0, 5, 300.0, 50.0)
        else:
            pot.step(n, 1.0, 5)
        pot.sync_status()

    straight = fresh()
    straight.build_neighbors(w.pos, w.species, w.box)
    straight.set_velocities(w.vel)
    advance(straight, 20)
    pos_a, vel_a, step_a = straight.state()
    th_a = straight.thermostat()

    first = fresh()
    first.build_neighbors(w.pos, w.species, w.box)
    first.set_velocities(w.vel)
    advance(first, 10)                                                # step 10 is a rebuild step (10 % 5 == 0)
    pos_s, vel_s, step_s = first.state()
    v_eta, eta, _ = first.thermostat()
    saved = (pos_s.cpu().numpy().copy(), vel_s.cpu().numpy().copy(), step_s, v_eta.copy(), eta.copy())
    first.close()

    resumed = fresh()
    resumed.build_neighbors(saved[0], w.species, w.box)
    resumed.set_state(vel=saved[1], step=saved[2], v_eta=saved[3], eta=saved[4])
    advance(resumed, 10)
    pos_b, vel_b, step_b = resumed.state()
    th_b = resumed.thermostat()
    assert step_a == step_b == 20
    assert pos_a.cpu().numpy().tobytes() == pos_b.cpu().numpy().tobytes()
    assert vel_a.cpu().numpy().tobytes() == vel_b.cpu().numpy().tobytes()
    assert th_a[0].tobytes() == th_b[0].tobytes() and th_a[1].tobytes() == th_b[1].tobytes()
    assert straight.energies().cpu().numpy().tobytes() == resumed.energies().cpu().numpy().tobytes()


def test_set_state_replaces_positions_velocities_and_step():
    w, model, pot = make_pair(5, 6, 1.0)
    pot.build_neighbors(w.pos, w.species, w.box)
    rng = np.random.default_rng(2)
    pos = w.pos + rng.uniform(-0.1, 0.1, w.pos.shape)
    pos -= np.floor(pos / w.box) * w.box
    pot.set_state(pos=pos, vel=w.vel, step=123)
    p, v, step = pot.state()
    assert step == 123 and np.array_equal(p.cpu().numpy(), pos) and np.array_equal(v.cpu().numpy(), w.vel)
    ref = oracle.evaluate(model, pos, w.species, w.box)
    out = pot.compute()
    pot.sync_status()
    assert np.abs(out["forces"].cpu().numpy() - ref["forces"]).max() <= 1e-4


def test_list_overflow_in_an_in_step_rebuild_is_reported_and_nothing_is_read_out_of_bounds():
    """Lists sized for the open lattice overflow when the same atoms are squeezed into a corner of the box and an in-step
    rebuild runs: the rebuild cuts the lists at the capacity, the fused kernel skips its evaluation, the status says why."""
    import paper_2608_16329_b200 as mlip
    C = mlip.binding.CODES
    w, model, pot = make_pair(5, 8, 1.0)
    pot.build_neighbors(w.pos, w.species, w.box)                       # capacity = entries of the open lattice + 12.5 %
    n_open = mlip.mlip_get_counters(pot.ctx)["list_entries"]
    blob = w.pos * 0.75                                                # same box, distances shrunk by a quarter
    n_blob = oracle.neighbors(blob, w.species, w.n_species, w.box, w.r_cut + w.skin).nbr.size
    assert n_blob > 1.125 * n_open + 1024
    pot.set_positions(blob)                                            # (the displacement check fires as well)
    pot.set_velocities(np.zeros_like(w.vel))
    pot.step(1, 1e-3, 1)                                               # one step with a rebuild
    assert pot.sync_status(raise_on_error=False) == C["MLIP_ERR_NEIGHBOR_OVERFLOW"]
    # the read above cleared the flags; the overflow shows again after the next rebuild, and the export refuses
    pot.step(1, 1e-3, 1)
    with pytest.raises(mlip.MlipError) as err:
        pot.neighbors()
    assert err.value.code == C["MLIP_ERR_NEIGHBOR_OVERFLOW"]
    out = pot.compute()                                                # skipped: cleared outputs, no out-of-bounds access
    assert float(out["forces"].abs().max().cpu()) == 0.0
    assert pot.sync_status(raise_on_error=False) == C["MLIP_ERR_NEIGHBOR_OVERFLOW"]
    # a synchronising build grows the array and everything works again
    pos, _, _ = pot.state()
    p = pos.cpu().numpy()
    pot.build_neighbors(p, w.species, w.box)
    seg, nbr = pot.neighbors()
    assert canonical_equal(oracle.neighbors(p, w.species, w.n_species, w.box, w.r_cut + w.skin), seg, nbr)
    ref = oracle.evaluate(model, p, w.species, w.box)
    assert np.abs(pot.compute()["forces"].cpu().numpy() - ref["forces"]).max() <= 1e-4 * max(1.0, np.abs(ref["forces"]).max())
    assert pot.sync_status(raise_on_error=False) == C["MLIP_OK"]


def test_a_look_back_wait_that_runs_out_ends_in_a_status_bit():
    """The offset scan of the one-pass list build waits for its predecessor tiles with a bounded number of polls.  A
    diagnostic rebuild in which one tile never publishes its word makes the successor's wait run out: the kernel must
    return promptly, report it, and leave the context usable."""
    import paper_2608_16329_b200 as mlip
    C = mlip.binding.CODES
    w, model, pot = make_pair(5, 12, 1.0)                                # 6,912 atoms = 108 tiles of 64
    pot.build_neighbors(w.pos, w.species, w.box)
    ref = pot.compute()["forces"].cpu().numpy()
    t0 = time.perf_counter()
    mlip.mlip_debug_rebuild(pot.ctx, 32, 40)
    assert pot.sync_status(raise_on_error=False) == C["MLIP_ERR_NEIGHBOR_OVERFLOW"]
    assert time.perf_counter() - t0 < 5.0
    # without the omission the same rebuild is clean, and the lists are those of the oracle
    mlip.mlip_debug_rebuild(pot.ctx, 1 << 18, -1)
    assert pot.sync_status(raise_on_error=False) == C["MLIP_OK"]
    seg, nbr = pot.neighbors()
    assert canonical_equal(oracle.neighbors(w.pos, w.species, w.n_species, w.box, w.r_cut + w.skin), seg, nbr)
    again = pot.compute()["forces"].cpu().numpy()
    assert np.abs(again - ref).max() < 2e-5


def test_a_diverged_configuration_stops_the_rebuild_instead_of_sorting_one_giant_cell():
    """A non-finite velocity sends an atom to NaN in the drift; the next rebuilds must return at once with the flag set
    (the broken configuration is neither sorted nor traversed), and so must the evaluations that follow."""
    import paper_2608_16329_b200 as mlip
    C = mlip.binding.CODES
    w, model, pot = make_pair(1, 4, 1.0)
    pot.build_neighbors(w.pos, w.species, w.box)
    vel = w.vel.copy()
    vel[17, 0] = np.nan
    pot.set_velocities(vel)
    t0 = time.perf_counter()
    pot.step(3, 1.0, 1)
    assert pot.sync_status(raise_on_error=False) == C["MLIP_ERR_NONFINITE"]
    assert time.perf_counter() - t0 < 5.0
    pot.build_neighbors(np.zeros_like(w.pos), w.species, w.box)         # 256 atoms in one cell can still be sorted
    with pytest.raises(mlip.MlipError) as err:
        pot.build_neighbors(np.zeros((2000, 3)), np.zeros(2000, dtype=np.int32), w.box)   # 2,000 cannot
    assert err.value.code == C["MLIP_ERR_NONFINITE"]
    pot.build_neighbors(w.pos, w.species, w.box)
    pot.compute()
    assert pot.sync_status(raise_on_error=False) == C["MLIP_OK"]
