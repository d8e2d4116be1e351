"""Pins for the oracle's velocity-Verlet NVE loop (spec invariants)."""
import numpy as np

import oracle
import workloads as wl


def _setup():
    w = wl.make_workload(2, n_cells=5)          # 250 atoms, box 16.5 A >= 2 * 7
    enc, head = wl.workload_weights(2, 1)
    return w, oracle.Model(1, 6.0, enc, head)


def test_energy_drift_scales_with_dt_squared_and_momentum_is_conserved():
    w, m = _setup()
    vel = w.vel * 3.0                            # ~2700 K: large enough that the error is far above round-off
    runs = {}
    for dt, steps in ((2.0, 8), (1.0, 16)):
        runs[dt] = oracle.nve(m, w.pos, vel, w.species, w.masses, w.box, steps, dt, r_list=7.0, rebuild_every=4)
    err = {dt: np.abs((r["e_pot"] + r["e_kin"]) - (r["e_pot"][0] + r["e_kin"][0])).max() for dt, r in runs.items()}
    kin_fluct = np.ptp(runs[1.0]["e_kin"])
    assert err[1.0] < 0.05 * kin_fluct           # the drift is far below the energy actually exchanged
    assert 2.5 < err[2.0] / err[1.0] < 6.0       # second-order integrator
    mom = (w.masses[w.species][:, None] * runs[1.0]["vel"]).sum(0)
    assert np.abs(mom).max() < 1e-9


def test_time_reversibility():
    w, m = _setup()
    fwd = oracle.nve(m, w.pos, w.vel, w.species, w.masses, w.box, 6, 1.0, r_list=7.0, rebuild_every=3)
    back = oracle.nve(m, fwd["pos"], -fwd["vel"], w.species, w.masses, w.box, 6, 1.0, r_list=7.0, rebuild_every=3)
    d = back["pos"] - w.pos
    d -= w.box * np.round(d / w.box)
    assert np.abs(d).max() < 1e-10 and np.abs(back["vel"] + w.vel).max() < 1e-10


def test_kinetic_energy_of_the_maxwell_draw_matches_the_temperature():
    w = wl.make_workload(2, n_cells=12)
    ke = oracle.kinetic_energy(w.vel, w.species, w.masses)
    t = 2.0 * ke / (3.0 * w.n_atoms * oracle.KB_EV_PER_K)
    assert abs(t - 300.0) < 10.0
    assert abs(oracle.ACC_UNIT / wl.ACC_UNIT - 1.0) < 1e-9
