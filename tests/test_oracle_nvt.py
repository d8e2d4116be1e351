"""Pins for the oracle's Nose-Hoover-chain NVT loop."""
import numpy as np
from scipy.integrate import solve_ivp

import oracle
import workloads as wl


def _setup():
    w = wl.make_workload(2, n_cells=5)          # 250 atoms, box 16.5 A >= 2 * 7
    enc, head = wl.workload_weights(2, 1)
    return w, oracle.Model(1, 6.0, enc, head)


def _chain_rhs(q, n_f, kT):
    """The chain's equations of motion for force-free particles: y = (sum m v^2, v_eta_1..M, eta_1..M)."""
    M = len(q)

    def rhs(t, y):
        ke2, v, dy = y[0], y[1:1 + M], np.zeros_like(y)
        dy[0] = -2.0 * v[0] * ke2
        for k in range(M):
            G = (ke2 - n_f * kT) / q[0] if k == 0 else (q[k - 1] * v[k - 1] ** 2 - kT) / q[k]
            dy[1 + k] = G - (v[k + 1] * v[k] if k + 1 < M else 0.0)
        dy[1 + M:] = v
        return dy
    return rhs


def test_chain_integrator_converges_to_the_ode_solution_at_second_order():
    """Force-free particles: the kinetic energy only feels the thermostat, so the splitting integrator must approach
    a high-accuracy solution of the chain's differential equations, with error ~ dt^2."""
    n_f, kT, tau = 297, oracle.KB_EV_PER_K * 300.0, 25.0
    q = oracle.nhc_masses(n_f, kT, tau)
    ke2_0 = 2.5 * n_f * kT                          # start well above the target
    ref = solve_ivp(_chain_rhs(q, n_f, kT), (0.0, 40.0), np.concatenate([[ke2_0], np.zeros(6)]), rtol=1e-12, atol=1e-14)
    want_ke2, want_v, want_eta = ref.y[0, -1], ref.y[1:4, -1], ref.y[4:7, -1]
    err = {}
    for dt in (1.0, 0.5):
        ke2, v_eta, eta = ke2_0, np.zeros(3), np.zeros(3)
        for _ in range(int(round(40.0 / dt))):
            for _half in range(2):
                s = oracle.nhc_half_step(ke2, v_eta, eta, q, n_f, kT, dt)
                ke2 *= s * s
        err[dt] = max(abs(ke2 - want_ke2) / want_ke2, np.abs(v_eta - want_v).max() / np.abs(want_v).max(),
                      np.abs(eta - want_eta).max() / np.abs(want_eta).max())
    assert want_ke2 < 0.9 * ke2_0                    # the thermostat has really acted
    assert err[1.0] < 2e-3
    assert 3.0 < err[1.0] / err[0.5] < 5.0           # second order


def test_infinitely_heavy_thermostat_is_nve():
    w, m = _setup()
    a = oracle.nvt(m, w.pos, w.vel, w.species, w.masses, w.box, 6, 1.0, 7.0, t_target=300.0, t_damp_fs=1e9, rebuild_every=3)
    b = oracle.nve(m, w.pos, w.vel, w.species, w.masses, w.box, 6, 1.0, r_list=7.0, rebuild_every=3)
    d = a["pos"] - b["pos"]
    d -= w.box * np.round(d / w.box)
    assert np.abs(d).max() < 1e-11 and np.abs(a["vel"] - b["vel"]).max() < 1e-12


def test_conserved_quantity_and_pull_towards_the_target_temperature():
    w, m = _setup()
    vel = w.vel * 2.0                               # four times the target kinetic energy
    r = oracle.nvt(m, w.pos, vel, w.species, w.masses, w.box, 40, 1.0, 7.0, t_target=w.temperature, t_damp_fs=20.0,
                   rebuild_every=5)
    drift = np.abs(r["conserved"] - r["conserved"][0]).max()
    moved = np.ptp(r["e_kin"])
    assert moved > 0.3 * r["e_kin"][0]              # the thermostat removes a large part of the excess
    assert r["e_kin"][-1] < r["e_kin"][0]
    assert drift < 0.01 * moved                     # while the extended energy stays put
    # physical energy alone is NOT conserved
    assert abs((r["e_pot"] + r["e_kin"])[-1] - (r["e_pot"] + r["e_kin"])[0]) > 20 * drift
    mom = (w.masses[w.species][:, None] * r["vel"]).sum(0)
    assert np.abs(mom).max() < 1e-9                 # uniform scaling keeps the total momentum at zero
