"""NVT (Nose-Hoover chain) through the C ABI against the oracle's NVT loop."""
import numpy as np
import pytest

import oracle
from helpers import make_pair

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("precision,x_tol,v_tol", [(1, 1e-10, 1e-11), (0, 1e-6, 1e-7)])
def test_nvt_follows_the_oracle_trajectory(precision, x_tol, v_tol):
    w, model, pot = make_pair(2, 6, 1.0, precision=precision)
    vel0 = w.vel * 2.0                                   # four times the target kinetic energy
    pot.build_neighbors(w.pos, w.species, w.box)
    pot.set_velocities(vel0)
    ref = oracle.nvt(model, w.pos, vel0, w.species, w.masses, w.box, 10, 1.0, w.r_cut + w.skin, t_target=w.temperature,
                     t_damp_fs=20.0, rebuild_every=5)
    pot.step_nvt(10, 1.0, 5, w.temperature, 20.0)
    pot.sync_status()
    pos, vel, step = pot.state()
    e = pot.energies().cpu().numpy()
    v_eta, eta, e_th = pot.thermostat()
    d = pos.cpu().numpy() - ref["pos"]
    d -= w.box * np.round(d / w.box)
    print(f"NVT precision {precision}: max|dx|={np.abs(d).max():.2e} max|dv|={np.abs(vel.cpu().numpy() - ref['vel']).max():.2e} "
          f"v_eta err={np.abs(v_eta - ref['v_eta']).max():.2e}")
    assert step == 10
    assert np.abs(d).max() < x_tol
    assert np.abs(vel.cpu().numpy() - ref["vel"]).max() < v_tol
    assert np.abs(v_eta - ref["v_eta"]).max() < 1e-6 * np.abs(ref["v_eta"]).max() + (0 if precision else 1e-9)
    assert np.abs(eta - ref["eta"]).max() < 1e-6 * np.abs(ref["eta"]).max() + (0 if precision else 1e-9)
    assert abs(e[1] - ref["e_kin"][-1]) < 1e-6 * ref["e_kin"][-1]
    assert abs((e.sum() + e_th) - ref["conserved"][-1]) < 2e-6 * abs(ref["e_pot"][-1])


def test_nvt_conserves_the_extended_energy_while_the_bath_takes_energy_out():
    """Random-weight networks release potential energy into motion; at fixed temperature the thermostat carries it away."""
    w, model, pot = make_pair(3, 8, 1.0)
    pot.build_neighbors(w.pos, w.species, w.box)
    pot.set_velocities(w.vel)
    pot.compute()
    e0 = pot.energies().cpu().numpy()
    pot.step_nvt(30, 1.0, -2, w.temperature, 25.0)
    assert pot.sync_status(raise_on_error=False) == 0
    e1 = pot.energies().cpu().numpy()
    _, _, e_th = pot.thermostat()
    drift = abs((e1.sum() + e_th) - e0.sum())
    assert e_th > 0.1 * e0[1]                                   # the bath has absorbed energy
    assert drift < 0.005 * abs(e_th) + 2e-6 * abs(e0[0])
    assert abs(e1.sum() - e0.sum()) > 100 * drift               # the physical energy alone is not conserved
