"""Measure the weight output scales recorded in the workload recipe.

Run `python -m oracle.calibrate_workloads` from the repository root.  For each
workload (a small instance of it) it prints the RMS of the invariants and of
the force magnitude with the scales currently stored in
`workloads/__init__.py`, and the head scale that would bring the
RMS force to 1 eV/Angstrom.  Calls only the oracle.
"""
import numpy as np

import oracle
import workloads as wl

SMALL = {1: 4, 2: 6, 3: 4, 4: 8, 5: 4}


def main():
    for cfg in (1, 2, 3, 4, 5):
        w = wl.make_workload(cfg, n_cells=SMALL[cfg])
        enc, head = wl.workload_weights(cfg, w.n_species)
        model = oracle.Model(w.n_species, w.r_cut, enc, head)
        nl = oracle.neighbors(w.pos, w.species, w.n_species, w.box, w.r_cut)
        out = oracle.compute(model, w.pos, w.species, w.box, nl, want_G=True)
        G = out["G"]
        rms_g = [float(np.sqrt((G[:, l * model.k:(l + 1) * model.k] ** 2).mean())) for l in range(model.l_max + 1)]
        rms_f = float(np.sqrt((out["forces"] ** 2).sum(axis=1).mean()))
        print(f"cfg {cfg} ({w.name}, {w.n_atoms} atoms, {nl.nbr.size / w.n_atoms:.1f} nbrs): "
              f"rms G per l = {np.round(rms_g, 3)}, rms|F| = {rms_f:.4f}, E/N = {out['energy'] / w.n_atoms:.4f}; "
              f"head scale for rms|F| = 1: {wl.HEAD_OUT_SCALE[cfg] / rms_f:.4f}")


if __name__ == "__main__":
    main()
