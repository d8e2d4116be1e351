"""Shared test helpers: build the oracle model and the CUDA potential from one workload."""
import numpy as np

import oracle
import workloads as wl


def make_pair(cfg, n_cells=None, skin=None, table_knots=0, precision=0, list_format=0, force_mode=0):
    """(workload, oracle model, CUDA potential) fed from the same seeded blobs."""
    import paper_2608_16329_b200 as mlip
    w = wl.make_workload(cfg, n_cells=n_cells)
    if skin is not None:
        w.skin = skin
    enc, head = wl.workload_weights(cfg, w.n_species)
    model = oracle.Model(w.n_species, w.r_cut, enc, head)
    pot = mlip.Potential(w.n_species, w.r_cut, w.skin, enc, head, w.masses, table_knots=table_knots, precision=precision, list_format=list_format,
                         force_mode=force_mode)
    return w, model, pot


def canonical_equal(nl, seg, nbr):
    return np.array_equal(nl.seg_ptr, seg.cpu().numpy()) and np.array_equal(nl.nbr, nbr.cpu().numpy())
