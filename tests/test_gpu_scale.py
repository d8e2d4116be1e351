"""Parity at the sizes the kernels run at: every warp group walks many tiles, lists hold billions of entries.

The small cases of test_gpu_parity.py give each persistent warp group at most one tile per species, so the steady
state of the fused kernels (prefetched list indices, tile indices carried by barriers, tables re-staged per species)
and the 64-bit offsets of the list build are compared with the oracle here: every atom of a mid-size system, blocks
of atoms of the full-size workloads (a block's interior atoms need only the block's surroundings on the oracle side),
and sampled list rows at 8 and 34 million atoms.
"""
import functools

import numpy as np
import pytest

import oracle
import workloads as wl
from helpers import make_pair

pytestmark = pytest.mark.gpu

E_RTOL, F_ATOL = 1e-6, 1e-4          # fp32 path (spec tolerances)
E_RTOL_F64, F_ATOL_F64 = 1e-10, 2e-9


def head_offsets(head, species, n_species, n_inv=128):
    """Sum over atoms of the regression networks' output biases: the part of E that no kernel arithmetic touches."""
    b_out = head.reshape(n_species, wl.head_net_size(n_inv))[:, -1]
    return b_out[species]


@functools.lru_cache(maxsize=None)
def _midsize_reference():
    w = wl.make_workload(5, n_cells=24)                      # 55,296 atoms: ~1,150 tiles of 8 per species, 296 warp groups
    enc, head = wl.workload_weights(5, w.n_species)
    model = oracle.Model(w.n_species, w.r_cut, enc, head)
    return w, enc, head, oracle.evaluate(model, w.pos, w.species, w.box)


@pytest.mark.parametrize("precision,force_mode", [(0, 0), (0, 1), (1, 0)])
def test_every_atom_of_a_many_tiles_per_group_system_matches_oracle(precision, force_mode):
    import paper_2608_16329_b200 as mlip
    w, enc, head, ref = _midsize_reference()
    pot = mlip.Potential(w.n_species, w.r_cut, 1.0, enc, head, w.masses, precision=precision, force_mode=force_mode)
    pot.build_neighbors(w.pos, w.species, w.box)
    out = pot.compute(want_e_atom=True)
    pot.sync_status()
    e = float(out["energy"].cpu())
    f = out["forces"].cpu().numpy().astype(np.float64)
    ea = out["e_atom"].cpu().numpy().astype(np.float64)
    xi = out["virial"].cpu().numpy().reshape(3, 3)
    off = head_offsets(head, w.species, w.n_species)
    interaction = np.abs(ref["e_atom"] - off)
    print(f"N={w.n_atoms} precision={precision} force_mode={force_mode}: rel dE={abs(e - ref['energy']) / abs(ref['energy']):.2e} "
          f"dE/sum|E_i - b|={abs(e - ref['energy']) / interaction.sum():.2e} max|dF|={np.abs(f - ref['forces']).max():.2e} "
          f"max|dE_i|={np.abs(ea - ref['e_atom']).max():.2e} (mean |E_i - b| = {interaction.mean():.3f} eV)")
    e_tol, f_tol, ea_tol, xi_tol = (E_RTOL_F64, F_ATOL_F64, 1e-9, 1e-9) if precision == 1 else (E_RTOL, F_ATOL, 2e-5, 1e-5)
    assert abs(e - ref["energy"]) <= e_tol * abs(ref["energy"])
    # the same bound without the constant per-species offsets that dominate the total
    assert abs(e - ref["energy"]) <= e_tol * interaction.sum()
    assert np.abs(f - ref["forces"]).max() <= f_tol
    assert np.abs(ea - ref["e_atom"]).max() <= ea_tol * max(1.0, interaction.max())
    assert np.abs(xi - ref["virial"]).max() <= xi_tol * np.abs(ref["virial"]).max()
    pot.close()


def lattice_block(cells, n_basis, origin, size):
    """Caller indices of the atoms on the lattice sites of a block of unit cells (periodic), sites in (ix, iy, iz, basis) order."""
    ax = [(origin[a] + np.arange(size[a])) % cells[a] for a in range(3)]
    ix, iy, iz, b = np.meshgrid(ax[0], ax[1], ax[2], np.arange(n_basis), indexing="ij")
    return (((ix * cells[1] + iy) * cells[2] + iz) * n_basis + b).ravel().astype(np.int64)


def blocks_spread_over(cells, n_basis, size, n_blocks, seed):
    """Blocks at the two box corners (the first wraps around all three periodic faces), the centre and random places."""
    rng = np.random.default_rng(seed)
    origins = [tuple(c - size[a] // 2 for a, c in enumerate(cells)), tuple(c - 3 * size[a] for a, c in enumerate(cells)),
               tuple(c // 2 for c in cells)]
    while len(origins) < n_blocks:
        origins.append(tuple(int(rng.integers(0, c)) for c in cells))
    return np.unique(np.concatenate([lattice_block(cells, n_basis, o, size) for o in origins[:n_blocks]]))


def compare_sampled(pot, model, w, atoms, head, precision=0):
    out = pot.compute(want_e_atom=True)
    pot.sync_status()
    ref = oracle.sampled(model, w.pos, w.species, w.box, atoms)
    idx = pot.torch.as_tensor(atoms, device=pot.device)
    f = out["forces"][idx].cpu().numpy().astype(np.float64)
    ea = out["e_atom"][idx].cpu().numpy().astype(np.float64)
    interaction = np.abs(ref["e_atom"] - head_offsets(head, w.species[atoms], w.n_species))
    print(f"{w.name}: {atoms.size} sampled atoms of {w.n_atoms}: max|dF|={np.abs(f - ref['forces']).max():.2e} "
          f"max|dE_i|={np.abs(ea - ref['e_atom']).max():.2e}")
    f_tol, ea_tol = (F_ATOL_F64, 1e-9) if precision == 1 else (F_ATOL, 2e-5)
    assert np.abs(f - ref["forces"]).max() <= f_tol
    assert np.abs(ea - ref["e_atom"]).max() <= ea_tol * max(1.0, interaction.max())
    return out


def list_rows_equal(pot, w, rows, pos=None):
    """Canonical lists of the sampled rows, exported on the device, against the oracle's lists of the same rows."""
    t = pot.torch
    seg, nbr = pot.neighbors()
    C = w.n_species
    nl = oracle.neighbors(w.pos if pos is None else pos, w.species, C, w.box, w.r_cut + w.skin, rows=rows)
    rows_t = t.as_tensor(rows, device=pot.device)
    seg_rows = seg[(rows_t[:, None] * C + t.arange(C + 1, device=pot.device)[None, :])]     # [rows][C + 1] absolute offsets
    lens = (seg_rows[:, 1:] - seg_rows[:, :-1]).reshape(-1).cpu().numpy()
    if not np.array_equal(lens, np.diff(nl.seg_ptr)):
        return False
    total = seg_rows[:, -1] - seg_rows[:, 0]
    first = t.cumsum(total, 0) - total
    within = t.arange(int(total.sum()), device=pot.device) - t.repeat_interleave(first, total)
    got = nbr[t.repeat_interleave(seg_rows[:, 0], total) + within].cpu().numpy()
    return np.array_equal(got, nl.nbr)


def sampled_rows(n, count, seed):
    """First and last tiles of the index range plus rows spread at random."""
    rng = np.random.default_rng(seed)
    return np.unique(np.concatenate([np.arange(1024), np.arange(n - 2048, n), rng.integers(0, n, count)])).astype(np.int64)


def test_benchmark_size_blocks_of_atoms_and_sampled_lists_match_oracle():
    """8,001,504 atoms, the benchmark's launch configuration: E_i and forces of 2,048 atoms in eight blocks spread over the
    box (all six species), and 6,000 list rows bit for bit -- after the first build and again after an in-step rebuild."""
    import paper_2608_16329_b200 as mlip
    w, model, pot = make_pair(5, 126, 1.0)
    enc, head = wl.workload_weights(5, w.n_species)
    pot.build_neighbors(w.pos, w.species, w.box)
    atoms = blocks_spread_over((126, 126, 126), 4, (4, 4, 4), 8, seed=5)
    assert atoms.size >= 1900 and np.bincount(w.species[atoms], minlength=6).min() > 200
    out = compare_sampled(pot, model, w, atoms, head)
    e = float(out["energy"].cpu())
    assert abs(e - float(out["e_atom"].double().sum().cpu())) <= 1e-6 * abs(e)
    assert np.abs(out["forces"].double().sum(0).cpu().numpy()).max() < 1e-3 * np.sqrt(w.n_atoms)
    del out
    rows = sampled_rows(w.n_atoms, 3000, seed=6)
    assert list_rows_equal(pot, w, rows)
    c = mlip.mlip_get_counters(pot.ctx)
    assert c["list_entries"] > 10 ** 9
    # two steps with a rebuild on the second: the one-pass traversal with its look-back scan over 125,024 tiles
    pot.set_velocities(w.vel)
    pot.step(2, 1.0, 2)
    assert pot.sync_status(raise_on_error=False) == 0 and pot.rebuilds() == 2
    pos, _, _ = pot.state()
    assert list_rows_equal(pot, w, rows, pos=pos.cpu().numpy())
    pot.close()


@functools.lru_cache(maxsize=1)
def _workload_34m():
    return wl.make_workload(5, n_cells=204, with_velocities=False)


@pytest.mark.parametrize("list_format", [0, 1])
def test_list_offsets_beyond_32_bits_match_oracle(list_format):
    """33,957,312 atoms: 4.55e9 list entries, so the offsets of the upper rows pass 2^31 and 2^32 -- with plain indices and
    with the 16-bit cell-relative codes."""
    import paper_2608_16329_b200 as mlip
    w = _workload_34m()
    enc, head = wl.workload_weights(5, w.n_species)
    pot = mlip.Potential(w.n_species, w.r_cut, w.skin, enc, head, w.masses, list_format=list_format)
    pot.build_neighbors(w.pos, w.species, w.box)
    assert mlip.mlip_get_counters(pot.ctx)["list_entries"] > 2 ** 32
    rows = sampled_rows(w.n_atoms, 2000, seed=7)
    assert list_rows_equal(pot, w, rows)
    # an in-step (single-traversal) rebuild at the same size
    pot.step(1, 1.0, 1)
    assert pot.sync_status(raise_on_error=False) == 0
    pos, _, _ = pot.state()
    assert list_rows_equal(pot, w, rows, pos=pos.cpu().numpy())
    pot.close()


def test_unary_workload_at_its_stated_size_every_atom():
    """Workload 2 in full: 65,536 atoms of one species, so a single table set and ~8,000 tiles of one species."""
    w, model, pot = make_pair(2, None, 1.0)
    assert w.n_atoms == 65536
    pot.build_neighbors(w.pos, w.species, w.box)
    out = pot.compute(want_e_atom=True)
    pot.sync_status()
    ref = oracle.evaluate(model, w.pos, w.species, w.box)
    e = float(out["energy"].cpu())
    assert abs(e - ref["energy"]) <= E_RTOL * abs(ref["energy"])
    assert np.abs(out["forces"].cpu().numpy() - ref["forces"]).max() <= F_ATOL
    assert np.abs(out["e_atom"].cpu().numpy() - ref["e_atom"]).max() <= 2e-5 * max(1.0, np.abs(ref["e_atom"]).max())
    seg, nbr = pot.neighbors()
    nl = oracle.neighbors(w.pos, w.species, 1, w.box, w.r_cut + w.skin)
    assert np.array_equal(nl.seg_ptr, seg.cpu().numpy()) and np.array_equal(nl.nbr, nbr.cpu().numpy())
    pot.close()


@pytest.mark.parametrize("cfg,cells,n_basis,size", [(3, (64, 64, 64), 4, (4, 4, 4)), (4, (125, 125, 128), 1, (6, 6, 6))])
def test_alloy_and_ionic_workloads_at_their_stated_sizes_sampled(cfg, cells, n_basis, size):
    """Workloads 3 (1,048,576 atoms, 90/5/5 alloy: tiles of the minority species are rare) and 4 (2,000,000 atoms)."""
    w, model, pot = make_pair(cfg, None, 1.0)
    enc, head = wl.workload_weights(cfg, w.n_species)
    assert w.n_atoms == int(np.prod(cells)) * n_basis
    pot.build_neighbors(w.pos, w.species, w.box)
    atoms = blocks_spread_over(cells, n_basis, size, 6, seed=cfg)
    compare_sampled(pot, model, w, atoms, head)
    assert list_rows_equal(pot, w, sampled_rows(w.n_atoms, 2000, seed=cfg))
    pot.close()
