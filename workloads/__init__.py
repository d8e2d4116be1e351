"""Seeded synthetic inputs: lattices, species, velocities and random network weights.

This module only *draws inputs*. It contains none of the potential's arithmetic
(no descriptor, network, force or neighbor-list code) and imports neither the
CUDA binding nor the CPU oracle, so both sides can be fed from it.

The five workloads stand in for the paper's bulk systems (Section 4.1.2: a
unary metal, a 3-component alloy, a 6-component high-entropy alloy): same
species counts, 6 Angstrom cutoff, crystalline neighbor counts.  Units:
Angstrom, eV, amu, fs, K.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

BASE_SEED = 260816329

KB_EV_PER_K = 8.617333262e-5
# 1 eV/(Angstrom amu) expressed in Angstrom/fs^2
ACC_UNIT = 9.6485332157e-3

# Network architecture (Section 4.1.3): radial encoder with three hidden layers
# of width 128, energy head with four hidden layers of width 64.
ENC_HIDDEN, ENC_LAYERS = 128, 3
HEAD_HIDDEN, HEAD_LAYERS = 64, 4
K_RADIAL = 32
L_MAX = 3

# Output scales folded into the random weights so that moments are O(1) and
# forces are O(1) eV/Angstrom (raw N(0, 1/fan_in) nets summed over ~78 neighbors
# give invariants of order 1e2-1e3).  The numbers were measured once with
# oracle/calibrate_workloads.py and are fixed constants of the recipe.
ENC_OUT_SCALE = {1: 0.1, 2: 0.1, 3: 0.1, 4: 0.1, 5: 0.1}
HEAD_OUT_SCALE = {1: 0.87, 2: 5.9, 3: 0.54, 4: 1.75, 5: 0.72}
# Per-species reference energy (eV) added to the head's output bias, standing in
# for the cohesive-energy offset a trained model carries.
E_REF = -4.0

MASSES = {
    1: [180.95, 92.91, 183.84, 95.95, 50.94, 26.98],
    2: [118.71],
    3: [26.98, 63.55, 24.31],
    4: [6.94, 30.97, 32.06],
    5: [180.95, 92.91, 183.84, 95.95, 50.94, 26.98],
}


@dataclass
class Workload:
    name: str
    cfg: int
    pos: np.ndarray        # [N,3] float64, inside [0, L)
    species: np.ndarray    # [N] int32
    box: np.ndarray        # [3] float64 orthorhombic edge lengths
    masses: np.ndarray     # [C] float64 amu
    n_species: int
    r_cut: float
    skin: float
    temperature: float
    dt_fs: float
    n_steps: int
    rebuild_every: int
    seed: int
    vel: np.ndarray | None = field(default=None)  # [N,3] float64 Angstrom/fs

    @property
    def n_atoms(self) -> int:
        return int(self.pos.shape[0])


_FCC_BASIS = np.array([[0, 0, 0], [0.5, 0.5, 0], [0.5, 0, 0.5], [0, 0.5, 0.5]], dtype=np.float64)
_BCC_BASIS = np.array([[0, 0, 0], [0.5, 0.5, 0.5]], dtype=np.float64)
_SC_BASIS = np.array([[0, 0, 0]], dtype=np.float64)


def lattice_sites(cells, a, basis) -> np.ndarray:
    """Sites in row-major (ix, iy, iz, basis) order, in Angstrom."""
    nx, ny, nz = cells
    ix, iy, iz = np.meshgrid(np.arange(nx), np.arange(ny), np.arange(nz), indexing="ij")
    origin = np.stack([ix, iy, iz], axis=-1).reshape(-1, 1, 3).astype(np.float64)
    return ((origin + basis[None, :, :]) * a).reshape(-1, 3)


def maxwell_velocities(rng, species, masses, temperature) -> np.ndarray:
    """Gaussian velocities at `temperature`, centre-of-mass motion removed."""
    m = np.asarray(masses, dtype=np.float64)[species]
    sigma = np.sqrt(KB_EV_PER_K * temperature / m * ACC_UNIT)
    v = rng.standard_normal((species.shape[0], 3)) * sigma[:, None]
    v -= (m[:, None] * v).sum(axis=0) / m.sum()
    return v


def make_workload(cfg: int, n_cells: int | None = None, seed: int | None = None,
                  with_velocities: bool = True) -> Workload:
    """Build workload `cfg` in 1..5.  `n_cells` overrides the lattice repeat
    (cubic) so tests can make small instances of the same recipe."""
    if seed is None:
        seed = BASE_SEED + cfg
    rng = np.random.default_rng(seed)
    if cfg == 1:
        n = n_cells or 4
        a, basis, cells, sigma, nsp = 3.6, _FCC_BASIS, (n, n, n), 0.05, 6
        fractions, T, skin, steps, rebuild = None, 300.0, 0.0, 0, 0
        name = f"hea6_fcc{n}"
    elif cfg == 2:
        n = n_cells or 32
        a, basis, cells, sigma, nsp = 3.3, _BCC_BASIS, (n, n, n), 0.08, 1
        fractions, T, skin, steps, rebuild = None, 300.0, 1.0, 100, 10
        name = f"unary_bcc{n}"
    elif cfg == 3:
        n = n_cells or 64
        a, basis, cells, sigma, nsp = 4.05, _FCC_BASIS, (n, n, n), 0.05, 3
        fractions, T, skin, steps, rebuild = [0.90, 0.05, 0.05], 300.0, 1.0, 100, 10
        name = f"alloy3_fcc{n}"
    elif cfg == 4:
        a, basis, sigma, nsp = 20.0 ** (1.0 / 3.0), _SC_BASIS, 0.10, 3
        cells = (125, 125, 128) if n_cells is None else (n_cells, n_cells, n_cells)
        fractions, T, skin, steps, rebuild = "exact", 600.0, 1.0, 100, 10
        name = f"ionic3_sc{cells[0]}x{cells[1]}x{cells[2]}"
    elif cfg == 5:
        n = n_cells or 126
        a, basis, cells, sigma, nsp = 3.6, _FCC_BASIS, (n, n, n), 0.05, 6
        fractions, T, skin, steps, rebuild = None, 300.0, 1.0, 50, 10
        name = f"hea6_fcc{n}"
    else:
        raise ValueError(f"unknown workload {cfg}")

    box = np.array(cells, dtype=np.float64) * a
    pos = lattice_sites(cells, a, basis)
    pos += rng.standard_normal(pos.shape) * sigma
    pos -= np.floor(pos / box) * box
    pos[pos >= box] = 0.0  # x = L after rounding belongs at 0
    n_atoms = pos.shape[0]

    if fractions is None:
        species = rng.integers(0, nsp, size=n_atoms).astype(np.int32)
    elif fractions == "exact":
        counts = np.array([round(0.47 * n_atoms), round(0.12 * n_atoms), 0])
        counts[2] = n_atoms - counts[:2].sum()
        species = np.repeat(np.arange(nsp, dtype=np.int32), counts)
        rng.shuffle(species)
    else:
        species = rng.choice(nsp, size=n_atoms, p=fractions).astype(np.int32)

    masses = np.array(MASSES[cfg], dtype=np.float64)
    vel = maxwell_velocities(rng, species, masses, T) if with_velocities else None
    return Workload(name=name, cfg=cfg, pos=pos, species=species, box=box, masses=masses,
                    n_species=nsp, r_cut=6.0, skin=skin, temperature=T, dt_fs=1.0,
                    n_steps=steps, rebuild_every=rebuild, seed=seed, vel=vel)


def enc_net_size(k=K_RADIAL, hidden=ENC_HIDDEN, layers=ENC_LAYERS) -> int:
    return hidden + hidden + (layers - 1) * (hidden * hidden + hidden) + k * hidden + k


def head_net_size(n_in, hidden=HEAD_HIDDEN, layers=HEAD_LAYERS) -> int:
    return n_in * hidden + hidden + (layers - 1) * (hidden * hidden + hidden) + hidden + 1


def _draw_net(rng, widths) -> list[np.ndarray]:
    """Layers W [out][in] then b [out], every entry N(0, 1/fan_in)."""
    parts = []
    for fan_in, fan_out in zip(widths[:-1], widths[1:]):
        s = 1.0 / np.sqrt(fan_in)
        parts.append(rng.standard_normal((fan_out, fan_in)) * s)
        parts.append(rng.standard_normal(fan_out) * s)
    return parts


def make_weights(n_species: int, seed: int, enc_out_scale: float = 1.0, head_out_scale: float = 1.0,
                 e_ref: float = E_REF, k: int = K_RADIAL, l_max: int = L_MAX,
                 enc_hidden: int = ENC_HIDDEN, enc_layers: int = ENC_LAYERS,
                 head_hidden: int = HEAD_HIDDEN, head_layers: int = HEAD_LAYERS):
    """Random-init weights as two flat float64 blobs.

    enc: [C*C] nets, net index = s_i * C + s_j (central species major); each
         net is W1[h][1], b1[h], W2[h][h], b2[h], ..., W_out[k][h], b_out[k].
    head: [C] nets, index = s_i; each net is W1[h][(l_max+1)*k], b1, W2[h][h],
          b2, ..., w_out[h], b_out[1].
    All matrices are row-major [out][in].
    """
    rng = np.random.default_rng(seed)
    enc_widths = [1] + [enc_hidden] * enc_layers + [k]
    head_widths = [(l_max + 1) * k] + [head_hidden] * head_layers + [1]
    enc = []
    for _ in range(n_species * n_species):
        parts = _draw_net(rng, enc_widths)
        parts[-2] = parts[-2] * enc_out_scale
        parts[-1] = parts[-1] * enc_out_scale
        enc.extend(p.ravel() for p in parts)
    head = []
    for _ in range(n_species):
        parts = _draw_net(rng, head_widths)
        parts[-2] = parts[-2] * head_out_scale
        parts[-1] = parts[-1] * head_out_scale + e_ref
        head.extend(p.ravel() for p in parts)
    enc = np.ascontiguousarray(np.concatenate(enc), dtype=np.float64)
    head = np.ascontiguousarray(np.concatenate(head), dtype=np.float64)
    assert enc.size == n_species * n_species * enc_net_size(k, enc_hidden, enc_layers)
    assert head.size == n_species * head_net_size((l_max + 1) * k, head_hidden, head_layers)
    return enc, head


def workload_weights(cfg: int, n_species: int, seed: int | None = None):
    """The weight blobs used with workload `cfg` (seed = workload seed + 1000)."""
    if seed is None:
        seed = BASE_SEED + cfg + 1000
    return make_weights(n_species, seed, ENC_OUT_SCALE[cfg], HEAD_OUT_SCALE[cfg])
