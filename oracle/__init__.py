"""CPU fp64 oracle (test infrastructure only).

Thin ctypes wrapper over `mlip_oracle.c` plus the few steps that are plainer in
numpy (harmonic projection matrices, the velocity-Verlet loop).  Only tests,
the smoke check and the benchmark's CPU-baseline leg may import this package;
it imports nothing from the CUDA package and the CUDA package never imports it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

from . import harmonic_projection

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mlip_oracle.c")
_LIB = os.path.join(_HERE, "libmlip_oracle.so")

# 1 eV/(Angstrom amu) in Angstrom/fs^2 (CODATA eV and atomic mass unit)
ACC_UNIT = 1.602176634e-19 / 1.66053906660e-27 * 1e-10
KB_EV_PER_K = 8.617333262e-5


def build(force: bool = False) -> str:
    """Compile the C core with gcc (no FMA contraction, OpenMP over atoms)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
                               "-o", _LIB, _SRC, "-lm"])
    return _LIB


class _CModel(ctypes.Structure):
    _fields_ = [("n_species", ctypes.c_int), ("k", ctypes.c_int), ("l_max", ctypes.c_int),
                ("enc_hidden", ctypes.c_int), ("enc_layers", ctypes.c_int),
                ("head_hidden", ctypes.c_int), ("head_layers", ctypes.c_int),
                ("r_cut", ctypes.c_double),
                ("enc_w", ctypes.c_void_p), ("head_w", ctypes.c_void_p), ("q", ctypes.c_void_p),
                ("chi_e", ctypes.c_int), ("chi_r", ctypes.c_int), ("envelope", ctypes.c_int),
                ("basis", ctypes.c_int), ("metric", ctypes.c_void_p)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_neighbors_brute.restype = ctypes.c_int64
        _lib.oracle_neighbors_cell.restype = ctypes.c_int64
        _lib.oracle_head.restype = ctypes.c_double
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


@dataclass
class Model:
    n_species: int
    r_cut: float
    enc_w: np.ndarray
    head_w: np.ndarray
    k: int = 32
    l_max: int = 3
    enc_hidden: int = 128
    enc_layers: int = 3
    head_hidden: int = 64
    head_layers: int = 4
    q: np.ndarray | None = None   # override the projection matrices (tests)
    chi_e: int = 0   # encoder conditioning (Section 3.2.2): 0 = species pair, C*C nets; 1 = neighbor species, C nets; 2 = none, 1 net
    chi_r: int = 0   # regression-network conditioning: 0 = central species, C nets; 1 = none, 1 net
    envelope: int = 0   # smooth cutoff: 0 = cosine, 1 = quintic polynomial 1 - 10 x^3 + 15 x^4 - 6 x^5
    basis: int = 0      # angular basis (Section 3.3): 0 = irreducible harmonics (C_l = I), 1 = canonical monomials (C_l = multiplicities)

    def __post_init__(self):
        self.enc_w = np.ascontiguousarray(self.enc_w, dtype=np.float64)
        self.head_w = np.ascontiguousarray(self.head_w, dtype=np.float64)
        if self.q is None:
            self.q = harmonic_projection.canonical_table(self.l_max) if self.basis == 1 else harmonic_projection.q_table(self.l_max)
        self.q = np.ascontiguousarray(self.q, dtype=np.float64)
        self.metric = np.ascontiguousarray(harmonic_projection.metric_diagonal(self.l_max, self.basis), dtype=np.float64)
        self._c = _CModel(self.n_species, self.k, self.l_max, self.enc_hidden, self.enc_layers,
                          self.head_hidden, self.head_layers, float(self.r_cut),
                          _p(self.enc_w), _p(self.head_w), _p(self.q), self.chi_e, self.chi_r, self.envelope,
                          self.basis, _p(self.metric))

    @property
    def d(self) -> int:
        return harmonic_projection.reducible_dim(self.l_max) if self.basis == 1 else (self.l_max + 1) ** 2

    @property
    def n_inv(self) -> int:
        return (self.l_max + 1) * self.k

    @property
    def n_enc_nets(self) -> int:
        return {0: self.n_species ** 2, 1: self.n_species, 2: 1}[self.chi_e]

    @property
    def n_head_nets(self) -> int:
        return {0: self.n_species, 1: 1}[self.chi_r]

    def ref(self):
        return ctypes.byref(self._c)


@dataclass
class NeighborList:
    rows: np.ndarray | None   # central atom of each list row (None: row q is atom q)
    seg_ptr: np.ndarray       # int64 [n_rows*C + 1]
    nbr: np.ndarray           # int32
    n_species: int

    @property
    def n_rows(self) -> int:
        return (self.seg_ptr.size - 1) // self.n_species


def neighbors(pos, species, n_species, box, r_list, rows=None, method="cell") -> NeighborList:
    """Species-segmented, ascending neighbor lists (strict d^2 < r_list^2)."""
    pos = np.ascontiguousarray(pos, dtype=np.float64)
    species = np.ascontiguousarray(species, dtype=np.int32)
    box = np.ascontiguousarray(box, dtype=np.float64)
    assert np.all(box >= 2.0 * r_list), "box must hold two list radii per edge (unique minimum image)"
    n = pos.shape[0]
    rows_a = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    n_rows = n if rows_a is None else rows_a.size
    fn = lib().oracle_neighbors_cell if method == "cell" else lib().oracle_neighbors_brute
    seg_ptr = np.zeros(n_rows * n_species + 1, dtype=np.int64)
    cap = max(64, int(n_rows * 160))
    while True:
        nbr = np.empty(cap, dtype=np.int32)
        total = fn(ctypes.c_int64(n), _p(pos), _p(species), ctypes.c_int(n_species), _p(box),
                   ctypes.c_double(r_list), ctypes.c_int64(n_rows), _p(rows_a), _p(seg_ptr), _p(nbr),
                   ctypes.c_int64(cap))
        if total <= cap:
            return NeighborList(rows_a, seg_ptr, nbr[:total].copy(), n_species)
        cap = int(total)


def compute(model: Model, pos, species, box, nl: NeighborList, want_G=False):
    """E, per-atom E_i, forces, virial from the central atoms of `nl`."""
    pos = np.ascontiguousarray(pos, dtype=np.float64)
    species = np.ascontiguousarray(species, dtype=np.int32)
    box = np.ascontiguousarray(box, dtype=np.float64)
    n = pos.shape[0]
    e_atom = np.zeros(n)
    forces = np.zeros((n, 3))
    virial = np.zeros(9)
    energy = ctypes.c_double(0.0)
    G = np.zeros((nl.n_rows, model.n_inv)) if want_G else None
    lib().oracle_compute(model.ref(), ctypes.c_int64(n), _p(pos), _p(species), _p(box),
                         ctypes.c_int64(nl.n_rows), _p(nl.rows), _p(nl.seg_ptr), _p(nl.nbr),
                         _p(e_atom), _p(forces), _p(virial), ctypes.byref(energy), _p(G))
    out = {"energy": energy.value, "e_atom": e_atom, "forces": forces, "virial": virial.reshape(3, 3)}
    if want_G:
        out["G"] = G
    return out


def evaluate(model: Model, pos, species, box, r_list=None, method="cell"):
    """Neighbor search + full evaluation of every atom."""
    nl = neighbors(pos, species, model.n_species, box, model.r_cut if r_list is None else r_list, method=method)
    return compute(model, pos, species, box, nl)


def sampled(model: Model, pos, species, box, atoms):
    """E_i and the full force for a few `atoms` of a large system.

    The force on atom a needs E_i of a itself and of every i that lists a, so the
    central-atom set is the union of the atoms and their neighbors within r_cut.
    """
    atoms = np.asarray(atoms, dtype=np.int64)
    first = neighbors(pos, species, model.n_species, box, model.r_cut, rows=atoms)
    centres = np.unique(np.concatenate([atoms, first.nbr.astype(np.int64)]))
    nl = neighbors(pos, species, model.n_species, box, model.r_cut, rows=centres)
    out = compute(model, pos, species, box, nl)
    return {"atoms": atoms, "e_atom": out["e_atom"][atoms], "forces": out["forces"][atoms]}


def encoder(model: Model, si, sj, r):
    y = np.zeros(model.k)
    dy = np.zeros(model.k)
    lib().oracle_encoder(model.ref(), ctypes.c_int(si), ctypes.c_int(sj), ctypes.c_double(r), _p(y), _p(dy))
    return y, dy


def radial(model: Model, si, sj, r):
    g = np.zeros(model.k)
    dg = np.zeros(model.k)
    lib().oracle_radial(model.ref(), ctypes.c_int(si), ctypes.c_int(sj), ctypes.c_double(r), _p(g), _p(dg))
    return g, dg


def angular(model: Model, u):
    u = np.ascontiguousarray(u, dtype=np.float64)
    h = np.zeros(model.d)
    dh = np.zeros((model.d, 3))
    lib().oracle_angular(model.ref(), _p(u), _p(h), _p(dh))
    return h, dh


def head(model: Model, s, G, want_grad=False):
    G = np.ascontiguousarray(G, dtype=np.float64)
    dG = np.zeros_like(G) if want_grad else None
    e = lib().oracle_head(model.ref(), ctypes.c_int(s), _p(G), _p(dG))
    return (e, dG) if want_grad else e


def kinetic_energy(vel, species, masses):
    m = np.asarray(masses, dtype=np.float64)[species]
    return 0.5 * float((m[:, None] * vel * vel).sum()) / ACC_UNIT


def nve(model: Model, pos, vel, species, masses, box, n_steps, dt_fs, r_list, rebuild_every=1):
    """Velocity-Verlet NVE: half kick, drift, wrap, forces, half kick.

    Lists of radius r_list are rebuilt every `rebuild_every` steps (step 0
    included).  Returns final positions, velocities and the per-step potential
    and kinetic energies (index 0 = initial state).
    """
    pos = np.array(pos, dtype=np.float64)
    vel = np.array(vel, dtype=np.float64)
    box = np.asarray(box, dtype=np.float64)
    inv_m = (ACC_UNIT / np.asarray(masses, dtype=np.float64))[species][:, None]
    nl = neighbors(pos, species, model.n_species, box, r_list)
    out = compute(model, pos, species, box, nl)
    e_pot, e_kin = [out["energy"]], [kinetic_energy(vel, species, masses)]
    for step in range(1, n_steps + 1):
        vel += 0.5 * dt_fs * out["forces"] * inv_m
        pos += dt_fs * vel
        pos -= np.floor(pos / box) * box
        if rebuild_every > 0 and step % rebuild_every == 0:
            nl = neighbors(pos, species, model.n_species, box, r_list)
        out = compute(model, pos, species, box, nl)
        vel += 0.5 * dt_fs * out["forces"] * inv_m
        e_pot.append(out["energy"])
        e_kin.append(kinetic_energy(vel, species, masses))
    return {"pos": pos, "vel": vel, "e_pot": np.array(e_pot), "e_kin": np.array(e_kin), "forces": out["forces"]}


def nhc_masses(n_f, kT, t_damp_fs, chain=3):
    """Thermostat masses of a Nose-Hoover chain: Q_1 = N_f kT tau^2, Q_k = kT tau^2 (eV fs^2)."""
    q = np.full(chain, kT * t_damp_fs ** 2)
    q[0] *= n_f
    return q


def nhc_half_step(ke2, v_eta, eta, q, n_f, kT, dt_fs):
    """Advance a Nose-Hoover chain by dt/2 at fixed particle positions and return the factor by which the
    particle velocities are scaled (Martyna, Tuckerman, Tobias and Klein 1996: one Suzuki-Yoshida term, one
    sub-cycle).  ke2 = sum m v^2 (twice the kinetic energy, eV); v_eta, eta are updated in place.

    Equations of motion: dv_i/dt = -v_eta1 v_i;  dv_eta_k/dt = G_k - v_eta_{k+1} v_eta_k,
    G_1 = (sum m v^2 - N_f kT) / Q_1,  G_k = (Q_{k-1} v_eta_{k-1}^2 - kT) / Q_k;  d eta_k/dt = v_eta_k.
    """
    M = len(q)
    d = 0.5 * dt_fs
    G = np.empty(M)
    G[0] = (ke2 - n_f * kT) / q[0]
    for k in range(1, M):
        G[k] = (q[k - 1] * v_eta[k - 1] ** 2 - kT) / q[k]
    v_eta[M - 1] += 0.5 * d * G[M - 1]
    for k in range(M - 2, -1, -1):
        a = np.exp(-0.25 * d * v_eta[k + 1])
        v_eta[k] = (v_eta[k] * a + 0.5 * d * G[k]) * a
    scale = np.exp(-d * v_eta[0])
    ke2 = ke2 * scale * scale
    eta += d * v_eta
    G[0] = (ke2 - n_f * kT) / q[0]
    for k in range(M - 1):
        a = np.exp(-0.25 * d * v_eta[k + 1])
        v_eta[k] = (v_eta[k] * a + 0.5 * d * G[k]) * a
        G[k + 1] = (q[k] * v_eta[k] ** 2 - kT) / q[k + 1]
    v_eta[M - 1] += 0.5 * d * G[M - 1]
    return scale


def nhc_energy(v_eta, eta, q, n_f, kT):
    """Thermostat part of the conserved quantity of Nose-Hoover-chain dynamics."""
    return float(0.5 * np.sum(q * v_eta ** 2) + n_f * kT * eta[0] + kT * np.sum(eta[1:]))


def nvt(model: Model, pos, vel, species, masses, box, n_steps, dt_fs, r_list, t_target, t_damp_fs, rebuild_every=1,
        chain=3, n_f=None):
    """Nose-Hoover-chain NVT: thermostat half step, velocity-Verlet step, thermostat half step.

    Section 4.2 runs NVT at 300 K through LAMMPS without naming the thermostat; this is the reading taken (the
    chain thermostat of LAMMPS's own NVT integrator, chain length 3).  N_f defaults to 3 N - 3.
    Returns positions, velocities, per-step energies and the conserved quantity (index 0 = initial state).
    """
    pos = np.array(pos, dtype=np.float64)
    vel = np.array(vel, dtype=np.float64)
    box = np.asarray(box, dtype=np.float64)
    n = pos.shape[0]
    n_f = 3 * n - 3 if n_f is None else n_f
    kT = KB_EV_PER_K * t_target
    q = nhc_masses(n_f, kT, t_damp_fs, chain)
    v_eta, eta = np.zeros(chain), np.zeros(chain)
    inv_m = (ACC_UNIT / np.asarray(masses, dtype=np.float64))[species][:, None]
    nl = neighbors(pos, species, model.n_species, box, r_list)
    out = compute(model, pos, species, box, nl)
    ke = kinetic_energy(vel, species, masses)
    e_pot, e_kin = [out["energy"]], [ke]
    conserved = [out["energy"] + ke + nhc_energy(v_eta, eta, q, n_f, kT)]
    for step in range(1, n_steps + 1):
        vel *= nhc_half_step(2.0 * kinetic_energy(vel, species, masses), v_eta, eta, q, n_f, kT, dt_fs)
        vel += 0.5 * dt_fs * out["forces"] * inv_m
        pos += dt_fs * vel
        pos -= np.floor(pos / box) * box
        if rebuild_every > 0 and step % rebuild_every == 0:
            nl = neighbors(pos, species, model.n_species, box, r_list)
        out = compute(model, pos, species, box, nl)
        vel += 0.5 * dt_fs * out["forces"] * inv_m
        vel *= nhc_half_step(2.0 * kinetic_energy(vel, species, masses), v_eta, eta, q, n_f, kT, dt_fs)
        ke = kinetic_energy(vel, species, masses)
        e_pot.append(out["energy"])
        e_kin.append(ke)
        conserved.append(out["energy"] + ke + nhc_energy(v_eta, eta, q, n_f, kT))
    return {"pos": pos, "vel": vel, "e_pot": np.array(e_pot), "e_kin": np.array(e_kin), "conserved": np.array(conserved),
            "v_eta": v_eta, "eta": eta, "forces": out["forces"]}
