"""Host-side slab decomposition for contexts with ghost atoms (mlip_build_neighbors_ghost).

A periodic orthorhombic box is cut along one axis into `n_domains` slabs.  A domain owns the atoms inside its slab and
receives copies ("ghosts") of the atoms within `halo` = r_cut + skin outside either face.  Each domain evaluates its own
central atoms; the forces that come back for its ghosts belong to other domains' atoms and are returned to them by index
(Section 4.4 runs the potential this way through the MD code's domain decomposition, one domain per GPU).  Index
bookkeeping only: no arithmetic of the potential lives here.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass
class Domain:
    pos: np.ndarray        # [n_owned + n_ghost, 3] slab-local coordinates, owned atoms first
    species: np.ndarray    # [n_owned + n_ghost]
    box: np.ndarray        # [3] local box: split axis = slab + halos + padding, other axes as given
    index: np.ndarray      # [n_owned + n_ghost] index of each local atom in the undivided system
    n_owned: int
    shift: float           # local coordinate on the split axis = (global - shift) mod L


def slab_domain(pos, species, box, rank, n_domains, halo, axis=0, margin=0.25) -> Domain:
    """Domain `rank` of `n_domains` equal slabs along `axis`.  `margin` (Angstrom) of extra room on both sides lets the
    outermost ghosts move between list builds without leaving the local box."""
    pos = np.asarray(pos, dtype=np.float64)
    box = np.asarray(box, dtype=np.float64)
    L = box[axis]
    width = L / n_domains
    lo = rank * width
    hi = L if rank == n_domains - 1 else lo + width
    if n_domains > 1 and width + 2 * halo > L:
        raise ValueError("slabs narrower than the box minus two halos would list an atom twice")
    x = pos[:, axis]
    own = (x >= lo) & (x < hi)
    shift = lo - halo - margin
    rel = (x - shift) % L
    if n_domains == 1:
        ghost = np.zeros_like(own)
        local_box = box.copy()
        rel = x.copy()
        shift = 0.0
    else:
        reach = (rel >= margin) & (rel < margin + (hi - lo) + 2 * halo)
        ghost = reach & ~own
        local_box = box.copy()
        local_box[axis] = (hi - lo) + 2 * halo + 2 * margin + halo       # + halo of empty space: open along the axis
    index = np.concatenate([np.nonzero(own)[0], np.nonzero(ghost)[0]])
    local = pos[index].copy()
    local[:, axis] = rel[index]
    return Domain(local, np.asarray(species)[index].copy(), local_box, index, int(own.sum()), float(shift))


def to_local(domain: Domain, pos, box, axis=0):
    """Current coordinates of the domain's atoms in its local frame (for mlip_set_positions between list builds)."""
    pos = np.asarray(pos, dtype=np.float64)
    out = pos[domain.index].copy()
    if domain.box[axis] != box[axis]:
        # stay next to where the atom was at the build, even if it crossed the whole box's periodic boundary
        d = (out[:, axis] - domain.shift) % box[axis] - domain.pos[:, axis]
        d -= box[axis] * np.round(d / box[axis])
        out[:, axis] = domain.pos[:, axis] + d
    return out


def scatter_forces(domain: Domain, local_forces, total):
    """Add a domain's result (owned parts and ghost reaction forces) into the undivided system's force array."""
    np.add.at(total, domain.index, np.asarray(local_forces, dtype=total.dtype))
    return total
