"""The allocation-free neighbor export against the allocating one, through the C ABI.

Some users of this library cannot allocate device memory at the point where they need the
canonical lists (an MD driver that owns all device memory through its own pools, a plug-in inside
another application, code that must not stall other streams with cudaMalloc).
`mlip_get_neighbors_noalloc` serves them from a static device array; here it must reproduce
`mlip_get_neighbors` bit for bit, twice in a row (the array keeps the first call's contents), and
refuse systems beyond its fixed size.  Collected last on purpose.
"""
import numpy as np
import pytest

from helpers import make_pair

pytestmark = pytest.mark.gpu


def _export(pot, fn):
    import torch
    seg = torch.empty(pot.n * pot.n_species + 1, dtype=torch.int64, device=pot.device)
    _, total = fn(pot.ctx, seg, None)
    nbr = torch.empty(max(total, 1), dtype=torch.int32, device=pot.device)
    rc, total = fn(pot.ctx, seg, nbr)
    assert rc == 0
    return seg.cpu().numpy(), nbr[:total].cpu().numpy()


def test_noalloc_export_matches_the_allocating_export_twice_in_a_row():
    import paper_2608_16329_b200 as mlip
    w, _, pot = make_pair(5, 6, 1.0)
    pot.build_neighbors(w.pos, w.species, w.box)
    seg_ref, nbr_ref = _export(pot, mlip.mlip_get_neighbors)
    assert nbr_ref.size == seg_ref[-1] > 100 * w.n_atoms
    for _ in range(2):
        seg, nbr = _export(pot, mlip.mlip_get_neighbors_noalloc)
        assert np.array_equal(seg, seg_ref) and np.array_equal(nbr, nbr_ref)
    # a different, smaller system afterwards: stale scratch contents must not leak into the result
    w2, _, pot2 = make_pair(3, 5, 1.0)
    pot2.build_neighbors(w2.pos, w2.species, w2.box)
    seg_ref2, nbr_ref2 = _export(pot2, mlip.mlip_get_neighbors)
    seg2, nbr2 = _export(pot2, mlip.mlip_get_neighbors_noalloc)
    assert np.array_equal(seg2, seg_ref2) and np.array_equal(nbr2, nbr_ref2)
    assert pot.sync_status(raise_on_error=False) == 0


def test_noalloc_export_rejects_sizes_beyond_its_static_scratch():
    import torch
    import paper_2608_16329_b200 as mlip
    w, _, pot = make_pair(5, 36, 1.0)            # 186,624 atoms x 6 species > 1,048,576 segments
    assert w.n_atoms * w.n_species > 1 << 20
    pot.build_neighbors(w.pos, w.species, w.box)
    seg = torch.empty(w.n_atoms * w.n_species + 1, dtype=torch.int64, device=pot.device)
    with pytest.raises(mlip.MlipError) as err:
        mlip.mlip_get_neighbors_noalloc(pot.ctx, seg, None)
    assert err.value.code == mlip.binding.CODES["MLIP_ERR_UNSUPPORTED"]
    assert "1048576" in str(err.value)
