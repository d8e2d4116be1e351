"""The decomposition's host logic with two ranks on CPU (gloo): each rank takes a slab with its ghosts, evaluates its own
central atoms (the oracle stands in for the GPU here), and the forces on ghosts travel back through a sum over ranks."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    import workloads as wl
    from paper_2608_16329_b200 import decomposition as dec
    w = wl.make_workload(5, n_cells=9)                # 2,916 atoms, box 32.4: two slabs of 16.2 + 2 x 7 halo
    enc, head = wl.make_weights(6, 5, 0.1, 0.7, enc_hidden=8, enc_layers=2)
    model = oracle.Model(6, w.r_cut, enc, head, enc_hidden=8, enc_layers=2)
    dom = dec.slab_domain(w.pos, w.species, w.box, rank, world, halo=w.r_cut + 1.0)
    assert dom.n_owned > 0 and dom.index.size > dom.n_owned
    # the domain's own evaluation in its local frame: central atoms = owned atoms only
    nl = oracle.neighbors(dom.pos, dom.species, 6, dom.box, w.r_cut, rows=np.arange(dom.n_owned))
    res = oracle.compute(model, dom.pos, dom.species, dom.box, nl)
    total = torch.zeros((w.n_atoms, 3), dtype=torch.float64)
    dec.scatter_forces(dom, res["forces"], total.numpy())
    scalars = torch.tensor([res["energy"], *res["virial"].ravel(), float(dom.n_owned)], dtype=torch.float64)
    dist.all_reduce(total)                            # ghost forces reach their owners
    dist.all_reduce(scalars)
    if rank == 0:
        ref = oracle.evaluate(model, w.pos, w.species, w.box)
        out.put((float(np.abs(total.numpy() - ref["forces"]).max()), abs(scalars[0].item() - ref["energy"]) / abs(ref["energy"]),
                 float(np.abs(scalars[1:10].numpy().reshape(3, 3) - ref["virial"]).max() / np.abs(ref["virial"]).max()),
                 int(scalars[10].item()), w.n_atoms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_each_with_a_slab_and_ghosts_reproduce_the_whole_system():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    d_force, d_energy, d_virial, owned, n = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert owned == n                                  # every atom is owned exactly once
    assert d_force < 1e-10 and d_energy < 1e-12 and d_virial < 1e-11


def test_slab_domains_partition_the_atoms_and_local_frames_round_trip():
    import workloads as wl
    from paper_2608_16329_b200 import decomposition as dec
    w = wl.make_workload(5, n_cells=12)
    halo = 7.0
    doms = [dec.slab_domain(w.pos, w.species, w.box, r, 3, halo) for r in range(3)]
    owned = np.concatenate([d.index[:d.n_owned] for d in doms])
    assert np.array_equal(np.sort(owned), np.arange(w.n_atoms))
    for r, d in enumerate(doms):
        assert (d.pos >= 0).all() and (d.pos < d.box).all()
        assert d.box[0] >= 2 * halo and d.pos[:, 0].max() < d.box[0] - halo     # the empty padding is there
        # every atom within the halo of an owned atom is present in the domain (checked on the split axis)
        x = w.pos[:, 0]
        lo, hi = w.box[0] / 3 * r, w.box[0] / 3 * (r + 1)
        near = ((x - lo) % w.box[0] < (hi - lo) + halo) | ((lo - x) % w.box[0] <= halo)
        assert np.isin(np.nonzero(near)[0], d.index).all()
        assert np.allclose(dec.to_local(d, w.pos, w.box), d.pos)
    one = dec.slab_domain(w.pos, w.species, w.box, 0, 1, halo)
    assert one.n_owned == w.n_atoms and np.array_equal(one.pos, w.pos)
