"""The benchmark's multi-rank bookkeeping (replicas, max-over-ranks timing) on CPU with gloo, world size 2."""
import os
import socket

import pytest
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
    import bench
    local_seconds = 2.0 if rank == 0 else 3.5            # rank 1 is the slow one
    slowest = bench.max_over_ranks(local_seconds, torch.device("cpu"))
    value = bench.whole_job_value(1000, 10, slowest, world)
    out.put((rank, slowest, value))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_sum_of_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, value in results:
        assert slowest == 3.5
        assert abs(value - 2 * 1000 * 10 / 3.5) < 1e-9


def test_single_process_is_a_no_op():
    import bench
    assert bench.max_over_ranks(1.25, torch.device("cpu")) == 1.25
    assert bench.whole_job_value(8, 5, 2.0, 1) == 20.0


def test_reference_arm_prints_one_json_line_with_the_contract_keys():
    import json
    import subprocess
    import sys
    from conftest import ROOT
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--cells", "6", "--steps", "2",
                        "--warmup", "1", "--cpu-centers", "64"], capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-500:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in line
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0


def _args(*flags):
    import sys
    import bench
    old = sys.argv
    sys.argv = ["bench.py"] + list(flags)
    try:
        return bench.parse_args()
    finally:
        sys.argv = old


def test_every_flag_combination_sets_up_its_problem_without_a_gpu():
    """Workload, weights (of the shape the flags ask for) and the work per unit for each mode the benchmark offers."""
    import bench
    import workloads as wl
    for precision in ("f32", "f64"):
        for k, lmax in [(32, 3), (16, 3), (64, 3), (32, 1), (32, 2)]:
            for extra in ([], ["--deterministic"], ["--ensemble", "nvt"]):
                args = _args("--cells", "4", "--precision", precision, "--k", str(k), "--lmax", str(lmax), *extra)
                prob = bench.problem_setup(args)
                w = prob["w"]
                assert w.n_atoms == 256 and prob["enc"].size == 36 * wl.enc_net_size(k)
                assert prob["head"].size == 6 * wl.head_net_size((lmax + 1) * k)
                assert prob["flop_pair"] > 0 and prob["flop_atom"] > 0
                if (k, lmax) == (32, 3):
                    assert prob["flop_pair"] == bench.FLOP_PER_PAIR and prob["flop_atom"] == bench.FLOP_PER_ATOM
    # the angular ablation's shapes: canonical basis and the higher orders
    can = bench.problem_setup(_args("--cells", "4", "--precision", "f64", "--basis", "canonical"))
    irr = bench.problem_setup(_args("--cells", "4", "--precision", "f64"))
    assert can["basis"] == 1 and can["flop_pair"] > irr["flop_pair"] and can["head"].size == irr["head"].size
    l5 = bench.problem_setup(_args("--cells", "4", "--precision", "f64", "--lmax", "5"))
    assert l5["head"].size == 6 * wl.head_net_size(6 * 32) and l5["flop_pair"] > can["flop_pair"]
    # the general count reduces to the default one at the default shape
    d, n_inv = 16, 128
    assert abs((60 + 150 + 512 + 6 * d * 32 + 168) - bench.FLOP_PER_PAIR) < 5
    assert abs((3 * d * 32 + 4 * (n_inv * 64 + 3 * 64 * 64) + 256 + 5000) - bench.FLOP_PER_ATOM) < 1e-3 * bench.FLOP_PER_ATOM


def test_sample_blocks_interior_atoms_have_their_whole_neighborhood_in_the_sample():
    import numpy as np
    import bench
    import oracle
    import workloads as wl
    w = wl.make_workload(5, n_cells=12)
    rows, inner = bench.sample_blocks((12, 12, 12), 4, 3.6, w.r_cut, 4 * 8 * 8 * 12)
    assert rows.size == 4 * 8 * 8 * 12 and 0 < inner.size < rows.size and np.isin(inner, rows).all()
    nl = oracle.neighbors(w.pos, w.species, w.n_species, w.box, w.r_cut, rows=inner)
    assert np.isin(nl.nbr, rows).all()
    # other lattices of the workload table
    for cfg, (cells, n_basis, a) in bench.LATTICES.items():
        r, i = bench.sample_blocks(cells, n_basis, a, 6.0, 49152)
        assert r.max() < np.prod(cells) * n_basis and r.size <= 49152 + 8 * 8 * 24 * n_basis


def test_traffic_record_is_tied_to_the_kernel_sources(tmp_path, monkeypatch):
    import bench
    rec = tmp_path / "t.txt"
    monkeypatch.setattr(bench, "TRAFFIC_RECORD", str(rec))
    assert bench.recorded_traffic()[0] is None
    rec.write_text(f"# comment\nkernel_revision: {bench.kernel_revision()}\ndram_bytes_per_atom: 700.5\n")
    assert bench.recorded_traffic()[0] == 700.5
    rec.write_text("kernel_revision: 0123456789abcdef\ndram_bytes_per_atom: 700.5\n")
    value, why = bench.recorded_traffic()
    assert value is None and "revision" in why


def test_time_step_shrinks_for_runs_beyond_the_stable_horizon_of_the_synthetic_potential():
    """The default run keeps the benchmark's 1 fs; a longer run covers the same simulated time in more, smaller steps."""
    import bench
    assert bench.time_step_fs(3 + 20) == 1.0
    assert bench.time_step_fs(5 + 100) == pytest.approx(bench.SAFE_TRAJECTORY_FS[5] / 105)
    assert bench.time_step_fs(0) == 1.0
    assert bench.time_step_fs(3 + 20, cfg=4) < 0.5   # the ionic stand-in's light species leave the tables' range sooner
