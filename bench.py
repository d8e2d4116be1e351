#!/usr/bin/env python
"""Benchmark of the hot path: velocity-Verlet NVE steps of the 6-component alloy on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--cells n]

A step is one pass of the whole path over all atoms: half kick + drift, neighbor rebuild
every 10th step (skin 1 A), one fused energy/force/virial kernel, half kick.  Prints one JSON
line.  With N > 1 (torchrun) every rank runs an independent replica of the workload on its
own GPU (the path has no exchange step on one node: replicas only) and the line reports the
aggregate over ranks using the slowest rank's time.

`--impl reference` times the CPU oracle (oracle/) as it stands on the host cores, on a
bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "atom_steps_per_s"
UNIT = "atom-steps/s"
CFG = 5
DEFAULT_CELLS = 126            # 4 * 126^3 = 8,001,504 atoms: the size the target is quoted on
REBUILD_EVERY = 10
DT_FS = 1.0
# A random-init network has no repulsive core: started from the lattice, NVE at 1 fs runs ~45 steps of the benchmark
# workload before a pair falls below the radial tables' lower end (measured: unary 270 fs, both alloys 45-50 fs, the ionic
# stand-in with its light species 18 fs).  A run that would leave this horizon takes a proportionally smaller time step; the
# work per step (lists, pairs, kernels, rebuild every 10 steps) does not depend on dt.
SAFE_TRAJECTORY_FS = {2: 120.0, 3: 24.0, 4: 8.0, 5: 24.0}


def time_step_fs(n_steps_total: int, cfg: int = CFG) -> float:
    return min(DT_FS, SAFE_TRAJECTORY_FS[cfg] / max(1, n_steps_total))

# Algorithmic work (fp32 operations, FMA = 2) of the fused kernel, per unit, with d = 16, k = 32:
#   pair: geometry 60 + harmonics 150 + spline value 192 and value + derivative 320 + Eq. 4 (2 d k = 1,024)
#         + Eq. 8-9 (4 d k = 2,048) + projection 168
#   atom: invariants and Eq. 7 (3 d k = 1,536) + head forward and reverse (82,176) + SiLU (~5,000)
FLOP_PER_PAIR = 3960.0         # pair inside r_cut: both neighbor loops (geometry, harmonics, spline, 6 d k contraction)
FLOP_PER_SKIN_ENTRY = 24.0     # list entry between r_cut and r_cut + skin: distance test in both loops
FLOP_PER_ATOM = 88700.0        # invariants, W_i, head forward + reverse, SiLU
FP32_LANES_PER_SM = 128
FP64_LANES_PER_SM = 64         # fp64 path: DFMA lanes per SM

# DRAM traffic of one fused-kernel launch comes from the committed ncu capture of a 500,000-atom launch
# (dram__bytes_read.sum + dram__bytes_write.sum per atom; the traffic is per-atom, so a launch of N atoms is reported as
# that figure times N).  The record names the kernel sources it was captured from; a different kernel prints no traffic.
TRAFFIC_RECORD = os.path.join(ROOT, "profiles", "k_mega_hea6_fcc50.traffic.txt")
KERNEL_SOURCES = ["megakernel.cu", "pair_math.cuh", "common.cuh"]


def kernel_revision() -> str:
    """Hash of the fused kernel's sources: ties a profiler record to the code it was taken from."""
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2608_16329_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def recorded_traffic():
    """(bytes per atom, note) from the ncu record, or (None, why) when it does not belong to the kernel as built."""
    try:
        rec = dict(line.split(":", 1) for line in open(TRAFFIC_RECORD) if ":" in line and not line.startswith("#"))
        rev, per_atom = rec["kernel_revision"].strip(), float(rec["dram_bytes_per_atom"])
    except (OSError, KeyError, ValueError):
        return None, "no ncu record"
    if rev != kernel_revision():
        return None, f"ncu record is of kernel revision {rev}, this kernel is {kernel_revision()}"
    return per_atom, f"ncu capture of a 500,000-atom launch scaled per atom (kernel revision {rev})"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cells", type=int, default=DEFAULT_CELLS, help="FCC cells per edge (N = 4 cells^3)")
    ap.add_argument("--cpu-centers", type=int, default=49152, help="central atoms in the CPU-oracle sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--cfg", type=int, default=CFG, choices=[2, 3, 4, 5],
                    help="workload: 5 = the 6-species alloy the metric is quoted on (default); 2, 3, 4 = the unary, "
                         "3-species alloy and ionic stand-ins at their full sizes (extra data points, not the contract line)")
    ap.add_argument("--precision", default="f32", choices=["f32", "f64"],
                    help="f64 runs the double-precision evaluation path instead (an extra data point, not the contract line)")
    ap.add_argument("--deterministic", action="store_true",
                    help="force_mode = 1: integer accumulation of forces, energy and virial (bit-reproducible): an extra data point")
    ap.add_argument("--ensemble", default="nve", choices=["nve", "nvt"],
                    help="nvt adds the Nose-Hoover-chain thermostat (the paper's ensemble) to every step: an extra data point")
    ap.add_argument("--k", type=int, default=32, choices=[16, 32, 64], help="radial channels (other than 32: --precision f64 only)")
    ap.add_argument("--lmax", type=int, default=3, choices=[1, 2, 3, 4, 5], help="angular order (other than 3: --precision f64 only; 4, 5: k = 32)")
    ap.add_argument("--basis", default="irreducible", choices=["irreducible", "canonical"],
                    help="canonical = all Cartesian monomials with the multiplicity metric, the descriptor before the "
                         "irreducible reduction (d = 20 at l_max = 3): --precision f64 only")
    ap.add_argument("--list16", action="store_true",
                    help="list_format = 1: neighbor lists as 16-bit cell-relative codes (half the list bytes): an extra data point")
    ap.add_argument("--sweep", default="", help="comma-separated FCC cell counts: size sweep of the 6-species workload "
                    "(inputs generated on the device), one JSON line per size; not the contract line")
    return ap.parse_args()


class ClockSampler:
    """nvidia-smi clock / throttle sampling in the background during the timed region."""

    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, sm_max, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                p = [x.strip() for x in line.split(",")]
                if len(p) < 9:
                    continue
                try:
                    sm.append(float(p[1])); sm_max.append(float(p[2])); power.append(float(p[3]))
                except ValueError:
                    continue
                for name, val in zip(names, p[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.path)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(sm_max)), "reasons": sorted(reasons),
                "power_w_max": float(max(power)), "samples": len(sm)}


def max_over_ranks(x: float, device) -> float:
    """Slowest rank's time: the number every rank reports against (no-op for a single process)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(atoms_per_rank: int, steps: int, seconds_max: float, world: int) -> float:
    """Replicas: every rank advances its own atoms; aggregate = all ranks' atom-steps over the slowest rank's time."""
    return world * atoms_per_rank * steps / seconds_max


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "sm_max_mhz": 1965.0}, "fallback"


LATTICES = {2: ((32, 32, 32), 2, 3.3), 3: ((64, 64, 64), 4, 4.05), 4: ((125, 125, 128), 1, 20.0 ** (1.0 / 3.0))}


def sample_blocks(cells, n_basis, a, r_cut, n_centers, seed=0):
    """Central atoms for the CPU leg: rectangular blocks of unit cells spread over the box (caller indices; lattice
    sites are numbered (ix, iy, iz, basis)).  Returns (all block atoms, those far enough inside a block that every atom
    within r_cut of them is in the block too -- the atoms whose complete force the block's evaluation gives)."""
    size = tuple(min(c, s) for c, s in zip(cells, (8, 8, 24)))
    per_block = size[0] * size[1] * size[2] * n_basis
    n_blocks = max(1, n_centers // per_block)
    margin = int(np.ceil((r_cut + 0.75) / a))
    rng = np.random.default_rng(seed)
    origins = [(0, 0, 0), tuple(c - s for c, s in zip(cells, size))]
    while len(origins) < n_blocks:
        origins.append(tuple(int(rng.integers(0, c - s + 1)) for c, s in zip(cells, size)))
    all_atoms, inner = [], []
    for o in origins[:n_blocks]:
        ix, iy, iz, b = np.meshgrid(*[o[d] + np.arange(size[d]) for d in range(3)], np.arange(n_basis), indexing="ij")
        idx = (((ix * cells[1] + iy) * cells[2] + iz) * n_basis + b)
        all_atoms.append(idx.ravel())
        if min(size) > 2 * margin:
            inner.append(idx[margin:size[0] - margin, margin:size[1] - margin, margin:size[2] - margin].ravel())
    all_atoms = np.unique(np.concatenate(all_atoms)).astype(np.int64)
    inner = np.unique(np.concatenate(inner)).astype(np.int64) if inner else np.empty(0, np.int64)
    return all_atoms, inner


def cpu_oracle_sample(w, enc, head, n_centers, repeats=1, rows=None, pos=None, k=32, l_max=3, basis=0):
    """Time the oracle (neighbor search + full evaluation) on `rows` (default: evenly spread central atoms).
    Returns (rows, seconds, threads, the oracle's outputs)."""
    import oracle
    model = oracle.Model(w.n_species, w.r_cut, enc, head, k=k, l_max=l_max, basis=basis)
    if rows is None:
        rows = np.unique(np.linspace(0, w.n_atoms - 1, n_centers).astype(np.int64))
    pos = w.pos if pos is None else pos
    best, out = None, None
    for _ in range(repeats):
        t0 = time.perf_counter()
        nl = oracle.neighbors(pos, w.species, w.n_species, w.box, w.r_cut + w.skin, rows=rows)
        out = oracle.compute(model, pos, w.species, w.box, nl)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return rows, best, oracle.num_threads(), out


def problem_setup(args, rank=0):
    """Workload, weights and the algorithmic work per unit for the flags given (no GPU needed)."""
    import workloads as wl
    cfg = args.cfg
    w = wl.make_workload(cfg, n_cells=args.cells if cfg == CFG else None, seed=wl.BASE_SEED + cfg + 17 * rank)
    canonical = args.basis == "canonical"
    default_shape = args.k == 32 and args.lmax == 3 and not canonical
    if default_shape:
        enc, head = wl.workload_weights(cfg, w.n_species)
    else:   # descriptor-shape variants of the paper's ablations: same recipe, networks of that shape
        enc, head = wl.make_weights(w.n_species, wl.BASE_SEED + cfg + 1000, wl.ENC_OUT_SCALE[cfg], wl.HEAD_OUT_SCALE[cfg],
                                    k=args.k, l_max=args.lmax)
    flop_pair, flop_atom = FLOP_PER_PAIR, FLOP_PER_ATOM
    if not default_shape:   # the same count written out in k and d = (l_max + 1)^2
        d_ang = (args.lmax + 1) * (args.lmax + 2) * (args.lmax + 3) // 6 if canonical else (args.lmax + 1) ** 2
        n_inv = (args.lmax + 1) * args.k
        flop_pair = 60 + 150 * d_ang / 16 + 512 * args.k / 32 + 6 * d_ang * args.k + 168 * d_ang / 16
        flop_atom = 3 * d_ang * args.k + 4 * (n_inv * 64 + 3 * 64 * 64) + 256 + 5000
    lattice = ((args.cells,) * 3, 4, 3.6) if cfg == CFG else LATTICES[cfg]
    return {"w": w, "enc": enc, "head": head, "default_shape": default_shape, "flop_pair": flop_pair, "flop_atom": flop_atom,
            "rebuild_every": REBUILD_EVERY if cfg != 4 else 3,   # the ionic stand-in is far from equilibrium under random weights
            "lattice": lattice, "f64": args.precision == "f64", "basis": 1 if canonical else 0}


def run_reference(args, rank, world):
    """CPU oracle arm: each step evaluates a bounded sample of central atoms of the same workload."""
    if rank != 0:
        return
    import workloads as wl
    w = wl.make_workload(CFG, n_cells=args.cells)
    enc, head = wl.workload_weights(CFG, w.n_species)
    n_centers = min(args.cpu_centers, 2048)
    for _ in range(args.warmup):
        cpu_oracle_sample(w, enc, head, 64)
    t0 = time.perf_counter()
    done, cores = 0, 1
    for _ in range(args.steps):
        rows, _, cores, _ = cpu_oracle_sample(w, enc, head, n_centers)
        done += rows.size
    dt = time.perf_counter() - t0
    value = done / dt
    sample = (f"{n_centers} central atoms spread evenly over the {w.n_atoms}-atom workload per step: cell-list "
              f"neighbor search for those atoms + full fp64 energy/force/virial evaluation of them")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * dt / max(args.steps, 1), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"cfg5 hea6 fcc{args.cells} ({w.n_atoms} atoms)", "sampled_atoms_per_step": n_centers},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def run_sweep(args):
    """Throughput and footprint versus system size up to what fits in HBM (the paper's Fig. 4(b) analogue).
    Lattice, displacements, species and velocities are drawn on the device with a seeded torch generator."""
    import torch
    import paper_2608_16329_b200 as mlip
    import workloads as wl
    dev = torch.device("cuda", 0)
    enc, head = wl.workload_weights(CFG, 6)
    masses = np.array(wl.MASSES[CFG])
    for cells in [int(x) for x in args.sweep.split(",") if x]:
        n = 4 * cells ** 3
        line = {"sweep": True, "cells": cells, "atoms": n}
        pot = None
        try:
            gen = torch.Generator(device=dev)
            gen.manual_seed(wl.BASE_SEED + cells)
            a = 3.6
            idx = torch.arange(n, device=dev, dtype=torch.int64)
            basis = torch.tensor(wl._FCC_BASIS, device=dev, dtype=torch.float64)[idx % 4]
            cell = torch.div(idx, 4, rounding_mode="floor")
            pos = torch.stack([torch.div(cell, cells * cells, rounding_mode="floor"), torch.div(cell, cells, rounding_mode="floor") % cells,
                               cell % cells], dim=1).to(torch.float64)
            del idx, cell
            pos = (pos + basis) * a
            del basis
            pos += 0.05 * torch.randn(pos.shape, generator=gen, device=dev, dtype=torch.float64)
            box = np.full(3, cells * a)
            pos -= torch.floor(pos / (cells * a)) * (cells * a)
            pos.clamp_(0.0, float(np.nextafter(cells * a, 0.0)))
            species = torch.randint(0, 6, (n,), generator=gen, device=dev, dtype=torch.int32)
            pot = mlip.Potential(6, 6.0, 1.0, enc, head, masses, list_format=1 if args.list16 else 0)
            pot.n = n
            mlip.mlip_build_neighbors(pot.ctx, pos, species, box)
            sig = torch.sqrt(torch.tensor(wl.KB_EV_PER_K * 300.0 * wl.ACC_UNIT / masses, device=dev))[species.long()]
            vel = torch.randn(pos.shape, generator=gen, device=dev, dtype=torch.float64) * sig[:, None]
            mlip.mlip_set_velocities(pot.ctx, vel)
            del pos, species, vel, sig
            torch.cuda.empty_cache()
            dt_fs = time_step_fs(args.warmup + args.steps, CFG)
            pot.step(args.warmup, dt_fs, REBUILD_EVERY)
            torch.cuda.synchronize()
            mlip.mlip_kernel_time(pot.ctx, reset=True)
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record()
            pot.step(args.steps, dt_fs, REBUILD_EVERY)
            ev1.record()
            torch.cuda.synchronize()
            ms = ev0.elapsed_time(ev1)
            k_n, k_ms = mlip.mlip_kernel_time(pot.ctx)
            status = pot.sync_status(raise_on_error=False)
            line.update({"atom_steps_per_s": n * args.steps / (ms * 1e-3), "ms_per_step": ms / args.steps,
                         "kernel_ms": k_ms / max(k_n, 1), "resident_GB": mlip.mlip_resident_bytes(pot.ctx) / 1e9,
                         "resident_bytes_per_atom": mlip.mlip_resident_bytes(pot.ctx) / n,
                         "status": mlip.binding.ERRORS.get(status, status)})
        except Exception as exc:   # out of memory ends the sweep
            line["error"] = str(exc)[:200]
        print(json.dumps(line), flush=True)
        if pot is not None:
            pot.close()
        torch.cuda.empty_cache()
        if "error" in line:
            break


def main():
    args = parse_args()
    if args.sweep:
        run_sweep(args)
        return
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import torch
    import torch.distributed as dist
    import paper_2608_16329_b200 as mlip
    import workloads as wl

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    cfg = args.cfg
    prob = problem_setup(args, rank)
    w, enc, head, default_shape, rebuild_every, f64 = (prob[q] for q in ("w", "enc", "head", "default_shape", "rebuild_every", "f64"))
    n = w.n_atoms
    pot = mlip.Potential(w.n_species, w.r_cut, w.skin, enc, head, w.masses, device=local_rank, precision=1 if f64 else 0,
                         k=args.k, l_max=args.lmax, force_mode=1 if args.deterministic else 0, basis=prob["basis"],
                         list_format=1 if args.list16 else 0)
    table_err = mlip.mlip_table_error(pot.ctx)

    # ---- device-resident run: inputs already in HBM when timing starts ----
    pot.build_neighbors(w.pos, w.species, w.box)
    pot.set_velocities(w.vel)
    dt_fs = time_step_fs(args.warmup + args.steps, cfg)
    def advance(n_steps):
        if args.ensemble == "nvt":
            pot.step_nvt(n_steps, dt_fs, rebuild_every, w.temperature, 100.0)
        else:
            pot.step(n_steps, dt_fs, rebuild_every)

    advance(args.warmup)
    pot.sync_status()
    barrier()
    mlip.mlip_get_timings(pot.ctx, reset=True)
    launches0 = mlip.mlip_get_counters(pot.ctx)["launches"]
    gpu_index = local_rank
    try:   # nvidia-smi numbers physical devices; honour a numeric CUDA_VISIBLE_DEVICES mapping
        gpu_index = int(os.environ.get("CUDA_VISIBLE_DEVICES", "").split(",")[local_rank])
    except (ValueError, IndexError):
        pass
    sampler = ClockSampler(gpu_index)
    if rank == 0:
        sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    advance(args.steps)
    ev1.record()
    barrier()
    ms = ev0.elapsed_time(ev1)
    clocks = sampler.stop() if rank == 0 else None
    status = pot.sync_status(raise_on_error=False)
    counters = mlip.mlip_get_counters(pot.ctx)
    t_build, t_kernel, t_integrate = mlip.mlip_get_timings(pot.ctx)
    k_launches, k_ms = mlip.mlip_kernel_time(pot.ctx, reset=True)
    e_final = pot.energies().cpu().numpy()
    ms_max = max_over_ranks(ms, dev)
    value = whole_job_value(n, args.steps, ms_max * 1e-3, world)

    # ---- end to end: host buffers through mlip_compute_host, copies inside the timed region ----
    e2e = None
    if not args.no_e2e:
        pos_a = torch.from_numpy(w.pos).pin_memory()
        rng = np.random.default_rng(1)
        shifted = w.pos + rng.uniform(-0.1, 0.1, w.pos.shape)
        shifted -= np.floor(shifted / w.box) * w.box
        shifted[shifted >= w.box] = 0.0
        pos_b = torch.from_numpy(shifted).pin_memory()
        species_h = torch.from_numpy(w.species).pin_memory()
        forces_h = torch.empty((n, 3), dtype=torch.float32).pin_memory()
        virial_h = np.zeros(9)
        mlip.mlip_compute_host(pot.ctx, pos_a, species_h, w.box, True, forces_h, virial_h)
        for i in range(2):
            mlip.mlip_compute_host(pot.ctx, pos_b if i % 2 == 0 else pos_a, None, None, False, forces_h, virial_h)
        barrier()
        e2e_steps = args.steps
        t0 = time.perf_counter()
        for i in range(e2e_steps):
            rebuild = (i % REBUILD_EVERY == 0)
            p = pos_a if i % 2 == 0 else pos_b
            mlip.mlip_compute_host(pot.ctx, p, species_h if rebuild else None, w.box if rebuild else None, rebuild,
                                   forces_h, virial_h)
        torch.cuda.synchronize()
        dt = max_over_ranks(time.perf_counter() - t0, dev)
        n_rebuilds = (e2e_steps + REBUILD_EVERY - 1) // REBUILD_EVERY
        e2e = {"value": whole_job_value(n, e2e_steps, dt, world), "unit": UNIT,
               "h2d_bytes_per_step": int(24 * n + 4 * n * n_rebuilds / e2e_steps),
               "d2h_bytes_per_step": int(12 * n + 80),
               "call": "mlip_compute_host (positions in, forces + energy + virial out, list rebuild every 10th call)"}

    if rank == 0:
        peaks, peak_kind = measured_peaks()
        props = torch.cuda.get_device_properties(local_rank)
        n_sm = props.multi_processor_count
        sm_max = (clocks or {}).get("sm_max_mhz") or peaks.get("sm_max_mhz", 1965.0)
        lanes = FP64_LANES_PER_SM if f64 else FP32_LANES_PER_SM
        peak_tflops = n_sm * lanes * 2 * sm_max * 1e6 / 1e12
        pairs = counters["pairs_in_cutoff"]
        entries = counters["list_entries"]
        flop_pair, flop_atom = prob["flop_pair"], prob["flop_atom"]
        flop = flop_pair * pairs + FLOP_PER_SKIN_ENTRY * max(entries - pairs, 0) + flop_atom * n
        k_avg_ms = k_ms / max(k_launches, 1)
        achieved = flop / (k_avg_ms * 1e-3) / 1e12
        roofline = {"bound": "alu", "kernel": "k_mega_f64" if f64 else "k_mega", "achieved": achieved, "peak": peak_tflops, "unit": "TFLOP/s",
                    "frac": achieved / peak_tflops,
                    "peak_source": f"{n_sm} SMs x {lanes} fp{args.precision[1:]} lanes x 2 x {sm_max:.0f} MHz (max SM clock)",
                    "kernel_ms_avg": k_avg_ms, "kernel_launches_timed": k_launches,
                    "kernel_share_of_step": k_ms / ms if ms > 0 else None,
                    "flop_per_launch": flop, "pairs_in_cutoff_per_atom": pairs / n, "list_entries_per_atom": entries / n,
                    "hbm_peak_gbs": peaks["hbm_gbs"], "hbm_peak_kind": f"of {peak_kind}"}
        per_atom, traffic_note = recorded_traffic() if (default_shape and not f64 and cfg == CFG and not args.list16) else (None, "no ncu record for this variant")
        roofline["traffic"] = None if per_atom is None else per_atom * n
        roofline["traffic_source"] = traffic_note
        if clocks and clocks.get("sm_mhz"):
            roofline["frac_at_sampled_clock"] = achieved / (n_sm * lanes * 2 * clocks["sm_mhz"] * 1e6 / 1e12)
        if not f64:   # the same fraction against an FMA-saturating kernel timed in this process
            ffma = mlip.mlip_measure_fp32_peak(local_rank)
            roofline["peak_measured_ffma"] = ffma
            roofline["frac_of_measured_ffma"] = achieved / ffma
        resident = mlip.mlip_resident_bytes(pot.ctx)
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                "ms_per_step": ms_max / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": args.precision, "data": "synthetic",
                "config": {"workload": f"cfg{cfg} {w.name}: {n} atoms, {w.n_species} species, r_cut 6 A, skin 1 A, "
                                       f"{args.ensemble.upper()} dt {dt_fs:.3g} fs, list rebuild every {rebuild_every} steps"
                                       + ("" if default_shape else f", k = {args.k}, l_max = {args.lmax}, {args.basis} basis")
                                       + (", deterministic force mode" if args.deterministic else "")
                                       + (", 16-bit neighbor codes" if args.list16 else ""),
                           "atoms_per_gpu": n, "parallelism": "replicas" if world > 1 else "single",
                           "l2": "inputs larger than L2 (positions + lists = %.1f GB per GPU)" % ((32 * n + 4 * entries) / 1e9)},
                "clocks": clocks, "e2e": e2e, "gpu_launches": counters["launches"] - launches0,
                "roofline": roofline,
                "device_ms_per_step": {"list_build": t_build / args.steps, "fused_kernel": t_kernel / args.steps,
                                       "integrator": t_integrate / args.steps},
                "resident_bytes_per_atom": resident / n,
                "max_atoms_in_180GB_extrapolated": int(180e9 / (resident / n)),
                "table_error": {"value": table_err[0], "deriv": table_err[1]},
                "status": mlip.binding.ERRORS.get(status, status),
                "energy_final_eV": {"potential": float(e_final[0]), "kinetic": float(e_final[1])}}
        if not args.no_cpu_baseline and world == 1:
            # The oracle on blocks of central atoms at the positions the run ended on; its outputs are then compared
            # with the GPU's evaluation of the same state: E_i of every sampled atom, the force of the blocks' interior
            # atoms (those whose whole r_cut neighborhood was evaluated).
            cells, n_basis, a_lat = prob["lattice"]
            rows, inner = sample_blocks(cells, n_basis, a_lat, w.r_cut, args.cpu_centers)
            pos_t, _, _ = pot.state()
            gpu = pot.compute(want_e_atom=True)
            pot.sync_status(raise_on_error=False)
            pos_now = pos_t.cpu().numpy()
            rows, sec, cores, ref = cpu_oracle_sample(w, enc, head, rows.size, rows=rows, pos=pos_now, k=args.k, l_max=args.lmax, basis=prob["basis"])
            line["cpu_baseline"] = {"value": rows.size / sec, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": f"{rows.size} central atoms in blocks of cells spread over the {n}-atom workload, one "
                                              f"energy/force/virial evaluation incl. their neighbor search ({sec:.1f} s)"}
            rows_t, inner_t = torch.as_tensor(rows, device=dev), torch.as_tensor(inner, device=dev)
            d_e = np.abs(gpu["e_atom"][rows_t].double().cpu().numpy() - ref["e_atom"][rows])
            d_f = np.abs(gpu["forces"][inner_t].double().cpu().numpy() - ref["forces"][inner]) if inner.size else np.zeros(1)
            e_tol, f_tol = (1e-9, 2e-9) if f64 else (2e-5, 1e-4)
            e_tol *= max(1.0, float(np.abs(ref["e_atom"][rows]).max()))
            if not default_shape and inner.size:   # networks of other shapes are not calibrated to forces of order 1 eV/Angstrom
                f_tol *= max(1.0, float(np.abs(ref["forces"][inner]).max()))
            line["parity"] = {"against": "oracle, same state (the positions the context held after the timed runs)", "n_atoms_e": int(rows.size),
                              "max_dE_i": float(d_e.max()), "n_atoms_f": int(inner.size), "max_dF": float(d_f.max()),
                              "tolerance": {"dE_i": e_tol, "dF": f_tol},
                              "ok": bool(d_e.max() <= e_tol and d_f.max() <= f_tol)}
        print(json.dumps(line), flush=True)
    pot.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
