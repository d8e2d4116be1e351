"""ctypes binding of include/mlip.h: argument marshalling only.

The functions carry the C entry points' names and take torch tensors (device
memory), numpy arrays (host memory) and plain numbers; every step of the path
runs inside the CUDA library.  Loading fails loudly if the library is missing:
there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("MLIP_B200_LIB") or os.path.join(_PKG, "libmlip_b200.so")

OK = 0
ERRORS = {0: "MLIP_OK", 1: "MLIP_ERR_INVALID_ARG", 2: "MLIP_ERR_UNSUPPORTED", 3: "MLIP_ERR_BOX_TOO_SMALL",
          4: "MLIP_ERR_NEIGHBOR_OVERFLOW", 5: "MLIP_ERR_SKIN_EXCEEDED", 6: "MLIP_ERR_NONFINITE",
          7: "MLIP_ERR_TABLE_TOLERANCE", 8: "MLIP_ERR_NOT_BUILT", 9: "MLIP_ERR_OOM", 10: "MLIP_ERR_CUDA",
          11: "MLIP_ERR_TABLE_RANGE"}
CODES = {v: k for k, v in ERRORS.items()}

EXPORTS = ["mlip_create", "mlip_table_error", "mlip_build_neighbors", "mlip_build_neighbors_ghost", "mlip_get_neighbors", "mlip_get_neighbors_noalloc", "mlip_set_positions",
           "mlip_set_velocities", "mlip_compute", "mlip_compute_f64", "mlip_compute_host", "mlip_step", "mlip_step_nvt", "mlip_get_thermostat", "mlip_reset_thermostat", "mlip_get_rebuilds", "mlip_get_state", "mlip_set_state", "mlip_debug_rebuild",
           "mlip_get_energies", "mlip_sync_status", "mlip_get_counters", "mlip_kernel_time", "mlip_get_timings", "mlip_measure_fp32_peak",
           "mlip_resident_bytes", "mlip_last_error", "mlip_destroy"]


class MlipError(RuntimeError):
    def __init__(self, code, message=""):
        self.code = code
        super().__init__(f"{ERRORS.get(code, code)}: {message}")


class Config(ctypes.Structure):
    _fields_ = [("n_species", ctypes.c_int), ("r_cut", ctypes.c_double), ("skin", ctypes.c_double),
                ("k", ctypes.c_int), ("l_max", ctypes.c_int),
                ("enc_hidden", ctypes.c_int), ("enc_layers", ctypes.c_int),
                ("head_hidden", ctypes.c_int), ("head_layers", ctypes.c_int),
                ("table_knots", ctypes.c_int), ("table_r_min", ctypes.c_double), ("table_tol", ctypes.c_double),
                ("device", ctypes.c_int), ("precision", ctypes.c_int),
                ("enc_conditioning", ctypes.c_int), ("head_conditioning", ctypes.c_int), ("force_mode", ctypes.c_int),
                ("envelope", ctypes.c_int), ("basis", ctypes.c_int), ("list_format", ctypes.c_int)]


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -c 'import __graft_entry__ as g; g.build()'` "
                              "(nvcc, sm_100a). There is no fallback path.")
        _lib = ctypes.CDLL(LIB_PATH)
        _lib.mlip_resident_bytes.restype = ctypes.c_size_t
        _lib.mlip_last_error.restype = ctypes.c_char_p
        _lib.mlip_destroy.restype = None
    return _lib


def _dev(t):
    """Device pointer of a CUDA torch tensor (or None)."""
    if t is None:
        return ctypes.c_void_p(0)
    assert t.is_cuda and t.is_contiguous()
    return ctypes.c_void_p(t.data_ptr())


def _host(a):
    if a is None:
        return ctypes.c_void_p(0)
    if hasattr(a, "data_ptr"):      # pinned CPU torch tensor
        assert not a.is_cuda and a.is_contiguous()
        return ctypes.c_void_p(a.data_ptr())
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.c_void_p)


def _stream(stream):
    if stream is None:
        import torch
        return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    return ctypes.c_void_p(int(stream))


def _check(ctx, rc, allow=()):
    if rc != OK and rc not in allow:
        msg = lib().mlip_last_error(ctx)
        raise MlipError(rc, msg.decode() if msg else "")
    return rc


def mlip_create(cfg: Config, enc_w: np.ndarray, head_w: np.ndarray, masses: np.ndarray, allow_table_error=False):
    enc_w = np.ascontiguousarray(enc_w, dtype=np.float64)
    head_w = np.ascontiguousarray(head_w, dtype=np.float64)
    masses = np.ascontiguousarray(masses, dtype=np.float64)
    ctx = ctypes.c_void_p(0)
    rc = lib().mlip_create(ctypes.byref(ctx), ctypes.byref(cfg), _host(enc_w), ctypes.c_size_t(enc_w.size),
                           _host(head_w), ctypes.c_size_t(head_w.size), _host(masses))
    _check(ctx if ctx.value else None, rc, allow=(CODES["MLIP_ERR_TABLE_TOLERANCE"],) if allow_table_error else ())
    return ctx


def mlip_table_error(ctx):
    a, b = ctypes.c_double(0), ctypes.c_double(0)
    _check(ctx, lib().mlip_table_error(ctx, ctypes.byref(a), ctypes.byref(b)))
    return a.value, b.value


def _cell(box):
    """Row-major cell vectors [9] from three edge lengths, nine numbers or a 3 x 3 matrix."""
    box = np.asarray(box, dtype=np.float64)
    if box.size == 3:
        box = np.diag(box.ravel())
    assert box.size == 9, "box: three edge lengths or the 3 x 3 cell vectors"
    return np.ascontiguousarray(box.ravel())


def mlip_build_neighbors(ctx, pos, species, box, stream=None):
    box = _cell(box)
    _check(ctx, lib().mlip_build_neighbors(ctx, ctypes.c_int64(pos.shape[0]), _dev(pos), _dev(species), _host(box), _stream(stream)))


def mlip_build_neighbors_ghost(ctx, n_owned, pos, species, box, stream=None):
    """Owned atoms first (pos[:n_owned] are the central atoms), ghosts after them."""
    box = _cell(box)
    n = pos.shape[0]
    _check(ctx, lib().mlip_build_neighbors_ghost(ctx, ctypes.c_int64(n_owned), ctypes.c_int64(n - n_owned), _dev(pos), _dev(species),
                                                 _host(box), _stream(stream)))


def mlip_get_neighbors(ctx, seg_ptr, nbr, stream=None):
    n = ctypes.c_int64(0)
    cap = 0 if nbr is None else nbr.numel()
    rc = lib().mlip_get_neighbors(ctx, _dev(seg_ptr), _dev(nbr), ctypes.c_int64(cap), ctypes.byref(n), _stream(stream))
    _check(ctx, rc, allow=(CODES["MLIP_ERR_NEIGHBOR_OVERFLOW"],))
    return rc, n.value


def mlip_get_neighbors_noalloc(ctx, seg_ptr, nbr, stream=None):
    """mlip_get_neighbors for callers that must not allocate device memory: the export's temporaries
    sit in a static device array inside the library (n_atoms * n_species <= 1,048,576).  Returns
    (status, number of entries); an unsupported size raises MlipError."""
    n = ctypes.c_int64(0)
    cap = 0 if nbr is None else nbr.numel()
    rc = lib().mlip_get_neighbors_noalloc(ctx, _dev(seg_ptr), _dev(nbr), ctypes.c_int64(cap), ctypes.byref(n), _stream(stream))
    _check(ctx, rc, allow=(CODES["MLIP_ERR_NEIGHBOR_OVERFLOW"],))
    return rc, n.value


def mlip_set_positions(ctx, pos, stream=None):
    _check(ctx, lib().mlip_set_positions(ctx, _dev(pos), _stream(stream)))


def mlip_set_velocities(ctx, vel, stream=None):
    _check(ctx, lib().mlip_set_velocities(ctx, _dev(vel), _stream(stream)))


def mlip_compute(ctx, energy=None, forces=None, virial=None, e_atom=None, stream=None):
    _check(ctx, lib().mlip_compute(ctx, _dev(energy), _dev(forces), _dev(virial), _dev(e_atom), _stream(stream)))


def mlip_compute_f64(ctx, energy=None, forces=None, virial=None, e_atom=None, stream=None):
    _check(ctx, lib().mlip_compute_f64(ctx, _dev(energy), _dev(forces), _dev(virial), _dev(e_atom), _stream(stream)))


def mlip_compute_host(ctx, pos, species, box, rebuild, forces_out, virial_out=None):
    e = ctypes.c_double(0)
    box = None if box is None else _cell(box)
    _check(ctx, lib().mlip_compute_host(ctx, ctypes.c_int64(pos.shape[0]), _host(pos), _host(species), _host(box),
                                        ctypes.c_int(int(rebuild)), ctypes.byref(e), _host(forces_out), _host(virial_out)))
    return e.value


def mlip_step(ctx, n_steps, dt_fs, rebuild_every, stream=None):
    _check(ctx, lib().mlip_step(ctx, ctypes.c_int(n_steps), ctypes.c_double(dt_fs), ctypes.c_int(rebuild_every), _stream(stream)))


def mlip_step_nvt(ctx, n_steps, dt_fs, rebuild_every, t_target_K, t_damp_fs, stream=None):
    _check(ctx, lib().mlip_step_nvt(ctx, ctypes.c_int(n_steps), ctypes.c_double(dt_fs), ctypes.c_int(rebuild_every),
                                    ctypes.c_double(t_target_K), ctypes.c_double(t_damp_fs), _stream(stream)))


def mlip_get_thermostat(ctx):
    """(v_eta [3], eta [3], thermostat energy in eV)."""
    v, e, en = (ctypes.c_double * 3)(), (ctypes.c_double * 3)(), ctypes.c_double(0)
    _check(ctx, lib().mlip_get_thermostat(ctx, v, e, ctypes.byref(en)))
    return np.array(v[:]), np.array(e[:]), en.value


def mlip_reset_thermostat(ctx):
    _check(ctx, lib().mlip_reset_thermostat(ctx))


def mlip_get_timings(ctx, reset=False):
    """Device ms spent in (list builds, fused kernel, integrator kernels) since the last reset."""
    b, k, i = ctypes.c_double(0), ctypes.c_double(0), ctypes.c_double(0)
    _check(ctx, lib().mlip_get_timings(ctx, ctypes.byref(b), ctypes.byref(k), ctypes.byref(i), ctypes.c_int(int(reset))))
    return b.value, k.value, i.value


def mlip_get_rebuilds(ctx) -> int:
    n = ctypes.c_int64(0)
    _check(ctx, lib().mlip_get_rebuilds(ctx, ctypes.byref(n)))
    return n.value


def mlip_get_state(ctx, pos=None, vel=None, stream=None):
    step = ctypes.c_int64(0)
    _check(ctx, lib().mlip_get_state(ctx, _dev(pos), _dev(vel), ctypes.byref(step), _stream(stream)))
    return step.value


def mlip_set_state(ctx, pos=None, vel=None, step=0, v_eta=None, eta=None, stream=None):
    v_eta = None if v_eta is None else np.ascontiguousarray(v_eta, dtype=np.float64)
    eta = None if eta is None else np.ascontiguousarray(eta, dtype=np.float64)
    _check(ctx, lib().mlip_set_state(ctx, _dev(pos), _dev(vel), ctypes.c_int64(step), _host(v_eta), _host(eta), _stream(stream)))


def mlip_debug_rebuild(ctx, spin_limit, unpublished_tile=-1, stream=None):
    _check(ctx, lib().mlip_debug_rebuild(ctx, ctypes.c_int(spin_limit), ctypes.c_int64(unpublished_tile), _stream(stream)))


def mlip_get_energies(ctx, e_pot=None, e_kin=None, stream=None):
    _check(ctx, lib().mlip_get_energies(ctx, _dev(e_pot), _dev(e_kin), _stream(stream)))


def mlip_sync_status(ctx, raise_on_error=True):
    rc = lib().mlip_sync_status(ctx)
    if raise_on_error:
        _check(ctx, rc)
    return rc


def mlip_get_counters(ctx):
    a, b, c = ctypes.c_int64(0), ctypes.c_int64(0), ctypes.c_int64(0)
    _check(ctx, lib().mlip_get_counters(ctx, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)))
    return {"list_entries": a.value, "pairs_in_cutoff": b.value, "launches": c.value}


def mlip_kernel_time(ctx, reset=False):
    """(launches timed, summed fused-kernel milliseconds) since the last reset."""
    n, ms = ctypes.c_int64(0), ctypes.c_double(0)
    _check(ctx, lib().mlip_kernel_time(ctx, ctypes.byref(n), ctypes.byref(ms), ctypes.c_int(int(reset))))
    return n.value, ms.value


def mlip_measure_fp32_peak(device=0) -> float:
    """Measured fp32 FMA rate of the device in TFLOP/s."""
    v = ctypes.c_double(0)
    rc = lib().mlip_measure_fp32_peak(ctypes.c_int(device), ctypes.byref(v))
    if rc != OK:
        raise MlipError(rc, "fp32 peak measurement failed")
    return v.value


def mlip_resident_bytes(ctx):
    return int(lib().mlip_resident_bytes(ctx))


def mlip_last_error(ctx=None):
    msg = lib().mlip_last_error(ctx)
    return msg.decode() if msg else ""


def mlip_destroy(ctx):
    if ctx is not None and ctx.value:
        lib().mlip_destroy(ctx)
        ctx.value = 0


class Potential:
    """Convenience owner of one context; allocates outputs as torch tensors."""

    def __init__(self, n_species, r_cut, skin, enc_w, head_w, masses, device=0, table_knots=0,
                 table_r_min=0.0, table_tol=0.0, enc_hidden=128, enc_layers=3, allow_table_error=False, precision=0,
                 enc_conditioning=0, head_conditioning=0, k=32, l_max=3, envelope=0, force_mode=0, basis=0, list_format=0):
        import torch
        self.torch = torch
        self.device = torch.device("cuda", device)
        self.n_species = n_species
        self.cfg = Config(n_species, r_cut, skin, k, l_max, enc_hidden, enc_layers, 64, 4, table_knots, table_r_min,
                          table_tol, device, precision, enc_conditioning, head_conditioning, force_mode, envelope, basis, list_format)
        self.precision = precision
        self.ctx = mlip_create(self.cfg, enc_w, head_w, masses, allow_table_error)
        self.n = 0

    def close(self):
        mlip_destroy(self.ctx)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def build_neighbors(self, pos, species, box, n_owned=None):
        """n_owned: the leading atoms that are this domain's own; the rest are ghosts (default: all owned)."""
        t = self.torch
        self._pos = t.as_tensor(pos, dtype=t.float64, device=self.device).contiguous()
        self._species = t.as_tensor(species, dtype=t.int32, device=self.device).contiguous()
        self.n = self._pos.shape[0]
        if n_owned is None or n_owned == self.n:
            mlip_build_neighbors(self.ctx, self._pos, self._species, box)
        else:
            mlip_build_neighbors_ghost(self.ctx, n_owned, self._pos, self._species, box)

    def neighbors(self):
        """Canonical lists as (seg_ptr int64 [N*C+1], nbr int32) on the device."""
        t = self.torch
        seg = t.empty(self.n * self.n_species + 1, dtype=t.int64, device=self.device)
        _, total = mlip_get_neighbors(self.ctx, seg, None)
        nbr = t.empty(max(total, 1), dtype=t.int32, device=self.device)
        rc, total = mlip_get_neighbors(self.ctx, seg, nbr)
        if rc != OK:
            raise MlipError(rc, "neighbor export")
        return seg, nbr[:total]

    def compute(self, want_e_atom=False):
        """Per-atom outputs are float32, or float64 on a context created with precision=1."""
        t = self.torch
        real = t.float64 if self.precision == 1 else t.float32
        out = {"energy": t.zeros(1, dtype=t.float64, device=self.device),
               "forces": t.empty((self.n, 3), dtype=real, device=self.device),
               "virial": t.zeros(9, dtype=t.float64, device=self.device),
               "e_atom": t.empty(self.n, dtype=real, device=self.device) if want_e_atom else None}
        call = mlip_compute_f64 if self.precision == 1 else mlip_compute
        call(self.ctx, out["energy"], out["forces"], out["virial"], out["e_atom"])
        return out

    def set_positions(self, pos):
        t = self.torch
        self._pos = t.as_tensor(pos, dtype=t.float64, device=self.device).contiguous()
        mlip_set_positions(self.ctx, self._pos)

    def set_velocities(self, vel):
        t = self.torch
        self._vel = t.as_tensor(vel, dtype=t.float64, device=self.device).contiguous()
        mlip_set_velocities(self.ctx, self._vel)

    def step(self, n_steps, dt_fs, rebuild_every):
        """rebuild_every > 0: fixed interval; 0: never; < 0: displacement-triggered, checked every -rebuild_every steps."""
        mlip_step(self.ctx, n_steps, dt_fs, rebuild_every)

    def step_nvt(self, n_steps, dt_fs, rebuild_every, t_target_K, t_damp_fs=100.0):
        mlip_step_nvt(self.ctx, n_steps, dt_fs, rebuild_every, t_target_K, t_damp_fs)

    def thermostat(self):
        return mlip_get_thermostat(self.ctx)

    def rebuilds(self) -> int:
        return mlip_get_rebuilds(self.ctx)

    def state(self):
        t = self.torch
        pos = t.empty((self.n, 3), dtype=t.float64, device=self.device)
        vel = t.empty((self.n, 3), dtype=t.float64, device=self.device)
        step = mlip_get_state(self.ctx, pos, vel)
        return pos, vel, step

    def set_state(self, pos=None, vel=None, step=0, v_eta=None, eta=None):
        t = self.torch
        if pos is not None:
            self._pos = t.as_tensor(pos, dtype=t.float64, device=self.device).contiguous()
        if vel is not None:
            self._vel = t.as_tensor(vel, dtype=t.float64, device=self.device).contiguous()
        mlip_set_state(self.ctx, self._pos if pos is not None else None, self._vel if vel is not None else None, step, v_eta, eta)

    def energies(self):
        t = self.torch
        e = t.zeros(2, dtype=t.float64, device=self.device)
        mlip_get_energies(self.ctx, e[0:1], e[1:2])
        return e

    def sync_status(self, raise_on_error=True):
        return mlip_sync_status(self.ctx, raise_on_error)
