"""The C-ABI library loads and exports every entry point the header declares (no GPU needed)."""
import ctypes
import os
import re

from conftest import ROOT


def _declared():
    text = open(os.path.join(ROOT, "include", "mlip.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mlip_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    import paper_2608_16329_b200 as mlip
    names = _declared()
    assert len(names) >= 15
    lib = ctypes.CDLL(mlip.binding.LIB_PATH)
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(mlip.binding.EXPORTS) == names


def test_binding_has_a_function_per_entry_point():
    import paper_2608_16329_b200 as mlip
    for name in _declared():
        assert callable(getattr(mlip.binding, name)), name


def test_argument_checks_need_no_device():
    import paper_2608_16329_b200 as mlip
    lib = mlip.binding.lib()
    assert lib.mlip_create(None, None, None, 0, None, 0, None) == mlip.binding.CODES["MLIP_ERR_INVALID_ARG"]
    assert lib.mlip_compute(None, None, None, None, None, None) == mlip.binding.CODES["MLIP_ERR_INVALID_ARG"]
    cfg = mlip.binding.Config(6, 6.0, 1.0, 64, 3, 128, 3, 64, 4, 0, 0.0, 0.0, 0)
    import numpy as np
    ctx = ctypes.c_void_p(0)
    w = np.zeros(8)
    rc = lib.mlip_create(ctypes.byref(ctx), ctypes.byref(cfg), w.ctypes.data_as(ctypes.c_void_p), ctypes.c_size_t(8),
                         w.ctypes.data_as(ctypes.c_void_p), ctypes.c_size_t(8), w.ctypes.data_as(ctypes.c_void_p))
    assert rc == mlip.binding.CODES["MLIP_ERR_UNSUPPORTED"] and not ctx.value     # k = 64 is not compiled into the fp32 path
    assert b"k = 32" in lib.mlip_last_error(None)
