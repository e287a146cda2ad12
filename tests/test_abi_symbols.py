"""The C-ABI library loads without a GPU and exports every symbol include/lq.h declares."""
import ctypes
import os
import re
import pytest

from paper_2604_18117_b200 import binding as B
from paper_2604_18117_b200 import build as BUILD

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "lq.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(lq_[a-z0-9_]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    BUILD.build()
    lib = ctypes.CDLL(B.LIB_PATH)
    names = _declared()
    assert "lq_calibrate" in names and "lq_quantize_act" in names and "lq_linear_forward" in names
    for n in names:
        assert hasattr(lib, n), f"missing symbol {n}"
    assert set(names) == set(B.EXPORTED)


def test_argument_errors_without_gpu():
    lib = B.lib()
    assert B.lq_version() >= 100
    assert lib.lq_status_string(1) == b"invalid argument"
    cfg = B.lq_config_default(128, 64, 8, "w8a8")
    assert (cfg.group, cfg.steps, cfg.rot_steps) == (64, 1000, 0) and abs(cfg.lr - 1e-4) < 1e-9
    out = ctypes.c_void_p()
    assert lib.lq_layer_import(ctypes.byref(cfg), None, None, None, None, None, None, None, ctypes.byref(out)) == 1
    bad = B.lq_config_default(128, 64, 200, "w8a8")
    import numpy as np
    z = np.zeros((128, 32), np.uint8)
    assert lib.lq_layer_import(ctypes.byref(bad), z.ctypes.data, z.ctypes.data, None, None, None, None, None,
                               ctypes.byref(out)) == 2
    assert lib.lq_quantize_act(None, None, 1, None, None) == 1
    assert lib.lq_set_option(b"no_such_option", 1) == 1


def test_option_names_and_values_are_checked():
    """lq_set_option knows its names and value ranges (no GPU needed: the switches are plain process-wide settings)."""
    from paper_2604_18117_b200 import binding as B
    for name, good, bad in (("overlap", (0, 1), (2, -1)), ("store_qb", (1, 0), ()), ("quant_ctas", (1, 0), (5,)),
                            ("quant_warps", (9, 0), (10,)), ("gemm_ctas", (7, 0), (-1,))):
        for v in good:
            B.lq_set_option(name, v)
        for v in bad:
            with pytest.raises(B.LqError):
                B.lq_set_option(name, v)
    with pytest.raises(B.LqError):
        B.lq_set_option("no_such_option", 1)
    B.lq_set_option("overlap", 1)
