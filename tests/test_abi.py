"""The C-ABI library loads, exports every symbol include/smtm.h declares, and rejects
bad arguments on the host (no device work is needed for any of this)."""
import ctypes

import numpy as np
import pytest

import paper_2112_02644_b200 as smtm
from paper_2112_02644_b200 import binding


def test_library_loads_and_exports_every_declared_symbol():
    lib = smtm.load_library()
    names = smtm.declared_symbols()
    assert {"smtm_cache_create", "smtm_encode", "smtm_lookup_exit", "smtm_cache_update",
            "smtm_cache_resize"} <= set(names)
    for name in names:
        assert getattr(lib, name) is not None


def test_status_strings():
    assert smtm.smtm_status_string(0) == "ok"
    seen = {smtm.smtm_status_string(i) for i in range(9)}
    assert len(seen) == 9 and "unknown status" not in seen
    assert smtm.smtm_status_string(99) == "unknown status"


def test_null_and_out_of_range_arguments_are_rejected_before_any_device_work():
    lib = smtm.load_library()
    out = ctypes.c_void_p()
    assert lib.smtm_cache_create(None, None, None, None, ctypes.byref(out)) == 1
    assert lib.smtm_cache_destroy(None) == 1
    assert lib.smtm_cache_resize(None, None) == 1
    assert lib.smtm_encode(None, 0, None, None, None, None, None) == 1
    dims = (ctypes.c_int32 * 1)(8)
    tau = (ctypes.c_float * 1)(0.8)
    cen = np.zeros((4, 8), np.float32)
    cen_p = (ctypes.c_void_p * 1)(cen.ctypes.data)
    bad = [dict(n_classes=0), dict(n_layers=17), dict(k_max=5), dict(k_min=0), dict(k_init=9),
           dict(window_W=0), dict(cl_num=21), dict(max_batch=0), dict(flags=4), dict(n_streams=0)]
    for kw in bad:
        f = dict(n_classes=4, n_layers=1, dims=dims, tau=tau, n_streams=1, k_init=2, k_min=2, k_max=4,
                 window_W=16, cl_num=19, cl_den=20, max_batch=8, flags=0)
        f.update(kw)
        cfg = binding._Config(*[f[name] for name, _ in binding._Config._fields_])
        assert lib.smtm_cache_create(ctypes.byref(cfg), cen_p, None, None, ctypes.byref(out)) == 1, kw
        assert out.value is None
    with pytest.raises(smtm.SmtmError):
        binding._check(4, "x")
