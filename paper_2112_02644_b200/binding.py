"""ctypes binding of include/smtm.h: same names, argument marshalling only.

Device arrays are torch CUDA tensors (torch is used for device memory and
streams, nothing else); host arrays are numpy arrays.  Every function raises
``SmtmError`` on a non-zero status.  Importing this module never touches the
GPU; the shared library is loaded on first use and a missing library is an
error, not a fallback.
"""
from __future__ import annotations

import ctypes
import os
import re
from typing import List, Optional, Sequence

import numpy as np

F32, F16, BF16 = 0, 1, 2
NCHW, NHWC = 0, 1
MAX_LAYERS = 16
FLAG_FORGET_FT = 1   # the frequency table itself forgets (fixed point, 10 fractional bits)
FLAG_MAPS_READY = 2  # the first lookup of a batch may read its maps while the previous update finishes (see smtm.h)
CTR_EXITS, CTR_NEAR, CTR_LOOKUPS, CTR_COUNT = 0, MAX_LAYERS, MAX_LAYERS + 1, MAX_LAYERS + 2

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libsmtm.so")
_HEADER = os.path.join(os.path.dirname(_HERE), "include", "smtm.h")
_lib = None


class SmtmError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {smtm_status_string(status)} (status {status})")


class _Config(ctypes.Structure):
    _fields_ = [("n_classes", ctypes.c_int32), ("n_layers", ctypes.c_int32),
                ("dims", ctypes.POINTER(ctypes.c_int32)), ("tau", ctypes.POINTER(ctypes.c_float)),
                ("n_streams", ctypes.c_int32), ("k_init", ctypes.c_int32), ("k_min", ctypes.c_int32),
                ("k_max", ctypes.c_int32), ("window_W", ctypes.c_int32), ("cl_num", ctypes.c_int32),
                ("cl_den", ctypes.c_int32), ("max_batch", ctypes.c_int32), ("flags", ctypes.c_uint32)]


class _Fmap(ctypes.Structure):
    _fields_ = [("d_data", ctypes.c_void_p), ("dtype", ctypes.c_int32), ("layout", ctypes.c_int32),
                ("B", ctypes.c_int32), ("C", ctypes.c_int32), ("H", ctypes.c_int32), ("W", ctypes.c_int32)]


class _Batch(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("d_stream_id", ctypes.c_void_p), ("d_sa", ctypes.c_void_p),
                ("d_done", ctypes.c_void_p), ("d_exit_layer", ctypes.c_void_p), ("d_pred", ctypes.c_void_p),
                ("d_ac", ctypes.c_void_p), ("d_sep", ctypes.c_void_p), ("d_top", ctypes.c_void_p),
                ("d_sv", ctypes.c_void_p * MAX_LAYERS)]


def library_path() -> str:
    return _LIB_PATH


def declared_symbols() -> List[str]:
    """Names of the functions include/smtm.h declares."""
    text = open(_HEADER).read()
    return sorted(set(re.findall(r"\b(smtm_[a-z_]+)\s*\(", text)))


def load_library():
    """Loads libsmtm.so (building it first if the sources are newer and nvcc is present)."""
    global _lib
    if _lib is not None:
        return _lib
    from . import build as _build
    if _build.stale():
        import shutil
        if shutil.which("nvcc"):
            _build.build()
        elif os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} was built from other sources than the ones present and nvcc is not "
                              "on PATH to rebuild it")
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: run `python -m paper_2112_02644_b200.build` "
                          "(there is no CPU fallback)")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i32 = ctypes.c_void_p, ctypes.c_int32
    lib.smtm_cache_create.argtypes = [ctypes.POINTER(_Config), ctypes.POINTER(vp), ctypes.POINTER(vp), vp,
                                      ctypes.POINTER(vp)]
    lib.smtm_cache_destroy.argtypes = [vp]
    lib.smtm_batch_reset.argtypes = [vp, ctypes.POINTER(_Batch), vp]
    lib.smtm_encode.argtypes = [vp, i32, ctypes.POINTER(_Fmap), vp, vp, vp, vp]
    lib.smtm_lookup_exit.argtypes = [vp, i32, ctypes.POINTER(_Fmap), ctypes.POINTER(_Batch), vp]
    lib.smtm_lookup_exit_begin.argtypes = [vp, i32, ctypes.POINTER(_Fmap), ctypes.POINTER(_Batch), vp]
    lib.smtm_lookup_exit_static.argtypes = [vp, i32, ctypes.POINTER(_Fmap), vp, vp, vp, vp, vp]
    lib.smtm_cache_update.argtypes = [vp, ctypes.POINTER(_Batch), vp, vp]
    lib.smtm_cache_resize.argtypes = [vp, vp]
    lib.smtm_cache_warmup.argtypes = [vp, i32, ctypes.POINTER(_Fmap), vp, vp]
    lib.smtm_cache_update_resize.argtypes = [vp, ctypes.POINTER(_Batch), vp, vp]
    lib.smtm_step_host.argtypes = [vp, ctypes.POINTER(_Fmap), ctypes.POINTER(vp), vp, vp, i32, vp, vp, vp, vp]
    lib.smtm_cache_get_members.argtypes = [vp, vp, vp]
    lib.smtm_cache_get_centers.argtypes = [vp, i32, vp, vp]
    lib.smtm_cache_get_tables.argtypes = [vp, vp, vp]
    lib.smtm_cache_get_counters.argtypes = [vp, vp]
    lib.smtm_cache_get_launches.argtypes = [vp, vp]
    lib.smtm_cache_get_routes.argtypes = [vp, vp]
    lib.smtm_cache_export_size.argtypes = [vp, vp]
    lib.smtm_cache_export.argtypes = [vp, vp, ctypes.c_uint64]
    lib.smtm_cache_import.argtypes = [vp, vp, ctypes.c_uint64]
    lib.smtm_cache_profile.argtypes = [vp, i32, i32]
    lib.smtm_cache_get_profile.argtypes = [vp, i32, vp, vp]
    lib.smtm_cache_get_profile_device.argtypes = [vp, vp, vp]
    lib.smtm_cache_get_profile_timeline.argtypes = [vp, ctypes.c_int64, vp, vp]
    lib.smtm_cache_status.argtypes = [vp]
    lib.smtm_cache_clear_status.argtypes = [vp]
    lib.smtm_cache_selftest_wait.argtypes = [vp, vp]
    lib.smtm_status_string.argtypes = [i32]
    lib.smtm_status_string.restype = ctypes.c_char_p
    for name in declared_symbols():
        fn = getattr(lib, name)
        if name != "smtm_status_string":
            fn.restype = ctypes.c_int
    _lib = lib
    return lib


def smtm_status_string(status: int) -> str:
    return load_library().smtm_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise SmtmError(status, where)


def _dptr(t) -> Optional[int]:
    """Device address of a torch CUDA tensor (None passes NULL)."""
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device arrays must be contiguous CUDA tensors"
    return t.data_ptr()


def _hptr(a: Optional[np.ndarray], dtype) -> Optional[int]:
    if a is None:
        return None
    assert isinstance(a, np.ndarray) and a.dtype == dtype and a.flags.c_contiguous
    return a.ctypes.data


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch

        return torch.cuda.current_stream().cuda_stream or None
    return getattr(stream, "cuda_stream", stream) or None


class Cache:
    """Handle of a device-resident semantic memory (smtm_cache_t)."""

    def __init__(self, handle: int, n: int, dims: Sequence[int], S: int, k_max: int, max_batch: int):
        self.handle, self.n, self.dims, self.S, self.k_max, self.max_batch = handle, n, list(dims), S, k_max, max_batch
        self.L = len(self.dims)

    def __del__(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.smtm_cache_destroy(self.handle)
            self.handle = None


class Fmap:
    """A batch of feature maps at one exit layer (smtm_fmap_t).  ``data`` is a CUDA tensor or None."""

    def __init__(self, data, dtype: int, layout: int, B: int, C: int, H: int, W: int):
        self.data = data
        self.c = _Fmap(_dptr(data), dtype, layout, B, C, H, W)


class Batch:
    """Per-batch carry (smtm_batch_t) holding torch CUDA tensors allocated by the caller side."""

    def __init__(self, cache: Cache, B: int, stream_id=None, device="cuda", with_diagnostics: bool = True):
        import torch

        self.B, self.cache = B, cache
        dev = torch.device(device)
        self.stream_id = None if stream_id is None else torch.as_tensor(stream_id, dtype=torch.int32, device=dev).contiguous()
        self.sa = torch.zeros((B, cache.k_max), dtype=torch.float32, device=dev)
        self.done = torch.zeros(B, dtype=torch.uint8, device=dev)
        self.exit_layer = torch.zeros(B, dtype=torch.int32, device=dev)
        self.pred = torch.full((B,), -1, dtype=torch.int32, device=dev)
        self.ac = torch.full((B, cache.L), float("nan"), dtype=torch.float32, device=dev) if with_diagnostics else None
        self.sep = torch.full((B, cache.L), float("nan"), dtype=torch.float32, device=dev) if with_diagnostics else None
        self.top = torch.full((B, 2), -1, dtype=torch.int32, device=dev) if with_diagnostics else None
        self.sv = [torch.zeros((B, d), dtype=torch.float32, device=dev) for d in cache.dims]
        sv = (ctypes.c_void_p * MAX_LAYERS)(*([t.data_ptr() for t in self.sv] + [None] * (MAX_LAYERS - cache.L)))
        self.c = _Batch(B, _dptr(self.stream_id), _dptr(self.sa), _dptr(self.done), _dptr(self.exit_layer),
                        _dptr(self.pred), _dptr(self.ac), _dptr(self.sep), _dptr(self.top), sv)



def smtm_cache_create(n_classes: int, dims: Sequence[int], tau: Sequence[float], centers: Sequence[np.ndarray],
                      counts: Optional[Sequence[np.ndarray]] = None, n_streams: int = 1, k_init: int = 5,
                      k_min: int = 2, k_max: int = 5, window_W: int = 16, cl_num: int = 19, cl_den: int = 20,
                      max_batch: int = 1024, init_members: Optional[np.ndarray] = None, flags: int = 0) -> Cache:
    lib = load_library()
    L = len(dims)
    dims_a = (ctypes.c_int32 * L)(*[int(d) for d in dims])
    tau_a = (ctypes.c_float * L)(*[float(t) for t in tau])
    cfg = _Config(n_classes, L, dims_a, tau_a, n_streams, k_init, k_min, k_max, window_W, cl_num, cl_den,
                  max_batch, flags)
    cen = [np.ascontiguousarray(c, np.float32) for c in centers]
    assert len(cen) == L and all(c.shape == (n_classes, d) for c, d in zip(cen, dims)), "centres: [L] x [n][C_l]"
    cen_p = (ctypes.c_void_p * L)(*[c.ctypes.data for c in cen])
    cnt_p = None
    if counts is not None:
        cnt = [np.ascontiguousarray(c, np.uint32) for c in counts]
        assert all(c.shape == (n_classes,) for c in cnt)
        cnt_p = (ctypes.c_void_p * L)(*[c.ctypes.data for c in cnt])
    mem = None
    if init_members is not None:
        mem = np.ascontiguousarray(init_members, np.int32)
        assert mem.size == n_streams * k_init
    out = ctypes.c_void_p()
    _check(lib.smtm_cache_create(ctypes.byref(cfg), cen_p, cnt_p, _hptr(mem, np.int32), ctypes.byref(out)),
           "smtm_cache_create")
    return Cache(out.value, n_classes, dims, n_streams, k_max, max_batch)


def smtm_cache_destroy(cache: Cache) -> None:
    if cache.handle:
        _check(load_library().smtm_cache_destroy(cache.handle), "smtm_cache_destroy")
        cache.handle = None


def smtm_batch_reset(cache: Cache, batch: Batch, stream=None) -> None:
    _check(load_library().smtm_batch_reset(cache.handle, ctypes.byref(batch.c), _stream(stream)), "smtm_batch_reset")


def smtm_encode(cache: Cache, layer: int, fmap: Fmap, sv, skip=None, sv_norm2=None, stream=None) -> None:
    _check(load_library().smtm_encode(cache.handle, layer, ctypes.byref(fmap.c), _dptr(skip), _dptr(sv),
                                      _dptr(sv_norm2), _stream(stream)), "smtm_encode")


def smtm_lookup_exit(cache: Cache, layer: int, fmap: Fmap, batch: Batch, stream=None) -> None:
    _check(load_library().smtm_lookup_exit(cache.handle, layer, ctypes.byref(fmap.c), ctypes.byref(batch.c),
                                           _stream(stream)), "smtm_lookup_exit")


def smtm_lookup_exit_begin(cache: Cache, layer: int, fmap: Fmap, batch: Batch, stream=None) -> None:
    _check(load_library().smtm_lookup_exit_begin(cache.handle, layer, ctypes.byref(fmap.c), ctypes.byref(batch.c),
                                                 _stream(stream)), "smtm_lookup_exit_begin")


def smtm_lookup_exit_static(cache: Cache, layer: int, fmap: Fmap, stream_id, exit_flags, pred, ac=None,
                            stream=None) -> None:
    """Single-layer lookup whose working memory is a fixed array inside the library (allocates nothing)."""
    _check(load_library().smtm_lookup_exit_static(cache.handle, layer, ctypes.byref(fmap.c), _dptr(stream_id),
                                                  _dptr(exit_flags), _dptr(pred), _dptr(ac), _stream(stream)),
           "smtm_lookup_exit_static")


def smtm_cache_update(cache: Cache, batch: Batch, fallback_label=None, stream=None) -> None:
    _check(load_library().smtm_cache_update(cache.handle, ctypes.byref(batch.c), _dptr(fallback_label),
                                            _stream(stream)), "smtm_cache_update")


def smtm_cache_update_resize(cache: Cache, batch: Batch, fallback_label=None, stream=None) -> None:
    _check(load_library().smtm_cache_update_resize(cache.handle, ctypes.byref(batch.c), _dptr(fallback_label),
                                                   _stream(stream)), "smtm_cache_update_resize")


def smtm_cache_warmup(cache: Cache, layer: int, fmap: Fmap, labels, stream=None) -> None:
    """Folds labelled frames into the centres of their classes at one layer (centre warm-up)."""
    _check(load_library().smtm_cache_warmup(cache.handle, layer, ctypes.byref(fmap.c), _dptr(labels),
                                            _stream(stream)), "smtm_cache_warmup")


def smtm_cache_resize(cache: Cache, stream=None) -> None:
    _check(load_library().smtm_cache_resize(cache.handle, _stream(stream)), "smtm_cache_resize")


def smtm_step_host(cache: Cache, fmaps: Sequence[Fmap], h_maps: Sequence, stream_id: Optional[np.ndarray],
                   fallback_label: Optional[np.ndarray], do_resize: bool, done: np.ndarray,
                   exit_layer: np.ndarray, pred: np.ndarray, stream=None) -> None:
    """One whole step from host memory; h_maps are host tensors/arrays (pinned for asynchronous copies)."""
    L = cache.L
    fm = (_Fmap * L)(*[f.c for f in fmaps])
    ptrs = (ctypes.c_void_p * L)(*[(m.data_ptr() if hasattr(m, "data_ptr") else m.ctypes.data) for m in h_maps])
    _check(load_library().smtm_step_host(cache.handle, fm, ptrs, _hptr(stream_id, np.int32),
                                         _hptr(fallback_label, np.int32), int(bool(do_resize)),
                                         _hptr(done, np.uint8), _hptr(exit_layer, np.int32),
                                         _hptr(pred, np.int32), _stream(stream)), "smtm_step_host")


def smtm_cache_get_members(cache: Cache):
    members = np.zeros((cache.S, cache.k_max), np.int32)
    k = np.zeros(cache.S, np.int32)
    _check(load_library().smtm_cache_get_members(cache.handle, members.ctypes.data, k.ctypes.data),
           "smtm_cache_get_members")
    return members, k


def smtm_cache_get_centers(cache: Cache, layer: int):
    cen = np.zeros((cache.n, cache.dims[layer]), np.float32)
    m = np.zeros(cache.n, np.uint32)
    _check(load_library().smtm_cache_get_centers(cache.handle, layer, cen.ctypes.data, m.ctypes.data),
           "smtm_cache_get_centers")
    return cen, m


def smtm_cache_get_tables(cache: Cache):
    ft = np.zeros((cache.S, cache.n), np.int32)
    ts = np.zeros((cache.S, cache.n), np.int32)
    _check(load_library().smtm_cache_get_tables(cache.handle, ft.ctypes.data, ts.ctypes.data),
           "smtm_cache_get_tables")
    return ft, ts


def smtm_cache_get_counters(cache: Cache) -> np.ndarray:
    out = np.zeros(CTR_COUNT, np.int64)
    _check(load_library().smtm_cache_get_counters(cache.handle, out.ctypes.data), "smtm_cache_get_counters")
    return out


def smtm_cache_get_launches(cache: Cache) -> int:
    out = np.zeros(1, np.int64)
    _check(load_library().smtm_cache_get_launches(cache.handle, out.ctypes.data), "smtm_cache_get_launches")
    return int(out[0])


ROUTE_FUSED, ROUTE_DENSE, ROUTE_PLAIN, ROUTE_PIPELINED, ROUTE_PIPELINED_DENSE, ROUTE_COUNT = 0, 1, 2, 3, 4, 5


def smtm_cache_get_routes(cache: Cache) -> np.ndarray:
    """Lookups served so far by the fused, the dense (tensor-core), the plain and the pipelined route."""
    out = np.zeros(ROUTE_COUNT, np.int64)
    _check(load_library().smtm_cache_get_routes(cache.handle, out.ctypes.data), "smtm_cache_get_routes")
    return out


def smtm_cache_export(cache: Cache) -> np.ndarray:
    """Snapshot of the memory (centres, counts, tables, fast memories, counters) as a host byte array."""
    size = ctypes.c_uint64(0)
    _check(load_library().smtm_cache_export_size(cache.handle, ctypes.byref(size)), "smtm_cache_export_size")
    blob = np.zeros(size.value, np.uint8)
    _check(load_library().smtm_cache_export(cache.handle, blob.ctypes.data, blob.nbytes), "smtm_cache_export")
    return blob


def smtm_cache_import(cache: Cache, blob: np.ndarray) -> None:
    """Puts a cache of the same shape back into the state a snapshot holds."""
    assert isinstance(blob, np.ndarray) and blob.dtype == np.uint8 and blob.flags.c_contiguous
    _check(load_library().smtm_cache_import(cache.handle, blob.ctypes.data, blob.nbytes), "smtm_cache_import")


def smtm_cache_profile(cache: Cache, max_lookups: int, every: int = 1) -> None:
    _check(load_library().smtm_cache_profile(cache.handle, int(max_lookups), int(every)), "smtm_cache_profile")


def smtm_cache_get_profile(cache: Cache, layer: int):
    """(total milliseconds, launches) of the streaming kernel at ``layer`` since profiling was switched on."""
    total = ctypes.c_double(0.0)
    count = ctypes.c_int64(0)
    _check(load_library().smtm_cache_get_profile(cache.handle, layer, ctypes.byref(total), ctypes.byref(count)),
           "smtm_cache_get_profile")
    return total.value, count.value


PROF_SCORE = MAX_LAYERS   # + layer: the scoring kernel of a layer whose pooling is a kernel of its own
PROF_PLAN, PROF_CENTERS, PROF_TABLES, PROF_SCORE_TC, PROF_FINISH_DENSE, PROF_REFRESH, PROF_KERNELS = (
    2 * MAX_LAYERS + i for i in range(7))


def smtm_cache_get_profile_device(cache: Cache):
    """(total milliseconds [PROF_KERNELS], steps [PROF_KERNELS]) by the device's own clock: index l < MAX_LAYERS is
    the fused lookup kernel of layer l, then PROF_PLAN, PROF_CENTERS, PROF_TABLES."""
    total = np.zeros(PROF_KERNELS, np.float64)
    count = np.zeros(PROF_KERNELS, np.int64)
    _check(load_library().smtm_cache_get_profile_device(cache.handle, total.ctypes.data, count.ctypes.data),
           "smtm_cache_get_profile_device")
    return total, count


def smtm_cache_get_profile_timeline(cache: Cache, step: int):
    """(begin ns [PROF_KERNELS], end ns [PROF_KERNELS]) of the step-th profiled step by the device's global timer;
    both 0 for a kernel that did not run in it."""
    begin = np.zeros(PROF_KERNELS, np.uint64)
    end = np.zeros(PROF_KERNELS, np.uint64)
    _check(load_library().smtm_cache_get_profile_timeline(cache.handle, int(step), begin.ctypes.data, end.ctypes.data),
           "smtm_cache_get_profile_timeline")
    return begin, end


def smtm_cache_status(cache: Cache) -> int:
    return int(load_library().smtm_cache_status(cache.handle))


def smtm_cache_clear_status(cache: Cache) -> None:
    _check(load_library().smtm_cache_clear_status(cache.handle), "smtm_cache_clear_status")


def smtm_cache_selftest_wait(cache: Cache, stream=None) -> None:
    """Enqueues a kernel whose bounded wait runs out (about a second); the status word then reads SMTM_ERR_TIMEOUT."""
    _check(load_library().smtm_cache_selftest_wait(cache.handle, _stream(stream)), "smtm_cache_selftest_wait")
