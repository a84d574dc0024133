"""CPU oracle of the SMTM semantic-memory hot path (arxiv 2112.02644).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's
CPU-baseline leg use it.  The CUDA library and its Python binding never import
it.  The arithmetic lives in ``smtm_oracle.c`` (plain C, double precision);
this module compiles that file with gcc, binds it with ctypes and adds
``OracleMemory``, which holds the memory state in numpy arrays and strings the
C functions together into the paper's per-frame procedure extended to a batch
of frames per step.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "smtm_oracle.c")
_LIB = os.path.join(_HERE, "libsmtm_oracle.so")

F32, F16, BF16 = 0, 1, 2
NCHW, NHWC = 0, 1
NEAR_BAND = 1e-4
FT_MAX = 1 << 20

_lib = None


def build(force: bool = False) -> str:
    """Compile smtm_oracle.c into a shared object next to it (gcc, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c99", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _p(a, t):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(t))


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.orc_cosine.restype = ctypes.c_double
        lib.orc_score.restype = ctypes.c_uint64
        lib.orc_score.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_int]
        _lib = lib
    return _lib


def _raw(x) -> np.ndarray:
    """Bytes of a feature map as a C-contiguous numpy array (torch CPU tensors accepted)."""
    if hasattr(x, "detach"):
        import torch

        x = x.detach().cpu().contiguous()
        if x.dtype in (torch.bfloat16, torch.float16):
            x = x.view(torch.int16)
        x = x.numpy()
    return np.ascontiguousarray(x)


def gap(x, dtype: int, layout: int, B: int, C: int, H: int, W: int,
        skip: Optional[np.ndarray] = None, out: Optional[np.ndarray] = None) -> np.ndarray:
    """Sec. 4.1: SV[b][c] = mean over H x W of the feature map.  Returns float64 [B][C]."""
    raw = _raw(x)
    es = 4 if dtype == F32 else 2
    assert raw.nbytes == B * C * H * W * es, "feature-map size does not match its shape"
    sv = np.zeros((B, C), np.float64) if out is None else out
    sk = None if skip is None else np.ascontiguousarray(skip, np.uint8)
    rc = _load().orc_gap(raw.ctypes.data_as(ctypes.c_void_p), dtype, layout, B, C, H, W,
                         _p(sk, ctypes.c_uint8), _p(sv, ctypes.c_double))
    assert rc == 0, rc
    return sv


def cosine(a: np.ndarray, b: np.ndarray) -> float:
    """Eq. 1."""
    a = np.ascontiguousarray(a, np.float64)
    b = np.ascontiguousarray(b, np.float64)
    assert a.shape == b.shape and a.ndim == 1
    return float(_load().orc_cosine(_p(a, ctypes.c_double), _p(b, ctypes.c_double), a.size))


def score(ft: int, ts: int, W: int) -> int:
    """Eq. 5 as the exact integer FT * 4^(12 - min(floor(TS / W), 12))."""
    return int(_load().orc_score(int(ft), int(ts), int(W)))


def lookup_layer(layer: int, sv, centers, stream_id, members, k, tau: float, sa, done,
                 exit_layer, pred, force=None, near_band: float = NEAR_BAND):
    """Eq. 1, 3, 4 and the exit rule at 1-based ``layer``; updates sa/done/exit_layer/pred in place.

    Returns (ac[B], sep[B], top[B][2], near[B])."""
    B, D = sv.shape
    n = centers.shape[0]
    k_max = members.shape[1]
    ac = np.full(B, np.nan)
    sep = np.full(B, np.nan)
    top = np.full((B, 2), -1, np.int32)
    near = np.zeros(B, np.uint8)
    for a, t in ((sv, np.float64), (centers, np.float64), (stream_id, np.int32), (members, np.int32),
                 (k, np.int32), (sa, np.float64), (done, np.uint8), (exit_layer, np.int32),
                 (pred, np.int32)):
        assert a.dtype == t and a.flags.c_contiguous
    assert sa.shape == (B, k_max) and centers.shape[1] == D
    fr = None if force is None else np.ascontiguousarray(force, np.int8)
    rc = _load().orc_lookup_layer(
        int(layer), B, D, _p(sv, ctypes.c_double), _p(centers, ctypes.c_double), n,
        _p(stream_id, ctypes.c_int32), _p(members, ctypes.c_int32), _p(k, ctypes.c_int32), k_max,
        ctypes.c_double(tau), ctypes.c_double(near_band), _p(sa, ctypes.c_double),
        _p(done, ctypes.c_uint8), _p(exit_layer, ctypes.c_int32), _p(pred, ctypes.c_int32),
        _p(ac, ctypes.c_double), _p(sep, ctypes.c_double), _p(top, ctypes.c_int32),
        _p(near, ctypes.c_uint8), _p(fr, ctypes.c_int8))
    assert rc == 0, rc
    return ac, sep, top, near


FT_FRAC = 10   # fractional bits of FT in the forgetting variant


def tables_update(stream_id, final_label, ft, ts, forgetting_W: int = 0) -> None:
    """Sec. 6.1 frequency / time-stamp tables, frames applied in ascending index.

    forgetting_W > 0: the variant of Sec. 7.1 that decays FT itself every W unseen frames."""
    S, n = ft.shape
    for a in (stream_id, final_label, ft, ts):
        assert a.dtype == np.int32 and a.flags.c_contiguous
    if forgetting_W:
        rc = _load().orc_tables_update_forgetting(len(final_label), _p(stream_id, ctypes.c_int32),
                                                  _p(final_label, ctypes.c_int32), S, n, int(forgetting_W),
                                                  _p(ft, ctypes.c_int32), _p(ts, ctypes.c_int32))
    else:
        rc = _load().orc_tables_update(len(final_label), _p(stream_id, ctypes.c_int32),
                                       _p(final_label, ctypes.c_int32), S, n,
                                       _p(ft, ctypes.c_int32), _p(ts, ctypes.c_int32))
    assert rc == 0, rc


def centers_update(l0: int, sv, final_label, stop_layer, centers, m) -> None:
    """Eq. 7 at 1-based layer ``l0`` for every frame in ascending index."""
    B, D = sv.shape
    assert sv.dtype == np.float64 and centers.dtype == np.float64 and m.dtype == np.uint32
    assert final_label.dtype == np.int32 and stop_layer.dtype == np.int32
    for a in (sv, final_label, stop_layer, centers, m):
        assert a.flags.c_contiguous
    rc = _load().orc_centers_update(int(l0), B, D, _p(sv, ctypes.c_double),
                                    _p(final_label, ctypes.c_int32), _p(stop_layer, ctypes.c_int32),
                                    centers.shape[0], _p(centers, ctypes.c_double),
                                    _p(m, ctypes.c_uint32))
    assert rc == 0, rc


def resize(ft, ts, W: int, k_min: int, k_max: int, cl_num: int, cl_den: int, members, k,
           forgetting: bool = False) -> None:
    """Eq. 5 ranking + Eq. 6 adaptive size, per stream; members/k updated in place."""
    S, n = ft.shape
    assert members.shape == (S, k_max) and k.shape == (S,)
    for a in (ft, ts, members, k):
        assert a.dtype == np.int32 and a.flags.c_contiguous
    rc = _load().orc_resize(S, n, _p(ft, ctypes.c_int32), _p(ts, ctypes.c_int32), int(W), int(k_min),
                            int(k_max), int(cl_num), int(cl_den), int(bool(forgetting)), _p(members, ctypes.c_int32),
                            _p(k, ctypes.c_int32))
    assert rc == 0, rc


class OracleMemory:
    """Global memory + per-stream fast memories, and the per-step procedure.

    A step looks every frame of a batch up against the memory as it stood when
    the step began (layers 1..L in order, Sec. 5), then applies the after-
    inference updates (Sec. 6.1 tables, Eq. 7 centres) and, when asked, the
    replacement / adaptive-size refresh (Eq. 5, Eq. 6).  With one frame per
    stream per step this is the paper's frame-by-frame procedure.
    """

    def __init__(self, n_classes: int, dims: Sequence[int], tau: Sequence[float], centers,
                 counts=None, n_streams: int = 1, k_init: int = 5, k_min: int = 2,
                 k_max: int = 5, window_W: int = 16, cl_num: int = 19, cl_den: int = 20,
                 init_members=None, forgetting: bool = False):
        self.forgetting = bool(forgetting)
        self.n, self.L, self.S = int(n_classes), len(dims), int(n_streams)
        self.dims = [int(d) for d in dims]
        self.tau = [float(np.float32(t)) for t in tau]
        self.k_min, self.k_max, self.W = int(k_min), int(k_max), int(window_W)
        self.cl_num, self.cl_den = int(cl_num), int(cl_den)
        self.centers = [np.ascontiguousarray(np.asarray(c, np.float32), np.float64) for c in centers]
        for c, d in zip(self.centers, self.dims):
            assert c.shape == (self.n, d)
        if counts is None:
            self.m = [np.ones(self.n, np.uint32) for _ in self.dims]
        else:
            self.m = [np.ascontiguousarray(c, np.uint32).copy() for c in counts]
        self.ft = np.zeros((self.S, self.n), np.int32)
        self.ts = np.zeros((self.S, self.n), np.int32)
        self.members = np.zeros((self.S, self.k_max), np.int32)
        if init_members is None:
            self.members[:, :k_init] = np.arange(k_init, dtype=np.int32)[None, :]
        else:
            self.members[:, :k_init] = np.asarray(init_members, np.int32).reshape(self.S, k_init)
        self.k = np.full(self.S, int(k_init), np.int32)
        self.exits_per_layer = np.zeros(self.L, np.int64)
        self.near_count = 0

    # -- per-batch carry ---------------------------------------------------
    def new_batch(self, B: int, stream_id=None) -> dict:
        sid = np.zeros(B, np.int32) if stream_id is None else np.ascontiguousarray(stream_id, np.int32)
        return dict(B=B, stream_id=sid, sa=np.zeros((B, self.k_max)), done=np.zeros(B, np.uint8),
                    exit_layer=np.zeros(B, np.int32), pred=np.full(B, -1, np.int32),
                    ac=np.full((B, self.L), np.nan), sep=np.full((B, self.L), np.nan),
                    top=np.full((B, 2), -1, np.int32), near=np.zeros((B, self.L), np.uint8),
                    sv=[np.zeros((B, d)) for d in self.dims])

    def lookup_exit(self, layer: int, fmap, dtype: int, layout: int, shape, batch: dict,
                    force=None) -> None:
        """One candidate exit layer (0-based ``layer``): encode the not-yet-exited frames, score, decide."""
        B, C, H, W = shape
        assert B == batch["B"] and C == self.dims[layer]
        todo = batch["done"] == 0
        gap(fmap, dtype, layout, B, C, H, W, skip=batch["done"], out=batch["sv"][layer])
        ac, sep, top, near = lookup_layer(layer + 1, batch["sv"][layer], self.centers[layer],
                                          batch["stream_id"], self.members, self.k, self.tau[layer],
                                          batch["sa"], batch["done"], batch["exit_layer"],
                                          batch["pred"], force=force)
        batch["ac"][todo, layer] = ac[todo]
        batch["sep"][todo, layer] = sep[todo]
        batch["top"][todo] = top[todo]
        batch["near"][todo, layer] = near[todo]
        self.exits_per_layer[layer] += int(np.count_nonzero(todo & (batch["done"] == 1)))
        self.near_count += int(near[todo].sum())

    def warmup(self, layer: int, fmap, dtype: int, layout: int, shape, labels) -> None:
        """Centre warm-up (Sec. 5, Sec. 6.3): labelled frames folded into their classes' centres
        at one layer (0-based) by Eq. 7, in ascending frame order."""
        B, C, H, W = shape
        sv = gap(fmap, dtype, layout, B, C, H, W)
        lab = np.ascontiguousarray(labels, np.int32)
        lab = np.where(lab >= self.n, -1, lab).astype(np.int32)
        stop = np.full(B, self.L, np.int32)
        centers_update(layer + 1, sv, lab, stop, self.centers[layer], self.m[layer])

    def update(self, batch: dict, fallback_label=None) -> None:
        """After-inference updates for the whole batch (Sec. 6.1 tables, Eq. 7 centres)."""
        B = batch["B"]
        fb = np.full(B, -1, np.int32) if fallback_label is None else np.asarray(fallback_label, np.int32)
        fb = np.where(fb >= self.n, -1, fb)    # a label outside the memory counts as no label
        exited = batch["done"] == 1
        final = np.ascontiguousarray(np.where(exited, batch["pred"], fb), np.int32)
        stop = np.ascontiguousarray(np.where(exited, batch["exit_layer"], self.L), np.int32)
        tables_update(batch["stream_id"], final, self.ft, self.ts, self.W if self.forgetting else 0)
        for l0 in range(1, self.L + 1):
            centers_update(l0, batch["sv"][l0 - 1], final, stop, self.centers[l0 - 1], self.m[l0 - 1])

    def resize(self) -> None:
        resize(self.ft, self.ts, self.W, self.k_min, self.k_max, self.cl_num, self.cl_den,
               self.members, self.k, forgetting=self.forgetting)
