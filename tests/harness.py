"""Runs a synthetic workload through the CUDA library and the CPU oracle side by side.

Both sides see the same bytes: the feature maps are generated once (on the GPU),
handed to the library by device pointer and copied to the host for the oracle.
Decisions are compared layer by layer; a frame whose decision differs must lie in
the near-threshold band (|AC - tau| <= 1e-4), is counted, and the oracle is re-run
for that layer with the library's decision imposed so that the states stay comparable.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

import oracle
import paper_2112_02644_b200 as smtm
import smtm_inputs as si

SV_RTOL = 1e-5       # semantic vectors, relative to the channel's mean |x|
SCORE_ATOL = 1e-5    # cosines live in [-1, 1]
CENTER_RTOL = 2e-5


@dataclass
class Report:
    frames: int = 0
    lookups: int = 0
    exits: list = field(default_factory=list)
    band_mismatches: int = 0
    near_oracle: int = 0
    max_sv_err: float = 0.0
    max_sa_err: float = 0.0
    max_center_err: float = 0.0
    routes: list = field(default_factory=list)   # lookups served by the fused, dense and plain routes


def make_pair(w: si.Workload, max_batch=None):
    cents, counts = si.initial_centers(w)
    tau = [w.tau] * w.L
    mem = oracle.OracleMemory(w.n, w.dims, tau, cents, counts, w.S, w.k_init, w.k_min, w.k_max, w.window_W,
                              forgetting=w.forgetting)
    cache = smtm.smtm_cache_create(w.n, w.dims, tau, cents, counts, n_streams=w.S, k_init=w.k_init, k_min=w.k_min,
                                   k_max=w.k_max, window_W=w.window_W, max_batch=max_batch or w.B,
                                   flags=smtm.FLAG_FORGET_FT if w.forgetting else 0)
    return cache, mem


def abs_mean_scale(x: torch.Tensor, w: si.Workload, layer: int) -> np.ndarray:
    """Mean |x| per (frame, channel): the scale the fp32 summation error is relative to."""
    axes = (2, 3) if w.layout == si.NCHW else (1, 2)
    return x.float().abs().mean(dim=axes).cpu().numpy().astype(np.float64)


def same_specials(g: np.ndarray, o: np.ndarray) -> np.ndarray:
    """Asserts that NaN and +-inf sit in the same places on both sides; returns the mask of finite entries."""
    assert np.array_equal(np.isnan(g), np.isnan(o)), "NaN in different places"
    inf = np.isinf(o)
    assert np.array_equal(np.isinf(g), inf) and np.array_equal(g[inf], o[inf]), "infinities differ"
    return np.isfinite(o)


def compare_layer(w, layer, x, gb, ob, todo, rep: Report):
    """Element-wise comparison of everything one lookup produced for the frames in ``todo``.
    Non-finite values (a NaN or an infinite element in a map propagates) must sit in the same places."""
    sv_g = gb.sv[layer].cpu().numpy().astype(np.float64)[todo]
    sv_o = ob["sv"][layer][todo]
    fin = same_specials(sv_g, sv_o)
    scale = np.maximum(np.nan_to_num(abs_mean_scale(x, w, layer)[todo], nan=1.0, posinf=1.0), 1e-30)
    err = np.where(fin, np.abs(sv_g - np.where(fin, sv_o, 0.0)), 0.0) / scale
    rep.max_sv_err = max(rep.max_sv_err, float(err.max(initial=0.0)))
    assert err.max(initial=0.0) <= SV_RTOL, f"semantic vectors off by {err.max():.3g} (relative) at layer {layer}"
    # cumulative similarity: weights add up to 2^(layer+1) - 1, each cosine within SCORE_ATOL
    sa_g = gb.sa.cpu().numpy().astype(np.float64)[todo]
    sa_o = ob["sa"][todo]
    fin = same_specials(sa_g, sa_o)
    sa_err = np.where(fin, np.abs(sa_g - np.where(fin, sa_o, 0.0)), 0.0)
    rep.max_sa_err = max(rep.max_sa_err, float(sa_err.max(initial=0.0)))
    assert sa_err.max(initial=0.0) <= SCORE_ATOL * (2 ** (layer + 1) - 1), f"cumulative similarity off by {sa_err.max():.3g}"
    # accumulated confidence and separability where the ratio is well conditioned
    ac_g = gb.ac.cpu().numpy().astype(np.float64)[:, layer]
    ac_o = ob["ac"][:, layer]
    sep_g = gb.sep.cpu().numpy().astype(np.float64)[:, layer]
    sep_o = ob["sep"][:, layer]
    for g, o in ((ac_g, ac_o), (sep_g, sep_o)):
        assert np.array_equal(np.isnan(g[todo]), np.isnan(o[todo])), "AC / separability: NaN in different places"
        fin = todo & np.isfinite(o) & np.isfinite(g) & (np.abs(o) < 5.0)
        assert np.all(np.abs(g[fin] - o[fin]) <= 2e-3 * (1 + np.abs(o[fin]))), "AC / separability mismatch"
    # top-1 class wherever the oracle's lead is clear of rounding
    top_g = gb.top.cpu().numpy()
    sa_sorted = np.sort(np.where(np.isnan(ob["sa"]), -np.inf, ob["sa"]), axis=1)
    if sa_sorted.shape[1] >= 2:
        clear = todo & ((sa_sorted[:, -1] - sa_sorted[:, -2]) > 1e-4)
        assert np.array_equal(top_g[clear, 0], ob["top"][clear, 0]), "top-1 class differs"


def step_pair(w, cache, mem, gb, lab, step, rep: Report, device="cuda", compare_values=True, edit=None):
    """One step on both sides, compared layer by layer.  Returns the oracle's batch.
    edit(layer, x): optional, changes the maps of a layer in place before either side sees them."""
    sid = si.stream_ids(w) if w.S > 1 else None
    ob = mem.new_batch(w.B, sid)
    begin = step % 2 == 1      # odd steps start with smtm_lookup_exit_begin on a carry full of garbage
    if begin:
        gb.sa.fill_(7.0)
        gb.done.fill_(1)
        gb.exit_layer.fill_(5)
        gb.pred.fill_(3)
    else:
        smtm.smtm_batch_reset(cache, gb)
    fb = si.fallback_labels(w, lab)
    for l in range(w.L):
        x = si.frames(w, l, lab, step, device=device)
        if edit is not None:
            edit(l, x)
        torch.cuda.synchronize()   # the maps are complete before the lookup is enqueued (SMTM_FLAG_MAPS_READY asks for it)
        B, C, H, W = si.shape4(w, l)
        todo = ob["done"] == 0
        (smtm.smtm_lookup_exit_begin if begin and l == 0 else smtm.smtm_lookup_exit)(
            cache, l, smtm.Fmap(x, w.dtype, w.layout, B, C, H, W), gb)
        torch.cuda.synchronize()
        if begin and l == 0:   # nothing of the old carry survives
            assert not bool((gb.sa == 7.0).any()) and bool((gb.pred[gb.done == 0] == -1).all())
        snap = {k: ob[k].copy() for k in ("sa", "done", "exit_layer", "pred")}
        xh = x.cpu()
        mem_exits, mem_near = mem.exits_per_layer.copy(), mem.near_count
        mem.lookup_exit(l, xh, w.dtype, w.layout, (B, C, H, W), ob)
        done_g = gb.done.cpu().numpy()
        diff = np.nonzero(done_g != ob["done"])[0]
        if diff.size:
            ac_g = gb.ac.cpu().numpy()[:, l]
            in_band = (ob["near"][diff, l] == 1) | (np.abs(ac_g[diff] - np.float32(w.tau)) <= 1e-4)
            assert in_band.all(), f"decision mismatch outside the 1e-4 band at layer {l}: frames {diff[~in_band][:8]}"
            rep.band_mismatches += int(diff.size)
            for k, v in snap.items():
                ob[k][...] = v
            mem.exits_per_layer[:] = mem_exits
            mem.near_count = mem_near
            force = np.full(w.B, -1, np.int8)
            force[diff] = done_g[diff]
            mem.lookup_exit(l, xh, w.dtype, w.layout, (B, C, H, W), ob, force=force)
        assert np.array_equal(done_g, ob["done"])
        assert np.array_equal(gb.exit_layer.cpu().numpy(), ob["exit_layer"])
        # predicted labels are bit-exact wherever a frame exited
        ex = ob["done"] == 1
        assert np.array_equal(gb.pred.cpu().numpy()[ex], ob["pred"][ex])
        if compare_values:
            compare_layer(w, l, x, gb, ob, todo, rep)
        rep.lookups += int(todo.sum())
        del x
    fb_d = torch.from_numpy(fb).to(device)
    if step % 2 == 0:       # both forms of the after-inference update are exercised
        smtm.smtm_cache_update(cache, gb, fb_d)
        smtm.smtm_cache_resize(cache)
    else:
        smtm.smtm_cache_update_resize(cache, gb, fb_d)
    mem.update(ob, fb)
    mem.resize()
    rep.frames += w.B
    rep.near_oracle = mem.near_count
    return ob


def compare_state(w, cache, mem, rep: Report):
    """Tables, counts, fast memories bit-exact; centres within rounding."""
    ft, ts = smtm.smtm_cache_get_tables(cache)
    assert np.array_equal(ft, mem.ft), "frequency table differs"
    assert np.array_equal(ts, mem.ts), "time-stamp table differs"
    members, k = smtm.smtm_cache_get_members(cache)
    assert np.array_equal(k, mem.k), "fast-memory sizes differ"
    assert np.array_equal(members, mem.members), "fast-memory members differ"
    for l in range(w.L):
        cen, m = smtm.smtm_cache_get_centers(cache, l)
        assert np.array_equal(m, mem.m[l]), "update counts differ"
        fin = same_specials(cen.astype(np.float64), mem.centers[l])   # a NaN folded into a centre by Eq. 7 stays there
        ref = np.where(fin, mem.centers[l], 0.0)
        scale = np.maximum(np.abs(ref), np.abs(ref).mean(axis=1, keepdims=True))
        err = np.where(fin, np.abs(cen.astype(np.float64) - ref), 0.0) / np.maximum(scale, 1e-30)
        rep.max_center_err = max(rep.max_center_err, float(err.max()))
        assert err.max() <= CENTER_RTOL, f"centres off by {err.max():.3g} at layer {l}"
    assert smtm.smtm_cache_status(cache) == 0, "device status word set"


def run_workload(w: si.Workload, steps=None, device="cuda", compare_values=True, state_every=1) -> Report:
    cache, mem = make_pair(w)
    rep = Report()
    labs = si.labels(w)
    sid = si.stream_ids(w) if w.S > 1 else None
    gb = smtm.Batch(cache, w.B, stream_id=sid, device=device)
    T = w.T if steps is None else steps
    for t in range(T):
        step_pair(w, cache, mem, gb, labs[t], t, rep, device, compare_values)
        if (t + 1) % state_every == 0 or t == T - 1:
            compare_state(w, cache, mem, rep)
    ctr = smtm.smtm_cache_get_counters(cache)
    rep.exits = [int(v) for v in ctr[: w.L]]
    assert rep.exits == [int(v) for v in mem.exits_per_layer], (rep.exits, mem.exits_per_layer)
    assert int(ctr[smtm.CTR_LOOKUPS]) == rep.lookups
    rep.routes = [int(v) for v in smtm.smtm_cache_get_routes(cache)]
    smtm.smtm_cache_destroy(cache)
    return rep
