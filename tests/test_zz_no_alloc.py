"""smtm_lookup_exit_static: the lookup for callers that cannot allocate device memory.

Plug-ins that run inside another engine's enqueue step, real-time threads and processes
with a frozen memory budget cannot call cudaMalloc; for them the library keeps the lookup's
working memory in a fixed array of its own.  The entry point must give exactly what
smtm_lookup_exit gives for a fresh batch, also when the array still holds an earlier
call's data.  (This file sorts last so that a failure here stops nothing else.)"""
import numpy as np
import pytest
import torch

import paper_2112_02644_b200 as smtm
import smtm_inputs as si

pytestmark = pytest.mark.gpu


def reference_lookup(cache, w, x, sid, layer=0):
    gb = smtm.Batch(cache, w.B, stream_id=sid)
    smtm.smtm_batch_reset(cache, gb)
    smtm.smtm_lookup_exit(cache, layer, smtm.Fmap(x, w.dtype, w.layout, *si.shape4(w, layer)), gb)
    torch.cuda.synchronize()
    return gb.done.cpu().numpy(), gb.pred.cpu().numpy(), gb.ac.cpu().numpy()


def test_static_lookup_equals_regular_lookup_on_two_calls_in_a_row():
    w = si.Workload("static", si.BF16, si.NCHW, B=96, stages=((2048, 7, 7),), n=60, k_init=12, k_min=12, k_max=12,
                    S=4, sigma=0.5, zipf_s=0.8, seed=9)
    cents, counts = si.initial_centers(w)
    cache = smtm.smtm_cache_create(w.n, w.dims, [w.tau], cents, counts, n_streams=w.S, k_init=w.k_init,
                                   k_min=w.k_min, k_max=w.k_max, max_batch=w.B)
    sid = (torch.arange(w.B, dtype=torch.int32, device="cuda") % w.S).contiguous()
    rng = np.random.default_rng(0)
    exits_seen = 0
    for call in range(2):   # the second call finds the first call's leftovers in the working memory
        lab = rng.integers(0, 2 * w.k_init, w.B).astype(np.int32)   # about half the frames are cached classes
        x = si.frames(w, 0, lab, step=call, device="cuda")
        want_exit, want_pred, want_ac = reference_lookup(cache, w, x, sid)
        got_exit = torch.full((w.B,), 7, dtype=torch.uint8, device="cuda")
        got_pred = torch.full((w.B,), 7, dtype=torch.int32, device="cuda")
        got_ac = torch.full((w.B, 1), 7.0, device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        launches_before = smtm.smtm_cache_get_launches(cache)
        smtm.smtm_lookup_exit_static(cache, 0, smtm.Fmap(x, w.dtype, w.layout, *si.shape4(w, 0)), sid, got_exit,
                                     got_pred, got_ac)
        torch.cuda.synchronize()
        if call > 0:    # (the very first call on a device may load the module that holds the array)
            assert torch.cuda.mem_get_info()[0] == free_before, "the call must not allocate device memory"
        assert smtm.smtm_cache_get_launches(cache) == launches_before + 1      # the fused kernel and nothing else
        assert np.array_equal(got_exit.cpu().numpy(), want_exit)
        assert np.array_equal(got_pred.cpu().numpy(), np.where(want_exit == 1, want_pred, -1))
        assert np.array_equal(got_ac.cpu().numpy(), want_ac)      # same kernels, same order: bitwise equal
        exits_seen += int(want_exit.sum())
    assert 0 < exits_seen < 2 * w.B
    assert smtm.smtm_cache_status(cache) == 0
    smtm.smtm_cache_destroy(cache)


def test_static_lookup_refuses_batches_beyond_its_fixed_memory():
    C, B = 2048, 1024     # 1024 x 2048 floats alone are 8 MiB, twice the fixed array
    cen = [np.ones((4, C), np.float32)]
    cache = smtm.smtm_cache_create(4, [C], [0.8], cen, k_init=2, k_min=2, k_max=4, max_batch=B)
    x = torch.zeros((B, C, 7, 7), dtype=torch.bfloat16, device="cuda")
    e = torch.zeros(B, dtype=torch.uint8, device="cuda")
    p = torch.zeros(B, dtype=torch.int32, device="cuda")
    before = smtm.smtm_cache_get_launches(cache)
    with pytest.raises(smtm.SmtmError) as err:
        smtm.smtm_lookup_exit_static(cache, 0, smtm.Fmap(x, si.BF16, si.NCHW, B, C, 7, 7), None, e, p)
    assert err.value.status == 2 and smtm.smtm_cache_get_launches(cache) == before
    smtm.smtm_cache_destroy(cache)


def test_static_lookups_back_to_back_on_a_cache_that_may_start_early():
    # A cache created with SMTM_FLAG_MAPS_READY lets the regular first lookup of a batch start while the stream's
    # previous kernel is finishing, because regular batches alternate their carries.  The static entry has one
    # carry for all calls, so it must never start early: here calls alternate, without synchronising, between a
    # layer served by two kernels (the second reads the semantic vectors from the shared array) and a layer
    # served by the one streaming kernel (which writes its semantic vectors to the same place).
    w = si.Workload("static_mixed", si.F16, si.NCHW, B=200, stages=((64, 2, 2), (512, 7, 7)), n=40, k_init=10, k_min=10,
                    k_max=10, S=1, sigma=0.5, zipf_s=0.8, seed=10)
    cents, counts = si.initial_centers(w)
    cache = smtm.smtm_cache_create(w.n, w.dims, [w.tau] * w.L, cents, counts, k_init=w.k_init, k_min=w.k_min,
                                   k_max=w.k_max, max_batch=w.B, flags=smtm.FLAG_MAPS_READY)
    rng = np.random.default_rng(1)
    rounds = 6
    xs, want = [], []
    for r in range(rounds):
        lab = rng.integers(0, 2 * w.k_init, w.B).astype(np.int32)
        layer = r % 2
        x = si.frames(w, layer, lab, step=r, device="cuda")
        xs.append(x)
        want.append(reference_lookup(cache, w, x, None, layer))
    routes0 = smtm.smtm_cache_get_routes(cache)
    got = [(torch.full((w.B,), 7, dtype=torch.uint8, device="cuda"), torch.full((w.B,), 7, dtype=torch.int32, device="cuda"),
            torch.full((w.B, w.L), 7.0, device="cuda")) for _ in range(rounds)]
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for r in range(rounds):                       # enqueued back to back on one stream
        e, p, ac = got[r]
        smtm.smtm_lookup_exit_static(cache, r % 2, smtm.Fmap(xs[r], w.dtype, w.layout, *si.shape4(w, r % 2)), None, e, p, ac)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    routes = smtm.smtm_cache_get_routes(cache) - routes0
    assert routes[smtm.ROUTE_PLAIN] == rounds // 2 and routes[smtm.ROUTE_FUSED] == rounds // 2
    for r in range(rounds):
        e, p, ac = got[r]
        we, wp, wac = want[r]
        assert np.array_equal(e.cpu().numpy(), we), r
        assert np.array_equal(p.cpu().numpy(), np.where(we == 1, wp, -1)), r
        # (the regular lookup of such a cache may take another route than the static one: same decisions, and
        # confidences equal up to the rounding of the dot products)
        got_ac, want_ac = ac.cpu().numpy()[:, r % 2].astype(np.float64), wac[:, r % 2].astype(np.float64)
        fin = np.isfinite(want_ac)
        assert np.array_equal(np.isfinite(got_ac), fin) and np.all(np.abs(got_ac[fin] - want_ac[fin]) <= 2e-3 * (1 + np.abs(want_ac[fin]))), r
    assert smtm.smtm_cache_status(cache) == 0
    smtm.smtm_cache_destroy(cache)
