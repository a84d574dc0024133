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


def reference_lookup(cache, w, x, sid):
    gb = smtm.Batch(cache, w.B, stream_id=sid)
    smtm.smtm_batch_reset(cache, gb)
    smtm.smtm_lookup_exit(cache, 0, smtm.Fmap(x, w.dtype, w.layout, *si.shape4(w, 0)), gb)
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
        smtm.smtm_lookup_exit_static(cache, 0, smtm.Fmap(x, w.dtype, w.layout, *si.shape4(w, 0)), sid, got_exit,
                                     got_pred, got_ac)
        torch.cuda.synchronize()
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
