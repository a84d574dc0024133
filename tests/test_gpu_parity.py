"""CUDA library vs CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import paper_2112_02644_b200 as smtm
import smtm_inputs as si
from harness import run_workload

pytestmark = pytest.mark.gpu

TORCH_DT = {si.F32: torch.float32, si.F16: torch.float16, si.BF16: torch.bfloat16}


def dummy_cache(C, n=4, max_batch=4096):
    cen = [np.ones((n, C), np.float32)]
    return smtm.smtm_cache_create(n, [C], [0.8], cen, k_init=2, k_min=2, k_max=n, max_batch=max_batch)


# ---------------------------------------------------------------------------- encode

ENCODE_SHAPES = [
    # (dtype, layout, B, C, H, W): the five workloads' stages, ragged channel counts, odd shapes
    (si.F32, si.NCHW, 8, 64, 56, 56),
    (si.BF16, si.NCHW, 5, 256, 56, 56), (si.BF16, si.NCHW, 5, 512, 28, 28),
    (si.BF16, si.NCHW, 7, 1024, 14, 14), (si.BF16, si.NCHW, 9, 2048, 7, 7),
    (si.BF16, si.NCHW, 3, 2048 + 8 * 5, 7, 7),      # ragged last chunk, unit-per-lane
    (si.BF16, si.NCHW, 3, 70, 14, 14), (si.F16, si.NCHW, 3, 24, 7, 7), (si.F32, si.NCHW, 3, 36, 7, 7),
    (si.F16, si.NCHW, 2, 33, 28, 28),               # ragged, team-per-channel
    (si.F32, si.NCHW, 2, 5, 2, 2), (si.F32, si.NCHW, 2, 3, 112, 112),  # 16-byte channels; channel > one stage
    (si.BF16, si.NCHW, 2, 7, 5, 3), (si.F16, si.NCHW, 1, 1, 1, 1),     # nothing aligned: plain path
    (si.F16, si.NHWC, 6, 24, 56, 56), (si.F16, si.NHWC, 6, 32, 28, 28),
    (si.F16, si.NHWC, 6, 96, 14, 14), (si.F16, si.NHWC, 6, 320, 7, 7),
    (si.BF16, si.NHWC, 2, 4096, 3, 3), (si.F32, si.NHWC, 3, 20, 9, 5), (si.F16, si.NHWC, 3, 12, 4, 4),
    (si.F32, si.NHWC, 2, 7, 3, 3),
]


@pytest.mark.parametrize("dt,layout,B,C,H,W", ENCODE_SHAPES)
def test_encode_matches_oracle(dt, layout, B, C, H, W):
    g = torch.Generator(device="cuda").manual_seed(B * 1000 + C)
    shape = (B, C, H, W) if layout == si.NCHW else (B, H, W, C)
    x = (torch.randn(shape, generator=g, device="cuda") * 0.7 + 0.2).to(TORCH_DT[dt]).contiguous()
    cache = dummy_cache(C)
    skip = torch.zeros(B, dtype=torch.uint8, device="cuda")
    if B > 2:
        skip[1] = 1
    sv = torch.full((B, C), -7.0, device="cuda")
    n2 = torch.full((B,), -7.0, device="cuda")
    smtm.smtm_encode(cache, 0, smtm.Fmap(x, dt, layout, B, C, H, W), sv, skip=skip, sv_norm2=n2)
    torch.cuda.synchronize()
    ref = oracle.gap(x.cpu(), dt, layout, B, C, H, W)
    axes = (2, 3) if layout == si.NCHW else (1, 2)
    scale = x.float().abs().mean(dim=axes).cpu().numpy().astype(np.float64)
    got = sv.cpu().numpy().astype(np.float64)
    keep = skip.cpu().numpy() == 0
    assert np.all(np.abs(got - ref)[keep] <= 1e-5 * scale[keep] + 1e-30)
    assert np.all(got[~keep] == -7.0)                       # skipped rows are not written
    n2h = n2.cpu().numpy().astype(np.float64)
    np.testing.assert_allclose(n2h[keep], (ref ** 2).sum(axis=1)[keep], rtol=1e-5)
    assert np.all(n2h[~keep] == -7.0)
    assert smtm.smtm_cache_status(cache) == 0
    # same bytes twice: bitwise identical (fixed reduction order)
    sv2 = torch.zeros_like(sv)
    smtm.smtm_encode(cache, 0, smtm.Fmap(x, dt, layout, B, C, H, W), sv2)
    torch.cuda.synchronize()
    assert torch.equal(sv2[keep], sv[keep])
    smtm.smtm_cache_destroy(cache)


def test_encode_constant_map_and_layout_equivalence():
    B, C, H, W = 4, 64, 14, 14
    cache = dummy_cache(C)
    x = torch.full((B, C, H, W), 0.625, dtype=torch.bfloat16, device="cuda")
    sv = torch.zeros((B, C), device="cuda")
    smtm.smtm_encode(cache, 0, smtm.Fmap(x, si.BF16, si.NCHW, B, C, H, W), sv)
    assert torch.all(sv == 0.625)
    g = torch.Generator(device="cuda").manual_seed(1)
    y = torch.randn((B, C, H, W), generator=g, device="cuda").half()
    a = torch.zeros((B, C), device="cuda")
    b = torch.zeros((B, C), device="cuda")
    smtm.smtm_encode(cache, 0, smtm.Fmap(y, si.F16, si.NCHW, B, C, H, W), a)
    yn = y.permute(0, 2, 3, 1).contiguous()
    smtm.smtm_encode(cache, 0, smtm.Fmap(yn, si.F16, si.NHWC, B, C, H, W), b)
    torch.cuda.synchronize()
    assert torch.allclose(a, b, rtol=0, atol=2e-6)
    smtm.smtm_cache_destroy(cache)


def test_argument_errors_launch_nothing():
    C = 64
    cache = dummy_cache(C, max_batch=8)
    x = torch.zeros((4, C, 7, 7), dtype=torch.bfloat16, device="cuda")
    sv = torch.zeros((4, C), device="cuda")
    before = smtm.smtm_cache_get_launches(cache)
    for fm, code in ((smtm.Fmap(x, si.BF16, si.NCHW, 4, C + 8, 7, 7), 2), (smtm.Fmap(x, 7, si.NCHW, 4, C, 7, 7), 3),
                     (smtm.Fmap(x, si.BF16, si.NCHW, 9, C, 7, 7), 2), (smtm.Fmap(None, si.BF16, si.NCHW, 4, C, 7, 7), 1)):
        with pytest.raises(smtm.SmtmError) as e:
            smtm.smtm_encode(cache, 0, fm, sv)
        assert e.value.status == code
    mis = torch.zeros(4 * C * 49 + 8, dtype=torch.bfloat16, device="cuda")[1:1 + 4 * C * 49]
    fm = smtm.Fmap(None, si.BF16, si.NCHW, 4, C, 7, 7)
    fm.c.d_data = mis.data_ptr()
    with pytest.raises(smtm.SmtmError) as e:
        smtm.smtm_encode(cache, 0, fm, sv)
    assert e.value.status == 4
    with pytest.raises(smtm.SmtmError):
        smtm.smtm_encode(cache, 1, smtm.Fmap(x, si.BF16, si.NCHW, 4, C, 7, 7), sv)
    assert smtm.smtm_cache_get_launches(cache) == before
    smtm.smtm_cache_destroy(cache)


# ---------------------------------------------------------------------------- whole path

def test_c1_single_layer_fp32():
    rep = run_workload(si.C1)
    assert rep.exits == [8] and rep.band_mismatches == 0
    assert rep.routes == [1, 0, 0, 0, 0]       # one fused launch: pooling, Eq. 1, Eq. 3, Eq. 4 and the decision


def test_c2_resnet50_bf16_four_layers():
    rep = run_workload(si.C2)
    assert sum(rep.exits) > 30 and rep.frames == 64
    assert rep.routes == [4, 0, 0, 0, 0]


def test_c2_exits_disabled_streams_every_layer():
    rep = run_workload(si.C2.scaled(tau=float("inf")))
    assert rep.exits == [0, 0, 0, 0] and rep.lookups == 4 * 64


def test_c3_mobilenetv2_fp16_nhwc_novel_classes_do_not_exit():
    w = si.C3
    rep = run_workload(w)
    assert sum(rep.exits) > 100
    lab = si.labels(w)[0]
    # the oracle (and therefore the library, which matched it) lets no novel frame exit
    cache_exits = sum(rep.exits)
    assert cache_exits <= int((lab < w.n).sum())


def test_c4_large_cache_straddles_threshold():
    rep = run_workload(si.C4)
    assert 100 < rep.exits[0] < 900
    assert rep.routes == [0, 1, 0, 0, 0], "the 1000-entry fast memory must be scored on the tensor cores (Eq. 1 as a dense contraction)"
    print("c4 max |SA error|:", rep.max_sa_err, "max SV error:", rep.max_sv_err)
    print("c4 near-threshold lookups (oracle):", rep.near_oracle, "band mismatches:", rep.band_mismatches)


@pytest.mark.parametrize("T", [6])
def test_c5_streaming_full_width(T):
    rep = run_workload(si.C5, steps=T)
    assert rep.frames == 512 * T and rep.exits[0] > 0
    assert rep.routes == [2 * T, 0, 0, 0, 0]


def test_c5_full_length_64_steps_state_only():
    # all 64 steps at full width; values are compared on every step, state every 8 steps
    rep = run_workload(si.C5, state_every=8)
    assert rep.frames == 512 * 64
    print("c5 exits per layer:", rep.exits, "never:", rep.frames - sum(rep.exits), "band:", rep.band_mismatches)


def test_adaptive_size_moves_and_ragged_small_cases():
    # small classes / streams / odd batch: exercises k growing and shrinking, ties, fallback -1
    w = si.Workload("tiny", si.F16, si.NCHW, B=37, stages=((24, 7, 7), (40, 5, 3)), n=23, k_init=3, k_min=2,
                    k_max=9, S=1, T=12, tau=0.3, window_W=3, sigma=0.4, zipf_s=0.7, novel_frac=0.15, n_novel=5,
                    repeat_p=0.5, seed=3)
    rep = run_workload(w)
    assert rep.frames == 37 * 12
    w2 = si.Workload("tiny_streams", si.BF16, si.NHWC, B=19, stages=((16, 6, 6),), n=11, k_init=2, k_min=2,
                     k_max=11, S=19, T=20, tau=0.2, window_W=2, sigma=0.5, zipf_s=1.0, repeat_p=0.6, seed=4)
    rep2 = run_workload(w2)
    assert rep2.frames == 19 * 20


def test_large_fast_memory_over_several_layers_uses_tensor_cores():
    # fast memories above 64 entries take the tensor-core scorer; ragged batch, class count that is not a
    # multiple of the tile, two exit layers (cumulative similarity over all slots), two streams, updates
    w = si.Workload("dense", si.BF16, si.NCHW, B=70, stages=((256, 14, 14), (512, 7, 7)), n=196, k_init=100,
                    k_min=70, k_max=196, S=1, T=4, tau=0.8, window_W=2, sigma=0.6, zipf_s=0.9, repeat_p=0.3, seed=6)
    rep = run_workload(w)
    assert rep.frames == 70 * 4 and rep.lookups > 70
    assert rep.routes == [0, 8, 0, 0, 0]       # both layers of all four steps on the tensor-core route
    w3 = si.Workload("dense_nhwc", si.F16, si.NHWC, B=33, stages=((320, 7, 7),), n=72, k_init=72, k_min=72, k_max=72,
                     S=1, T=2, tau=0.8, sigma=1.0, zipf_s=1.0, seed=8)
    rep3 = run_workload(w3)
    assert rep3.frames == 66 and rep3.routes == [0, 2, 0, 0, 0]


def test_forgetting_frequency_table_rapid_scene_change():
    # the paper's long-tail / rapid-change setting: FT itself decays every W unseen frames
    w = si.Workload("forget", si.BF16, si.NCHW, B=24, stages=((64, 7, 7), (128, 7, 7)), n=30, k_init=4, k_min=2,
                    k_max=12, S=24, T=30, tau=0.4, window_W=3, sigma=0.5, zipf_s=0.8, repeat_p=0.3, forgetting=True,
                    seed=12)
    rep = run_workload(w)
    assert rep.frames == 24 * 30
    w1 = w.scaled(name="forget_one_stream", S=1, B=50, T=8, window_W=5)   # many frames of one stream per step
    rep1 = run_workload(w1)
    assert rep1.frames == 400


def test_centre_warm_up_on_the_gpu_matches_oracle_and_feeds_lookups():
    # Sec. 5: centres = per-class mean semantic vector of labelled frames, built on the GPU from count 0,
    # in two batches, then used by a normal step
    w = si.Workload("warm", si.BF16, si.NCHW, B=96, stages=((256, 14, 14), (512, 7, 7)), n=12, k_init=12, k_min=12,
                    k_max=12, S=1, T=3, tau=0.5, sigma=0.5, zipf_s=0.5, seed=14)
    zeros = [np.zeros((w.n, d), np.float32) for d in w.dims]
    m0 = [np.zeros(w.n, np.uint32) for _ in w.dims]
    tau = [w.tau] * w.L
    cache = smtm.smtm_cache_create(w.n, w.dims, tau, zeros, m0, k_init=w.k_init, k_min=w.k_min, k_max=w.k_max,
                                   max_batch=w.B)
    mem = oracle.OracleMemory(w.n, w.dims, tau, zeros, m0, 1, w.k_init, w.k_min, w.k_max, w.window_W)
    labs = si.labels(w)
    for t in range(2):
        lab = labs[t].copy()
        lab[::7] = -1                      # unlabelled frames
        lab[3::11] = w.n + 2               # labels outside the memory
        for l in range(w.L):
            x = si.frames(w, l, labs[t], 100 + t, device="cuda")
            smtm.smtm_cache_warmup(cache, l, smtm.Fmap(x, w.dtype, w.layout, *si.shape4(w, l)),
                                   torch.from_numpy(lab).cuda())
            mem.warmup(l, x.cpu(), w.dtype, w.layout, si.shape4(w, l), lab)
    for l in range(w.L):
        cen, m = smtm.smtm_cache_get_centers(cache, l)
        assert np.array_equal(m, mem.m[l]) and m.sum() > 100
        np.testing.assert_allclose(cen, mem.centers[l], rtol=2e-5, atol=1e-6)
    ft, ts = smtm.smtm_cache_get_tables(cache)
    assert not ft.any() and not ts.any()
    # a normal step on the warmed-up memory: most frames find their class
    from harness import Report, step_pair, compare_state
    gb = smtm.Batch(cache, w.B)
    rep = Report()
    step_pair(w, cache, mem, gb, labs[2], 2, rep)
    compare_state(w, cache, mem, rep)
    assert int(gb.done.sum()) > w.B // 2
    smtm.smtm_cache_destroy(cache)


def test_c6_vgg16_shaped_thirteen_shallow_exits():
    # many layers, tiny maps (down to 2x2, which no 16-byte grouping serves), forgetting tables
    rep = run_workload(si.C6, steps=4)
    assert rep.frames == 128 * 4 and len(rep.exits) == 13
    print("c6 exits per layer:", rep.exits)


def test_step_host_matches_device_path():
    w = si.C5.scaled(B=32, S=32, T=3)
    cents, counts = si.initial_centers(w)
    tau = [w.tau] * w.L
    mk = lambda: smtm.smtm_cache_create(w.n, w.dims, tau, cents, counts, n_streams=w.S, k_init=w.k_init,
                                        k_min=w.k_min, k_max=w.k_max, window_W=w.window_W, max_batch=w.B)
    a, b = mk(), mk()
    gb = smtm.Batch(a, w.B, stream_id=si.stream_ids(w))
    labs = si.labels(w)
    sid = si.stream_ids(w)
    for t in range(w.T):
        maps = [si.frames(w, l, labs[t], t, device="cuda") for l in range(w.L)]
        fb = si.fallback_labels(w, labs[t])
        smtm.smtm_batch_reset(a, gb)
        for l in range(w.L):
            smtm.smtm_lookup_exit(a, l, smtm.Fmap(maps[l], w.dtype, w.layout, *si.shape4(w, l)), gb)
        smtm.smtm_cache_update(a, gb, torch.from_numpy(fb).cuda())
        smtm.smtm_cache_resize(a)
        hm = [m.cpu().pin_memory() for m in maps]
        done = np.zeros(w.B, np.uint8); el = np.zeros(w.B, np.int32); pred = np.zeros(w.B, np.int32)
        fmaps = [smtm.Fmap(None, w.dtype, w.layout, *si.shape4(w, l)) for l in range(w.L)]
        smtm.smtm_step_host(b, fmaps, hm, sid, fb, True, done, el, pred)
        assert np.array_equal(done, gb.done.cpu().numpy())
        assert np.array_equal(el, gb.exit_layer.cpu().numpy())
        assert np.array_equal(pred, gb.pred.cpu().numpy())
    for x, y in zip(smtm.smtm_cache_get_tables(a), smtm.smtm_cache_get_tables(b)):
        assert np.array_equal(x, y)
    for l in range(w.L):
        ca, cb = smtm.smtm_cache_get_centers(a, l), smtm.smtm_cache_get_centers(b, l)
        assert np.array_equal(ca[0], cb[0]) and np.array_equal(ca[1], cb[1])


# ---------------------------------------------------------------------------- the fused kernel's cluster sizes

@pytest.mark.parametrize("B", [5, 37, 148, 151])
def test_fused_lookup_every_cluster_size(B):
    # The fused lookup cuts a frame into 1, 2, 4 or 8 parts (CTAs of a cluster) depending on how many frames there
    # are: 5 frames -> 8 parts, 37 -> 4, 148 -> 1 at the first layer (2 at the second, whose 2048 channels do not
    # fit one part), 151 -> a ragged last round.  Fast memories of up to 64 entries use both slots of every lane.
    w = si.Workload(f"clusters_{B}", si.BF16, si.NCHW, B=B, stages=((1024, 14, 14), (2048, 7, 7)), n=90, k_init=40,
                    k_min=33, k_max=64, S=B if B < 100 else 1, T=2, tau=0.8, window_W=2, sigma=0.5, zipf_s=1.0, repeat_p=0.5,
                    seed=20 + B)
    rep = run_workload(w)
    assert rep.frames == 2 * B and rep.lookups >= 2 * B


def test_update_of_a_batch_too_large_for_the_single_cta_plan():
    # up to 4096 frames the update lists the (layer, class) pairs of Eq. 7 with one CTA and a bitmap in shared
    # memory; beyond that many CTAs elect them through tags in global memory.  4200 small frames of one stream
    # take the second way (every other test takes the first).
    w = si.Workload("big_batch", si.F16, si.NCHW, B=4200, stages=((64, 4, 4), (128, 2, 2)), n=60, k_init=10, k_min=6,
                    k_max=24, S=1, T=3, tau=0.8, window_W=4, sigma=0.5, zipf_s=1.0, repeat_p=0.3, seed=77)
    rep = run_workload(w)
    assert rep.frames == 3 * 4200 and sum(rep.exits) > 0


def test_fused_lookup_exact_ties_go_to_the_lower_class():
    # two classes with the same centre at every layer: their similarities tie bit for bit, the lower class id
    # ranks first (top-1 / top-2 are selected through 64-bit keys in the fused kernel) and such a frame never exits
    from harness import Report, step_pair

    w = si.Workload("ties", si.BF16, si.NCHW, B=40, stages=((256, 14, 14), (512, 7, 7)), n=12, k_init=12, k_min=12,
                    k_max=12, S=1, T=1, tau=0.5, window_W=4, sigma=0.3, zipf_s=0.5, seed=31)
    cents, counts = si.initial_centers(w)
    for l in range(w.L):
        cents[l][1] = cents[l][0]
        cents[l][7] = cents[l][0]
    tau = [w.tau] * w.L
    mem = oracle.OracleMemory(w.n, w.dims, tau, cents, counts, w.S, w.k_init, w.k_min, w.k_max, w.window_W)
    cache = smtm.smtm_cache_create(w.n, w.dims, tau, cents, counts, n_streams=w.S, k_init=w.k_init, k_min=w.k_min,
                                   k_max=w.k_max, window_W=w.window_W, max_batch=w.B)
    gb = smtm.Batch(cache, w.B)
    lab = si.labels(w)[0]
    ob = step_pair(w, cache, mem, gb, lab, 0, Report())
    tied = lab == 0          # frames drawn around class 0: classes 0, 1 and 7 score the same for them
    assert tied.sum() >= 3
    top = gb.top.cpu().numpy()
    assert np.array_equal(top, ob["top"])
    assert np.all(top[tied, 0] == 0) and np.all(top[tied, 1] == 1)
    assert not gb.done.cpu().numpy()[tied].any()
    ac = gb.ac.cpu().numpy()
    assert np.all(ac[tied] == 0.0)
    smtm.smtm_cache_destroy(cache)


def test_device_clock_profile_reports_every_kernel_of_a_step():
    # every `every`-th step carries stamps of the device's clock: each kernel of the step reports a duration
    w = si.C5.scaled(B=64, S=64, T=3)
    cents, counts = si.initial_centers(w)
    cache = smtm.smtm_cache_create(w.n, w.dims, [w.tau] * w.L, cents, counts, n_streams=w.S, k_init=w.k_init,
                                   k_min=w.k_min, k_max=w.k_max, window_W=w.window_W, max_batch=w.B)
    gb = smtm.Batch(cache, w.B, stream_id=si.stream_ids(w))
    labs = si.labels(w)
    smtm.smtm_cache_profile(cache, 8, 2)          # steps 0 and 2 are profiled, step 1 is not
    for t in range(3):
        for l in range(w.L):
            x = si.frames(w, l, labs[t], t, device="cuda")
            (smtm.smtm_lookup_exit_begin if l == 0 else smtm.smtm_lookup_exit)(
                cache, l, smtm.Fmap(x, w.dtype, w.layout, *si.shape4(w, l)), gb)
        smtm.smtm_cache_update_resize(cache, gb, torch.from_numpy(si.fallback_labels(w, labs[t])).cuda())
    total, count = smtm.smtm_cache_get_profile_device(cache)
    for i in (0, 1, smtm.PROF_PLAN, smtm.PROF_CENTERS, smtm.PROF_TABLES):
        assert count[i] == 2 and 0.0 < total[i] < 100.0, (i, count[i], total[i])   # milliseconds
    assert count[2:smtm.MAX_LAYERS].sum() == 0
    ev_ms, ev_n = smtm.smtm_cache_get_profile(cache, 0)
    assert ev_n == 2 and ev_ms >= total[0] * 0.5
    # the stamps themselves: the kernels of a step in the order of their dependencies, the durations the same ones
    spans = np.zeros(smtm.PROF_KERNELS)
    for step in range(2):
        begin, end = smtm.smtm_cache_get_profile_timeline(cache, step)
        ran = [0, 1, smtm.PROF_PLAN, smtm.PROF_CENTERS, smtm.PROF_TABLES]
        assert (begin[ran] > 0).all() and (end[ran] >= begin[ran]).all()
        assert not begin[2:smtm.MAX_LAYERS].any() and not end[2:smtm.MAX_LAYERS].any()
        assert end[0] <= begin[1] and end[1] <= begin[smtm.PROF_PLAN] and end[1] <= begin[smtm.PROF_TABLES]
        assert end[smtm.PROF_PLAN] <= begin[smtm.PROF_CENTERS]
        spans += (end - begin).astype(np.float64) * 1e-6
    assert np.allclose(spans, total)
    with pytest.raises(smtm.SmtmError):
        smtm.smtm_cache_get_profile_timeline(cache, 2)
    # stamps alone (negative period): no events, the device clock still reports the step
    smtm.smtm_cache_profile(cache, 8, -1)
    for l in range(w.L):
        x = si.frames(w, l, labs[0], 0, device="cuda")
        (smtm.smtm_lookup_exit_begin if l == 0 else smtm.smtm_lookup_exit)(
            cache, l, smtm.Fmap(x, w.dtype, w.layout, *si.shape4(w, l)), gb)
    smtm.smtm_cache_update_resize(cache, gb, torch.from_numpy(si.fallback_labels(w, labs[0])).cuda())
    assert smtm.smtm_cache_get_profile(cache, 0)[1] == 0
    assert list(smtm.smtm_cache_get_profile_device(cache)[1][[0, 1, smtm.PROF_PLAN]]) == [1, 1, 1]
    smtm.smtm_cache_profile(cache, 0, 1)
    assert smtm.smtm_cache_get_profile_device(cache)[1].sum() == 0
    smtm.smtm_cache_destroy(cache)


def test_maps_ready_flag_with_alternating_batches():
    # SMTM_FLAG_MAPS_READY: the first lookup of a step may read its maps and write its batch's SV stash while the
    # previous step's update is still running; the caller alternates two carries.  Results are those of the oracle.
    from harness import Report, compare_state, step_pair

    w = si.C5.scaled(B=96, S=96, T=6)
    cents, counts = si.initial_centers(w)
    tau = [w.tau] * w.L
    mem = oracle.OracleMemory(w.n, w.dims, tau, cents, counts, w.S, w.k_init, w.k_min, w.k_max, w.window_W)
    cache = smtm.smtm_cache_create(w.n, w.dims, tau, cents, counts, n_streams=w.S, k_init=w.k_init, k_min=w.k_min,
                                   k_max=w.k_max, window_W=w.window_W, max_batch=w.B, flags=smtm.FLAG_MAPS_READY)
    sid = si.stream_ids(w)
    gbs = [smtm.Batch(cache, w.B, stream_id=sid), smtm.Batch(cache, w.B, stream_id=sid)]
    labs = si.labels(w)
    rep = Report()
    for t in range(w.T):
        step_pair(w, cache, mem, gbs[t % 2], labs[t], t, rep)
    compare_state(w, cache, mem, rep)
    # back to back without the harness's synchronisation in between: steps overlap on the device
    maps = [[si.frames(w, l, labs[t], t, device="cuda") for l in range(w.L)] for t in range(w.T)]
    torch.cuda.synchronize()
    for t in range(w.T):
        gb = gbs[t % 2]
        smtm.smtm_lookup_exit_begin(cache, 0, smtm.Fmap(maps[t][0], w.dtype, w.layout, *si.shape4(w, 0)), gb)
        smtm.smtm_lookup_exit(cache, 1, smtm.Fmap(maps[t][1], w.dtype, w.layout, *si.shape4(w, 1)), gb)
        smtm.smtm_cache_update_resize(cache, gb, torch.from_numpy(si.fallback_labels(w, labs[t])).cuda())
    for t in range(w.T):
        ob = mem.new_batch(w.B, sid)
        for l in range(w.L):
            mem.lookup_exit(l, maps[t][l].cpu(), w.dtype, w.layout, si.shape4(w, l), ob)
        mem.update(ob, si.fallback_labels(w, labs[t]))
        mem.resize()
    torch.cuda.synchronize()
    assert np.array_equal(gbs[(w.T - 1) % 2].done.cpu().numpy(), ob["done"])
    assert np.array_equal(gbs[(w.T - 1) % 2].pred.cpu().numpy(), ob["pred"])
    compare_state(w, cache, mem, rep)
    routes = smtm.smtm_cache_get_routes(cache)
    assert routes[smtm.ROUTE_PIPELINED] == 2 * 2 * w.T and routes.sum() == routes[smtm.ROUTE_PIPELINED]
    smtm.smtm_cache_destroy(cache)


def _run_steps_against_oracle(w, S, sid, forgetting=False, split_refresh=False):
    """Steps of workload w on a cache of S streams with the given stream ids, library and oracle side by side;
    decisions of every step and the state after the last one must agree."""
    from harness import Report, compare_state

    cents, counts = si.initial_centers(w)
    tau = [w.tau] * w.L
    mem = oracle.OracleMemory(w.n, w.dims, tau, cents, counts, S, w.k_init, w.k_min, w.k_max, w.window_W,
                              forgetting=forgetting)
    cache = smtm.smtm_cache_create(w.n, w.dims, tau, cents, counts, n_streams=S, k_init=w.k_init, k_min=w.k_min,
                                   k_max=w.k_max, window_W=w.window_W, max_batch=w.B,
                                   flags=smtm.FLAG_FORGET_FT if forgetting else 0)
    gb = smtm.Batch(cache, w.B, stream_id=sid)
    labs = si.labels(w)
    for t in range(w.T):
        maps = [si.frames(w, l, labs[t], t, device="cuda") for l in range(w.L)]
        fb = si.fallback_labels(w, labs[t])
        for l in range(w.L):
            (smtm.smtm_lookup_exit_begin if l == 0 else smtm.smtm_lookup_exit)(
                cache, l, smtm.Fmap(maps[l], w.dtype, w.layout, *si.shape4(w, l)), gb)
        if split_refresh:
            smtm.smtm_cache_update(cache, gb, torch.from_numpy(fb).cuda())
            smtm.smtm_cache_resize(cache)
        else:
            smtm.smtm_cache_update_resize(cache, gb, torch.from_numpy(fb).cuda())
        ob = mem.new_batch(w.B, sid)
        for l in range(w.L):
            mem.lookup_exit(l, maps[l].cpu(), w.dtype, w.layout, si.shape4(w, l), ob)
        mem.update(ob, fb)
        mem.resize()
        torch.cuda.synchronize()
        assert np.array_equal(gb.done.cpu().numpy(), ob["done"]), "step %d" % t
        assert np.array_equal(gb.pred.cpu().numpy(), ob["pred"]), "step %d" % t
        assert np.array_equal(gb.exit_layer.cpu().numpy(), ob["exit_layer"]), "step %d" % t
    compare_state(w, cache, mem, Report())
    members, k = smtm.smtm_cache_get_members(cache)
    assert smtm.smtm_cache_status(cache) == 0
    smtm.smtm_cache_destroy(cache)
    return k


@pytest.mark.parametrize("forgetting", [False, True], ids=["counts", "forgetting"])
def test_several_frames_per_stream_interleaved(forgetting):
    # Six streams whose frames are interleaved in the batch, several frames each (two streams have a single
    # frame): Sec. 6.1 applies a stream's frames in ascending index, so each frame's position counts among
    # its own stream's frames only.
    w = si.C5.scaled(B=37, S=37, T=5, n=40, k_init=6, k_min=3, k_max=12)
    S = 6
    sid = np.array([(b * 7 + 3) % 4 for b in range(w.B)], np.int32)   # streams 0..3, interleaved
    sid[11], sid[20] = 4, 5                                             # streams 4 and 5: one frame each
    _run_steps_against_oracle(w, S, sid, forgetting=forgetting)


@pytest.mark.parametrize("split_refresh", [False, True], ids=["in-update", "stand-alone"])
def test_memory_of_six_hundred_classes_with_adaptive_size(split_refresh):
    # A memory of 513 .. 1024 classes: the refresh ranks by a sort in registers (inside the update's tables CTA,
    # or a thread per class in the stand-alone refresh); most classes have a zero score and follow the others in
    # ascending id; the fast memory's size moves between its bounds (Eq. 6).
    w = si.Workload("six_hundred", si.BF16, si.NCHW, B=48, stages=((256, 14, 14),), n=600, k_init=20, k_min=8,
                    k_max=100, S=1, T=5, tau=0.8, window_W=2, sigma=0.6, zipf_s=1.1, repeat_p=0.3, seed=11)
    k = _run_steps_against_oracle(w, 1, None, split_refresh=split_refresh)
    assert w.k_min <= int(k[0]) <= w.k_max


def test_maps_ready_flag_with_nhwc_maps():
    # SMTM_FLAG_MAPS_READY with NHWC maps: the first layer of a step is pooled on the library's stream beside the
    # previous step's other kernels and scored on the caller's stream; the later layers keep their one kernel
    # per layer.  Steps run back to back with two alternating carries; results are those of the oracle.
    from harness import Report, compare_state

    w = si.C3.scaled(B=40, S=40, T=5, k_min=4, k_max=16, k_init=8)
    cents, counts = si.initial_centers(w)
    tau = [w.tau] * w.L
    mem = oracle.OracleMemory(w.n, w.dims, tau, cents, counts, w.S, w.k_init, w.k_min, w.k_max, w.window_W)
    cache = smtm.smtm_cache_create(w.n, w.dims, tau, cents, counts, n_streams=w.S, k_init=w.k_init, k_min=w.k_min,
                                   k_max=w.k_max, window_W=w.window_W, max_batch=w.B, flags=smtm.FLAG_MAPS_READY)
    sid = si.stream_ids(w)
    gbs = [smtm.Batch(cache, w.B, stream_id=sid), smtm.Batch(cache, w.B, stream_id=sid)]
    labs = si.labels(w)
    maps = [[si.frames(w, l, labs[t], t, device="cuda") for l in range(w.L)] for t in range(w.T)]
    fbs = [torch.from_numpy(si.fallback_labels(w, labs[t])).cuda() for t in range(w.T)]
    torch.cuda.synchronize()
    for t in range(w.T):
        gb = gbs[t % 2]
        for l in range(w.L):
            (smtm.smtm_lookup_exit_begin if l == 0 else smtm.smtm_lookup_exit)(
                cache, l, smtm.Fmap(maps[t][l], w.dtype, w.layout, *si.shape4(w, l)), gb)
        smtm.smtm_cache_update_resize(cache, gb, fbs[t])
    torch.cuda.synchronize()
    for t in range(w.T):
        ob = mem.new_batch(w.B, sid)
        for l in range(w.L):
            mem.lookup_exit(l, maps[t][l].cpu(), w.dtype, w.layout, si.shape4(w, l), ob)
        mem.update(ob, si.fallback_labels(w, labs[t]))
        mem.resize()
    last = gbs[(w.T - 1) % 2]
    assert np.array_equal(last.done.cpu().numpy(), ob["done"])
    assert np.array_equal(last.pred.cpu().numpy(), ob["pred"])
    assert np.array_equal(last.exit_layer.cpu().numpy(), ob["exit_layer"])
    compare_state(w, cache, mem, Report())
    routes = smtm.smtm_cache_get_routes(cache)
    assert routes[smtm.ROUTE_PIPELINED] == w.T and routes[smtm.ROUTE_FUSED] == w.T * (w.L - 1), routes
    assert smtm.smtm_cache_status(cache) == 0
    smtm.smtm_cache_destroy(cache)


DENSE_GRAPH = si.Workload("dense_graph", si.BF16, si.NCHW, B=70, stages=((256, 14, 14), (512, 7, 7)), n=196, k_init=100,
                           k_min=70, k_max=196, S=1, T=8, tau=0.8, window_W=2, sigma=0.6, zipf_s=0.9, repeat_p=0.3, seed=6)


@pytest.mark.gpu
@pytest.mark.parametrize("graph", [False, True], ids=["eager", "graph"])
def test_maps_ready_flag_with_a_large_fast_memory(graph):
    # SMTM_FLAG_MAPS_READY on a cache whose fast memory is scored on the tensor cores: the first layer's pooling
    # of a step runs on the library's stream beside the previous step's decision kernel and update, into the
    # other of two split buffers.  Steps run back to back (eagerly, or captured in one graph and replayed from
    # a restored memory); results are those of the oracle.
    from harness import Report, compare_state

    w = DENSE_GRAPH
    cents, counts = si.initial_centers(w)
    tau = [w.tau] * w.L
    mem = oracle.OracleMemory(w.n, w.dims, tau, cents, counts, w.S, w.k_init, w.k_min, w.k_max, w.window_W)
    cache = smtm.smtm_cache_create(w.n, w.dims, tau, cents, counts, n_streams=w.S, k_init=w.k_init, k_min=w.k_min,
                                   k_max=w.k_max, window_W=w.window_W, max_batch=w.B, flags=smtm.FLAG_MAPS_READY)
    sid = si.stream_ids(w)
    gbs = [smtm.Batch(cache, w.B, stream_id=sid), smtm.Batch(cache, w.B, stream_id=sid)]
    labs = si.labels(w)
    maps = [[si.frames(w, l, labs[t], t, device="cuda") for l in range(w.L)] for t in range(w.T)]
    fbs = [torch.from_numpy(si.fallback_labels(w, labs[t])).cuda() for t in range(w.T)]
    torch.cuda.synchronize()

    def steps(stream=None):
        for t in range(w.T):
            gb = gbs[t % 2]
            smtm.smtm_lookup_exit_begin(cache, 0, smtm.Fmap(maps[t][0], w.dtype, w.layout, *si.shape4(w, 0)), gb, stream)
            smtm.smtm_lookup_exit(cache, 1, smtm.Fmap(maps[t][1], w.dtype, w.layout, *si.shape4(w, 1)), gb, stream)
            smtm.smtm_cache_update_resize(cache, gb, fbs[t], stream)

    if graph:
        blob = smtm.smtm_cache_export(cache)
        st = torch.cuda.Stream()
        with torch.cuda.stream(st):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=st):
                steps(st.cuda_stream)
            g.replay()
            st.synchronize()                      # (the import below is not ordered on this stream)
            smtm.smtm_cache_import(cache, blob)   # the replay that counts starts from the initial memory
            g.replay()
        st.synchronize()
    else:
        steps()
    torch.cuda.synchronize()
    for t in range(w.T):
        ob = mem.new_batch(w.B, sid)
        for l in range(w.L):
            mem.lookup_exit(l, maps[t][l].cpu(), w.dtype, w.layout, si.shape4(w, l), ob)
        mem.update(ob, si.fallback_labels(w, labs[t]))
        mem.resize()
    last = gbs[(w.T - 1) % 2]
    assert np.array_equal(last.done.cpu().numpy(), ob["done"])
    assert np.array_equal(last.pred.cpu().numpy(), ob["pred"])
    assert np.array_equal(last.exit_layer.cpu().numpy(), ob["exit_layer"])
    compare_state(w, cache, mem, Report())
    routes = smtm.smtm_cache_get_routes(cache)
    assert routes[smtm.ROUTE_PIPELINED_DENSE] == w.T and routes[smtm.ROUTE_DENSE] == w.T, routes
    assert smtm.smtm_cache_status(cache) == 0
    smtm.smtm_cache_destroy(cache)



@pytest.mark.parametrize("w", [si.C5.scaled(T=8), DENSE_GRAPH], ids=["c5_full_width", "tensor_core_route"])
def test_bench_launch_configuration_matches_oracle(w):
    # The benchmark's own launch configuration at full width: 512 streams, CUDA graphs of several steps, chained
    # launches, SMTM_FLAG_MAPS_READY with two alternating carries, no diagnostics.  The graphs are replayed twice
    # over; decisions of every step (read back from copies taken inside the graphs), counters and the final
    # state must be the oracle's.
    from harness import Report, compare_state

    G, passes = 4, 2
    cents, counts = si.initial_centers(w)
    tau = [w.tau] * w.L
    mem = oracle.OracleMemory(w.n, w.dims, tau, cents, counts, w.S, w.k_init, w.k_min, w.k_max, w.window_W)
    cache = smtm.smtm_cache_create(w.n, w.dims, tau, cents, counts, n_streams=w.S, k_init=w.k_init, k_min=w.k_min,
                                   k_max=w.k_max, window_W=w.window_W, max_batch=w.B, flags=smtm.FLAG_MAPS_READY)
    sid = si.stream_ids(w)
    gbs = [smtm.Batch(cache, w.B, stream_id=sid, with_diagnostics=False) for _ in range(2)]
    labs = si.labels(w)
    maps = [[si.frames(w, l, labs[t], t, device="cuda") for l in range(w.L)] for t in range(w.T)]
    fbs = [torch.from_numpy(si.fallback_labels(w, labs[t])).cuda() for t in range(w.T)]
    kept = [dict(done=torch.zeros(w.B, dtype=torch.uint8, device="cuda"),
                 pred=torch.zeros(w.B, dtype=torch.int32, device="cuda"),
                 el=torch.zeros(w.B, dtype=torch.int32, device="cuda")) for _ in range(w.T)]
    stream = torch.cuda.Stream()
    sh = stream.cuda_stream

    def step(t):
        gb = gbs[t % 2]
        smtm.smtm_lookup_exit_begin(cache, 0, smtm.Fmap(maps[t][0], w.dtype, w.layout, *si.shape4(w, 0)), gb, sh)
        smtm.smtm_lookup_exit(cache, 1, smtm.Fmap(maps[t][1], w.dtype, w.layout, *si.shape4(w, 1)), gb, sh)
        smtm.smtm_cache_update_resize(cache, gb, fbs[t], sh)
        kept[t]["done"].copy_(gb.done, non_blocking=True)      # a copy node of the graph
        kept[t]["pred"].copy_(gb.pred, non_blocking=True)
        kept[t]["el"].copy_(gb.exit_layer, non_blocking=True)

    with torch.cuda.stream(stream):
        graphs = []
        step(0)                      # eager once: one-time attributes are not set inside a capture
        stream.synchronize()
        smtm.smtm_cache_destroy(cache)
        cache = smtm.smtm_cache_create(w.n, w.dims, tau, cents, counts, n_streams=w.S, k_init=w.k_init,
                                       k_min=w.k_min, k_max=w.k_max, window_W=w.window_W, max_batch=w.B,
                                       flags=smtm.FLAG_MAPS_READY)
        gbs[:] = [smtm.Batch(cache, w.B, stream_id=sid, with_diagnostics=False) for _ in range(2)]
        for g0 in range(0, w.T, G):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for t in range(g0, g0 + G):
                    step(t)
            graphs.append(g)
        rep = Report()
        for p in range(passes):
            for gi, g in enumerate(graphs):
                g.replay()
                stream.synchronize()
                for t in range(gi * G, gi * G + G):   # the oracle, step by step, on the same maps
                    ob = mem.new_batch(w.B, sid)
                    for l in range(w.L):
                        mem.lookup_exit(l, maps[t][l].cpu(), w.dtype, w.layout, si.shape4(w, l), ob)
                    assert mem.near_count == 0, "a decision within 1e-4 of the threshold: pick another seed"
                    assert np.array_equal(kept[t]["done"].cpu().numpy(), ob["done"]), (p, t)
                    assert np.array_equal(kept[t]["el"].cpu().numpy(), ob["exit_layer"]), (p, t)
                    ex = ob["done"] == 1
                    assert np.array_equal(kept[t]["pred"].cpu().numpy()[ex], ob["pred"][ex]), (p, t)
                    mem.update(ob, si.fallback_labels(w, labs[t]))
                    mem.resize()
                    rep.frames += w.B
            compare_state(w, cache, mem, rep)
    ctr = smtm.smtm_cache_get_counters(cache)
    assert [int(v) for v in ctr[: w.L]] == [int(v) for v in mem.exits_per_layer]
    smtm.smtm_cache_destroy(cache)


# ---------------------------------------------------------------------------- degenerate inputs on every route

EDGE_ROUTES = {
    # route -> (workload, index into Report.routes that must serve every lookup)
    "fused": (si.Workload("edge_fused", si.BF16, si.NCHW, B=40, stages=((256, 14, 14), (512, 7, 7)), n=24, k_init=6,
                          k_min=2, k_max=9, S=1, T=3, tau=0.8, window_W=2, sigma=0.5, zipf_s=0.6, repeat_p=0.3, seed=41), 0),
    "dense": (si.Workload("edge_dense", si.BF16, si.NCHW, B=40, stages=((256, 14, 14), (512, 7, 7)), n=80, k_init=72,
                          k_min=66, k_max=80, S=1, T=3, tau=0.8, window_W=2, sigma=0.5, zipf_s=0.6, repeat_p=0.3, seed=42), 1),
    "plain": (si.Workload("edge_plain", si.F32, si.NHWC, B=40, stages=((21, 9, 5), (38, 3, 3)), n=24, k_init=6,
                          k_min=2, k_max=9, S=1, T=3, tau=0.8, window_W=2, sigma=0.5, zipf_s=0.6, repeat_p=0.3, seed=43), 2),
}


@pytest.mark.parametrize("one_entry", [False, True], ids=["k6", "k1"])
@pytest.mark.parametrize("route", list(EDGE_ROUTES))
def test_degenerate_frames_match_the_oracle_on_every_route(route, one_entry):
    # Sec. 5 is silent on these inputs; the readings are pinned on the oracle (tests/test_oracle_pins.py) and the
    # kernels must follow them element by element: an all-zero map (post-ReLU features make it a real input:
    # zero-length SV, similarity 0 to everything, no exit), a map with one NaN element and one with one +Inf
    # element (they propagate: NaN similarities rank last, the frame never exits, Eq. 7 carries the NaN into the
    # centre of the frame's class, which then ranks last for every later frame), and a fast memory with a single
    # entry (no runner-up: never exits).  Three steps, so that the poisoned centres are looked up as well.
    from harness import Report, compare_state, make_pair, step_pair

    w, served = EDGE_ROUTES[route]
    if one_entry:
        w = w.scaled(name=w.name + "_k1", k_init=1, k_min=1, k_max=max(w.k_max, 70) if route == "dense" else 3)
    cache, mem = make_pair(w)
    gb = smtm.Batch(cache, w.B)
    labs = si.labels(w)

    def poison(step):
        def edit(layer, x):
            flat = x.view(w.B, -1)
            flat[0].zero_()                                  # every layer: nothing to pool
            flat[21 + step, 5] = float("-inf")               # every layer
            if layer == 0:                                   # first layer only: the NaN then rides on in SA
                flat[1 + step, 17] = float("nan")
                flat[11 + step, flat.shape[1] - 3] = float("inf")
        return edit

    rep = Report()
    for t in range(w.T):
        ob = step_pair(w, cache, mem, gb, labs[t], t, rep, edit=poison(t))
        compare_state(w, cache, mem, rep)
        done = gb.done.cpu().numpy()
        assert not done[[0, 1 + t, 11 + t, 21 + t]].any()       # none of the degenerate frames exits
        assert np.isnan(ob["sa"][[1 + t, 11 + t, 21 + t], 0]).all()
        assert gb.ac.cpu().numpy()[0, w.L - 1] == 0.0
        if one_entry and t == 0:
            assert not done.any() and (gb.top.cpu().numpy()[:, 1] == -1).all()
    routes = smtm.smtm_cache_get_routes(cache)
    assert routes[served] == w.T * w.L and routes.sum() == w.T * w.L, routes
    assert np.isnan(mem.centers[0]).any()                        # Eq. 7 did carry a NaN into a centre
    smtm.smtm_cache_destroy(cache)


def test_stream_id_outside_the_cache_skips_the_frame_and_sets_the_status_word():
    # a frame that names a stream the cache does not have is scored against nothing, stays in, takes no part in
    # the update, and the sticky status word reports an invalid argument; the other frames are served as usual
    from harness import Report, compare_state

    w = si.C5.scaled(name="bad_sid", B=24, S=24, T=2)
    cents, counts = si.initial_centers(w)
    tau = [w.tau] * w.L
    good = si.stream_ids(w)
    bad = good.copy()
    bad[5], bad[17] = w.S, -3
    for fused in (True, False):       # the second cache is fed maps in a shape only the plain route serves
        ww = w if fused else w.scaled(name="bad_sid_plain", dtype=si.F32, layout=si.NHWC, stages=((21, 3, 3), (38, 2, 2)))
        cents, counts = si.initial_centers(ww)
        cache = smtm.smtm_cache_create(ww.n, ww.dims, tau, cents, counts, n_streams=ww.S, k_init=ww.k_init, k_min=ww.k_min,
                                       k_max=ww.k_max, window_W=ww.window_W, max_batch=ww.B)
        mem = oracle.OracleMemory(ww.n, ww.dims, tau, cents, counts, ww.S, ww.k_init, ww.k_min, ww.k_max, ww.window_W)
        gb = smtm.Batch(cache, ww.B, stream_id=bad)
        labs = si.labels(ww)
        for t in range(ww.T):
            fb = si.fallback_labels(ww, labs[t])
            ob = mem.new_batch(ww.B, good)
            for l in range(ww.L):
                x = si.frames(ww, l, labs[t], t, device="cuda")
                (smtm.smtm_lookup_exit_begin if l == 0 else smtm.smtm_lookup_exit)(
                    cache, l, smtm.Fmap(x, ww.dtype, ww.layout, *si.shape4(ww, l)), gb)
                mem.lookup_exit(l, x.cpu(), ww.dtype, ww.layout, si.shape4(ww, l), ob)
            smtm.smtm_cache_update_resize(cache, gb, torch.from_numpy(fb).cuda())
            # the oracle is told what the library is documented to do with such a frame: it does not exit and is
            # left out of the update (no label); its stream's tables (which it does not name) see nothing
            for b in (5, 17):
                ob["done"][b], ob["exit_layer"][b], ob["pred"][b] = 0, 0, -1
            fb2 = fb.copy(); fb2[[5, 17]] = -1
            sid_o = good.copy()
            keep = np.ones(ww.B, bool); keep[[5, 17]] = False
            sub = {k: (v[keep] if isinstance(v, np.ndarray) and v.shape[:1] == (ww.B,) else v) for k, v in ob.items()}
            sub["sv"] = [v[keep] for v in ob["sv"]]
            sub["B"] = int(keep.sum()); sub["stream_id"] = np.ascontiguousarray(sid_o[keep])
            mem.update(sub, fb2[keep])
            mem.resize()
            done = gb.done.cpu().numpy()
            assert not done[[5, 17]].any() and np.array_equal(done[keep], ob["done"][keep])
            assert np.array_equal(gb.pred.cpu().numpy()[keep & (done == 1)], ob["pred"][keep & (done == 1)])
            assert (gb.ac.cpu().numpy()[[5, 17]] == 0.0).all()
        assert smtm.smtm_cache_status(cache) == 1                 # SMTM_ERR_INVALID_ARG, sticky
        ft, ts = smtm.smtm_cache_get_tables(cache)
        assert np.array_equal(ft, mem.ft) and np.array_equal(ts, mem.ts)
        assert not ft[[5, 17]].any() and not ts[[5, 17]].any()    # the streams those frames should have named saw nothing
        members, k = smtm.smtm_cache_get_members(cache)
        assert np.array_equal(k, mem.k)
        for s_ in range(ww.S):      # (slots beyond k are unspecified in a fast memory that was never refreshed)
            assert np.array_equal(members[s_, : k[s_]], mem.members[s_, : k[s_]]), s_
        for l in range(ww.L):
            cen, m = smtm.smtm_cache_get_centers(cache, l)
            assert np.array_equal(m, mem.m[l])
            np.testing.assert_allclose(cen, mem.centers[l], rtol=2e-5, atol=1e-7)
        assert smtm.smtm_cache_get_routes(cache)[0 if fused else 2] == ww.T * ww.L
        smtm.smtm_cache_destroy(cache)


def test_export_then_import_puts_the_cache_back_bit_for_bit():
    # snapshot after two steps, run three more, import the snapshot, run the same three again: identical decisions
    # and an identical final state; the snapshot also moves to a second cache of the same shape, and is refused
    # by a cache of another shape
    w = si.C5.scaled(name="snapshot", B=64, S=64, T=5)
    cents, counts = si.initial_centers(w)
    tau = [w.tau] * w.L
    mk = lambda ww=w: smtm.smtm_cache_create(ww.n, ww.dims, tau, cents, counts, n_streams=ww.S, k_init=ww.k_init,
                                              k_min=ww.k_min, k_max=ww.k_max, window_W=ww.window_W, max_batch=ww.B)
    labs = si.labels(w)
    sid = si.stream_ids(w)
    maps = [[si.frames(w, l, labs[t], t, device="cuda") for l in range(w.L)] for t in range(w.T)]

    def run(cache, steps):
        gb = smtm.Batch(cache, w.B, stream_id=sid)
        out = []
        for t in steps:
            for l in range(w.L):
                (smtm.smtm_lookup_exit_begin if l == 0 else smtm.smtm_lookup_exit)(
                    cache, l, smtm.Fmap(maps[t][l], w.dtype, w.layout, *si.shape4(w, l)), gb)
            smtm.smtm_cache_update_resize(cache, gb, torch.from_numpy(si.fallback_labels(w, labs[t])).cuda())
            torch.cuda.synchronize()
            out.append((gb.done.cpu().numpy().copy(), gb.pred.cpu().numpy().copy(), gb.sa.cpu().numpy().copy()))
        return out

    def state(cache):
        return [smtm.smtm_cache_get_tables(cache), smtm.smtm_cache_get_members(cache),
                [smtm.smtm_cache_get_centers(cache, l) for l in range(w.L)], smtm.smtm_cache_get_counters(cache)]

    def same(a, b):
        flat = lambda x: [x] if isinstance(x, np.ndarray) else [z for y in x for z in flat(y)]
        return all(np.array_equal(p, q) for p, q in zip(flat(a), flat(b)))

    a = mk()
    run(a, [0, 1])
    blob = smtm.smtm_cache_export(a)
    at_snapshot = state(a)
    first = run(a, [2, 3, 4])
    after = state(a)
    assert not same(at_snapshot, after)
    smtm.smtm_cache_import(a, blob)
    assert same(state(a), at_snapshot)
    second = run(a, [2, 3, 4])
    assert same(first, second) and same(state(a), after)
    b = mk()                                     # a fresh cache of the same shape takes the snapshot too
    smtm.smtm_cache_import(b, blob)
    assert same(run(b, [2, 3, 4]), first) and same(state(b), after)
    other = mk(w.scaled(S=32, B=32))
    with pytest.raises(smtm.SmtmError) as e:
        smtm.smtm_cache_import(other, blob)
    assert e.value.status == 2
    bad = blob.copy(); bad[:8] = 0
    with pytest.raises(smtm.SmtmError) as e:
        smtm.smtm_cache_import(b, bad)
    assert e.value.status == 1 and same(state(b), after)          # nothing was changed
    for c in (a, b, other):
        smtm.smtm_cache_destroy(c)


def test_a_wait_that_runs_out_sets_the_status_word_and_leaves_the_context_usable():
    # The streaming kernels wait for their copies with a limit (about a second); a wait that runs out records
    # SMTM_ERR_TIMEOUT in the sticky status word and the kernel returns.  The self-test waits on a barrier that
    # nobody arrives on: nothing traps or hangs, the status reads 8, and after clearing it the same cache
    # serves a step that matches the oracle.
    from harness import Report, compare_state, make_pair, step_pair

    w = si.C5.scaled(name="after_timeout", B=24, S=24, T=2)
    cache, mem = make_pair(w)
    assert smtm.smtm_cache_status(cache) == 0
    smtm.smtm_cache_selftest_wait(cache)
    assert smtm.smtm_cache_status(cache) == 8            # SMTM_ERR_TIMEOUT
    assert smtm.smtm_status_string(8) == "device-side wait timed out"
    assert smtm.smtm_cache_status(cache) == 8            # sticky
    smtm.smtm_cache_clear_status(cache)
    assert smtm.smtm_cache_status(cache) == 0
    gb = smtm.Batch(cache, w.B, stream_id=si.stream_ids(w))
    rep = Report()
    labs = si.labels(w)
    for t in range(w.T):
        step_pair(w, cache, mem, gb, labs[t], t, rep)
    compare_state(w, cache, mem, rep)                    # also asserts that the status word is clear
    smtm.smtm_cache_destroy(cache)
