"""The oracle's batch step against a second, independent statement of the paper's
frame-by-frame procedure written with numpy library routines, and the batch /
stream equivalences the step semantics promise."""
import math

import numpy as np
import torch

import oracle
import smtm_inputs as si


class FrameByFrame:
    """One stream, one frame at a time, straight from Sec. 5 and Sec. 6 with numpy routines."""

    def __init__(self, centers, counts, members, tau, W, k_min, k_max, cl):
        self.c = [np.array(c, np.float64) for c in centers]
        self.m = [np.array(x, np.int64) for x in counts]
        self.members = list(members)
        self.tau, self.W, self.k_min, self.k_max, self.cl = tau, W, k_min, k_max, cl
        n = self.c[0].shape[0]
        self.ft = np.zeros(n, np.int64)
        self.ts = np.zeros(n, np.int64)

    def infer(self, maps, fallback):
        """maps: list over layers of float64 [C,H,W].  Returns (label, stop layer, exited)."""
        L = len(maps)
        sa = np.zeros(len(self.members))
        svs = []
        label, stop, exited = fallback, L, False
        for l, x in enumerate(maps, start=1):
            sv = x.mean(axis=(1, 2))
            svs.append(sv)
            cen = self.c[l - 1][self.members]
            s = cen @ sv / (np.linalg.norm(cen, axis=1) * np.linalg.norm(sv))
            sa += s * 2.0 ** (l - 1)
            order = sorted(range(len(sa)), key=lambda j: (-sa[j], self.members[j]))
            h, sh = sa[order[0]], sa[order[1]]
            if h > 0 and (h - sh) > self.tau * max(sh, 0.0):
                label, stop, exited = self.members[order[0]], l, True
                break
        # after-inference updates
        if label >= 0:
            self.ft[label] += 1
        self.ts += 1
        if label >= 0:
            self.ts[label] = 0
            for l0 in range(1, stop + 1):
                c, m = self.c[l0 - 1], self.m[l0 - 1]
                c[label] = (c[label] * m[label] + svs[l0 - 1]) / (m[label] + 1)
                m[label] += 1
        score = self.ft * 0.25 ** (self.ts // self.W)
        if score.sum() > 0:
            rank = sorted(range(len(score)), key=lambda i: (-score[i], i))
            k = self.k_max
            for kk in range(self.k_min, self.k_max + 1):
                if score[rank[:kk]].sum() / score.sum() > self.cl:
                    k = kk
                    break
            self.members = rank[:k]
        return label, stop, exited


def small_workload(**kw):
    base = dict(name="tiny", dtype=si.F32, layout=si.NCHW, B=1, stages=((12, 3, 2), (20, 2, 2)), n=9,
                k_init=3, k_min=2, k_max=6, S=1, T=40, tau=0.35, window_W=4, sigma=0.4, relu=True,
                zipf_s=1.0, repeat_p=0.7, seed=5)
    base.update(kw)
    return si.Workload(**base)


def test_single_stream_step_equals_frame_by_frame_procedure():
    w = small_workload()
    cents, counts = si.initial_centers(w)
    mem = oracle.OracleMemory(w.n, w.dims, [w.tau] * w.L, cents, counts, 1, w.k_init, w.k_min, w.k_max,
                              w.window_W)
    ref = FrameByFrame(cents, counts, range(w.k_init), float(np.float32(w.tau)), w.window_W, w.k_min,
                       w.k_max, 0.95)
    labs = si.labels(w)
    exits = 0
    for t in range(w.T):
        lab = labs[t]
        fb = si.fallback_labels(w, lab)
        maps = [si.frames(w, l, lab, t) for l in range(w.L)]
        batch = mem.new_batch(1)
        for l in range(w.L):
            mem.lookup_exit(l, maps[l], w.dtype, w.layout, si.shape4(w, l), batch)
        mem.update(batch, fb)
        mem.resize()
        label, stop, exited = ref.infer([m[0].double().numpy() for m in maps], int(fb[0]))
        exits += exited
        assert bool(batch["done"][0]) == exited
        assert (batch["exit_layer"][0] if exited else w.L) == stop
        assert (batch["pred"][0] if exited else fb[0]) == label
        assert list(mem.members[0, : mem.k[0]]) == list(ref.members)
        assert np.array_equal(mem.ft[0], ref.ft) and np.array_equal(mem.ts[0], ref.ts)
        for l in range(w.L):
            np.testing.assert_allclose(mem.centers[l], ref.c[l], rtol=1e-12, atol=1e-14)
            assert np.array_equal(mem.m[l], ref.m[l])
    assert 5 < exits < w.T          # the scenario exercises both outcomes
    assert mem.k.min() >= w.k_min and len(set(map(int, mem.members[0]))) == w.k_max


def test_streams_are_independent_except_through_the_shared_centres():
    # S streams x 1 frame per step: tables and fast memories equal those of S separate
    # single-stream runs when the centres are held fixed (tau high enough that nothing
    # exits would still move centres, so compare tables only, which do not depend on them).
    w = small_workload(B=4, S=4, T=25, tau=1e9)
    cents, counts = si.initial_centers(w)
    labs = si.labels(w)
    sid = si.stream_ids(w)
    mem = oracle.OracleMemory(w.n, w.dims, [w.tau] * w.L, cents, counts, w.S, w.k_init, w.k_min, w.k_max,
                              w.window_W)
    solo = [oracle.OracleMemory(w.n, w.dims, [w.tau] * w.L, cents, counts, 1, w.k_init, w.k_min, w.k_max,
                                w.window_W) for _ in range(w.S)]
    for t in range(w.T):
        fb = si.fallback_labels(w, labs[t])
        maps = [si.frames(w, l, labs[t], t) for l in range(w.L)]
        batch = mem.new_batch(w.B, sid)
        for l in range(w.L):
            mem.lookup_exit(l, maps[l], w.dtype, w.layout, si.shape4(w, l), batch)
        mem.update(batch, fb)
        mem.resize()
        for s in range(w.S):
            b1 = solo[s].new_batch(1)
            for l in range(w.L):
                solo[s].lookup_exit(l, maps[l][s:s + 1], w.dtype, w.layout, si.shape4(w, l, 1), b1)
            solo[s].update(b1, fb[s:s + 1])
            solo[s].resize()
            assert np.array_equal(mem.ft[s], solo[s].ft[0]) and np.array_equal(mem.ts[s], solo[s].ts[0])
            assert mem.k[s] == solo[s].k[0] and np.array_equal(mem.members[s], solo[s].members[0])


def test_batch_of_one_stream_updates_tables_like_consecutive_frames():
    # B frames of one stream in one step: tables as if the frames had come one by one;
    # centres as Eq. 7 applied once per frame in ascending order.
    w = small_workload(B=16, S=1, T=1, tau=0.35)
    cents, counts = si.initial_centers(w)
    lab = si.labels(w)[0]
    fb = si.fallback_labels(w, lab)
    mem = oracle.OracleMemory(w.n, w.dims, [w.tau] * w.L, cents, counts, 1, w.k_init, w.k_min, w.k_max,
                              w.window_W)
    maps = [si.frames(w, l, lab, 0) for l in range(w.L)]
    batch = mem.new_batch(w.B)
    for l in range(w.L):
        mem.lookup_exit(l, maps[l], w.dtype, w.layout, si.shape4(w, l), batch)
    mem.update(batch, fb)
    final = np.where(batch["done"] == 1, batch["pred"], fb)
    stop = np.where(batch["done"] == 1, batch["exit_layer"], w.L)
    assert mem.ft[0].sum() == (final >= 0).sum()
    for i in range(w.n):
        pos = [b for b in range(w.B) if final[b] == i]
        assert mem.ft[0, i] == len(pos)
        assert mem.ts[0, i] == (w.B - 1 - pos[-1] if pos else w.B)
    for l in range(w.L):
        sv = maps[l].double().numpy().mean(axis=(2, 3))
        for j in range(w.n):
            F = [b for b in range(w.B) if final[b] == j and stop[b] >= l + 1]
            want = (counts[l][j] * cents[l][j].astype(np.float64) + sv[F].sum(axis=0)) / (counts[l][j] + len(F))
            np.testing.assert_allclose(mem.centers[l][j], want, rtol=1e-12, atol=1e-14)
            assert mem.m[l][j] == counts[l][j] + len(F)


def test_workload_recipes_have_the_stated_statistics():
    p = si.zipf_pmf(100, 1.1)
    assert math.isclose(p.sum(), 1.0) and math.isclose(p[0] / p[9], 10 ** 1.1, rel_tol=1e-12)
    lab = si.labels(si.C5)
    assert lab.shape == (64, 512) and lab.min() >= 0 and lab.max() < 500
    rep = (lab[1:] == lab[:-1]).mean()
    assert 0.85 < rep < 0.90            # 0.85 + 0.15 * P(resample hits the same class)
    lab3 = si.labels(si.C3)[0]
    assert 0.12 < (lab3 >= 200).mean() < 0.28 and lab3.max() < 250
    x = si.frames(si.C3.scaled(B=4), 3, lab3[:4])
    assert x.shape == (4, 7, 7, 320) and x.dtype == torch.float16 and x.min() >= 0
    x = si.frames(si.C1, 0, si.labels(si.C1)[0])
    assert x.shape == (8, 64, 56, 56) and x.dtype == torch.float32 and x.min() < 0
    c1 = si.initial_centers(si.C1)[0][0]
    np.testing.assert_allclose(np.linalg.norm(c1, axis=1), 1.0, rtol=1e-6)


def test_centre_warm_up_from_zero_is_the_class_mean():
    # Sec. 5: centres start as the average semantic vector per class over labelled frames.
    n, C, H, W, B = 5, 12, 3, 4, 40
    rng = np.random.default_rng(21)
    x = torch.from_numpy(rng.standard_normal((B, C, H, W)).astype(np.float32))
    lab = rng.integers(-1, n + 2, B).astype(np.int32)          # -1 and labels >= n are skipped
    mem = oracle.OracleMemory(n, [C], [0.8], [np.zeros((n, C), np.float32)], [np.zeros(n, np.uint32)], k_init=2,
                              k_min=2, k_max=3)
    mem.warmup(0, x[:25], oracle.F32, oracle.NCHW, (25, C, H, W), lab[:25])
    mem.warmup(0, x[25:], oracle.F32, oracle.NCHW, (15, C, H, W), lab[25:])   # in two batches: same mean
    sv = x.double().numpy().mean(axis=(2, 3))
    for j in range(n):
        rows = sv[lab == j]
        assert mem.m[0][j] == len(rows)
        if len(rows):
            np.testing.assert_allclose(mem.centers[0][j], rows.mean(axis=0), rtol=1e-12, atol=1e-14)
        else:
            assert not mem.centers[0][j].any()
    assert not mem.ft.any() and not mem.ts.any()               # tables untouched
