"""Pins for the CPU oracle: closed forms, invariants, library routines, brute force.

Each test fixes the oracle to something other than itself, chosen so that a
dropped term, a wrong sign or index, or a transposed operand fails somewhere.
"""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from oracle import BF16, F16, F32, NCHW, NHWC

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")


def golden():
    out = {}
    for line in open(GOLDEN):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split()
            out[k] = float(v)
    return out


def torch_dtype(dt):
    return {F32: torch.float32, F16: torch.float16, BF16: torch.bfloat16}[dt]


# --------------------------------------------------------------------------- GAP (Sec. 4.1)

@pytest.mark.parametrize("dt", [F32, F16, BF16])
@pytest.mark.parametrize("layout", [NCHW, NHWC])
def test_gap_constant_map_returns_the_constant(dt, layout):
    B, C, H, W = 3, 5, 7, 4
    x = torch.full((B, C, H, W), 0.625, dtype=torch_dtype(dt))  # exactly representable
    sv = oracle.gap(x, dt, layout, B, C, H, W)
    assert np.array_equal(sv, np.full((B, C), 0.625))


@pytest.mark.parametrize("dt", [F32, F16, BF16])
def test_gap_matches_numpy_mean_both_layouts(dt):
    g = torch.Generator().manual_seed(1)
    B, C, H, W = 4, 6, 5, 3  # all different: an index mix-up changes the result
    x = torch.randn((B, C, H, W), generator=g).to(torch_dtype(dt))
    ref = x.double().numpy().mean(axis=(2, 3))
    sv = oracle.gap(x, dt, NCHW, B, C, H, W)
    np.testing.assert_allclose(sv, ref, rtol=1e-14, atol=1e-15)
    sv2 = oracle.gap(x.permute(0, 2, 3, 1).contiguous(), dt, NHWC, B, C, H, W)
    np.testing.assert_allclose(sv2, ref, rtol=1e-14, atol=1e-15)


def test_gap_channel_identity_and_linearity():
    B, C, H, W = 2, 9, 3, 5
    # channel c of frame b holds the value 10*b + c everywhere
    x = (10 * torch.arange(B)[:, None, None, None] + torch.arange(C)[None, :, None, None]).float()
    x = x.expand(B, C, H, W).contiguous()
    sv = oracle.gap(x, F32, NCHW, B, C, H, W)
    assert np.array_equal(sv, 10 * np.arange(B)[:, None] + np.arange(C)[None, :])
    g = torch.Generator().manual_seed(2)
    y = torch.randn((B, C, H, W), generator=g)
    z = torch.randn((B, C, H, W), generator=g)
    lhs = oracle.gap((2 * y + 0.5 * z), F32, NCHW, B, C, H, W)
    rhs = 2 * oracle.gap(y, F32, NCHW, B, C, H, W) + 0.5 * oracle.gap(z, F32, NCHW, B, C, H, W)
    np.testing.assert_allclose(lhs, rhs, rtol=0, atol=1e-6)


def test_gap_skip_mask_leaves_rows_untouched():
    B, C, H, W = 4, 3, 2, 2
    x = torch.ones((B, C, H, W))
    out = np.full((B, C), -7.0)
    oracle.gap(x, F32, NCHW, B, C, H, W, skip=np.array([0, 1, 0, 1], np.uint8), out=out)
    assert np.array_equal(out[[0, 2]], np.ones((2, C))) and np.array_equal(out[[1, 3]], np.full((2, C), -7.0))


def test_half_and_bfloat_widening_all_bit_patterns():
    bits = np.arange(65536, dtype=np.uint16)
    ref16 = bits.view(np.float16).astype(np.float64)
    got16 = oracle.gap(bits.view(np.int16), F16, NCHW, 65536, 1, 1, 1)[:, 0]
    assert np.array_equal(np.isnan(ref16), np.isnan(got16))
    ok = ~np.isnan(ref16)
    assert np.array_equal(ref16[ok], got16[ok])   # (-0 pools to +0: the sum starts from +0)
    refb = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).double().numpy()
    gotb = oracle.gap(bits.view(np.int16), BF16, NCHW, 65536, 1, 1, 1)[:, 0]
    okb = ~np.isnan(refb)
    assert np.array_equal(np.isnan(refb), np.isnan(gotb)) and np.array_equal(refb[okb], gotb[okb])


def test_gap_of_rectified_gaussian_matches_closed_form():
    # E[max(mu + s z, 0)] = mu Phi(mu/s) + s phi(mu/s); the sample mean over H*W = 4096
    # pixels stays within 5 standard errors.
    mu, s, H = 0.3, 0.5, 64
    g = torch.Generator().manual_seed(3)
    x = (mu + s * torch.randn((1, 8, H, H), generator=g)).clamp_(min=0)
    sv = oracle.gap(x, F32, NCHW, 1, 8, H, H)[0]
    t = mu / s
    want = mu * 0.5 * (1 + math.erf(t / math.sqrt(2))) + s * math.exp(-t * t / 2) / math.sqrt(2 * math.pi)
    assert np.all(np.abs(sv - want) < 5 * s / H)


# --------------------------------------------------------------------------- cosine (Eq. 1)

def test_cosine_closed_forms():
    gold = golden()
    v = np.array([0.3, -1.2, 2.5, 0.7])
    assert oracle.cosine(v, v) == pytest.approx(1.0, abs=1e-15)
    assert oracle.cosine(v, -v) == pytest.approx(-1.0, abs=1e-15)
    assert oracle.cosine(np.array([1.0, 0, 0]), np.array([0, 1.0, 0])) == 0.0
    assert oracle.cosine(np.array([1.0, 0.0]), np.array([3.0, 4.0])) == pytest.approx(0.6, abs=1e-15)
    assert oracle.cosine(np.zeros(4), v) == 0.0 and oracle.cosine(v, np.zeros(4)) == 0.0
    rng = np.random.default_rng(0)
    for _ in range(50):
        a, b = rng.standard_normal(17), rng.standard_normal(17)
        c = oracle.cosine(a, b)
        assert gold["cosine_min"] <= c <= gold["cosine_max"]
        assert c == pytest.approx(oracle.cosine(b, a), abs=1e-15)                   # symmetric
        assert c == pytest.approx(oracle.cosine(3.5 * a, 0.01 * b), abs=1e-14)      # scale invariant
        assert c == pytest.approx(a @ b / (np.linalg.norm(a) * np.linalg.norm(b)), abs=1e-14)


# --------------------------------------------------------------------------- lookup helpers

def run_lookup(sv_layers, centers_layers, members, tau, k=None, force=None, stream_id=None):
    """Feed already-encoded semantic vectors through layers 1..L; returns the carry dict."""
    B = sv_layers[0].shape[0]
    members = np.ascontiguousarray(np.atleast_2d(members), np.int32)
    S, k_max = members.shape
    kk = np.full(S, k_max if k is None else k, np.int32)
    sid = np.zeros(B, np.int32) if stream_id is None else np.asarray(stream_id, np.int32)
    st = dict(sa=np.zeros((B, k_max)), done=np.zeros(B, np.uint8), exit_layer=np.zeros(B, np.int32),
              pred=np.full(B, -1, np.int32), ac=[], sep=[], top=[], near=[], sa_hist=[])
    for l, (sv, cen) in enumerate(zip(sv_layers, centers_layers), start=1):
        ac, sep, top, near = oracle.lookup_layer(
            l, np.ascontiguousarray(sv, np.float64), np.ascontiguousarray(cen, np.float64), sid,
            members, kk, tau, st["sa"], st["done"], st["exit_layer"], st["pred"],
            force=None if force is None else force[l - 1])
        st["ac"].append(ac); st["sep"].append(sep); st["top"].append(top); st["near"].append(near)
        st["sa_hist"].append(st["sa"].copy())
    return st


def test_cumulative_similarity_weights_and_identity():
    # Sec. 5 below Eq. 3: weight_l = 2^(l-1); constant similarity c at every layer gives
    # SA^l = c (2^l - 1), i.e. the earlier weights add up to weight_l - 1.
    gold = golden()
    L = 6
    e = np.array([[1.0, 0.0], [1.0, 0.0], [0.0, 1.0]])   # classes 0 and 1 share a centre: a tie, no exit
    sv = [np.array([[1.0, 0.0]])] * L               # cos = (1, 1, 0) at every layer
    st = run_lookup(sv, [e] * L, [0, 1, 2], tau=1e9)
    assert st["done"][0] == 0
    for l in range(1, L + 1):
        assert st["sa_hist"][l - 1][0, 0] == gold["weight_base"] ** l + gold["weight_sum_identity_offset"]
        assert st["sa_hist"][l - 1][0, 1] == st["sa_hist"][l - 1][0, 0]
        assert st["sa_hist"][l - 1][0, 2] == 0.0
    # distinct similarity per layer: SA = sum s_l 2^(l-1) with s_l = cos(theta_l)
    th = [0.3, 1.1, 0.7]
    svs = [np.array([[math.cos(t), math.sin(t)]]) for t in th]
    st = run_lookup(svs, [np.eye(2)] * 3, [0, 1], tau=1e9)
    want0 = sum(math.cos(t) * 2 ** i for i, t in enumerate(th))
    want1 = sum(math.sin(t) * 2 ** i for i, t in enumerate(th))
    np.testing.assert_allclose(st["sa"][0], [want0, want1], rtol=1e-14)


def test_accumulated_confidence_hand_example_and_strictness():
    # cosines proportional to (3, 2, 1): AC = (3 - 2) / 2 = 0.5 at a single layer, and sep = AC.
    sv = [np.array([[3.0, 2.0, 1.0]])]
    st = run_lookup(sv, [np.eye(3)], [0, 1, 2], tau=0.49)
    assert st["ac"][0][0] == pytest.approx(0.5, abs=1e-14) and st["sep"][0][0] == pytest.approx(0.5, abs=1e-14)
    assert st["done"][0] == 1 and st["pred"][0] == 0 and st["exit_layer"][0] == 1
    assert list(st["top"][0][0]) == [0, 1]
    assert run_lookup(sv, [np.eye(3)], [0, 1, 2], tau=0.51)["done"][0] == 0
    # exactly on the threshold: cosines (2, 1)/sqrt 5 give AC = 1 exactly -> "exceeds" is strict
    sv = [np.array([[2.0, 1.0]])]
    st = run_lookup(sv, [np.eye(2)], [0, 1], tau=1.0)
    assert st["ac"][0][0] == pytest.approx(1.0, abs=1e-15) and st["done"][0] == 0
    assert run_lookup(sv, [np.eye(2)], [0, 1], tau=0.999)["done"][0] == 1
    # AC is invariant to a positive scaling of the frame's vector (cosine is)
    a = run_lookup([np.array([[3.0, 2.0, 1.0]])], [np.eye(3)], [0, 1, 2], tau=9)["ac"][0][0]
    b = run_lookup([np.array([[30.0, 20.0, 10.0]])], [np.eye(3)], [0, 1, 2], tau=9)["ac"][0][0]
    assert a == pytest.approx(b, abs=1e-14)


def test_exit_happens_at_the_first_layer_that_exceeds_tau_and_label_is_class_of_top():
    # layer 1 ambiguous (cos equal-ish), layer 2 decisive for class 7 (slot 1)
    members = [4, 7]
    l1 = np.array([[1.0, 0.9]])
    l2 = np.array([[0.1, 1.0]])
    st = run_lookup([l1, l2], [np.eye(2)] * 2, [0, 1], tau=0.3)  # ids are rows of centres: remap below
    # with class ids 0/1: SA after layer 2 = (c1a + 2 c2a, c1b + 2 c2b)
    c1 = l1[0] / np.linalg.norm(l1); c2 = l2[0] / np.linalg.norm(l2)
    sa = c1 + 2 * c2
    assert st["exit_layer"][0] == 2 and st["pred"][0] == 1
    assert st["ac"][1][0] == pytest.approx((sa[1] - sa[0]) / sa[0], rel=1e-13)
    # same thing with non-trivial class ids: centres live at rows 4 and 7 of a 9-class memory
    cen = np.zeros((9, 2)); cen[4] = [1, 0]; cen[7] = [0, 1]
    st = run_lookup([l1, l2], [cen] * 2, members, tau=0.3)
    assert st["pred"][0] == 7 and list(st["top"][1][0]) == [7, 4]
    # a done frame is not touched by later layers
    st = run_lookup([np.array([[1.0, 0.0]]), np.array([[0.0, 1.0]])], [np.eye(2)] * 2, [0, 1], tau=0.5)
    assert st["exit_layer"][0] == 1 and st["pred"][0] == 0 and st["sa"][0, 0] == 1.0 and st["sa"][0, 1] == 0.0


def test_top2_brute_force_with_ties_on_tiny_caches():
    rng = np.random.default_rng(5)
    for trial in range(200):
        k, D = int(rng.integers(2, 7)), 4
        cen = rng.integers(-2, 3, (8, D)).astype(np.float64)   # small integers: exact ties occur
        cen[np.all(cen == 0, axis=1)] = 1.0
        members = rng.permutation(8)[:k].astype(np.int32)
        sv = rng.integers(-2, 3, (1, D)).astype(np.float64)
        if not sv.any():
            sv[0, 0] = 1.0
        st = run_lookup([sv], [cen], members, tau=1e9)
        cos = np.array([sv[0] @ cen[c] / (np.linalg.norm(sv[0]) * np.linalg.norm(cen[c])) for c in members])
        # all k^2 ordered pairs: top is the one nobody beats, second the best of the rest
        order = sorted(range(k), key=lambda j: (-round(cos[j], 12), members[j]))
        assert st["top"][0][0, 0] == members[order[0]]
        assert st["top"][0][0, 1] == members[order[1]]
        top, sec = cos[order[0]], cos[order[1]]
        want = 0.0 if top <= 1e-12 else (math.inf if sec <= 1e-12 else (top - sec) / sec)
        if abs(sec) > 1e-9 and abs(top) > 1e-9:
            assert st["ac"][0][0] == pytest.approx(want, rel=1e-9)


def test_sign_cases_of_the_exit_rule():
    e = np.eye(2)
    # second-highest negative, top positive: confident match, AC reported as +inf
    st = run_lookup([np.array([[1.0, -0.5]])], [e], [0, 1], tau=0.8)
    assert st["done"][0] == 1 and math.isinf(st["ac"][0][0])
    # top itself not positive: nothing resembles the frame, no exit, AC = 0
    st = run_lookup([np.array([[-1.0, -2.0]])], [e], [0, 1], tau=0.0)
    assert st["done"][0] == 0 and st["ac"][0][0] == 0.0
    # exact tie: AC = 0, lower class id reported first, no exit for tau >= 0
    st = run_lookup([np.array([[1.0, 1.0]])], [e], [1, 0], tau=0.0)
    assert st["done"][0] == 0 and st["ac"][0][0] == 0.0 and list(st["top"][0][0]) == [0, 1]
    # a single cached class has no second-highest: never exits
    st = run_lookup([np.array([[1.0, 0.0]])], [e], [0, 1], tau=0.0, k=1)
    assert st["done"][0] == 0 and st["ac"][0][0] == 0.0 and list(st["top"][0][0]) == [0, -1]
    # zero-length semantic vector: all similarities 0
    st = run_lookup([np.zeros((1, 2))], [e], [0, 1], tau=0.0)
    assert st["done"][0] == 0 and np.all(st["sa"] == 0)


def test_only_fast_memory_is_looked_up_and_streams_use_their_own():
    cen = np.eye(4)
    sv = np.array([[0.0, 0.0, 1.0, 0.1], [0.0, 0.0, 1.0, 0.1]])
    members = np.array([[0, 3], [2, 3]], np.int32)   # stream 0 does not cache class 2
    st = run_lookup([sv], [cen], members, tau=0.8, stream_id=[0, 1])
    assert st["pred"][1] == 2 and st["done"][1] == 1
    assert st["pred"][0] in (-1, 3) and list(st["top"][0][0]) == [3, 0]


def test_forced_decisions_and_near_band():
    sv = [np.array([[3.0, 2.0, 1.0]] * 2)]
    st = run_lookup(sv, [np.eye(3)], [0, 1, 2], tau=0.5 + 5e-5, force=[np.array([-1, 1], np.int8)])
    assert list(st["done"]) == [0, 1] and list(st["near"][0]) == [1, 1]
    st = run_lookup(sv, [np.eye(3)], [0, 1, 2], tau=0.4, force=[np.array([0, -1], np.int8)])
    assert list(st["done"]) == [0, 1] and list(st["near"][0]) == [0, 0]


# --------------------------------------------------------------------------- tables (Sec. 6.1)

def test_frequency_and_timestamp_tables_replay():
    rng = np.random.default_rng(7)
    S, n, B = 3, 6, 40
    sid = rng.integers(0, S, B).astype(np.int32)
    lab = rng.integers(-1, n, B).astype(np.int32)
    ft = np.zeros((S, n), np.int32); ts = np.zeros((S, n), np.int32)
    oracle.tables_update(sid, lab, ft, ts)
    for s in range(S):
        seq = [int(l) for l, q in zip(lab, sid) if q == s]
        for i in range(n):
            assert ft[s, i] == seq.count(i)                                  # appearances
            since = len(seq) - 1 - max([p for p, l in enumerate(seq) if l == i], default=-1)
            assert ts[s, i] == (since if i in seq else len(seq))            # frames since last seen
        assert ft[s].sum() == sum(1 for l in seq if l >= 0)
    # splitting the batch in two calls gives the same tables (frame-by-frame semantics)
    ft2 = np.zeros((S, n), np.int32); ts2 = np.zeros((S, n), np.int32)
    oracle.tables_update(sid[:13].copy(), lab[:13].copy(), ft2, ts2)
    oracle.tables_update(sid[13:].copy(), lab[13:].copy(), ft2, ts2)
    assert np.array_equal(ft, ft2) and np.array_equal(ts, ts2)


# --------------------------------------------------------------------------- Eq. 5 / Eq. 6

def test_replacement_score_is_eq5_exactly():
    gold = golden()
    W = 16
    unit = 4 ** 12
    for ft, ts in itertools.product([0, 1, 3, 17, 1000], [0, 1, 15, 16, 31, 32, 100, 191]):
        want = Fraction(ft) * Fraction(gold["decay_base"]) ** (ts // W)
        assert Fraction(oracle.score(ft, ts, W), unit) == want
    assert oracle.score(5, 15, 16) == 5 * unit          # inside the window: no decay
    assert oracle.score(8, 16, 16) * 4 == 8 * unit      # one window elapsed: a quarter


def brute_resize(ft, ts, W, k_min, k_max, cl):
    sc = [Fraction(int(f)) * Fraction(1, 4) ** (int(t) // W) for f, t in zip(ft, ts)]
    total = sum(sc)
    if total == 0:
        return None
    order = sorted(range(len(sc)), key=lambda i: (-sc[i], i))
    k = k_max
    for kk in range(k_min, k_max + 1):
        if sum(sc[i] for i in order[:kk]) / total > cl:
            k = kk
            break
    return order[:k_max], k


def test_resize_matches_exact_rational_brute_force():
    rng = np.random.default_rng(11)
    for trial in range(100):
        S, n = 2, int(rng.integers(4, 30))
        k_min = int(rng.integers(1, 4)); k_max = int(rng.integers(k_min, min(n, 12) + 1))
        ft = (rng.integers(0, 6, (S, n)) * (rng.random((S, n)) < 0.6)).astype(np.int32)
        ts = rng.integers(0, 80, (S, n)).astype(np.int32)
        members = np.full((S, k_max), -5, np.int32); k = np.full(S, -5, np.int32)
        oracle.resize(ft, ts, 16, k_min, k_max, 19, 20, members, k)
        for s in range(S):
            want = brute_resize(ft[s], ts[s], 16, k_min, k_max, Fraction(19, 20))
            if want is None:
                assert k[s] == -5 and np.all(members[s] == -5)   # all-zero scores: state kept
            else:
                assert list(members[s]) == want[0] and k[s] == want[1]


def test_adaptive_size_closed_forms():
    gold = golden()
    n = 40
    cl = Fraction(gold["confidence_level"]).limit_denominator(100)
    assert cl == Fraction(19, 20)
    ts = np.zeros((1, n), np.int32)
    # uniform scores: smallest k with k/n > 0.95 is floor(0.95 n) + 1
    ft = np.full((1, n), 3, np.int32)
    members = np.zeros((1, n), np.int32); k = np.zeros(1, np.int32)
    oracle.resize(ft, ts, 16, 1, n, 19, 20, members, k)
    assert k[0] == math.floor(0.95 * n) + 1 and list(members[0]) == list(range(n))
    # ... clipped by k_max
    m2 = np.zeros((1, 10), np.int32)
    oracle.resize(ft, ts, 16, 1, 10, 19, 20, m2, k)
    assert k[0] == 10
    # one dominant class: k_min is enough
    ft = np.ones((1, n), np.int32); ft[0, 17] = 100000
    m3 = np.zeros((1, 8), np.int32)
    oracle.resize(ft, ts, 16, 2, 8, 19, 20, m3, k)
    assert k[0] == 2 and m3[0, 0] == 17 and m3[0, 1] == 0
    # k = n covers everything: P(A) = 1 exceeds any CL below 1, raising CL never shrinks k
    rng = np.random.default_rng(3)
    ft = rng.integers(0, 50, (1, n)).astype(np.int32); ts = rng.integers(0, 64, (1, n)).astype(np.int32)
    last = 0
    for num in (10, 14, 17, 19):
        mm = np.zeros((1, n), np.int32)
        oracle.resize(ft, ts, 16, 1, n, num, 20, mm, k)
        assert k[0] >= last
        last = k[0]
    # recency beats frequency once a window has elapsed: FT 10 seen 40 frames ago (10/16) < FT 1 now
    ft = np.array([[10, 1, 0]], np.int32); ts = np.array([[40, 0, 0]], np.int32)
    mm = np.zeros((1, 2), np.int32)
    oracle.resize(ft, ts, 16, 1, 2, 19, 20, mm, k)
    assert list(mm[0]) == [1, 0]


# --------------------------------------------------------------------------- Eq. 7

def test_centre_update_closed_form_and_fixed_point():
    rng = np.random.default_rng(13)
    n, D, B = 5, 7, 12
    c0 = rng.standard_normal((n, D)); m0 = rng.integers(1, 40, n).astype(np.uint32)
    sv = rng.standard_normal((B, D))
    final = rng.integers(-1, n, B).astype(np.int32)
    stop = rng.integers(1, 4, B).astype(np.int32)
    for l0 in (1, 2, 3):
        c = c0.copy(); m = m0.copy()
        oracle.centers_update(l0, sv, final, stop, c, m)
        for j in range(n):
            F = [b for b in range(B) if final[b] == j and stop[b] >= l0]
            want = (m0[j] * c0[j] + sv[F].sum(axis=0)) / (m0[j] + len(F))   # mean of m old + q new samples
            np.testing.assert_allclose(c[j], want, rtol=1e-12, atol=1e-14)
            assert m[j] == m0[j] + len(F)
    # identical vector: the centre does not move, the count does
    c = np.tile(np.array([[0.25, -1.5, 3.0]]), (2, 1)); m = np.array([4, 9], np.uint32)
    sv = np.tile(np.array([[0.25, -1.5, 3.0]]), (6, 1))
    oracle.centers_update(1, sv, np.zeros(6, np.int32), np.ones(6, np.int32), c, m)
    assert np.array_equal(c, np.tile(np.array([[0.25, -1.5, 3.0]]), (2, 1))) and list(m) == [10, 9]
    # a single update with m = 1 is the midpoint
    c = np.array([[2.0, 4.0]]); m = np.array([1], np.uint32)
    oracle.centers_update(1, np.array([[4.0, 0.0]]), np.zeros(1, np.int32), np.ones(1, np.int32), c, m)
    assert np.array_equal(c, [[3.0, 2.0]]) and m[0] == 2


# --------------------------------------------------------------------------- forgetting variant (Sec. 6.1 / 7.1)

def test_forgetting_tables_equal_eq5_score_until_a_class_reappears_and_forget_afterwards():
    W, n = 4, 3
    unit = 1 << oracle.FT_FRAC
    # class 0 seen five times, then class 1 for 9 frames: class 0 has TS = 9 -> two windows elapsed
    seq = np.array([0] * 5 + [1] * 9, np.int32)
    sid = np.zeros(len(seq), np.int32)
    ft = np.zeros((1, n), np.int32); ts = np.zeros((1, n), np.int32)
    oracle.tables_update(sid, seq, ft, ts, forgetting_W=W)
    plain_ft = np.zeros((1, n), np.int32); plain_ts = np.zeros((1, n), np.int32)
    oracle.tables_update(sid, seq, plain_ft, plain_ts)
    assert np.array_equal(ts, plain_ts)
    for i in range(n):   # FT of the forgetting table = Eq. 5's score of the plain tables (exact here: no rounding)
        want = Fraction(int(plain_ft[0, i])) * Fraction(1, 4) ** (int(plain_ts[0, i]) // W)
        assert Fraction(int(ft[0, i]), unit) == want
    assert ft[0, 0] == 5 * unit // 16 and ft[0, 1] == 9 * unit and ft[0, 2] == 0
    # class 0 reappears once: the plain count is 6, the forgetting table only remembers 5/16 + 1
    more = np.array([0], np.int32)
    oracle.tables_update(np.zeros(1, np.int32), more, ft, ts, forgetting_W=W)
    oracle.tables_update(np.zeros(1, np.int32), more, plain_ft, plain_ts)
    assert plain_ft[0, 0] == 6 and ft[0, 0] == 5 * unit // 16 + unit and ts[0, 0] == 0
    # ranking with forgetting uses FT as the score: class 1 (9) > class 0 (21/16) > class 2
    members = np.zeros((1, 3), np.int32); k = np.zeros(1, np.int32)
    oracle.resize(ft, ts, W, 1, 3, 19, 20, members, k, forgetting=True)
    assert list(members[0]) == [1, 0, 2] and k[0] == 2   # 9 / (9 + 21/16) = 0.873 < 0.95 -> two entries
    # decay rounds down in fixed point: one appearance survives five windows (1024 >> 10 = 1), not six
    ft = np.zeros((1, 2), np.int32); ts = np.zeros((1, 2), np.int32)
    seq = np.array([0] + [1] * (5 * W), np.int32)
    oracle.tables_update(np.zeros(len(seq), np.int32), seq, ft, ts, forgetting_W=W)
    assert ft[0, 0] == 1
    oracle.tables_update(np.zeros(W, np.int32), np.ones(W, np.int32), ft, ts, forgetting_W=W)
    assert ft[0, 0] == 0


# --------------------------------------------------------------------------- branches the paper is silent on

def test_nan_similarity_ranks_below_every_number_and_an_all_nan_frame_never_exits():
    # Sec. 5, Eq. 4 says nothing about non-finite similarities.  Reading: a NaN ranks after every
    # number in top-1 / top-2 (ties among NaN by class id) and a frame whose SA are all NaN
    # reports AC = 0 and stays in.  A NaN component in the semantic vector makes every cosine NaN;
    # a NaN in one centre makes only that class's similarity NaN.
    e = np.eye(3)
    cen = e.copy()
    cen[0, 1] = np.nan                       # class 0's centre is broken: its similarity is NaN
    sv = np.array([[0.9, 0.5, 0.2]])
    st = run_lookup([sv], [cen], [0, 1, 2], tau=0.8)
    assert math.isnan(st["sa"][0, 0]) and not math.isnan(st["sa"][0, 1])
    # the numbers rank first, in their own order: class 1 (0.5/|sv|) then class 2; the NaN is last
    assert list(st["top"][0][0]) == [1, 2]
    want = (0.5 - 0.2) / 0.2                 # cosines share the denominator |sv|
    assert st["ac"][0][0] == pytest.approx(want, rel=1e-12) and st["done"][0] == 1 and st["pred"][0] == 1
    # one number among NaNs: the number is top-1, a NaN (lowest class id) second.  Eq. 4 with a NaN
    # runner-up is NaN, and a NaN confidence exceeds no threshold: the frame stays in
    cen2 = e.copy(); cen2[0, 0] = np.nan; cen2[2, 2] = np.nan
    for tau in (0.8, 0.0, -1.0):
        st = run_lookup([np.array([[0.1, 0.7, 0.1]])], [cen2], [0, 1, 2], tau=tau)
        assert list(st["top"][0][0]) == [1, 0] and math.isnan(st["ac"][0][0])
        assert st["done"][0] == 0 and st["pred"][0] == -1 and st["near"][0][0] == 0
    # every similarity NaN (a NaN in the frame itself): top-1 is the lowest class id by the tie rule,
    # AC = 0, no exit at any threshold, and nothing is predicted
    svn = np.array([[np.nan, 1.0, 0.0]])
    for tau in (0.8, 0.0, -1.0):
        st = run_lookup([svn], [e], [2, 0, 1], tau=tau)
        assert np.isnan(st["sa"]).all()
        assert st["done"][0] == 0 and st["ac"][0][0] == 0.0 and st["pred"][0] == -1
        assert list(st["top"][0][0]) == [0, 1]
    # an infinite component: inf / inf in Eq. 1 is NaN as well, same outcome
    st = run_lookup([np.array([[np.inf, 1.0, 0.0]])], [e], [0, 1, 2], tau=0.5)
    assert np.isnan(st["sa"]).all() and st["done"][0] == 0 and st["ac"][0][0] == 0.0


def test_replacement_score_exponent_is_clamped_at_twelve_windows():
    # Eq. 5's 0.25^floor(TS / W) is held as the integer FT * 4^(12 - e): beyond e = 12 the factor
    # would drop below one unit, so e stops there (a stated deviation: FT * 4^0 = FT from 12 W on).
    W, unit = 16, 4 ** 12
    assert oracle.score(7, 11 * W + W - 1, W) == 7 * 4          # e = 11: the last exact window
    assert Fraction(oracle.score(7, 11 * W, W), unit) == Fraction(7) * Fraction(1, 4) ** 11
    for ts in (12 * W, 12 * W + 5, 13 * W, 40 * W, 2 ** 31 - 1):
        assert oracle.score(7, ts, W) == 7                       # e clamped: never below FT * 4^0
        assert oracle.score(1 << 20, ts, W) == 1 << 20
    assert oracle.score(0, 40 * W, W) == 0
    # the clamp keeps the order of Eq. 5 among old classes (monotone in FT) and against fresh ones
    assert oracle.score(3, 40 * W, W) < oracle.score(4, 40 * W, W) < oracle.score(2, 11 * W, W)


def test_frequency_count_saturates_and_time_stamp_stops_at_its_ceiling():
    # FT stops at 2^20 (so that Eq. 6's sums of FT * 4^12 over up to 8192 classes fit 64 bits) and TS at
    # INT32_MAX; neither wraps.
    sid = np.zeros(3, np.int32)
    ft = np.array([[(1 << 20) - 1, 5]], np.int32)
    ts = np.array([[9, 2 ** 31 - 2]], np.int32)
    oracle.tables_update(sid, np.array([0, 0, 0], np.int32), ft, ts)
    assert ft[0, 0] == 1 << 20 and ts[0, 0] == 0            # one more appearance reaches the cap, two more stay
    assert ft[0, 1] == 5 and ts[0, 1] == 2 ** 31 - 1        # aged once to the ceiling, then held
    oracle.tables_update(sid, np.array([1, -1, 0], np.int32), ft, ts)
    assert ft[0, 0] == 1 << 20 and ft[0, 1] == 6 and ts[0, 1] == 2 and ts[0, 0] == 0
    # the score of a saturated count is the cap times the window factor, still exact in 64 bits
    assert oracle.score(1 << 20, 0, 16) == (1 << 20) * 4 ** 12
    assert oracle.score((1 << 20) + 123, 0, 16) == (1 << 20) * 4 ** 12    # a larger stored value reads as the cap
    # the forgetting table saturates at the same count in its fixed-point unit and ages to the same ceiling
    ft = np.array([[((1 << 20) << oracle.FT_FRAC) - 1, 0]], np.int32)
    ts = np.array([[0, 2 ** 31 - 2]], np.int32)
    oracle.tables_update(np.zeros(2, np.int32), np.array([0, 0], np.int32), ft, ts, forgetting_W=1 << 30)
    assert ft[0, 0] == (1 << 20) << oracle.FT_FRAC and ts[0, 1] == 2 ** 31 - 1
