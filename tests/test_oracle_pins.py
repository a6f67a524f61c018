"""Pins for the CPU oracle: closed forms, invariants, hand-derived values, library
special cases and brute force.  None of these tests re-types the oracle's loops;
each checks it against something the paper or the mathematics fixes.
"""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import sharpv_oracle as orc
from paper_2511_08003_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split()
            out[k] = float(v)
    return out


# ---------------------------------------------------------------- Eq. 1 identities
def test_dissim_identities():
    rng = np.random.default_rng(10)
    v = rng.standard_normal(257)
    assert orc.dissim(v, v) == 0.0
    assert orc.dissim(v, 3.7 * v) < 1e-15               # direction only: scale invariant
    assert abs(orc.dissim(v, -v) - 2.0) < 1e-15         # antipodal unit vectors
    u = rng.standard_normal(257)
    u -= (u @ v) / (v @ v) * v                          # orthogonal to v
    assert abs(orc.dissim(v, u) - math.sqrt(2.0)) < 1e-14


@pytest.mark.parametrize("theta", [1e-6, 0.01, 0.3, math.pi / 4, 1.0, math.pi / 2, 2.5, math.pi])
def test_dissim_is_chord_of_angle(theta):
    """Eq. 1: the distance between unit vectors at angle theta is the chord 2 sin(theta/2)."""
    rng = np.random.default_rng(11)
    d = 64
    q, _ = np.linalg.qr(rng.standard_normal((d, d)))    # random rotation
    a = q @ np.r_[5.0, 0.0, np.zeros(d - 2)]
    b = q @ np.r_[0.25 * math.cos(theta), 0.25 * math.sin(theta), np.zeros(d - 2)]
    assert abs(orc.dissim(a, b) - 2.0 * math.sin(theta / 2)) < 1e-13
    assert abs(orc.cosine(a, b) - math.cos(theta)) < 1e-13
    assert abs(orc.one_minus_cos(a, b) - (1 - math.cos(theta))) < 1e-13


def test_dissim_both_sides_of_eq1_agree():
    """||v1^ - v2^|| (what the oracle evaluates) against sqrt(2 - 2 cos) with cos from numpy."""
    rng = np.random.default_rng(12)
    for _ in range(50):
        a, b = rng.standard_normal(100), rng.standard_normal(100)
        c = float(a @ b / (np.linalg.norm(a) * np.linalg.norm(b)))
        assert abs(orc.dissim(a, b) - math.sqrt(2 - 2 * c)) < 1e-12
        assert abs(orc.cosine(a, b) - c) < 1e-14
        assert abs(orc.cosine(a, a) - 1.0) < 1e-14      # self-similarity
        assert abs(orc.cosine(2.5 * a, 0.1 * b) - c) < 1e-14


def test_zero_vector_convention():
    z = np.zeros(8)
    v = np.arange(1.0, 9.0)
    assert orc.dissim(z, z) == 0.0
    assert abs(orc.dissim(z, v) - 1.0) < 1e-15          # |0 - v^| = 1
    assert orc.cosine(z, v) == 0.0


# ---------------------------------------------------------------- hand-derived example
def test_hand_case_f2_d2():
    g = _golden("hand_case_f2_d2.txt")
    tokens = np.array([[1, 0], [0, 1], [0, 1], [0, 1]], dtype=np.float32)
    r = orc.score_frames(tokens, [0, 2], f=2, w=1.0)
    S, T, I = r["spatial"], r["temporal"], r["importance"]
    tol = 1e-14
    assert abs(S[0] - g["S1_0"]) < tol and abs(S[1] - g["S1_1"]) < tol
    assert abs(T[0] - g["T1_0"]) < tol
    assert abs(I[0] - g["I1_0"]) < tol
    assert abs(r["ratio"][0] - g["ratio_1"]) < tol
    assert abs(S[2] - g["S2_0"]) < tol and abs(S[3] - g["S2_1"]) < tol
    assert abs(T[2] - g["T2_0"]) < tol and abs(T[3] - g["T2_1"]) < tol
    assert abs(I[2] - g["I2_0"]) < tol and abs(I[3] - g["I2_1"]) < tol
    assert abs(r["ratio"][1] - g["ratio_2"]) < tol
    # budgets: floor(0.3827*2)=0, floor(0.5*2)=1; ceil gives 1,1; nearest gives 1,1
    assert list(r["k"]) == [0, 1]
    assert list(orc.score_frames(tokens, [0, 2], f=2, round_mode=orc.ROUND_CEIL)["k"]) == [1, 1]
    assert list(orc.score_frames(tokens, [0, 2], f=2, round_mode=orc.ROUND_NEAREST)["k"]) == [1, 1]
    assert list(orc.score_frames(tokens, [0, 2], f=2, min_keep=1)["k"]) == [1, 1]
    idx, off = orc.select_tokens(I, [1, 1], f=2)
    assert list(idx) == [0, 2] and list(off) == [0, 1, 2]   # frame 1 tie -> lower index; frame 2 token 0


def test_w_weights_the_spatial_term():
    """Eq. 4: I = T + w S, so I(w=2) - I(w=1) = S and I(w=0) = T."""
    wl = W.fill_tokens(W.custom("w", 5, W.F32, 3, 16, 0, [W.make_video_spec(3, 0.5)]))
    r0 = orc.score_frames(wl.tokens, wl.video_frame_offsets, wl.f, w=0.0)
    r1 = orc.score_frames(wl.tokens, wl.video_frame_offsets, wl.f, w=1.0)
    r2 = orc.score_frames(wl.tokens, wl.video_frame_offsets, wl.f, w=2.0)
    np.testing.assert_allclose(r0["importance"], r0["temporal"], rtol=0, atol=0)
    np.testing.assert_allclose(r2["importance"] - r1["importance"], r1["spatial"], rtol=0, atol=1e-15)
    np.testing.assert_array_equal(r1["ratio"], r2["ratio"])          # the budget does not depend on w


# ---------------------------------------------------------------- Section 3.1.3 equivalence
def test_first_frame_equals_virtual_mean_frame():
    """Eq. 6 must equal Eq. 5 applied after prepending a frame whose tokens all equal the
    first frame's mean (the paper's stated equivalence)."""
    rng = np.random.default_rng(13)
    d = 40
    # integer-valued tokens and f a power of two: the mean is exactly representable in fp32,
    # so the virtual frame can be handed to the oracle without rounding
    f2 = 8
    xi = rng.integers(-8, 9, size=(2 * f2, d)).astype(np.float32)
    base = orc.score_frames(xi, [0, 2], f2)
    virt = np.repeat(xi[:f2].astype(np.float64).mean(axis=0, keepdims=True), f2, axis=0).astype(np.float32)
    assert np.array_equal(virt.astype(np.float64).mean(axis=0), xi[:f2].astype(np.float64).mean(axis=0))
    ext = orc.score_frames(np.concatenate([virt, xi]), [0, 3], f2)
    # frame index 1 of the extended video is the original frame 1, now scored by the t>=2 rule
    assert abs(ext["ratio"][1] - base["ratio"][0]) < 1e-14
    np.testing.assert_allclose(ext["temporal"][f2:2 * f2], base["spatial"][:f2], atol=1e-14)
    np.testing.assert_allclose(ext["ratio"][2], base["ratio"][1], atol=0)


def test_first_frame_kept_set_independent_of_T1_convention():
    """With T_1 := S_1, I_1 = (1+w) S_1: the kept set equals the top-k of S_1 alone."""
    wl = W.fill_tokens(W.custom("c", 6, W.F32, 5, 32, 0, [W.make_video_spec(2, 0.8)]))
    r = orc.score_frames(wl.tokens, wl.video_frame_offsets, wl.f, w=0.7)
    k = [7, 0]
    a, _ = orc.select_tokens(r["importance"], k, wl.f)
    b, _ = orc.select_tokens(r["spatial"], k, wl.f)
    assert np.array_equal(a, b)


# ---------------------------------------------------------------- bounds and special cases
def test_bounds_and_static_video():
    wl = W.fill_tokens(W.tiny(d=64))
    r = orc.score_frames(wl.tokens, wl.video_frame_offsets, wl.f)
    for key in ("spatial", "temporal"):
        assert r[key].min() >= 0.0 and r[key].max() <= 2.0
    assert r["importance"].max() <= 4.0
    assert r["ratio"].min() >= 0.0 and r["ratio"].max() <= 1.0
    assert np.all(r["k"] >= 0) and np.all(r["k"] <= wl.f)
    np.testing.assert_array_equal(r["k"], np.floor(r["ratio"].astype(np.float32) * np.float32(wl.f)).astype(np.int32))
    # all frames identical: T = 0, threshold 0, nothing kept after the first frame
    frame = wl.tokens[:wl.f]
    static = np.concatenate([frame] * 4)
    rs = orc.score_frames(static, [0, 4], wl.f)
    assert np.all(rs["temporal"][wl.f:] == 0.0)
    assert np.all(rs["ratio"][1:] == 0.0) and np.all(rs["k"][1:] == 0)
    assert rs["ratio"][0] == r["ratio"][0]
    # spatial score of every copy equals the first frame's
    for t in range(1, 4):
        np.testing.assert_array_equal(rs["spatial"][t * wl.f:(t + 1) * wl.f], rs["spatial"][:wl.f])


def test_frame_scale_invariance():
    """Scaling a whole frame by a positive constant changes no direction: S, T, r unchanged."""
    wl = W.fill_tokens(W.custom("s", 7, W.F32, 4, 48, 0, [W.make_video_spec(3, 0.6)]))
    x = wl.tokens.copy()
    r0 = orc.score_frames(x, [0, 3], wl.f)
    x[wl.f:2 * wl.f] *= np.float32(4.0)     # power of two: exact in fp32
    r1 = orc.score_frames(x, [0, 3], wl.f)
    for key in ("spatial", "temporal", "importance", "ratio"):
        np.testing.assert_allclose(r1[key], r0[key], atol=1e-14)


def test_temporal_term_is_position_aligned_and_video_local():
    """T compares token i of frame t with token i of frame t-1 (Eq. 3), never across videos."""
    rng = np.random.default_rng(14)
    f, d = 6, 32
    f1 = rng.standard_normal((f, d)).astype(np.float32)
    f2 = np.roll(f1, 1, axis=0)             # token i of frame 2 is token i-1 of frame 1
    x = np.concatenate([f1, f2])
    r = orc.score_frames(x, [0, 2], f)
    for i in range(f):
        a, b = f2[i].astype(np.float64), f1[i].astype(np.float64)
        c = a @ b / np.linalg.norm(a) / np.linalg.norm(b)
        assert abs(r["temporal"][f + i] - math.sqrt(2 - 2 * c)) < 1e-12
    # as two one-frame videos the second frame is a first frame: T := S
    r2 = orc.score_frames(x, [0, 1, 2], f)
    np.testing.assert_array_equal(r2["temporal"][f:], r2["spatial"][f:])
    np.testing.assert_array_equal(r2["spatial"], r["spatial"])
    # the spatial score of a permuted frame is the permuted spatial score
    np.testing.assert_allclose(np.roll(r["spatial"][:f], 1), r["spatial"][f:], atol=1e-14)


def test_scores_against_numpy_library_routines():
    """Whole small workload against numpy's norm / matmul (library special case)."""
    wl = W.fill_tokens(W.custom("n", 8, W.BF16, 4, 96, 0,
                                [W.make_video_spec(3, 0.9), W.make_video_spec(2, 0.5)]))
    x = wl.tokens_as_f32().astype(np.float64).reshape(5, wl.f, wl.d)
    xn = x / np.linalg.norm(x, axis=2, keepdims=True)
    m = x.mean(axis=1, keepdims=True)
    mn = m / np.linalg.norm(m, axis=2, keepdims=True)
    S = np.sqrt(np.maximum(0, 2 - 2 * np.einsum("tfd,tfd->tf", xn, np.broadcast_to(mn, x.shape))))
    T = np.empty_like(S)
    first = {0, 3}
    for t in range(5):
        T[t] = S[t] if t in first else np.sqrt(np.maximum(0, 2 - 2 * np.einsum("fd,fd->f", xn[t], xn[t - 1])))
    r = orc.score_frames(wl.tokens, wl.video_frame_offsets, wl.f, w=1.0)
    np.testing.assert_allclose(r["spatial"], S.ravel(), atol=1e-12)
    np.testing.assert_allclose(r["temporal"], T.ravel(), atol=1e-12)
    np.testing.assert_allclose(r["importance"], (T + S).ravel(), atol=1e-12)
    np.testing.assert_allclose(r["ratio"], np.linalg.norm(T, axis=1) / (2 * math.sqrt(wl.f)), atol=1e-13)


# ---------------------------------------------------------------- manual variant (1 - cos), Section 3.1.1
def test_hand_case_f2_d2_one_minus_cos():
    """The hand-derived example under the manual variant's dissimilarity: S, T, I and both ratios."""
    g = _golden("hand_case_f2_d2_one_minus_cos.txt")
    tokens = np.array([[1, 0], [0, 1], [0, 1], [0, 1]], dtype=np.float32)
    r = orc.score_frames(tokens, [0, 2], f=2, w=1.0, dissim_kind=orc.ONE_MINUS_COS)
    S, T, I = r["spatial"], r["temporal"], r["importance"]
    tol = 1e-14
    for i, (ks, kt) in enumerate([("S1_0", "T1_0"), ("S1_1", "T1_1"), ("S2_0", "T2_0"), ("S2_1", "T2_1")]):
        assert abs(S[i] - g[ks]) < tol, (i, S[i])
        assert abs(T[i] - g[kt]) < tol, (i, T[i])
    assert abs(I[0] - g["I1_0"]) < tol and abs(I[2] - g["I2_0"]) < tol and abs(I[3] - g["I2_1"]) < tol
    assert abs(r["ratio"][0] - g["ratio_1"]) < tol and abs(r["ratio"][1] - g["ratio_2"]) < tol
    assert list(r["k"]) == [0, 0]                                   # floor(0.29), floor(0.71)
    kn = orc.score_frames(tokens, [0, 2], f=2, dissim_kind=orc.ONE_MINUS_COS, round_mode=orc.ROUND_NEAREST)["k"]
    assert list(kn) == [0, 1]
    kc = orc.score_frames(tokens, [0, 2], f=2, dissim_kind=orc.ONE_MINUS_COS, round_mode=orc.ROUND_CEIL)["k"]
    assert list(kc) == [1, 1]


def test_one_minus_cos_scores_against_numpy_and_dissim_identity():
    """Manual variant on a whole small workload (two videos, so two first frames): S, T, I and the
    ratio against numpy's 1 - a.b / (|a||b|), and element-wise 1 - cos = Dissim^2 / 2 against the
    default variant (Eq. 1: Dissim^2 = 2 - 2 cos)."""
    wl = W.fill_tokens(W.custom("n", 8, W.BF16, 4, 96, 0,
                                [W.make_video_spec(3, 0.9), W.make_video_spec(2, 0.5)]))
    x = wl.tokens_as_f32().astype(np.float64).reshape(5, wl.f, wl.d)
    m = x.mean(axis=1)

    def omc(a, b):
        return 1.0 - np.sum(a * b, axis=-1) / (np.linalg.norm(a, axis=-1) * np.linalg.norm(b, axis=-1))

    S = np.stack([omc(x[t], m[t][None, :]) for t in range(5)])
    T = np.stack([S[t] if t in (0, 3) else omc(x[t], x[t - 1]) for t in range(5)])
    w = 0.7
    r = orc.score_frames(wl.tokens, wl.video_frame_offsets, wl.f, w=w, dissim_kind=orc.ONE_MINUS_COS)
    np.testing.assert_allclose(r["spatial"], S.ravel(), atol=1e-12)
    np.testing.assert_allclose(r["temporal"], T.ravel(), atol=1e-12)
    np.testing.assert_allclose(r["importance"], (T + w * S).ravel(), atol=1e-12)
    np.testing.assert_allclose(r["ratio"], np.linalg.norm(T, axis=1) / (2 * math.sqrt(wl.f)), atol=1e-13)
    # temporal and spatial terms differ on non-first frames, so a swap of kinds in either shows
    assert np.max(np.abs(T[1] - S[1])) > 1e-3
    q = orc.score_frames(wl.tokens, wl.video_frame_offsets, wl.f, w=w, dissim_kind=orc.DISSIM)
    np.testing.assert_allclose(r["spatial"], q["spatial"] ** 2 / 2, atol=1e-14)
    np.testing.assert_allclose(r["temporal"], q["temporal"] ** 2 / 2, atol=1e-14)
    # the two kinds really differ (1 - cos != Dissim away from 0 and 2)
    assert np.max(np.abs(r["temporal"] - q["temporal"])) > 0.1


# ---------------------------------------------------------------- statistical closed forms
def test_statistical_closed_forms_on_generator():
    """Large d, unit-variance tokens: AR(1) rho gives cos ~ rho, T ~ sqrt(2-2rho),
    r_t ~ sqrt((1-rho)/2); an iid first frame gives r_1 ~ sqrt(2 - 2/sqrt(f))/2;
    a scene cut gives r ~ 1/sqrt(2)."""
    d = 2048
    for rho in (0.9, 0.95, 0.97):
        v = W.make_video_spec(5, rho, cuts=[3])
        wl = W.fill_tokens(W.custom("stat", 20, W.F32, 7, d, 0, [v]))
        r = orc.score_frames(wl.tokens, wl.video_frame_offsets, wl.f)
        f = wl.f
        tol = 4.0 / math.sqrt(d)
        for t in (1, 2, 4):
            assert abs(r["ratio"][t] - math.sqrt((1 - rho) / 2)) < tol * 0.2
            assert abs(r["temporal"][t * f:(t + 1) * f].mean() - math.sqrt(2 - 2 * rho)) < tol * 0.2
        assert abs(r["ratio"][3] - 1 / math.sqrt(2)) < tol * 0.2
        assert abs(r["ratio"][0] - math.sqrt(2 - 2 / math.sqrt(f)) / 2) < tol * 0.2


def test_static_video_prunes_at_least_as_much_as_one_with_cuts():
    """Section 3.1.3: static content is pruned harder than content with scene changes."""
    kept = {}
    for name, cuts, rho in (("static", [], 1.0), ("smooth", [], 0.97), ("cuts", [2, 5, 9], 0.97)):
        v = W.make_video_spec(12, rho, cuts=cuts)
        wl = W.fill_tokens(W.custom(name, 21, W.F32, 6, 256, 0, [v]))
        r = orc.score_frames(wl.tokens, wl.video_frame_offsets, wl.f)
        kept[name] = int(r["k"].sum())
        idx, off = orc.select_tokens(r["importance"], r["k"], wl.f)
        assert idx.size == kept[name]
    assert kept["static"] <= kept["smooth"] <= kept["cuts"]
    assert kept["static"] < kept["cuts"]


# ---------------------------------------------------------------- selection
def test_select_against_stable_argsort_and_invariants():
    rng = np.random.default_rng(15)
    F, f = 11, 37
    imp = rng.standard_normal(F * f).astype(np.float32)
    imp[rng.integers(0, F * f, 60)] = 0.5          # many ties
    imp[3 * f:4 * f] = 1.25                        # a frame of all-equal scores
    k = rng.integers(0, f + 1, F).astype(np.int32)
    k[0], k[1] = 0, f
    idx, off = orc.select_tokens(imp, k, f)
    assert idx.size == int(k.sum())                               # kept count = sum of budgets
    np.testing.assert_array_equal(off, np.concatenate([[0], np.cumsum(k)]))
    assert np.all(np.diff(idx) > 0)                               # strictly ascending
    for t in range(F):
        mine = idx[off[t]:off[t + 1]]
        assert np.all(mine // f == t)                             # inside its frame
        order = np.argsort(-imp[t * f:(t + 1) * f].astype(np.float64), kind="stable")
        np.testing.assert_array_equal(mine - t * f, np.sort(order[:k[t]]))
    np.testing.assert_array_equal(idx[off[3]:off[4]] - 3 * f, np.arange(k[3]))   # ties -> lowest indices


def test_select_brute_force_tiny():
    """For f <= 7 enumerate every k-subset: the kept set has the maximum score sum and is
    the lexicographically smallest among the maximisers."""
    rng = np.random.default_rng(16)
    for f in range(1, 8):
        for _ in range(6):
            imp = rng.integers(0, 4, f).astype(np.float32) / 2      # few distinct values: ties
            for k in range(f + 1):
                idx, _ = orc.select_tokens(imp, [k], f)
                best, best_set = None, None
                for comb in itertools.combinations(range(f), k):
                    s = float(sum(imp[list(comb)]))
                    if best is None or s > best:
                        best, best_set = s, comb
                assert tuple(idx) == tuple(best_set if k else ())


def test_select_threshold_variant():
    imp = np.array([0.1, 1.7, 1.6, 2.0, 1.61, 0.0], dtype=np.float32)
    idx, off = orc.select_threshold(imp, 1.6, F=2, f=3)
    assert list(idx) == [1, 3, 4] and list(off) == [0, 1, 3]


def test_gather_rows_is_fancy_indexing():
    rng = np.random.default_rng(17)
    x = rng.integers(0, 65536, (50, 24)).astype(np.uint16)
    idx = np.array([0, 3, 4, 17, 49], np.int32)
    np.testing.assert_array_equal(orc.gather_rows(x, idx), x[idx])
    wide = rng.standard_normal((20, 40)).astype(np.float32)
    view = wide[:, :16]                                  # row stride larger than the row
    np.testing.assert_array_equal(orc.gather_rows(view, idx[:3]), view[idx[:3]])


# ---------------------------------------------------------------- stage two
def _stage2(wl, M, **kw):
    return orc.kv_calibrate_prune(wl.hidden, wl.tokens, wl.seq_offsets, wl.vis_begin, wl.vis_count,
                                  wl.vis_offsets, M, **kw)


def test_calibration_cos_and_keep_rule():
    wl = W.fill_hidden(W.fill_tokens(W.custom(
        "c2", 30, W.BF16, 5, 128, 7, [W.make_video_spec(2, 0.9), W.make_video_spec(3, 0.8)])))
    M = 0.7
    r = _stage2(wl, M)
    h = wl.hidden_as_f32().astype(np.float64)
    v = wl.tokens_as_f32().astype(np.float64)
    keep = np.ones(wl.total_seq_tokens, bool)
    for b in range(wl.num_videos):
        s0, vo, nv = wl.seq_offsets[b], wl.vis_offsets[b], wl.vis_count[b]
        hh, vv = h[s0:s0 + nv], v[vo:vo + nv]
        c = np.einsum("nd,nd->n", hh, vv) / np.linalg.norm(hh, axis=1) / np.linalg.norm(vv, axis=1)
        np.testing.assert_allclose(r["cos"][vo:vo + nv], c, atol=1e-13)
        keep[s0:s0 + nv] = c.astype(np.float32) >= np.float32(M)     # discard iff cos < M (Eq. 7)
    np.testing.assert_array_equal(r["kept_pos"], np.nonzero(keep)[0])
    n_text = wl.num_videos * wl.n_text
    assert r["kept_pos"].size == n_text + int((r["cos"].astype(np.float32) >= np.float32(M)).sum())
    for b in range(wl.num_videos):                                   # every text token survives
        text = np.arange(wl.seq_offsets[b] + wl.vis_count[b], wl.seq_offsets[b + 1])
        assert np.all(np.isin(text, r["kept_pos"]))
        lo, hi = r["kept_seq_offsets"][b], r["kept_seq_offsets"][b + 1]
        seg = r["kept_pos"][lo:hi]
        assert np.all((seg >= wl.seq_offsets[b]) & (seg < wl.seq_offsets[b + 1]))
    assert r["kept_seq_offsets"][0] == 0 and r["kept_seq_offsets"][-1] == r["kept_pos"].size


def test_calibration_threshold_boundary_and_extremes():
    d = 16
    v = np.zeros((3, d), np.float32)
    v[:, 0] = 1.0
    h = np.zeros((3, d), np.float32)
    h[0, 0] = 1.0                    # cos = 1
    h[1, 0], h[1, 1] = 3.0, 4.0      # cos = 0.6 exactly in real arithmetic
    h[2, 0] = -2.0                   # cos = -1
    args = ([0, 3], [0], [3], [0])
    r = orc.kv_calibrate_prune(h, v, *args, M=0.5)
    np.testing.assert_allclose(r["cos"], [1.0, 0.6, -1.0], atol=1e-15)
    assert list(r["kept_pos"]) == [0, 1]
    assert list(orc.kv_calibrate_prune(h, v, *args, M=-1.0)["kept_pos"]) == [0, 1, 2]   # cos == M is kept
    assert list(orc.kv_calibrate_prune(h, v, *args, M=1.0)["kept_pos"]) == [0]
    assert list(orc.kv_calibrate_prune(h, v, *args, M=1.5)["kept_pos"]) == []


def test_calibration_statistics_of_generator():
    """h = v + s N(0,1), unit-variance v: cos ~ 1/sqrt(1+s^2); with s ~ U[0,2] the kept share at
    threshold M is min(1, sqrt(1/M^2 - 1)/2): everything at M = 0.2, about 39 % at M = 0.788."""
    wl = W.fill_hidden(W.fill_tokens(W.custom("c3", 31, W.F32, 10, 1024, 16, [W.make_video_spec(12, 0.9)])))
    n = wl.n_visual
    r = _stage2(wl, 0.2)
    assert r["kept_pos"].size == wl.total_seq_tokens
    for M in (0.788, 0.95):
        r = _stage2(wl, M)
        share = (r["kept_pos"].size - wl.n_text) / n
        assert abs(share - math.sqrt(1 / M ** 2 - 1) / 2) < 3.5 / math.sqrt(n) + 0.02
    s = np.random.default_rng([31, 2]).uniform(0, 2, n)        # the generator's first draw of stream 2
    np.testing.assert_allclose(r["cos"], 1 / np.sqrt(1 + s ** 2), atol=5.0 / math.sqrt(wl.d))


def test_nonzero_vis_begin():
    """System tokens before the visual block (the (S, V, I) order of Section 3.2.1)."""
    rng = np.random.default_rng(32)
    d, ns, nv, npmt = 24, 3, 5, 2
    vis = rng.standard_normal((nv, d)).astype(np.float32)
    hid = rng.standard_normal((ns + nv + npmt, d)).astype(np.float32)
    hid[ns:ns + nv] = vis
    hid[ns + 1] = -vis[1]
    hid[ns + 3] = -vis[3]
    r = orc.kv_calibrate_prune(hid, vis, [0, ns + nv + npmt], [ns], [nv], [0], M=0.2)
    assert list(r["kept_pos"]) == [0, 1, 2, 3, 5, 7, 8, 9]
    np.testing.assert_allclose(r["cos"], [1, -1, 1, -1, 1], atol=1e-14)


def test_kv_compact_is_fancy_indexing():
    rng = np.random.default_rng(33)
    L, H, T, Dh = 3, 2, 29, 8
    kv = rng.integers(0, 65536, (L, 2, H, T, Dh)).astype(np.uint16)
    kept = np.array([0, 1, 5, 6, 7, 20, 28], np.int32)
    out = orc.kv_compact(kv, kept)
    np.testing.assert_array_equal(out[:, :, :, :kept.size], kv[:, :, :, kept])
    assert np.all(out[:, :, :, kept.size:] == 0)                   # untouched beyond the kept prefix
    # layer range
    out2 = orc.kv_compact(kv, kept, layer_begin=1, layer_end=2)
    assert np.all(out2[0] == 0) and np.all(out2[2] == 0)
    np.testing.assert_array_equal(out2[1, :, :, :kept.size], kv[1][:, :, kept])
    # token-major source layout [L,2,T,H,Dh] viewed as [L,2,H,T,Dh]
    tm = np.ascontiguousarray(kv.transpose(0, 1, 3, 2, 4))
    view = tm.transpose(0, 1, 3, 2, 4)
    out3 = orc.kv_compact(view, kept)
    np.testing.assert_array_equal(out3, out)


def test_layer_by_layer_pruning_is_eq7_per_layer_in_numpy():
    """The layer-by-layer reading of Eq. 7 (Section 3.2.3) against plain numpy: every layer's kept set is
    {text} + {visual: cos(h_l, v) >= M} of its own hidden state, and only that layer's planes are compacted."""
    rng = np.random.default_rng(12)
    L, H, Dh, d, nv, ntext, M = 3, 2, 8, 16, 10, 3, 0.5
    T = nv + ntext
    visual = rng.standard_normal((nv, d)).astype(np.float32)
    hidden = [np.concatenate([visual + (0.3 + 0.6 * l) * rng.standard_normal((nv, d)).astype(np.float32),
                              rng.standard_normal((ntext, d)).astype(np.float32)]) for l in range(L)]
    kv = rng.standard_normal((L + 1, 2, H, T, Dh)).astype(np.float32)
    so, vb, vc, vo = (np.array(x, np.int32) for x in ([0, T], [0], [nv], [0]))
    res, out = orc.kv_prune_layers(hidden, visual, so, vb, vc, vo, M, kv, layer_begin=1)
    np.testing.assert_array_equal(out[0], kv[0])                    # a layer outside the range is untouched
    sizes = []
    for l in range(L):
        h = hidden[l][:nv].astype(np.float64)
        v = visual.astype(np.float64)
        cos = (h * v).sum(1) / (np.linalg.norm(h, axis=1) * np.linalg.norm(v, axis=1))
        np.testing.assert_allclose(res[l]["cos"], cos, rtol=1e-12)
        kept = np.concatenate([np.nonzero(cos.astype(np.float32) >= np.float32(M))[0], np.arange(nv, T)])
        np.testing.assert_array_equal(res[l]["kept_pos"], kept)
        np.testing.assert_array_equal(out[1 + l][:, :, :kept.size], kv[1 + l][:, :, kept])
        np.testing.assert_array_equal(out[1 + l][:, :, kept.size:], kv[1 + l][:, :, kept.size:])
        sizes.append(kept.size)
    assert len(set(sizes)) > 1                                      # the layers really differ


def test_layer_level_discard_is_eq7_on_the_layer_average_in_numpy():
    """Eq. 7 as printed, against numpy on a stack of hidden states whose similarity to the visual features
    decays with depth: per-layer average cosine, the first layer under M, and "that layer and every deeper
    one lose their visual rows, text rows stay" (Section 3.2.3, Section 1)."""
    rng = np.random.default_rng(31)
    d, n_layers = 48, 7
    lens_sys, lens_vis, lens_txt = [2, 0, 1], [11, 6, 0], [3, 2, 4]
    so = np.concatenate([[0], np.cumsum(np.add(np.add(lens_sys, lens_vis), lens_txt))]).astype(np.int32)
    vb = np.array(lens_sys, np.int32)
    vc = np.array(lens_vis, np.int32)
    vo = np.concatenate([[0], np.cumsum(lens_vis)])[:-1].astype(np.int32)
    T = int(so[-1])
    vis = rng.standard_normal((int(vc.sum()), d)).astype(np.float32)
    # the second sequence drifts three times as fast as the first: it crosses the threshold earlier
    drift = {0: [0.1, 0.3, 0.5, 0.9, 1.4, 0.6, 3.0], 1: [0.3, 0.9, 1.5, 2.7, 4.2, 1.8, 9.0]}
    hid = rng.standard_normal((n_layers, T, d)).astype(np.float32)
    for l in range(n_layers):
        for b in (0, 1):
            r0 = so[b] + vb[b]
            hid[l, r0:r0 + vc[b]] = vis[vo[b]:vo[b] + vc[b]] + drift[b][l] * rng.standard_normal((vc[b], d))
    M = 0.6
    o = orc.kv_discard_layers(hid, vis, so, vb, vc, vo, M)
    # numpy, written independently
    mean = np.zeros((n_layers, 3))
    for l in range(n_layers):
        for b in (0, 1):
            h = hid[l, so[b] + vb[b]:so[b] + vb[b] + vc[b]].astype(np.float64)
            v = vis[vo[b]:vo[b] + vc[b]].astype(np.float64)
            mean[l, b] = np.mean(np.sum(h * v, 1) / (np.linalg.norm(h, axis=1) * np.linalg.norm(v, axis=1)))
    np.testing.assert_allclose(o["mean_cos"], mean, atol=1e-12)
    first = [int(np.argmax(mean[:, b] < M)) if (mean[:, b] < M).any() else n_layers for b in (0, 1)] + [n_layers]
    assert list(o["first_discard"]) == first
    assert 0 < first[1] < first[0] < n_layers              # the faster drift is cut earlier; both are cut somewhere
    # layer 5 of sequence 0 drifts less than layer 4: a layer behind the first failing one stays dropped
    assert mean[5, 0] > mean[4, 0]
    for l in range(n_layers):
        want = [p for b in range(3) for p in range(so[b], so[b + 1])
                if not (l >= first[b] and so[b] + vb[b] <= p < so[b] + vb[b] + vc[b])]
        assert list(o["kept_pos"][l]) == want
        assert list(o["kept_seq_offsets"][l]) == [int(np.searchsorted(want, so[b])) for b in range(4)]
    # M below every average keeps everything at every layer; M above every average drops all visual rows at layer 0
    lo = orc.kv_discard_layers(hid, vis, so, vb, vc, vo, -1.0)
    assert all(k.size == T for k in lo["kept_pos"]) and list(lo["first_discard"]) == [n_layers] * 3
    hi = orc.kv_discard_layers(hid, vis, so, vb, vc, vo, 1.5)
    assert list(hi["first_discard"]) == [0, 0, n_layers]    # the sequence without visual tokens is never cut
    assert all(k.size == T - int(vc.sum()) for k in hi["kept_pos"])
    # thread count does not change anything but rounding order of the mean
    o4 = orc.kv_discard_layers(hid, vis, so, vb, vc, vo, M, nthreads=4)
    np.testing.assert_allclose(o4["mean_cos"], o["mean_cos"], atol=1e-14)
    assert list(o4["first_discard"]) == first


def test_kv_compact_inplace_equals_out_of_place_prefix():
    rng = np.random.default_rng(35)
    L, H, T, Dh = 2, 3, 41, 8
    kv = rng.integers(0, 65536, (L, 2, H, T, Dh)).astype(np.uint16)
    kept = np.array([0, 1, 2, 9, 10, 30, 39, 40], np.int32)       # a leading run that stays where it is
    ref = kv.copy()
    out = orc.kv_compact_inplace(kv.copy(), kept)
    np.testing.assert_array_equal(out[:, :, :, :kept.size], ref[:, :, :, kept])     # fancy indexing
    np.testing.assert_array_equal(out[:, :, :, kept.size:], ref[:, :, :, kept.size:])   # tail untouched
    # a token-major cache and a layer range
    tm = np.ascontiguousarray(ref.transpose(0, 1, 3, 2, 4))
    orc.kv_compact_inplace(tm.transpose(0, 1, 3, 2, 4), kept, layer_begin=1, layer_end=2)
    np.testing.assert_array_equal(tm[0], ref[0].transpose(0, 2, 1, 3))
    np.testing.assert_array_equal(tm[1][:, :kept.size], ref[1][:, :, kept].transpose(0, 2, 1, 3))


def test_rope_reencoding_pins():
    """Rotary re-encoding of compacted keys: (1) tokens that do not move are untouched and values never
    change; (2) keys built as R(p_old) k come out as R(p_new) k; (3) pair norms are preserved;
    (4) dimensions beyond rotary_dim are copied."""
    rng = np.random.default_rng(36)
    L, H, Dh, R, base = 2, 2, 16, 12, 10000.0
    so = np.array([0, 9, 20], np.int32)                      # two sequences of 9 and 11 tokens
    T = 20
    kept = np.array([0, 1, 2, 5, 8, 9, 10, 14, 19], np.int32)
    kso = np.array([0, 5, 9], np.int32)
    half = R // 2
    inv = base ** (-2.0 * np.arange(half) / R)

    def rot(x, pos):                                         # textbook rotary embedding, half-split pairs
        ang = np.asarray(pos, np.float64)[..., None] * inv
        x1, x2 = x[..., :half], x[..., half:R]
        return np.concatenate([x1 * np.cos(ang) - x2 * np.sin(ang), x2 * np.cos(ang) + x1 * np.sin(ang), x[..., R:]],
                              axis=-1)

    raw = rng.standard_normal((L, 2, H, T, Dh))
    pos_old = np.concatenate([np.arange(9), np.arange(11)])
    cache = raw.copy()
    cache[:, 0] = rot(raw[:, 0], pos_old)                    # keys carry their old positions
    cache32 = cache.astype(np.float32)
    out = orc.kv_compact_rope(cache32, kept, kso, so, R, base)
    pos_new = np.concatenate([np.arange(5), np.arange(4)])
    expect_k = rot(raw[:, 0][:, :, kept], pos_new)
    np.testing.assert_allclose(out[:, 0], expect_k, atol=2e-6)            # fp32 storage of the cache
    np.testing.assert_array_equal(out[:, 1], cache32[:, 1][:, :, kept].astype(np.float64))   # values: bit copy
    # tokens 0, 1, 2 of sequence 0 and token 9 (first of sequence 1) keep their positions
    for j in (0, 1, 2, 5):
        np.testing.assert_array_equal(out[:, 0, :, j], cache32[:, 0, :, kept[j]].astype(np.float64))
    np.testing.assert_array_equal(out[:, 0, :, :, R:], cache32[:, 0][:, :, kept][..., R:].astype(np.float64))
    kin = cache32[:, 0][:, :, kept].astype(np.float64)
    n_in = np.hypot(kin[..., :half], kin[..., half:R])
    n_out = np.hypot(out[:, 0][..., :half], out[:, 0][..., half:R])
    np.testing.assert_allclose(n_out, n_in, rtol=1e-12)
    # rotary_dim = 0 is plain compaction
    np.testing.assert_array_equal(orc.kv_compact_rope(cache32, kept, kso, so, 0, base),
                                  cache32[:, :, :, kept].astype(np.float64))


def test_multithreaded_oracle_is_identical():
    wl = W.fill_hidden(W.fill_tokens(W.custom("mt", 34, W.BF16, 4, 64, 5, [W.make_video_spec(6, 0.9, cuts=[3])])))
    a = orc.score_frames(wl.tokens, wl.video_frame_offsets, wl.f, nthreads=1)
    b = orc.score_frames(wl.tokens, wl.video_frame_offsets, wl.f, nthreads=4)
    for key in a:
        np.testing.assert_array_equal(a[key], b[key])
    c1, c4 = _stage2(wl, 0.7, nthreads=1), _stage2(wl, 0.7, nthreads=4)
    for key in c1:
        np.testing.assert_array_equal(c1[key], c4[key])
