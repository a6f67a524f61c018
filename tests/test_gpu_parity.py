"""GPU parity: every C-ABI entry point against the CPU oracle, element by element, on the same
seeded inputs.  Runs on a B200 (`-m gpu`)."""
import functools

import numpy as np
import pytest
import torch

from helpers import (BOUNDARY_TOL, TIGHT_TOL, TOL, DeviceWorkload, Guarded, assert_scores, check_budgets, check_kept_sets, rel_err,
                     to_dev, to_host)
from oracle import sharpv_oracle as orc
from paper_2511_08003_b200 import binding as sv
from paper_2511_08003_b200 import workloads as W

pytestmark = pytest.mark.gpu

NT = 8  # oracle threads


def _small_ragged():
    vids = [W.make_video_spec(5, 0.9, cuts=[2]), W.make_video_spec(1, 0.5), W.make_video_spec(9, 0.75, cuts=[3, 4]),
            W.make_video_spec(2, 0.99)]
    return W.custom("small_ragged", 40, W.BF16, 14, 3584, 64, vids, 0.0, 3, 4, 128)


def _odd_shapes():
    # f = 37 (not a multiple of anything), d = 8 fp32 (one 32-byte row), head_dim 8
    vids = [W.make_video_spec(7, 0.6, cuts=[5], duplicates=[2]), W.make_video_spec(3, 0.3)]
    wl = W.custom("odd", 41, W.F32, 6, 8, 3, vids, 0.0, 2, 3, 8)
    return wl


CASES = {
    "tiny": lambda: W.tiny(),
    "onevision_small": lambda: W.onevision_7b(n_frames=8, num_layers=2),
    "video7b_small": lambda: W.video_7b(n_frames=16, num_layers=2),
    "small_ragged": _small_ragged,
    "odd_shapes": _odd_shapes,
    "pllava_like": lambda: W.custom("pllava", 42, W.BF16, 12, 4096, 20, [W.make_video_spec(4, 0.9)], 0.0, 2, 8, 128),
    "onevision_7b": lambda: W.onevision_7b(),
    "video_7b": lambda: W.video_7b(),
}


@functools.lru_cache(maxsize=None)
def _case(name):
    wl = CASES[name]()
    W.fill_tokens(wl)
    W.fill_hidden(wl)
    if wl.kv_bytes() <= 1 << 30:
        W.fill_kv(wl)
    return wl, DeviceWorkload(wl, kv=True)


@pytest.mark.parametrize("name", list(CASES))
def test_stage_one_scores_budgets_selection_gather(name):
    wl, dw = _case(name)
    F, f = wl.total_frames, wl.f
    o = orc.score_frames(wl.tokens, wl.video_frame_offsets, f, w=1.0, nthreads=NT)
    g = sv.sharpv_score_frames(dw.tokens, dw.video_frame_offsets, F, f, w=1.0, want_spatial=True,
                               want_temporal=True)
    torch.cuda.synchronize()
    assert_scores(g, o, f, min(TOL[wl.dtype], TIGHT_TOL))      # bf16 inputs widen exactly: the fp32 bound holds
    k_gpu = to_host(g["k"])
    exempt_frames = check_budgets(k_gpu, o, f)
    assert len(exempt_frames) <= max(1, F // 50)

    # exact duplicates give exactly zero temporal importance and an empty budget
    for v, off in zip(wl.videos, wl.video_frame_offsets[:-1]):
        for t in np.nonzero(v.duplicate)[0]:
            assert np.all(to_host(g["temporal"])[(off + t) * f:(off + t + 1) * f] == 0.0)
            assert k_gpu[off + t] == 0

    sel = sv.sharpv_select_tokens(g["importance"], g["k"], F, f, tokens=dw.tokens)
    torch.cuda.synchronize()
    n = int(sel["num_kept"].item())
    assert n == int(k_gpu.sum())                                   # kept count = sum of budgets
    idx = to_host(sel["kept_index"])[:n]
    off = to_host(sel["kept_offsets"])
    exempt = check_kept_sets(idx, off, o["importance"], k_gpu, f, orc.select_tokens)
    assert exempt <= max(2, n // 1000)
    # gathered rows are a bit copy of the rows the GPU selected
    np.testing.assert_array_equal(to_host(sel["tokens"])[:n], orc.gather_rows(wl.tokens, idx))


@pytest.mark.parametrize("name", ["tiny", "small_ragged", "odd_shapes"])
@pytest.mark.parametrize("kind", [sv.DISSIM, sv.ONE_MINUS_COS])
@pytest.mark.parametrize("round_mode,min_keep,w", [(sv.ROUND_FLOOR, 0, 1.0), (sv.ROUND_NEAREST, 3, 0.5),
                                                   (sv.ROUND_CEIL, 0, 2.0)])
def test_score_variants(name, kind, round_mode, min_keep, w):
    wl, dw = _case(name)
    F, f = wl.total_frames, wl.f
    o = orc.score_frames(wl.tokens, wl.video_frame_offsets, f, w=w, round_mode=round_mode, min_keep=min_keep,
                         dissim_kind=kind, nthreads=NT)
    g = sv.sharpv_score_frames(dw.tokens, dw.video_frame_offsets, F, f, w=w, dissim_kind=kind,
                               round_mode=round_mode, min_keep=min_keep)
    torch.cuda.synchronize()
    assert "spatial" not in g and "temporal" not in g
    assert_scores(g, o, f, keys=("importance", "ratio"))
    check_budgets(to_host(g["k"]), o, f)


def test_select_alone_is_bit_exact_with_ties():
    """Same fp32 scores and budgets on both sides: no tolerance, ties included."""
    rng = np.random.default_rng(50)
    for F, f in ((1, 1), (3, 7), (40, 196), (5, 1000), (2, 8192), (300, 169)):
        imp = rng.standard_normal(F * f).astype(np.float32)
        imp[rng.integers(0, F * f, F * f // 3)] = 0.25           # heavy ties
        imp[rng.integers(0, F * f, 5)] = -0.0
        imp[rng.integers(0, F * f, 5)] = 0.0
        if F > 2:
            imp[f:2 * f] = 1.0                                   # a frame of equal scores
        k = rng.integers(0, f + 1, F).astype(np.int32)
        k[0] = f if F > 1 else k[0]
        k[-1] = 0 if F > 1 else k[-1]
        idx_o, off_o = orc.select_tokens(imp, k, f)
        g = sv.sharpv_select_tokens(torch.from_numpy(imp).cuda(), torch.from_numpy(k).cuda(), F, f, gather=False)
        torch.cuda.synchronize()
        n = int(g["num_kept"].item())
        np.testing.assert_array_equal(to_host(g["kept_offsets"]), off_o)
        np.testing.assert_array_equal(to_host(g["kept_index"])[:n], idx_o)
        # budgets out of range are clamped to [0, f]
        k2 = k.copy()
        k2[0] = f + 5
        k2[-1] = -3
        g2 = sv.sharpv_select_tokens(torch.from_numpy(imp).cuda(), torch.from_numpy(k2).cuda(), F, f, gather=False)
        idx_o2, off_o2 = orc.select_tokens(imp, k2, f)
        np.testing.assert_array_equal(to_host(g2["kept_offsets"]), off_o2)
        np.testing.assert_array_equal(to_host(g2["kept_index"])[:off_o2[-1]], idx_o2)


def test_random_selectors_of_the_ablation():
    """The two random selectors of the ablation (Section 4.3.1: random choice under the per-frame
    budgets of the method, and random choice video-wide under the total budget only) are the
    per-frame top-k run on random scores; the random numbers are inputs, drawn on the host."""
    wl, dw = _case("tiny")
    F, f = wl.total_frames, wl.f
    o = orc.score_frames(wl.tokens, wl.video_frame_offsets, f, w=1.0, nthreads=NT)
    g = sv.sharpv_score_frames(dw.tokens, dw.video_frame_offsets, F, f, w=1.0)
    torch.cuda.synchronize()
    check_budgets(to_host(g["k"]), o, f)
    rnd = np.random.default_rng(77).random(F * f).astype(np.float32)
    d_rnd = torch.from_numpy(rnd).cuda()
    # per-frame budgets of the method, random tokens inside each frame
    k = to_host(g["k"])
    s1 = sv.sharpv_select_tokens(d_rnd, g["k"], F, f, tokens=dw.tokens)
    torch.cuda.synchronize()
    idx_o, off_o = orc.select_tokens(rnd, k, f)
    n = int(s1["num_kept"].item())
    assert n == int(k.sum())
    np.testing.assert_array_equal(to_host(s1["kept_offsets"]), off_o)
    np.testing.assert_array_equal(to_host(s1["kept_index"])[:n], idx_o)
    np.testing.assert_array_equal(to_host(s1["tokens"])[:n], wl.tokens[idx_o])
    # one budget for the whole video: the video is one segment of F * f tokens
    k_all = np.array([int(k.sum())], np.int32)
    s2 = sv.sharpv_select_tokens(d_rnd, torch.from_numpy(k_all).cuda(), 1, F * f, tokens=dw.tokens)
    torch.cuda.synchronize()
    idx_o2, off_o2 = orc.select_tokens(rnd, k_all, F * f)
    assert int(s2["num_kept"].item()) == n
    np.testing.assert_array_equal(to_host(s2["kept_index"])[:n], idx_o2)
    np.testing.assert_array_equal(to_host(s2["tokens"])[:n], wl.tokens[idx_o2])
    # the same number of tokens, spread differently over the frames
    per_frame = np.bincount(idx_o2 // f, minlength=F)
    assert per_frame.sum() == n and not np.array_equal(per_frame, k)


def test_select_threshold_variant():
    wl, dw = _case("tiny")
    F, f = wl.total_frames, wl.f
    g = sv.sharpv_score_frames(dw.tokens, dw.video_frame_offsets, F, f, dissim_kind=sv.ONE_MINUS_COS)
    imp = to_host(g["importance"])
    for K in (0.0, 0.1, float(np.median(imp)), 1.6, 10.0):
        idx_o, off_o = orc.select_threshold(imp, K, F, f)
        s = sv.sharpv_select_tokens_threshold(g["importance"], K, F, f, tokens=dw.tokens)
        torch.cuda.synchronize()
        n = int(s["num_kept"].item())
        assert n == idx_o.size
        np.testing.assert_array_equal(to_host(s["kept_offsets"]), off_o)
        np.testing.assert_array_equal(to_host(s["kept_index"])[:n], idx_o)
        np.testing.assert_array_equal(to_host(s["tokens"])[:n], wl.tokens[idx_o])


@pytest.mark.parametrize("name", list(CASES))
@pytest.mark.parametrize("M", [0.2, 0.788, 0.95])
def test_stage_two_calibration_and_compaction(name, M):
    wl, dw = _case(name)
    T = wl.total_seq_tokens
    o = orc.kv_calibrate_prune(wl.hidden, wl.tokens, wl.seq_offsets, wl.vis_begin, wl.vis_count, wl.vis_offsets,
                               M, nthreads=NT)
    g = sv.sharpv_kv_calibrate_prune(dw.hidden, dw.tokens, dw.seq_offsets, dw.vis_begin, dw.vis_count,
                                     dw.vis_offsets, T, M=M, want_mean_cos=True)
    torch.cuda.synchronize()
    cos_g = to_host(g["cos"])[:wl.n_visual]
    e = rel_err(cos_g, o["cos"])
    assert e <= TIGHT_TOL, f"cos rel err {e}"
    kso = to_host(g["kept_seq_offsets"])
    n = int(kso[-1])
    kept = to_host(g["kept_pos"])[:n]
    assert np.all(np.diff(kept) > 0)
    sym = np.setxor1d(kept, o["kept_pos"])
    if sym.size:                                                   # only tokens at the threshold may differ
        vis_row = np.full(T, -1)
        for b in range(wl.num_videos):
            s0 = wl.seq_offsets[b] + wl.vis_begin[b]
            vis_row[s0:s0 + wl.vis_count[b]] = wl.vis_offsets[b] + np.arange(wl.vis_count[b])
        assert np.all(vis_row[sym] >= 0)
        assert np.all(np.abs(o["cos"][vis_row[sym]] - M) <= BOUNDARY_TOL)
        assert sym.size <= max(2, wl.n_visual // 1000)
    else:
        np.testing.assert_array_equal(kso, o["kept_seq_offsets"])
    # the flags the GPU used are consistent with its own cosines
    for b in range(wl.num_videos):
        seg = kept[kso[b]:kso[b + 1]]
        assert np.all((seg >= wl.seq_offsets[b]) & (seg < wl.seq_offsets[b + 1]))
    mean_o = [o["cos"][wl.vis_offsets[b]:wl.vis_offsets[b] + wl.vis_count[b]].mean() for b in range(wl.num_videos)]
    assert rel_err(to_host(g["mean_cos"]), np.array(mean_o)) <= 1e-5

    if wl.kv is None:
        return
    dst = torch.zeros_like(dw.kv)
    sv.sharpv_kv_compact(dw.kv, dst, g["kept_pos"], g["kept_seq_offsets"], capacity=T)
    torch.cuda.synchronize()
    expect = orc.kv_compact(wl.kv, kept, nthreads=NT)             # for the GPU's own index set
    np.testing.assert_array_equal(to_host(dst), expect)           # bit exact, rows beyond n untouched (zero)


def test_kv_compact_layouts_and_layer_range():
    wl, dw = _case("small_ragged")
    T = wl.total_seq_tokens
    rng = np.random.default_rng(51)
    kept = np.sort(rng.choice(T, size=T // 3, replace=False)).astype(np.int32)
    kept_d = torch.from_numpy(kept).cuda()
    kso = torch.tensor([0, kept.size], dtype=torch.int32, device="cuda")
    L, _, H, _, Dh = wl.kv_shape()
    # token-major source [L,2,T,H,Dh] viewed as [L,2,H,T,Dh]; smaller destination capacity
    src_tm = dw.kv.permute(0, 1, 3, 2, 4).contiguous()
    cap = kept.size + 5
    dst = torch.zeros((L, 2, H, cap, Dh), dtype=dw.kv.dtype, device="cuda")
    sv.sharpv_kv_compact(src_tm.permute(0, 1, 3, 2, 4), dst, kept_d, kso, capacity=cap, layer_begin=1, layer_end=3)
    torch.cuda.synchronize()
    out = to_host(dst)
    assert np.all(out[0] == 0)
    np.testing.assert_array_equal(out[1:3, :, :, :kept.size], wl.kv[1:3][:, :, :, kept])
    assert np.all(out[:, :, :, kept.size:] == 0)
    # token-major destination
    dst_tm = torch.zeros((L, 2, cap, H, Dh), dtype=dw.kv.dtype, device="cuda")
    sv.sharpv_kv_compact(dw.kv, dst_tm.permute(0, 1, 3, 2, 4), kept_d, kso, capacity=cap)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(to_host(dst_tm)[:, :, :kept.size], wl.kv[:, :, :, kept].transpose(0, 1, 3, 2, 4))


@pytest.mark.parametrize("dtype,Dh", [(torch.bfloat16, 96), (torch.float32, 40), (torch.bfloat16, 8), (torch.float32, 516)])
def test_kv_compact_row_sizes_that_are_not_a_power_of_two(dtype, Dh):
    """Rows of 12, 10, 1 and 129 16-byte vectors (a tile of the copy kernels then holds a number of rows that does
    not divide its vectors evenly): out of place, in place and with a capacity below the kept count, bit for bit
    against the oracle; several row tiles, a ragged last tile."""
    rng = np.random.default_rng(1200 + Dh)
    L, H, T = 3, 2, 1500
    kv = torch.randn((L, 2, H, T, Dh), dtype=torch.float32, device="cuda",
                     generator=torch.Generator(device="cuda").manual_seed(Dh)).to(dtype)
    kept = np.sort(rng.choice(T, size=701, replace=False)).astype(np.int32)
    kept[:30] = np.arange(30)
    kept = np.unique(kept)
    n = kept.size
    kept_d = torch.from_numpy(kept).cuda()
    kso = torch.tensor([0, 400, n], dtype=torch.int32, device="cuda")
    host = to_host(kv)
    dst = torch.zeros((L, 2, H, n + 3, Dh), dtype=dtype, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sv.sharpv_kv_compact(kv, dst, kept_d, kso, capacity=n + 3, status_word=status)
    torch.cuda.synchronize()
    out = to_host(dst)
    want = orc.kv_compact(host, kept)[:, :, :, :n]
    np.testing.assert_array_equal(out[:, :, :, :n], want)
    assert not out[:, :, :, n:].any() and int(status.item()) == 0
    small = torch.zeros((L, 2, H, 100, Dh), dtype=dtype, device="cuda")
    sv.sharpv_kv_compact(kv, small, kept_d, kso, capacity=100, layer_begin=1, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == sv.Status.ERR_CAPACITY
    np.testing.assert_array_equal(to_host(small)[1:], want[1:, :, :, :100])
    assert not to_host(small)[0].any()
    inplace = kv.clone()
    sv.sharpv_kv_compact(inplace, inplace, kept_d, kso, capacity=T)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(to_host(inplace), orc.kv_compact_inplace(host.copy(), kept))


def test_kv_compact_rejects_partial_overlap_accepts_neighbours():
    """Source and destination carved out of one allocation: caches that touch without sharing a byte are
    compacted, a destination that starts inside the source is refused before anything is launched."""
    wl, dw = _case("small_ragged")
    T = wl.total_seq_tokens
    L, _, H, _, Dh = wl.kv_shape()
    both = torch.zeros((2 * L, 2, H, T, Dh), dtype=dw.kv.dtype, device="cuda")
    both[:L] = dw.kv
    src, dst = both[:L], both[L:]                          # neighbours: dst starts where src ends
    kept = np.arange(1, T, 3, dtype=np.int32)
    kept_d = torch.from_numpy(kept).cuda()
    kso = torch.tensor([0, kept.size], dtype=torch.int32, device="cuda")
    sv.sharpv_kv_compact(src, dst, kept_d, kso, capacity=T)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(to_host(dst)[:, :, :, :kept.size], wl.kv[:, :, :, kept])
    np.testing.assert_array_equal(to_host(src), wl.kv)      # the source is untouched
    before = to_host(both).copy()
    shifted = both.view(-1)[Dh:Dh + src.numel()].view(src.shape)      # one row further on: shares bytes with src
    for bad in (shifted, both[1:L + 1]):
        with pytest.raises(sv.SharpVError) as e:
            sv.sharpv_kv_compact(src, bad, kept_d, kso, capacity=T)
        assert e.value.status == sv.Status.ERR_INVALID_ARG
    with pytest.raises(sv.SharpVError):
        ws = torch.empty(sv.sharpv_kv_compact_rope_workspace_bytes(T, Dh), dtype=torch.uint8, device="cuda")
        sv.sharpv_kv_compact_rope(src, shifted, kept_d, kso, torch.tensor([0, T], dtype=torch.int32, device="cuda"),
                                  T, Dh, 1.0e4, workspace=ws)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(to_host(both), before)    # nothing ran
    # a single layer of one cache into another layer of the same allocation is fine
    sv.sharpv_kv_compact(both, both, kept_d, kso, capacity=T, layer_begin=0, layer_end=1)     # in place
    torch.cuda.synchronize()


@pytest.mark.parametrize("name", ["tiny", "small_ragged", "odd_shapes", "onevision_7b"])
@pytest.mark.parametrize("M", [0.2, 0.788])
def test_kv_compact_in_place(name, M):
    """kv_dst == kv_src: the kept prefix of every plane equals the gathered rows, the tail keeps its old
    contents, bit for bit (oracle: copy each plane, gather from the copy)."""
    wl, dw = _case(name)
    T = wl.total_seq_tokens
    g = sv.sharpv_kv_calibrate_prune(dw.hidden, dw.tokens, dw.seq_offsets, dw.vis_begin, dw.vis_count,
                                     dw.vis_offsets, T, M=M)
    torch.cuda.synchronize()
    n = int(g["kept_seq_offsets"][-1].item())
    kept = to_host(g["kept_pos"])[:n]
    kv = dw.kv.clone()
    sv.sharpv_kv_compact(kv, kv, g["kept_pos"], g["kept_seq_offsets"], capacity=T)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(to_host(kv), orc.kv_compact_inplace(wl.kv.copy(), kept))
    # token-major cache, layers [1, L) only
    L = wl.num_layers
    if L > 1:
        tm = dw.kv.permute(0, 1, 3, 2, 4).contiguous()
        view = tm.permute(0, 1, 3, 2, 4)
        sv.sharpv_kv_compact(view, view, g["kept_pos"], g["kept_seq_offsets"], capacity=T, layer_begin=1)
        torch.cuda.synchronize()
        expect = np.ascontiguousarray(wl.kv.transpose(0, 1, 3, 2, 4))
        orc.kv_compact_inplace(expect.transpose(0, 1, 3, 2, 4), kept, layer_begin=1)
        np.testing.assert_array_equal(to_host(tm), expect)


def test_layer_wise_reading_of_eq7():
    """Eq. 7 read layer by layer (hierarchical cache pruning): every layer has its own hidden state, its own
    kept set and compacts only its own K/V.  Built from the same two entry points, one call per layer."""
    L = 4
    wl = W.custom("layers", 90, W.BF16, 8, 512, 16, [W.make_video_spec(6, 0.9, cuts=[3])], 0.0, L, 2, 64)
    W.fill_tokens(wl)
    W.fill_kv(wl)
    dw_tokens = to_dev(wl.tokens)
    i32 = lambda a: torch.from_numpy(a).cuda()
    tabs = [i32(wl.seq_offsets), i32(wl.vis_begin), i32(wl.vis_count), i32(wl.vis_offsets)]
    T, M = wl.total_seq_tokens, 0.6
    kv = to_dev(wl.kv)
    expect = wl.kv.copy()
    means, counts = [], []
    for l in range(L):
        W.fill_hidden(wl, s_max=0.5 + 1.0 * l)          # deeper layers drift further from the visual features
        hid = to_dev(wl.hidden)
        g = sv.sharpv_kv_calibrate_prune(hid, dw_tokens, *tabs, T, M=M, want_mean_cos=True)
        sv.sharpv_kv_compact(kv, kv, g["kept_pos"], g["kept_seq_offsets"], capacity=T, layer_begin=l, layer_end=l + 1)
        torch.cuda.synchronize()
        o = orc.kv_calibrate_prune(wl.hidden, wl.tokens, wl.seq_offsets, wl.vis_begin, wl.vis_count,
                                   wl.vis_offsets, M)
        n = int(g["kept_seq_offsets"][-1].item())
        kept = to_host(g["kept_pos"])[:n]
        assert np.setxor1d(kept, o["kept_pos"]).size <= 2
        orc.kv_compact_inplace(expect, kept, layer_begin=l, layer_end=l + 1)
        means.append(float(g["mean_cos"][0].item()))
        counts.append(n)
        assert abs(means[-1] - o["cos"].mean()) <= 1e-5
    np.testing.assert_array_equal(to_host(kv), expect)
    assert all(a > b for a, b in zip(means, means[1:]))     # similarity decays with depth ...
    assert all(a >= b for a, b in zip(counts, counts[1:]))  # ... and so does the kept cache
    assert counts[0] > counts[-1] >= wl.n_text


def test_layer_by_layer_entry_point():
    """sharpv_kv_prune_layers (Section 3.2.3 read per layer) against the oracle: per-layer cosines, kept
    lists and the cache whose layers are compacted with their own lists, in place and into a second cache,
    for a layer range that starts above layer 0."""
    L, lb = 5, 1
    wl = W.custom("layers", 92, W.BF16, 8, 512, 16, [W.make_video_spec(5, 0.9, cuts=[2]), W.make_video_spec(3, 0.8)],
                  0.0, L, 2, 64)
    W.fill_tokens(wl)
    W.fill_kv(wl)
    T, M = wl.total_seq_tokens, 0.6
    hidden = []
    for l in range(lb, L):
        W.fill_hidden(wl, s_max=0.4 + 0.8 * l)
        hidden.append(wl.hidden.copy())
    i32 = lambda a: torch.from_numpy(a).cuda()
    tabs = [i32(wl.seq_offsets), i32(wl.vis_begin), i32(wl.vis_count), i32(wl.vis_offsets)]
    d_hidden = torch.stack([to_dev(h) for h in hidden])
    res, expect = orc.kv_prune_layers(hidden, wl.tokens, wl.seq_offsets, wl.vis_begin, wl.vis_count, wl.vis_offsets,
                                      M, wl.kv, layer_begin=lb, nthreads=NT)
    kv = to_dev(wl.kv)
    g = sv.sharpv_kv_prune_layers(d_hidden, to_dev(wl.tokens), *tabs, T, kv, kv, M=M, layer_begin=lb,
                                  want_mean_cos=True)
    torch.cuda.synchronize()
    exempt = 0
    for i, o in enumerate(res):
        assert rel_err(to_host(g["cos"][i]), o["cos"], floor=1.0) <= TIGHT_TOL
        n = int(g["kept_seq_offsets"][i, -1].item())
        kept = to_host(g["kept_pos"][i])[:n]
        sym = np.setxor1d(kept, o["kept_pos"])
        exempt += sym.size
        vis_of = {int(p): int(v) for p, v in zip(np.concatenate([wl.seq_offsets[b] + wl.vis_begin[b] + np.arange(wl.vis_count[b])
                                                                 for b in range(len(wl.vis_count))]),
                                                 np.concatenate([wl.vis_offsets[b] + np.arange(wl.vis_count[b])
                                                                 for b in range(len(wl.vis_count))]))}
        for pos in sym:                     # only tokens whose cosine sits on the threshold may differ
            assert abs(o["cos"][vis_of[int(pos)]] - M) <= BOUNDARY_TOL
    assert exempt <= 2
    if exempt == 0:
        np.testing.assert_array_equal(to_host(kv), expect)
        # into a second cache: the prefix of every plane in the range, nothing else
        dst = torch.zeros_like(kv)
        g2 = sv.sharpv_kv_prune_layers(d_hidden, to_dev(wl.tokens), *tabs, T, to_dev(wl.kv), dst, M=M, layer_begin=lb)
        torch.cuda.synchronize()
        out = to_host(dst)
        assert np.all(out[:lb] == 0)
        for i, o in enumerate(res):
            n = o["kept_pos"].size
            np.testing.assert_array_equal(out[lb + i][:, :, :n], wl.kv[lb + i][:, :, o["kept_pos"]])
            assert np.all(out[lb + i][:, :, n:] == 0)
        np.testing.assert_array_equal(to_host(g2["kept_seq_offsets"]), to_host(g["kept_seq_offsets"]))
    counts = [int(x) for x in to_host(g["kept_seq_offsets"])[:, -1]]
    assert counts[0] > counts[-1] >= wl.n_text          # deeper layers keep less


def test_layer_level_discard_entry_point():
    """Eq. 7 as printed (SHARPV_PRUNE_PER_LAYER) against the oracle: per-layer average cosine, the first
    discarded layer of each sequence, kept lists that lose whole visual blocks from that layer on, and the
    cache compacted with them (in place, into a second cache, decisions only); 28 layers in one call."""
    L, lb = 30, 2
    wl = W.custom("discard", 93, W.BF16, 6, 256, 9, [W.make_video_spec(4, 0.9), W.make_video_spec(2, 0.8),
                                                       W.make_video_spec(3, 0.85)], 0.0, L, 2, 64)
    W.fill_tokens(wl)
    W.fill_kv(wl)
    T, M, n = wl.total_seq_tokens, 0.45, L - lb
    hidden = []
    for i in range(n):
        W.fill_hidden(wl, s_max=0.3 + 0.25 * i)           # the similarity decays with depth
        hidden.append(wl.hidden.copy())
    hid = np.stack(hidden)
    o = orc.kv_discard_layers(hid, wl.tokens, wl.seq_offsets, wl.vis_begin, wl.vis_count, wl.vis_offsets, M, nthreads=NT)
    first = o["first_discard"]
    assert 0 < first.min() and first.max() < n               # every sequence is cut somewhere inside the range
    i32 = lambda a: torch.from_numpy(a).cuda()
    tabs = [i32(wl.seq_offsets), i32(wl.vis_begin), i32(wl.vis_count), i32(wl.vis_offsets)]
    d_hidden = torch.from_numpy(hid.view(np.int16)).cuda().view(torch.bfloat16)
    kv = to_dev(wl.kv)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    g = sv.sharpv_kv_prune_layers(d_hidden, to_dev(wl.tokens), *tabs, T, kv, kv, M=M, mode=sv.PRUNE_PER_LAYER,
                                  layer_begin=lb, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    mean_g = to_host(g["mean_cos"]).astype(np.float64)
    assert np.max(np.abs(mean_g - o["mean_cos"])) <= 1e-5
    # a mean within 1e-5 of M may fall on either side; away from it the decisions are the oracle's
    assert np.all(np.abs(o["mean_cos"] - M) > 1e-5), "test data sits on the threshold: change the seed"
    np.testing.assert_array_equal(to_host(g["first_discard"]), lb + first)
    np.testing.assert_array_equal(to_host(g["kept_seq_offsets"]), o["kept_seq_offsets"])
    expect = wl.kv.copy()
    for i in range(n):
        kept = to_host(g["kept_pos"][i])[:o["kept_seq_offsets"][i, -1]]
        np.testing.assert_array_equal(kept, o["kept_pos"][i])
        orc.kv_compact_inplace(expect, o["kept_pos"][i], layer_begin=lb + i, layer_end=lb + i + 1)
    np.testing.assert_array_equal(to_host(kv), expect)
    # into a second cache; and decisions only
    dst = torch.zeros_like(kv)
    g2 = sv.sharpv_kv_prune_layers(d_hidden, to_dev(wl.tokens), *tabs, T, to_dev(wl.kv), dst, M=M,
                                   mode=sv.PRUNE_PER_LAYER, layer_begin=lb)
    g3 = sv.sharpv_kv_prune_layers(d_hidden, to_dev(wl.tokens), *tabs, T, None, None, M=M, mode=sv.PRUNE_PER_LAYER,
                                   layer_begin=lb, kv_layers=L)
    torch.cuda.synchronize()
    out = to_host(dst)
    assert np.all(out[:lb] == 0)
    for i in range(n):
        k = o["kept_pos"][i]
        np.testing.assert_array_equal(out[lb + i][:, :, :k.size], wl.kv[lb + i][:, :, k])
        assert np.all(out[lb + i][:, :, k.size:] == 0)
    for key in ("kept_seq_offsets", "first_discard", "mean_cos"):
        assert torch.equal(g2[key], g[key]) and torch.equal(g3[key], g[key])
    # the per-token reading of the same stack keeps a different, token-wise set
    g4 = sv.sharpv_kv_prune_layers(d_hidden, to_dev(wl.tokens), *tabs, T, None, None, M=M, layer_begin=lb, kv_layers=L)
    torch.cuda.synchronize()
    res = [orc.kv_calibrate_prune(h, wl.tokens, wl.seq_offsets, wl.vis_begin, wl.vis_count, wl.vis_offsets, M,
                                  nthreads=NT) for h in hidden]
    diff = sum(np.setxor1d(to_host(g4["kept_pos"][i])[:int(g4["kept_seq_offsets"][i, -1].item())],
                           res[i]["kept_pos"]).size for i in range(n))
    assert diff <= 4


def test_kv_compact_one_byte_cache():
    """An fp8-sized cache (one byte per element, 128-byte rows): compaction is a bit copy and needs no
    knowledge of the element format."""
    rng = np.random.default_rng(91)
    L, H, T, Dh = 3, 4, 1500, 128
    kv = rng.integers(0, 256, (L, 2, H, T, Dh), dtype=np.uint8)
    kept = np.sort(rng.choice(T, size=600, replace=False)).astype(np.int32)
    kept_d = torch.from_numpy(kept).cuda()
    kso = torch.tensor([0, kept.size], dtype=torch.int32, device="cuda")
    src = torch.from_numpy(kv).cuda()
    dst = torch.zeros_like(src)
    sv.sharpv_kv_compact(src, dst, kept_d, kso, capacity=T)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(dst.cpu().numpy(), orc.kv_compact(kv, kept))
    sv.sharpv_kv_compact(src, src, kept_d, kso, capacity=T)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(src.cpu().numpy(), orc.kv_compact_inplace(kv.copy(), kept))
    if hasattr(torch, "float8_e4m3fn"):
        f8 = torch.from_numpy(kv).cuda().view(torch.float8_e4m3fn)
        out = torch.zeros_like(f8)
        sv.sharpv_kv_compact(f8, out, kept_d, kso, capacity=T)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(out.view(torch.uint8).cpu().numpy()[:, :, :, :kept.size], kv[:, :, :, kept])


@pytest.mark.parametrize("dtype,Dh,R", [(W.BF16, 128, 128), (W.BF16, 128, 64), (W.F32, 64, 32), (W.F32, 64, 64),
                                         (W.BF16, 64, 0)])
def test_kv_compact_with_rotary_reencoding(dtype, Dh, R):
    """Keys are rotated by the distance they move, values are bit copies.  The result is compared with the
    fp64 oracle: fp32 caches to fp32 rounding, bf16 caches to half a bf16 ulp plus the fp32 error."""
    rng = np.random.default_rng(92)
    L, H = 2, 3
    so = np.array([0, 700, 700, 1500, 1530], np.int32)           # four sequences, one of them empty
    T = int(so[-1])
    kept = np.sort(rng.choice(T, size=600, replace=False)).astype(np.int32)
    kept[:40] = np.arange(40)                                    # a run that does not move at all
    kept = np.unique(kept)
    kso = np.searchsorted(kept, so).astype(np.int32)
    raw = rng.standard_normal((L, 2, H, T, Dh)).astype(np.float32)
    kv = W.f32_to_bf16_bits(raw) if dtype == W.BF16 else raw
    base = 1.0e6
    o = orc.kv_compact_rope(kv, kept, kso, so, R, base)
    src = to_dev(kv)
    cap = kept.size + 7
    dst = torch.zeros((L, 2, H, cap, Dh), dtype=src.dtype, device="cuda")
    i32 = lambda a: torch.from_numpy(a).cuda()
    sv.sharpv_kv_compact_rope(src, dst, i32(kept), i32(kso), i32(so), cap, R, base)
    torch.cuda.synchronize()
    out = to_host(dst)
    n = kept.size
    assert not out[:, :, :, n:].any()                              # nothing written beyond the kept prefix
    np.testing.assert_array_equal(out[:, 1, :, :n], kv[:, 1][:, :, kept])          # values: bit copy
    np.testing.assert_array_equal(out[:, 0, :, :n, R:], kv[:, 0][:, :, kept][..., R:])   # beyond the rotary part
    got = (W.bf16_bits_to_f32(out) if dtype == W.BF16 else out).astype(np.float64)[:, 0, :, :n, :R]
    want = o[:, 0, :, :, :R]
    if R:
        half = R // 2
        pair = np.hypot(want[..., :half], want[..., half:])
        pair = np.concatenate([pair, pair], axis=-1)
        # bf16 keeps 8 significant bits: half a unit in the last place is at most 2^-8 of the value
        half_ulp = 2.0 ** -8 if dtype == W.BF16 else 0.0
        assert np.all(np.abs(got - want) <= half_ulp * np.abs(want) * 1.001 + 4e-6 * pair + 1e-30)
        moved = np.nonzero(kept - so[np.searchsorted(so, kept, side="right") - 1] !=
                           np.arange(n) - kso[np.searchsorted(so, kept, side="right") - 1])[0]
        assert moved.size > 100                                    # most tokens do move
        still = np.setdiff1d(np.arange(n), moved)
        np.testing.assert_array_equal(out[:, 0][:, :, still], kv[:, 0][:, :, kept[still]])   # unmoved keys: bit copy


def test_capacity_overflow_is_reported_not_written():
    wl, dw = _case("tiny")
    F, f, T = wl.total_frames, wl.f, wl.total_seq_tokens
    g = sv.sharpv_score_frames(dw.tokens, dw.video_frame_offsets, F, f)
    full = sv.sharpv_select_tokens(g["importance"], g["k"], F, f, tokens=dw.tokens)
    n = int(full["num_kept"].item())
    cap = n - 7
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    guard = 12345
    out = {"kept_index": torch.full((cap + 16,), guard, dtype=torch.int32, device="cuda"),
           "tokens": torch.zeros((cap + 16, wl.d), dtype=dw.tokens.dtype, device="cuda")}
    s = sv.sharpv_select_tokens(g["importance"], g["k"], F, f, tokens=dw.tokens, capacity=cap, out=out,
                                status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == sv.Status.ERR_CAPACITY
    assert int(s["num_kept"].item()) == n                          # true count still reported
    np.testing.assert_array_equal(to_host(s["kept_index"])[:cap], to_host(full["kept_index"])[:cap])
    assert np.all(to_host(s["kept_index"])[cap:] == guard)         # nothing written beyond capacity
    assert np.all(to_host(s["tokens"])[cap:] == 0)
    np.testing.assert_array_equal(to_host(s["tokens"])[:cap], to_host(full["tokens"])[:cap])

    status.zero_()
    c = sv.sharpv_kv_calibrate_prune(dw.hidden, dw.tokens, dw.seq_offsets, dw.vis_begin, dw.vis_count,
                                     dw.vis_offsets, T, M=0.2, capacity=100,
                                     out={"kept_pos": torch.full((132,), guard, dtype=torch.int32, device="cuda")},
                                     status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == sv.Status.ERR_CAPACITY
    assert int(c["kept_seq_offsets"][-1].item()) == T              # everything survives M = 0.2 here
    np.testing.assert_array_equal(to_host(c["kept_pos"])[:100], np.arange(100))
    assert np.all(to_host(c["kept_pos"])[100:] == guard)
    status.zero_()
    dst = torch.zeros_like(dw.kv)
    sv.sharpv_kv_compact(dw.kv, dst, c["kept_pos"], c["kept_seq_offsets"], capacity=100, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == sv.Status.ERR_CAPACITY
    np.testing.assert_array_equal(to_host(dst)[:, :, :, :100], wl.kv[:, :, :, :100])
    assert np.all(to_host(dst)[:, :, :, 100:] == 0)


def test_degenerate_inputs():
    dev = "cuda"
    # no frames at all
    vfo = torch.zeros(2, dtype=torch.int32, device=dev)
    tok = torch.zeros((4, 8), dtype=torch.float32, device=dev)
    g = sv.sharpv_score_frames(tok, vfo, 0, 4)
    assert g["importance"].numel() == 0
    s = sv.sharpv_select_tokens(g["importance"], g["k"], 0, 4, gather=False)
    torch.cuda.synchronize()
    assert int(s["num_kept"].item()) == 0 and to_host(s["kept_offsets"]).tolist() == [0]
    # one token per frame, zero vectors, a uniform frame (every token equals the mean)
    f, d = 4, 16
    x = np.zeros((3 * f, d), np.float32)
    x[f:2 * f] = np.arange(1, d + 1, dtype=np.float32)             # uniform frame: S = 0 exactly in the oracle
    x[2 * f:3 * f] = np.random.default_rng(52).standard_normal((f, d)).astype(np.float32)
    x[2 * f + 1] = 0.0                                              # a zero token inside a normal frame
    o = orc.score_frames(x, [0, 3], f)
    g = sv.sharpv_score_frames(to_dev(x), torch.tensor([0, 3], dtype=torch.int32, device=dev), 3, f,
                               want_spatial=True, want_temporal=True)
    torch.cuda.synchronize()
    assert_scores(g, o, f)
    np.testing.assert_array_equal(to_host(g["k"]), o["k"])
    # a uniform frame of bf16 tokens whose fp32 mean is a rounded multiple of the token
    xb = W.f32_to_bf16_bits(np.tile(np.random.default_rng(53).standard_normal((1, 64)).astype(np.float32), (7, 1)))
    ob = orc.score_frames(xb, [0, 1], 7)
    gb = sv.sharpv_score_frames(to_dev(xb), torch.tensor([0, 1], dtype=torch.int32, device=dev), 1, 7,
                                want_spatial=True)
    torch.cuda.synchronize()
    assert_scores(gb, ob, 7, keys=("spatial",))
    # stage two with zero hidden rows and a sequence without visual tokens
    hid = np.random.default_rng(54).standard_normal((10, 16)).astype(np.float32)
    vis = hid[2:6].copy()
    hid[3] = 0.0
    so, vb, vc, vo = [0, 8, 10], [2, 0], [4, 0], [0, 4]
    oc = orc.kv_calibrate_prune(hid, vis, so, vb, vc, vo, M=0.5)
    t32 = lambda a: torch.tensor(a, dtype=torch.int32, device=dev)
    gc = sv.sharpv_kv_calibrate_prune(to_dev(hid), to_dev(vis), t32(so), t32(vb), t32(vc), t32(vo), 10, M=0.5,
                                      want_mean_cos=True)
    torch.cuda.synchronize()
    n = int(gc["kept_seq_offsets"][-1].item())
    np.testing.assert_array_equal(to_host(gc["kept_pos"])[:n], oc["kept_pos"])
    np.testing.assert_array_equal(to_host(gc["kept_seq_offsets"]), oc["kept_seq_offsets"])
    assert rel_err(to_host(gc["cos"]), oc["cos"]) <= TIGHT_TOL
    assert to_host(gc["mean_cos"])[1] == 0.0


@pytest.mark.parametrize("dtype,d", [(W.BF16, 128), (W.F32, 64), (W.BF16, 384), (W.F32, 256)])
@pytest.mark.parametrize("grid", [1, 3, 14, 15, 17])
def test_nearly_parallel_rows_and_frame_sizes(dtype, d, grid):
    """Rows that are almost parallel without being equal (a scaled copy of the previous frame, a frame of
    identical tokens next to its own rounded mean) in shapes on both sides of the fused kernel's limits
    (f = 1, 9, 196, 225)."""
    f = grid * grid
    rng = np.random.default_rng(70 + grid)
    base = rng.standard_normal((f, d)).astype(np.float32)
    frames = [base,
              base * np.float32(1.5),                                   # scaled copy: T ~ 0, not identical
              np.tile(rng.standard_normal((1, d)).astype(np.float32), (f, 1)),   # uniform frame: S ~ 0
              base + np.float32(1e-3) * rng.standard_normal((f, d)).astype(np.float32),
              base.copy()]
    x = np.concatenate(frames)
    if dtype == W.BF16:
        x = W.f32_to_bf16_bits(x)
    vfo = np.array([0, 3, 5], np.int32)
    o = orc.score_frames(x, vfo, f, nthreads=NT)
    g = sv.sharpv_score_frames(to_dev(x), torch.from_numpy(vfo).cuda(), 5, f, want_spatial=True, want_temporal=True)
    torch.cuda.synchronize()
    assert_scores(g, o, f)
    check_budgets(to_host(g["k"]), o, f)


def test_small_scores_meet_the_relative_bound_report(capsys):
    """Scores between 1e-4 and 5e-2 (frames that drift a little from their predecessor) in shapes of both
    score paths and both storage types: relative error against max(|oracle|, 1e-3), and the absolute error
    of the rows the oracle calls parallel.  Prints the worst values (run with -s to see them)."""
    rows = []
    for dtype, d in [(W.BF16, 128), (W.F32, 64), (W.BF16, 72), (W.F32, 200), (W.BF16, 3584)]:
        f = 49
        rng = np.random.default_rng(90 + d)
        base = rng.standard_normal((f, d)).astype(np.float32)
        frames = [base] + [base + np.float32(e) * rng.standard_normal((f, d)).astype(np.float32)
                           for e in (1e-4, 1e-3, 1e-2, 3e-2)] + [base * np.float32(0.75)]
        x = np.concatenate(frames)
        if dtype == W.BF16:
            x = W.f32_to_bf16_bits(x)
        F = len(frames)
        vfo = np.array([0, F], np.int32)
        o = orc.score_frames(x, vfo, f, nthreads=NT)
        g = sv.sharpv_score_frames(to_dev(x), torch.from_numpy(vfo).cuda(), F, f, want_spatial=True, want_temporal=True)
        torch.cuda.synchronize()
        errs = assert_scores(g, o, f)
        T_g, T_o = to_host(g["temporal"]).astype(np.float64), o["temporal"]
        par = T_o < 1e-6
        rows.append((dtype, d, errs["temporal"], errs["spatial"],
                     float(np.max(np.abs(T_g - T_o)[par])) if par.any() else 0.0))
    with capsys.disabled():
        for r in rows:
            print(f"\n  {r[0]:5s} d={r[1]:5d}: T rel {r[2]:.2e}  S rel {r[3]:.2e}  |T| of parallel rows {r[4]:.2e}", end="")


@pytest.mark.parametrize("seed", range(12))
def test_score_random_shapes(seed):
    """Random frame sizes, feature sizes, video counts (videos without frames included) and both
    storage types: exercises every way a CTA's range of tiles can start, cross a slice and end."""
    rng = np.random.default_rng(1000 + seed)
    bf16 = bool(rng.integers(2))
    f = int(rng.choice([1, 2, 3, 5, 17, 64, 100, 144, 169, 196, 201, 255, 256]))
    slices = int(rng.choice([1, 2, 3, 7, 28]))
    d = slices * (128 if bf16 else 64)
    counts = [int(c) for c in rng.choice([0, 1, 1, 2, 3, 5, 9, 20], size=int(rng.integers(1, 7)))]
    if sum(counts) == 0:
        counts[0] = 4
    vfo = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    F = int(vfo[-1])
    x = rng.standard_normal((F * f, d)).astype(np.float32)
    for t in range(1, F):                          # correlate consecutive frames, some exact duplicates
        r = rng.random()
        if r < 0.2:
            x[t * f:(t + 1) * f] = x[(t - 1) * f:t * f]
        elif r < 0.8:
            x[t * f:(t + 1) * f] = 0.9 * x[(t - 1) * f:t * f] + 0.436 * x[t * f:(t + 1) * f]
    xs = W.f32_to_bf16_bits(x) if bf16 else x
    w = float(rng.choice([0.0, 0.5, 1.0, 2.0]))
    o = orc.score_frames(xs, vfo, f, w=w, nthreads=NT)
    g = sv.sharpv_score_frames(to_dev(xs), torch.from_numpy(vfo).cuda(), F, f, w=w, want_spatial=True,
                               want_temporal=True)
    torch.cuda.synchronize()
    assert_scores(g, o, f, what=f"(f={f}, d={d}, frames={counts}, bf16={bf16})")
    check_budgets(to_host(g["k"]), o, f)
    # selection on the GPU's own scores and budgets against the oracle's selection of the same inputs
    sel = sv.sharpv_select_tokens(g["importance"], g["k"], F, f, gather=False)
    torch.cuda.synchronize()
    idx_o, off_o = orc.select_tokens(to_host(g["importance"]), to_host(g["k"]), f)
    np.testing.assert_array_equal(to_host(sel["kept_offsets"]), off_o)
    np.testing.assert_array_equal(to_host(sel["kept_index"])[:off_o[-1]], idx_o)


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("f", [1, 7, 24, 25, 49, 72, 97, 121, 145, 170, 193, 217, 241, 256])
def test_score_every_frame_size_class(f, bf16):
    """Frame sizes on both sides of every step in the number of rows a lane keeps in the fused score
    kernel (one instance of the kernel per step), for both storage types, with a range of tiles that
    starts inside a video, crosses slices and ends inside a video."""
    rng = np.random.default_rng(3000 + f)
    d = 3 * (128 if bf16 else 64)
    vfo = np.array([0, 4, 4, 9, 11], np.int32)
    F = int(vfo[-1])
    x = rng.standard_normal((F * f, d)).astype(np.float32)
    for t in range(1, F):
        x[t * f:(t + 1) * f] = 0.95 * x[(t - 1) * f:t * f] + 0.312 * x[t * f:(t + 1) * f]
    x[6 * f:7 * f] = x[5 * f:6 * f]                 # one exact duplicate frame
    xs = W.f32_to_bf16_bits(x) if bf16 else x
    o = orc.score_frames(xs, vfo, f, w=1.0, nthreads=NT)
    g = sv.sharpv_score_frames(to_dev(xs), torch.from_numpy(vfo).cuda(), F, f, w=1.0, want_spatial=True,
                               want_temporal=True)
    torch.cuda.synchronize()
    assert_scores(g, o, f, what=f"(f={f}, bf16={bf16})")
    check_budgets(to_host(g["k"]), o, f)
    assert np.all(to_host(g["temporal"])[6 * f:7 * f] == 0.0)      # the duplicate frame: exactly zero


@pytest.mark.parametrize("seed", range(10))
def test_stage_two_random_layouts(seed):
    """Random sequence layouts (system tokens before the visual block, sequences without visual tokens,
    empty sequences), feature sizes, K/V shapes and cache layouts, out of place and in place."""
    rng = np.random.default_rng(2000 + seed)
    bf16 = bool(rng.integers(2))
    d = int(rng.choice([8, 64, 200, 896])) * (1 if bf16 else 1)
    B = int(rng.integers(1, 6))
    n_sys = rng.integers(0, 4, B)
    n_vis = rng.choice([0, 1, 7, 40, 300], size=B)
    n_txt = rng.integers(0, 6, B)
    if rng.random() < 0.3:
        n_sys[-1] = n_vis[-1] = n_txt[-1] = 0              # a sequence without any token
    lens = n_sys + n_vis + n_txt
    if lens.sum() == 0:
        n_vis[0], lens[0] = 5, 5
    so = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    vo = np.concatenate([[0], np.cumsum(n_vis)])[:-1].astype(np.int32)
    T, NV = int(so[-1]), int(n_vis.sum())
    vis = rng.standard_normal((max(NV, 1), d)).astype(np.float32)
    hid = rng.standard_normal((T, d)).astype(np.float32)
    for b in range(B):
        s0 = so[b] + n_sys[b]
        drift = rng.uniform(0, 2, n_vis[b]).astype(np.float32)[:, None]
        hid[s0:s0 + n_vis[b]] = vis[vo[b]:vo[b] + n_vis[b]] + drift * hid[s0:s0 + n_vis[b]]
    if bf16:
        vis, hid = W.f32_to_bf16_bits(vis), W.f32_to_bf16_bits(hid)
    M = float(rng.choice([0.2, 0.6, 0.788, 0.95]))
    vb, vc = n_sys.astype(np.int32), n_vis.astype(np.int32)
    o = orc.kv_calibrate_prune(hid, vis, so, vb, vc, vo, M)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()
    g = sv.sharpv_kv_calibrate_prune(to_dev(hid), to_dev(vis), i32(so), i32(vb), i32(vc), i32(vo), T, M=M,
                                     want_mean_cos=True)
    torch.cuda.synchronize()
    if NV:
        assert rel_err(to_host(g["cos"])[:NV], o["cos"][:NV]) <= TIGHT_TOL
    kso = to_host(g["kept_seq_offsets"])
    n = int(kso[-1])
    kept = to_host(g["kept_pos"])[:n]
    sym = np.setxor1d(kept, o["kept_pos"])
    assert sym.size <= 1
    if sym.size == 0:
        np.testing.assert_array_equal(kso, o["kept_seq_offsets"])

    L, H, Dh = int(rng.integers(1, 4)), int(rng.integers(1, 4)), int(rng.choice([8, 16, 64, 128]))
    store = np.uint16 if bf16 else np.float32
    token_major = bool(rng.integers(2))
    shape = (L, 2, T, H, Dh) if token_major else (L, 2, H, T, Dh)
    raw = (rng.integers(0, 65536, shape).astype(np.uint16) if bf16
           else rng.standard_normal(shape).astype(np.float32))
    kv_h = raw.transpose(0, 1, 3, 2, 4) if token_major else raw            # [L,2,H,T,Dh] view
    kv_d = to_dev(raw)
    kv_v = kv_d.permute(0, 1, 3, 2, 4) if token_major else kv_d
    dst = torch.zeros((L, 2, H, max(n, 1) + 3, Dh), dtype=kv_d.dtype, device="cuda")
    sv.sharpv_kv_compact(kv_v, dst, g["kept_pos"], g["kept_seq_offsets"], capacity=T)
    torch.cuda.synchronize()
    out = to_host(dst)
    np.testing.assert_array_equal(out[:, :, :, :n], kv_h[:, :, :, kept])
    assert not out[:, :, :, n:].any()
    sv.sharpv_kv_compact(kv_v, kv_v, g["kept_pos"], g["kept_seq_offsets"], capacity=T)        # in place
    torch.cuda.synchronize()
    expect = np.ascontiguousarray(kv_h).copy()
    orc.kv_compact_inplace(expect, kept)
    got = to_host(kv_d)
    np.testing.assert_array_equal(got.transpose(0, 1, 3, 2, 4) if token_major else got, expect)
    assert store == got.dtype


@pytest.mark.parametrize("name", list(CASES))
def test_prune_frames_equals_score_then_select(name):
    """Stage one in one call against the oracle's composition score_frames -> select_tokens -> gather_rows,
    and bit for bit against the two entry points it replaces."""
    wl, dw = _case(name)
    F, f = wl.total_frames, wl.f
    tol = TOL[wl.dtype]
    o = orc.score_frames(wl.tokens, wl.video_frame_offsets, f, w=1.0, nthreads=NT)
    g = sv.sharpv_prune_frames(dw.tokens, dw.video_frame_offsets, F, f, w=1.0, want_spatial=True, want_temporal=True)
    torch.cuda.synchronize()
    assert_scores(g, o, f, min(tol, TIGHT_TOL))
    k_gpu = to_host(g["k"])
    check_budgets(k_gpu, o, f)
    off = to_host(g["kept_offsets"])
    n = int(g["num_kept"].item())
    assert n == off[-1] == int(np.clip(k_gpu, 0, f).sum())
    idx = to_host(g["kept_index"])[:n]
    exempt = check_kept_sets(idx, off, o["importance"], k_gpu, f, orc.select_tokens)
    assert exempt <= max(2, n // 1000)
    np.testing.assert_array_equal(to_host(g["tokens"])[:n], orc.gather_rows(wl.tokens, idx))
    # the two-call path on the same inputs: identical bits everywhere
    a = sv.sharpv_score_frames(dw.tokens, dw.video_frame_offsets, F, f, w=1.0)
    b = sv.sharpv_select_tokens(a["importance"], a["k"], F, f, tokens=dw.tokens)
    torch.cuda.synchronize()
    assert torch.equal(a["importance"], g["importance"]) and torch.equal(a["k"], g["k"])
    assert torch.equal(b["kept_offsets"], g["kept_offsets"]) and int(b["num_kept"].item()) == n
    assert torch.equal(b["kept_index"][:n], g["kept_index"][:n])
    assert torch.equal(b["tokens"][:n].view(torch.uint8), g["tokens"][:n].view(torch.uint8))


@pytest.mark.parametrize("seed", range(8))
def test_prune_frames_random_shapes_ties_and_capacity(seed):
    """Random shapes on both sides of the fused kernels' limits, frames of equal tokens (all scores tie),
    forced minimum budgets, a capacity smaller than the kept count, indices only."""
    rng = np.random.default_rng(4000 + seed)
    bf16 = bool(rng.integers(2))
    f = int(rng.choice([1, 3, 17, 100, 196, 256, 300]))
    d = int(rng.choice([1, 2, 3, 7])) * (64 if bf16 else 32) + (8 if seed % 4 == 3 else 0)
    counts = [int(c) for c in rng.choice([0, 1, 2, 3, 6], size=int(rng.integers(1, 5)))]
    if sum(counts) == 0:
        counts[0] = 2
    vfo = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    F = int(vfo[-1])
    x = rng.standard_normal((F * f, d)).astype(np.float32)
    for t in range(1, F):
        x[t * f:(t + 1) * f] = 0.9 * x[(t - 1) * f:t * f] + 0.436 * x[t * f:(t + 1) * f]
    if F > 2:
        x[2 * f:3 * f] = x[2 * f]                                  # a frame of identical tokens: every score ties
    xs = W.f32_to_bf16_bits(x) if bf16 else x
    mk = int(rng.integers(0, 3))
    o = orc.score_frames(xs, vfo, f, w=0.5, min_keep=mk, round_mode=orc.ROUND_NEAREST, nthreads=NT)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    g = sv.sharpv_prune_frames(to_dev(xs), torch.from_numpy(vfo).cuda(), F, f, w=0.5, min_keep=mk,
                               round_mode=sv.ROUND_NEAREST, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert_scores(g, o, f, keys=("importance", "ratio"))
    k_gpu = to_host(g["k"])
    check_budgets(k_gpu, o, f)
    # selection on the GPU's own fp32 scores and budgets: exact, ties included
    idx_o, off_o = orc.select_tokens(to_host(g["importance"]), k_gpu, f)
    n = int(g["num_kept"].item())
    np.testing.assert_array_equal(to_host(g["kept_offsets"]), off_o)
    np.testing.assert_array_equal(to_host(g["kept_index"])[:n], idx_o)
    np.testing.assert_array_equal(to_host(g["tokens"])[:n], orc.gather_rows(xs, idx_o))
    if n > 1:
        cap = n // 2
        small = sv.sharpv_prune_frames(to_dev(xs), torch.from_numpy(vfo).cuda(), F, f, w=0.5, min_keep=mk,
                                       round_mode=sv.ROUND_NEAREST, capacity=cap, gather=False, status_word=status)
        torch.cuda.synchronize()
        assert int(status.item()) == sv.Status.ERR_CAPACITY and int(small["num_kept"].item()) == n
        np.testing.assert_array_equal(to_host(small["kept_index"])[:cap], idx_o[:cap])
        assert "tokens" not in small


@pytest.mark.parametrize("F,f,bf16", [(149, 40, True), (300, 196, True), (700, 9, False), (5000, 6, True)])
def test_prune_frames_with_more_frames_than_sms(F, f, bf16):
    """Stage one in one call on batches with more frames than the GPU has SMs (the finaliser then runs as
    two smaller CTAs per SM) and with more frames than a CTA scans by itself (the kept lists' offsets then
    come from the one-CTA scan kernel): scores against the oracle, selection and gather exact on the GPU's
    own scores, several videos, ties, and a capacity below the kept count."""
    rng = np.random.default_rng(9000 + F)
    d = 128 if bf16 else 64
    cuts = np.sort(rng.choice(np.arange(1, F), size=5, replace=False))
    vfo = np.concatenate([[0], cuts, [F]]).astype(np.int32)
    x = rng.standard_normal((F * f, d)).astype(np.float32)
    for t in range(1, F):
        x[t * f:(t + 1) * f] = 0.9 * x[(t - 1) * f:t * f] + 0.436 * x[t * f:(t + 1) * f]
    x[3 * f:4 * f] = x[3 * f]                                      # a frame of identical tokens: every score ties
    xs = W.f32_to_bf16_bits(x) if bf16 else x
    o = orc.score_frames(xs, vfo, f, w=1.0, min_keep=1, nthreads=NT)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    g = sv.sharpv_prune_frames(to_dev(xs), torch.from_numpy(vfo).cuda(), F, f, w=1.0, min_keep=1, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert_scores(g, o, f, keys=("importance", "ratio"))
    k_gpu = to_host(g["k"])
    check_budgets(k_gpu, o, f)
    idx_o, off_o = orc.select_tokens(to_host(g["importance"]), k_gpu, f)
    n = int(g["num_kept"].item())
    assert n == idx_o.size
    np.testing.assert_array_equal(to_host(g["kept_offsets"]), off_o)
    np.testing.assert_array_equal(to_host(g["kept_index"])[:n], idx_o)
    np.testing.assert_array_equal(to_host(g["tokens"])[:n], orc.gather_rows(xs, idx_o))
    cap = n // 3
    small = sv.sharpv_prune_frames(to_dev(xs), torch.from_numpy(vfo).cuda(), F, f, w=1.0, min_keep=1, capacity=cap,
                                   status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == sv.Status.ERR_CAPACITY and int(small["num_kept"].item()) == n
    np.testing.assert_array_equal(to_host(small["kept_index"])[:cap], idx_o[:cap])
    np.testing.assert_array_equal(to_host(small["tokens"])[:cap], orc.gather_rows(xs, idx_o[:cap]))


def test_many_frames_and_many_positions_use_the_scan_kernels():
    """Batches beyond the sizes at which every CTA adds up the counts in front of it itself: 20,000 tiny
    frames through the selection, 1.2 million packed positions through the calibration (their offsets then
    come from the one-CTA scan kernel)."""
    rng = np.random.default_rng(77)
    F, f = 20_000, 5
    imp = rng.random(F * f).astype(np.float32)
    imp[rng.integers(0, F * f, 3000)] = 0.5                        # ties
    k = rng.integers(-1, f + 2, F).astype(np.int32)                # budgets outside [0, f] are clamped
    sel = sv.sharpv_select_tokens(to_dev(imp), to_dev(k), F, f, gather=False)
    torch.cuda.synchronize()
    idx_o, off_o = orc.select_tokens(imp, k, f)
    np.testing.assert_array_equal(to_host(sel["kept_offsets"]), off_o)
    assert int(sel["num_kept"].item()) == idx_o.size
    np.testing.assert_array_equal(to_host(sel["kept_index"])[:idx_o.size], idx_o)
    thr = sv.sharpv_select_tokens_threshold(to_dev(imp), 0.5, F, f, gather=False)
    torch.cuda.synchronize()
    idx_t, off_t = orc.select_threshold(imp, 0.5, F, f)
    np.testing.assert_array_equal(to_host(thr["kept_offsets"]), off_t)
    np.testing.assert_array_equal(to_host(thr["kept_index"])[:idx_t.size], idx_t)
    # capacity overflow is still reported by the scan
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    small = sv.sharpv_select_tokens(to_dev(imp), to_dev(k), F, f, gather=False, capacity=100, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == sv.Status.ERR_CAPACITY and int(small["num_kept"].item()) == idx_o.size
    np.testing.assert_array_equal(to_host(small["kept_index"])[:100], idx_o[:100])

    T, d = 1_200_000, 16
    lens = np.array([400_000, 0, 799_990, 10])
    so = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    vb = np.array([5, 0, 1000, 0], np.int32)
    vc = np.array([300_000, 0, 500_000, 10], np.int32)
    vo = np.concatenate([[0], np.cumsum(vc)])[:-1].astype(np.int32)
    vis = rng.standard_normal((int(vc.sum()), d)).astype(np.float32)
    hid = rng.standard_normal((T, d)).astype(np.float32)
    for b in range(4):
        r0 = so[b] + vb[b]
        hid[r0:r0 + vc[b]] += 1.5 * vis[vo[b]:vo[b] + vc[b]]
    t32 = lambda a: torch.from_numpy(np.asarray(a, np.int32)).cuda()
    g = sv.sharpv_kv_calibrate_prune(to_dev(hid), to_dev(vis), t32(so), t32(vb), t32(vc), t32(vo), T, M=0.8)
    torch.cuda.synchronize()
    o = orc.kv_calibrate_prune(hid, vis, so, vb, vc, vo, 0.8, nthreads=NT)
    assert rel_err(to_host(g["cos"]), o["cos"]) <= TIGHT_TOL
    kso = to_host(g["kept_seq_offsets"])
    kept = to_host(g["kept_pos"])[:kso[-1]]
    assert np.all(np.diff(kept) > 0)
    sym = np.setxor1d(kept, o["kept_pos"])
    for pos in sym:                                                 # only cosines at the threshold may differ
        b = int(np.searchsorted(so, pos, side="right") - 1)
        row = vo[b] + (pos - so[b] - vb[b])
        assert 0 <= pos - so[b] - vb[b] < vc[b] and abs(o["cos"][row] - 0.8) <= BOUNDARY_TOL
    assert sym.size <= 20
    if sym.size == 0:
        np.testing.assert_array_equal(kso, o["kept_seq_offsets"])
    assert 0.2 * T < kept.size < 0.9 * T


@pytest.mark.parametrize("name", ["tiny", "small_ragged", "odd_shapes"])
def test_outputs_stay_inside_their_buffers(name):
    """Every output and workspace of every entry point sits between two guard bands; capacities are exactly
    the kept counts.  After each call the bands must be untouched."""
    wl, dw = _case(name)
    F, f, d, T, B = wl.total_frames, wl.f, wl.d, wl.total_seq_tokens, wl.num_videos
    NV = F * f
    tdt = dw.tokens.dtype
    G = Guarded()
    u8, f32, i32 = torch.uint8, torch.float32, torch.int32
    # stage one, two calls
    o1 = {"importance": G.empty(NV, f32), "spatial": G.empty(NV, f32), "temporal": G.empty(NV, f32),
          "ratio": G.empty(F, f32), "k": G.empty(F, i32)}
    ws1 = G.empty(sv.sharpv_score_frames_workspace_bytes(F, f, d), u8)
    sv.sharpv_score_frames(dw.tokens, dw.video_frame_offsets, F, f, out=o1, workspace=ws1)
    G.check("score_frames")
    n1 = int(np.clip(to_host(o1["k"]), 0, f).sum())
    o2 = {"kept_index": G.empty(max(n1, 1), i32), "kept_offsets": G.empty(F + 1, i32), "num_kept": G.empty(1, i32),
          "tokens": G.empty((max(n1, 1), d), tdt)}
    ws2 = G.empty(sv.sharpv_select_tokens_workspace_bytes(F, f), u8)
    sv.sharpv_select_tokens(o1["importance"], o1["k"], F, f, tokens=dw.tokens, capacity=n1, out=o2, workspace=ws2)
    G.check("select_tokens")
    sv.sharpv_select_tokens_threshold(o1["importance"], 1.0, F, f, tokens=dw.tokens, capacity=n1, out=o2, workspace=ws2)
    G.check("select_tokens_threshold")
    # stage one, one call
    o3 = {"importance": G.empty(NV, f32), "ratio": G.empty(F, f32), "k": G.empty(F, i32),
          "kept_index": G.empty(max(n1, 1), i32), "kept_offsets": G.empty(F + 1, i32), "num_kept": G.empty(1, i32),
          "tokens": G.empty((max(n1, 1), d), tdt)}
    ws3 = G.empty(sv.sharpv_prune_frames_workspace_bytes(F, f, d), u8)
    sv.sharpv_prune_frames(dw.tokens, dw.video_frame_offsets, F, f, capacity=n1, out=o3, workspace=ws3)
    G.check("prune_frames")
    assert int(o3["num_kept"].item()) == n1
    # stage two
    M = 0.6
    tabs = (dw.seq_offsets, dw.vis_begin, dw.vis_count, dw.vis_offsets)
    probe = sv.sharpv_kv_calibrate_prune(dw.hidden, dw.tokens, *tabs, T, M=M)
    torch.cuda.synchronize()
    n2 = int(probe["kept_seq_offsets"][-1].item())
    o4 = {"cos": G.empty(NV, f32), "kept_pos": G.empty(max(n2, 1), i32), "kept_seq_offsets": G.empty(B + 1, i32),
          "mean_cos": G.empty(B, f32)}
    ws4 = G.empty(sv.sharpv_kv_calibrate_prune_workspace_bytes(T, B), u8)
    sv.sharpv_kv_calibrate_prune(dw.hidden, dw.tokens, *tabs, T, M=M, capacity=n2, want_mean_cos=True, out=o4,
                                 workspace=ws4)
    G.check("kv_calibrate_prune")
    sv.sharpv_kv_calibrate_prune_noalloc(dw.hidden, dw.tokens, *tabs, T, M=M, capacity=n2, want_mean_cos=True, out=o4)
    G.check("kv_calibrate_prune_noalloc")
    L, _, H, _, Dh = wl.kv_shape()
    dst = G.empty((L, 2, H, max(n2, 1), Dh), tdt)
    sv.sharpv_kv_compact(dw.kv, dst, o4["kept_pos"], o4["kept_seq_offsets"], capacity=n2)
    G.check("kv_compact")
    np.testing.assert_array_equal(to_host(dst)[:, :, :, :n2], wl.kv[:, :, :, to_host(o4["kept_pos"])[:n2]])
    cache = G.empty(wl.kv_shape(), tdt)
    cache.copy_(dw.kv)
    sv.sharpv_kv_compact(cache, cache, o4["kept_pos"], o4["kept_seq_offsets"], capacity=n2)
    G.check("kv_compact in place")
    if Dh * cache.element_size() % 32 == 0:
        wsr = G.empty(sv.sharpv_kv_compact_rope_workspace_bytes(max(n2, 1), Dh), u8)
        sv.sharpv_kv_compact_rope(dw.kv, dst, o4["kept_pos"], o4["kept_seq_offsets"], dw.seq_offsets, n2, Dh, 1.0e4,
                                  workspace=wsr)
        G.check("kv_compact_rope")
    hid = torch.stack([dw.hidden] * L)
    wsl = G.empty(sv.sharpv_kv_prune_layers_workspace_bytes(T, B, L), u8)
    for mode in (sv.PRUNE_PER_TOKEN, sv.PRUNE_PER_LAYER):
        cache.copy_(dw.kv)
        sv.sharpv_kv_prune_layers(hid, dw.tokens, *tabs, T, cache, cache, M=M, mode=mode, workspace=wsl)
        G.check(f"kv_prune_layers mode {mode}")


def test_run_to_run_bit_reproducible():
    wl, dw = _case("small_ragged")
    F, f = wl.total_frames, wl.f
    a = sv.sharpv_score_frames(dw.tokens, dw.video_frame_offsets, F, f, want_spatial=True, want_temporal=True)
    b = sv.sharpv_score_frames(dw.tokens, dw.video_frame_offsets, F, f, want_spatial=True, want_temporal=True)
    torch.cuda.synchronize()
    for key in a:
        assert torch.equal(a[key], b[key]), key


def test_strided_token_rows():
    """Row stride larger than d (tokens embedded in a wider buffer)."""
    wl, dw = _case("tiny")
    F, f, d = wl.total_frames, wl.f, wl.d
    wide = torch.zeros((wl.n_visual, d + 64), dtype=dw.tokens.dtype, device="cuda")
    wide[:, :d] = dw.tokens
    a = sv.sharpv_score_frames(dw.tokens, dw.video_frame_offsets, F, f)
    b = sv.sharpv_score_frames(wide[:, :d], dw.video_frame_offsets, F, f)
    torch.cuda.synchronize()
    assert torch.equal(a["importance"], b["importance"]) and torch.equal(a["k"], b["k"])
    sa = sv.sharpv_select_tokens(a["importance"], a["k"], F, f, tokens=dw.tokens)
    sb = sv.sharpv_select_tokens(b["importance"], b["k"], F, f, tokens=wide[:, :d])
    torch.cuda.synchronize()
    n = int(sa["num_kept"].item())
    assert torch.equal(sa["tokens"][:n], sb["tokens"][:n])


# ------------------------------------------------------------------------------------------------
# full-size workloads in the launch configuration the benchmark times
# ------------------------------------------------------------------------------------------------
def _device_kv(wl, seed):
    """N(0,1) K/V drawn on the device with torch's generator (values never influence a decision)."""
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    dt = torch.float32 if wl.dtype == W.F32 else torch.bfloat16
    kv = torch.empty(wl.kv_shape(), dtype=dt, device="cuda")
    for l in range(wl.num_layers):
        kv[l] = torch.randn(wl.kv_shape()[1:], dtype=torch.float32, device="cuda", generator=gen).to(dt)
    return kv


@pytest.mark.parametrize("name", ["ragged_batch", "long_video"])
def test_full_size_workloads(name):
    """The 16-video ragged batch (424 frames) and the 256-frame video at their full sizes: scores,
    budgets and kept sets element by element against the oracle; compacted K/V (4.8 GB / 2.9 GB) on
    sampled planes and rows plus properties that hold for every plane; then the single-call stage one, the
    rotary and the in-place compaction on the same inputs."""
    wl = W.PRESETS[name]()
    W.fill_tokens(wl)
    W.fill_hidden(wl)
    dw = DeviceWorkload(wl)
    F, f, T, M = wl.total_frames, wl.f, wl.total_seq_tokens, 0.788
    o = orc.score_frames(wl.tokens, wl.video_frame_offsets, f, nthreads=NT)
    g = sv.sharpv_score_frames(dw.tokens, dw.video_frame_offsets, F, f, want_spatial=True, want_temporal=True)
    torch.cuda.synchronize()
    assert_scores(g, o, f)
    k_gpu = to_host(g["k"])
    assert len(check_budgets(k_gpu, o, f)) <= max(1, F // 50)
    sel = sv.sharpv_select_tokens(g["importance"], g["k"], F, f, tokens=dw.tokens)
    torch.cuda.synchronize()
    n = int(sel["num_kept"].item())
    assert n == int(k_gpu.sum())
    idx = to_host(sel["kept_index"])[:n]
    exempt = check_kept_sets(idx, to_host(sel["kept_offsets"]), o["importance"], k_gpu, f, orc.select_tokens)
    assert exempt <= max(2, n // 1000)
    rows = np.random.default_rng(80).choice(n, size=min(n, 512), replace=False)
    got = sel["tokens"][torch.from_numpy(rows).cuda()]
    np.testing.assert_array_equal(to_host(got), wl.tokens[idx[rows]])

    oc = orc.kv_calibrate_prune(wl.hidden, wl.tokens, wl.seq_offsets, wl.vis_begin, wl.vis_count, wl.vis_offsets,
                                M, nthreads=NT)
    gc = sv.sharpv_kv_calibrate_prune(dw.hidden, dw.tokens, dw.seq_offsets, dw.vis_begin, dw.vis_count,
                                      dw.vis_offsets, T, M=M)
    torch.cuda.synchronize()
    assert rel_err(to_host(gc["cos"])[:wl.n_visual], oc["cos"]) <= TIGHT_TOL
    kso = to_host(gc["kept_seq_offsets"])
    nk = int(kso[-1])
    kept = to_host(gc["kept_pos"])[:nk]
    sym = np.setxor1d(kept, oc["kept_pos"])
    assert sym.size <= max(2, wl.n_visual // 1000)
    if sym.size == 0:
        np.testing.assert_array_equal(kso, oc["kept_seq_offsets"])

    kv = _device_kv(wl, 81)
    dst = torch.zeros_like(kv)
    sv.sharpv_kv_compact(kv, dst, gc["kept_pos"], gc["kept_seq_offsets"], capacity=T)
    torch.cuda.synchronize()
    L, _, H, _, Dh = wl.kv_shape()
    rng = np.random.default_rng(82)
    planes = {(0, 0, 0), (L - 1, 1, H - 1)} | {(int(rng.integers(L)), int(rng.integers(2)), int(rng.integers(H)))
                                               for _ in range(6)}
    for (l, kvi, h) in planes:                       # sampled planes against the oracle, whole plane
        src_plane = to_host(kv[l, kvi, h])[None, None, None]          # [1, 1, 1, T, Dh] ... one-plane cache
        src5 = np.ascontiguousarray(np.broadcast_to(src_plane, (1, 2, 1, T, Dh)))
        expect = orc.kv_compact(src5, kept)[0, 0, 0]
        np.testing.assert_array_equal(to_host(dst[l, kvi, h]), expect)
    # every plane: the kept prefix equals the gathered source rows, the rest is untouched
    kept_d = gc["kept_pos"][:nk].long()
    assert torch.equal(dst[:, :, :, :nk].view(torch.int16), kv[:, :, :, kept_d].view(torch.int16))
    assert int(dst[:, :, :, nk:].view(torch.int16).abs().max().item()) == 0

    # stage one in one call at the full size: bit for bit the two calls above
    pr = sv.sharpv_prune_frames(dw.tokens, dw.video_frame_offsets, F, f)
    torch.cuda.synchronize()
    assert torch.equal(pr["importance"], g["importance"]) and torch.equal(pr["k"], g["k"])
    assert int(pr["num_kept"].item()) == n and torch.equal(pr["kept_offsets"], sel["kept_offsets"])
    assert torch.equal(pr["kept_index"][:n], sel["kept_index"][:n])
    assert torch.equal(pr["tokens"][:n].view(torch.int16), sel["tokens"][:n].view(torch.int16))
    del pr, sel

    # rotary re-encoding at the full size: values and the keys that do not move are bit copies of the plain
    # compaction; sampled key planes against the oracle
    seqs = torch.from_numpy(wl.seq_offsets).cuda()
    dst.zero_()
    sv.sharpv_kv_compact_rope(kv, dst, gc["kept_pos"], gc["kept_seq_offsets"], seqs, T, Dh, 1.0e6)
    torch.cuda.synchronize()
    assert torch.equal(dst[:, 1, :, :nk].view(torch.int16), kv[:, 1][:, :, kept_d].view(torch.int16))
    assert int(dst[:, :, :, nk:].view(torch.int16).abs().max().item()) == 0
    b_of = np.searchsorted(wl.seq_offsets, kept, side="right") - 1
    still = np.nonzero(kept - wl.seq_offsets[b_of] == np.arange(nk) - kso[b_of])[0]
    still_d = torch.from_numpy(still).cuda()
    assert torch.equal(dst[:, 0][:, :, still_d].view(torch.int16), kv[:, 0][:, :, kept_d[still_d]].view(torch.int16))
    for (l, _, h) in sorted(planes)[:3]:
        src5 = np.ascontiguousarray(to_host(kv[l, :, h])[None, :, None])          # [1, 2, 1, T, Dh]
        want = orc.kv_compact_rope(src5, kept, kso, wl.seq_offsets, Dh, 1.0e6)[0, 0, 0]
        got = W.bf16_bits_to_f32(to_host(dst[l, 0, h, :nk])).astype(np.float64)
        pair = np.hypot(want[:, :Dh // 2], want[:, Dh // 2:])
        pair = np.concatenate([pair, pair], axis=-1)
        assert np.all(np.abs(got - want) <= 2.0 ** -8 * np.abs(want) * 1.001 + 4e-6 * pair + 1e-30)

    # in place at the full size: the kept prefix of every plane equals the rows gathered from the original,
    # the tail keeps its old contents
    dst.copy_(kv)
    sv.sharpv_kv_compact(dst, dst, gc["kept_pos"], gc["kept_seq_offsets"], capacity=T)
    torch.cuda.synchronize()
    assert torch.equal(dst[:, :, :, :nk].view(torch.int16), kv[:, :, :, kept_d].view(torch.int16))
    assert torch.equal(dst[:, :, :, nk:].view(torch.int16), kv[:, :, :, nk:].view(torch.int16))
