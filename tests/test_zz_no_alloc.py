"""Allocation-free calibration entry point against the workspace-taking one.

Collected last on purpose (file name): if it fails under `-x`, every other test has already run.

Who needs the variant: a serving engine that handed all spare device memory to its own cache pool,
a plug-in that is given tensors but no allocator, a process under a fixed memory budget.  Such a
caller passes inputs and outputs only; the library's scratch sits in a fixed device array.  The
test calls it twice in a row through the C ABI (second call on a different, smaller input, so
stale scratch from the first call would show) and demands the very same outputs as the existing
entry point, which runs the same kernels on caller-provided scratch.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import sharpv_oracle as orc
from paper_2511_08003_b200 import binding as sv
from paper_2511_08003_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _inputs(wl, dev):
    bits = lambda a: (torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16) if a.dtype == np.uint16
                      else torch.from_numpy(a).to(dev))
    i32 = lambda a: torch.from_numpy(a).to(dev)
    return (bits(wl.hidden), bits(wl.tokens), i32(wl.seq_offsets), i32(wl.vis_begin), i32(wl.vis_count),
            i32(wl.vis_offsets), wl.total_seq_tokens)


def _outputs(wl, dev):
    """Every output the call writes, allocated up front: the call under test is handed memory only."""
    B, T = wl.num_videos, wl.total_seq_tokens
    return {"cos": torch.empty(wl.n_visual, dtype=torch.float32, device=dev),
            "kept_pos": torch.empty(T, dtype=torch.int32, device=dev),
            "kept_seq_offsets": torch.empty(B + 1, dtype=torch.int32, device=dev),
            "mean_cos": torch.empty(B, dtype=torch.float32, device=dev)}


def _same(a, b, n_visual):
    n = int(a["kept_seq_offsets"][-1].item())
    assert torch.equal(a["kept_seq_offsets"], b["kept_seq_offsets"])
    assert torch.equal(a["kept_pos"][:n], b["kept_pos"][:n])
    # same kernels, same order of operations: the cosines agree to the last bit, which is inside
    # the 1e-5 relative tolerance the parity tests use
    assert torch.equal(a["cos"][:n_visual], b["cos"][:n_visual])
    assert torch.equal(a["mean_cos"], b["mean_cos"])
    return n


def test_noalloc_matches_workspace_entry_point_twice_in_a_row():
    dev = torch.device("cuda", 0)
    big = W.fill_hidden(W.fill_tokens(W.custom(
        "na_big", 60, W.BF16, 14, 1024, 48, [W.make_video_spec(7, 0.9, cuts=[3]), W.make_video_spec(4, 0.8)])))
    small = W.fill_hidden(W.fill_tokens(W.custom("na_small", 61, W.F32, 5, 64, 9, [W.make_video_spec(3, 0.7)])))
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    kept = []
    for wl, M in ((big, 0.788), (small, 0.6)):
        args = _inputs(wl, dev)
        ref = sv.sharpv_kv_calibrate_prune(*args, M=M, want_mean_cos=True)
        got = sv.sharpv_kv_calibrate_prune_noalloc(*args, M=M, want_mean_cos=True, out=_outputs(wl, dev),
                                                   status_word=status)
        torch.cuda.synchronize()
        kept.append(_same(got, ref, wl.n_visual))
        assert 0 < kept[-1] < wl.total_seq_tokens            # the threshold actually prunes something
        # and against the CPU oracle directly, so that this file stands on its own
        o = orc.kv_calibrate_prune(wl.hidden, wl.tokens, wl.seq_offsets, wl.vis_begin, wl.vis_count, wl.vis_offsets,
                                   M, nthreads=4)
        cos = got["cos"].cpu().numpy().astype(np.float64)
        assert np.max(np.abs(cos - o["cos"])) <= 1e-5
        away = np.abs(o["cos"] - M) > 1e-5                    # tokens whose oracle cosine is not at the threshold
        pos = np.concatenate([wl.seq_offsets[b] + wl.vis_begin[b] + np.arange(wl.vis_count[b])
                              for b in range(wl.num_videos)])
        mine = np.zeros(wl.total_seq_tokens, bool)
        mine[got["kept_pos"][:kept[-1]].cpu().numpy()] = True
        theirs = np.zeros(wl.total_seq_tokens, bool)
        theirs[o["kept_pos"]] = True
        assert np.array_equal(mine[pos][away], theirs[pos][away])
        assert np.array_equal(np.delete(mine, pos), np.delete(theirs, pos))      # text positions: all kept
    assert int(status.item()) == 0
    # and once more on the first input: the scratch now holds the small call's leftovers
    args = _inputs(big, dev)
    ref = sv.sharpv_kv_calibrate_prune(*args, M=0.788, want_mean_cos=True)
    got = sv.sharpv_kv_calibrate_prune_noalloc(*args, M=0.788, want_mean_cos=True, out=_outputs(big, dev))
    torch.cuda.synchronize()
    assert _same(got, ref, big.n_visual) == kept[0]


def test_noalloc_takes_the_largest_input_it_documents_and_allocates_nothing():
    """total_seq_tokens == SHARPV_NOALLOC_MAX_SEQ_TOKENS uses the fixed scratch to its last byte; with all
    outputs passed in, the device's free memory is the same before and after the call."""
    dev = torch.device("cuda", 0)
    T, d, n_vis = sv.NOALLOC_MAX_SEQ_TOKENS, 64, 200_000
    g = torch.Generator(device=dev)
    g.manual_seed(62)
    visual = torch.randn((n_vis, d), dtype=torch.float32, device=dev, generator=g)
    hidden = torch.randn((T, d), dtype=torch.float32, device=dev, generator=g)
    hidden[1000:1000 + n_vis] = visual + 0.9 * hidden[1000:1000 + n_vis]
    i32 = lambda v: torch.tensor(v, dtype=torch.int32, device=dev)
    tabs = (i32([0, T]), i32([1000]), i32([n_vis]), i32([0]))
    ref = sv.sharpv_kv_calibrate_prune(hidden, visual, *tabs, T, M=0.75, want_mean_cos=True)
    out = {"cos": torch.empty(n_vis, dtype=torch.float32, device=dev),
           "kept_pos": torch.empty(T, dtype=torch.int32, device=dev),
           "kept_seq_offsets": torch.empty(2, dtype=torch.int32, device=dev),
           "mean_cos": torch.empty(1, dtype=torch.float32, device=dev)}
    sv.sharpv_kv_calibrate_prune_noalloc(hidden, visual, *tabs, T, M=0.75, want_mean_cos=True, out=out)   # set-up call
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info(dev)
    got = sv.sharpv_kv_calibrate_prune_noalloc(hidden, visual, *tabs, T, M=0.75, want_mean_cos=True, out=out)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info(dev)
    assert free_after == free_before
    n = _same(got, ref, n_vis)
    assert T - n_vis < n < T


def test_noalloc_rejects_inputs_beyond_its_fixed_scratch():
    L = sv.lib()
    P = 0x10000
    too_many = sv.NOALLOC_MAX_SEQ_TOKENS + 1
    rc = L.sharpv_kv_calibrate_prune_noalloc(P, 64, P, 64, 1, 64, 1, P, P, P, P, too_many, 10, 0.2, P, None, P, P,
                                             too_many, None, None)
    assert rc == sv.Status.ERR_UNSUPPORTED
