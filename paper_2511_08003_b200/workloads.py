"""Seeded synthetic VideoLLM workloads for the SharpV pruning path.

This module only *draws inputs*: visual token matrices with the temporal and
spatial correlation structure of projected video frames, the hidden state of
the calibration layer, a K/V cache and the packing tables that say where each
video's tokens sit.  It holds none of the method's arithmetic (no similarity,
no score, no selection) and is the one module that both the CPU oracle's tests
and the CUDA path's tests/benchmark import, so that both see the same bytes.

Shapes follow the paper's Table 2 (LLaVA-OneVision-7B: d=3584, 28 layers,
196 tokens/frame, 32 frames; LLaVA-OneVision-0.5B: d=896).  The videos stand in
for the evaluation videos of the paper, which need datasets and trained
encoders that are not available offline.

Draw order (fixed; every stream is numpy ``default_rng([seed, stream])``):
  stream 0  structure: frame counts, scene cuts, rho values, duplicate frames
  stream 1  token noise, video by video, frame by frame
  stream 2  hidden state: per-token drift s, then noise, sequence by sequence
  stream 3  K/V cache values
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

F32 = "f32"
BF16 = "bf16"


# --------------------------------------------------------------------------
# bf16 <-> fp32 bit helpers (storage format conversion only)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round to nearest, ties to even); returns uint16."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to fp32."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------
# specification of one video and of one workload
# --------------------------------------------------------------------------
@dataclass
class VideoSpec:
    n_frames: int
    rho: np.ndarray            # [n_frames]; rho[0] unused; 0 at a scene cut
    duplicate: np.ndarray      # [n_frames] bool; frame is a bit copy of its predecessor


@dataclass
class Workload:
    """One packed batch of videos with everything both stages read."""
    name: str
    seed: int
    dtype: str                 # "f32" or "bf16"
    grid: int                  # tokens per frame f = grid*grid
    f: int
    d: int
    n_text: int                # text tokens appended after each video's visual tokens
    videos: List[VideoSpec]
    blur_sigma: float
    # K/V cache shape
    num_layers: int
    num_kv_heads: int
    head_dim: int
    # packing tables (int32)
    video_frame_offsets: np.ndarray = field(default=None)   # [B+1]
    seq_offsets: np.ndarray = field(default=None)           # [B+1] rows of the packed hidden state
    vis_begin: np.ndarray = field(default=None)             # [B] first visual row inside a sequence
    vis_count: np.ndarray = field(default=None)             # [B]
    vis_offsets: np.ndarray = field(default=None)           # [B] first row in the visual matrix
    # data (filled lazily)
    tokens: Optional[np.ndarray] = None    # [N_v, d] float32, or uint16 bf16 bit patterns
    hidden: Optional[np.ndarray] = None    # [T, d] same storage as tokens
    kv: Optional[np.ndarray] = None        # [L, 2, H, T, D_h] same storage

    @property
    def num_videos(self) -> int:
        return len(self.videos)

    @property
    def total_frames(self) -> int:
        return int(self.video_frame_offsets[-1])

    @property
    def n_visual(self) -> int:
        return self.total_frames * self.f

    @property
    def total_seq_tokens(self) -> int:
        return int(self.seq_offsets[-1])

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == F32 else 2

    @property
    def np_storage(self):
        return np.float32 if self.dtype == F32 else np.uint16

    def kv_shape(self):
        return (self.num_layers, 2, self.num_kv_heads, self.total_seq_tokens, self.head_dim)

    def kv_bytes(self) -> int:
        n = 1
        for s in self.kv_shape():
            n *= s
        return n * self.elem_bytes

    def tokens_as_f32(self) -> np.ndarray:
        return self.tokens if self.dtype == F32 else bf16_bits_to_f32(self.tokens)

    def hidden_as_f32(self) -> np.ndarray:
        return self.hidden if self.dtype == F32 else bf16_bits_to_f32(self.hidden)


# --------------------------------------------------------------------------
# spatial blur of the innovation noise on the token grid
# --------------------------------------------------------------------------
def _gauss_taps(sigma: float, radius: int = 3) -> np.ndarray:
    x = np.arange(-radius, radius + 1, dtype=np.float64)
    w = np.exp(-0.5 * (x / sigma) ** 2)
    return w / w.sum()


def _blur_axis(z: np.ndarray, axis: int, taps: np.ndarray) -> np.ndarray:
    """1-D Gaussian filter along a grid axis; at the border the taps that fall
    outside the grid are dropped and the rest renormalised to sum to one."""
    g = z.shape[axis]
    radius = (len(taps) - 1) // 2
    out = np.zeros_like(z)
    wsum = np.zeros(g, dtype=np.float64)
    for k in range(-radius, radius + 1):
        w = float(taps[k + radius])
        lo, hi = max(0, -k), min(g, g - k)   # destination range with source p+k in bounds
        if hi <= lo:
            continue
        dst = [slice(None)] * z.ndim
        src = [slice(None)] * z.ndim
        dst[axis] = slice(lo, hi)
        src[axis] = slice(lo + k, hi + k)
        out[tuple(dst)] += np.float32(w) * z[tuple(src)]
        wsum[lo:hi] += w
    shape = [1] * z.ndim
    shape[axis] = g
    out /= wsum.reshape(shape).astype(np.float32)
    return out


def blur_noise(z: np.ndarray, grid: int, sigma: float) -> np.ndarray:
    """z: [grid*grid, d] iid N(0,1).  Separable Gaussian blur (radius 3) over the
    grid for every channel, rescaled by 1/sqrt(sum w^2) of the interior 2-D
    kernel so interior elements keep unit variance."""
    if sigma <= 0:
        return z
    taps = _gauss_taps(sigma)
    zz = z.reshape(grid, grid, -1)
    zz = _blur_axis(zz, 0, taps)
    zz = _blur_axis(zz, 1, taps)
    k2 = np.outer(taps, taps)
    scale = np.float32(1.0 / np.sqrt((k2 ** 2).sum()))
    return (zz * scale).reshape(grid * grid, -1)


# --------------------------------------------------------------------------
# structure draws
# --------------------------------------------------------------------------
def make_video_spec(n_frames: int, rho, cuts: Sequence[int] = (),
                    duplicates: Sequence[int] = ()) -> VideoSpec:
    r = np.empty(n_frames, dtype=np.float64)
    r[:] = rho
    r[0] = 0.0
    for c in cuts:
        r[int(c)] = 0.0
    dup = np.zeros(n_frames, dtype=bool)
    for t in duplicates:
        dup[int(t)] = True
    return VideoSpec(n_frames=n_frames, rho=r, duplicate=dup)


def _pack(wl: Workload) -> Workload:
    B = wl.num_videos
    n = np.array([v.n_frames for v in wl.videos], dtype=np.int64)
    wl.video_frame_offsets = np.concatenate([[0], np.cumsum(n)]).astype(np.int32)
    vis = n * wl.f
    seq = vis + wl.n_text
    wl.seq_offsets = np.concatenate([[0], np.cumsum(seq)]).astype(np.int32)
    wl.vis_begin = np.zeros(B, dtype=np.int32)           # visual tokens first, text after
    wl.vis_count = vis.astype(np.int32)
    wl.vis_offsets = np.concatenate([[0], np.cumsum(vis)])[:-1].astype(np.int32)
    return wl


# --------------------------------------------------------------------------
# data draws
# --------------------------------------------------------------------------
def fill_tokens(wl: Workload) -> Workload:
    """AR(1) over frames, position aligned:  x_t = rho_t x_{t-1} + sqrt(1-rho_t^2) z_t."""
    rng = np.random.default_rng([wl.seed, 1])
    out = np.empty((wl.n_visual, wl.d), dtype=wl.np_storage)
    row = 0
    for v in wl.videos:
        prev = None
        for t in range(v.n_frames):
            if t > 0 and v.duplicate[t]:
                cur = prev
            else:
                z = rng.standard_normal((wl.f, wl.d), dtype=np.float32)
                z = blur_noise(z, wl.grid, wl.blur_sigma)
                if t == 0 or v.rho[t] == 0.0:
                    cur = z
                else:
                    r = np.float32(v.rho[t])
                    cur = r * prev + np.float32(np.sqrt(1.0 - float(v.rho[t]) ** 2)) * z
            out[row:row + wl.f] = cur if wl.dtype == F32 else f32_to_bf16_bits(cur)
            prev = cur
            row += wl.f
    wl.tokens = out
    return wl


def fill_hidden(wl: Workload, s_max: float = 2.0) -> Workload:
    """Calibration-layer hidden state: visual rows h = v + s*N(0,1) with a
    per-token s ~ U[0, s_max]; text rows N(0,1)."""
    assert wl.tokens is not None
    rng = np.random.default_rng([wl.seed, 2])
    T = wl.total_seq_tokens
    out = np.empty((T, wl.d), dtype=wl.np_storage)
    for b in range(wl.num_videos):
        s0 = int(wl.seq_offsets[b])
        nv = int(wl.vis_count[b])
        vb = int(wl.vis_begin[b])
        vo = int(wl.vis_offsets[b])
        nt = int(wl.seq_offsets[b + 1]) - s0
        chunk = 4096
        s_all = rng.uniform(0.0, s_max, size=nv).astype(np.float32)
        for c0 in range(0, nv, chunk):
            c1 = min(nv, c0 + chunk)
            v = wl.tokens[vo + c0:vo + c1]
            v = v if wl.dtype == F32 else bf16_bits_to_f32(v)
            h = v + s_all[c0:c1, None] * rng.standard_normal((c1 - c0, wl.d), dtype=np.float32)
            out[s0 + vb + c0:s0 + vb + c1] = h if wl.dtype == F32 else f32_to_bf16_bits(h)
        text_rows = [r for r in range(0, vb)] + [r for r in range(vb + nv, nt)]
        if text_rows:
            tx = rng.standard_normal((len(text_rows), wl.d), dtype=np.float32)
            out[s0 + np.array(text_rows)] = tx if wl.dtype == F32 else f32_to_bf16_bits(tx)
    wl.hidden = out
    return wl


def fill_kv(wl: Workload) -> Workload:
    """K/V ~ N(0,1), layout [L, 2, H, T, D_h].  The values never influence a
    decision; compaction is compared as raw words."""
    rng = np.random.default_rng([wl.seed, 3])
    shape = wl.kv_shape()
    out = np.empty(shape, dtype=wl.np_storage)
    for l in range(shape[0]):
        z = rng.standard_normal(shape[1:], dtype=np.float32)
        out[l] = z if wl.dtype == F32 else f32_to_bf16_bits(z)
    wl.kv = out
    return wl


# --------------------------------------------------------------------------
# the five named workloads (optionally shrunk for quick tests)
# --------------------------------------------------------------------------
def _new(name, seed, dtype, grid, d, n_text, videos, blur, L, H, Dh) -> Workload:
    wl = Workload(name=name, seed=seed, dtype=dtype, grid=grid, f=grid * grid, d=d, n_text=n_text,
                  videos=videos, blur_sigma=blur, num_layers=L, num_kv_heads=H, head_dim=Dh)
    return _pack(wl)


def tiny(d: int = 896) -> Workload:
    """8 frames x 196 tokens, fp32, rho=0.9, scene cut at frame 4, 32 text tokens,
    one layer, 2 KV heads x 64.  Seed 0."""
    v = make_video_spec(8, 0.9, cuts=[4])
    return _new("tiny", 0, F32, 14, d, 32, [v], 0.0, 1, 2, 64)


def onevision_7b(n_frames: int = 32, d: int = 3584, num_layers: int = 28) -> Workload:
    """32 frames x 196 tokens, bf16, rho=0.95, 3 scene cuts, blur sigma=1, 64 text tokens."""
    rng = np.random.default_rng([1, 0])
    ncut = min(3, max(0, n_frames - 1))
    cuts = np.sort(rng.choice(np.arange(1, n_frames), size=ncut, replace=False)) if ncut else []
    v = make_video_spec(n_frames, 0.95, cuts=cuts)
    return _new("onevision_7b", 1, BF16, 14, d, 64, [v], 1.0, num_layers, 4, 128)


def video_7b(n_frames: int = 64, d: int = 3584, num_layers: int = 28) -> Workload:
    """64 frames x 169 tokens (13x13), bf16; 5 cuts -> 6 segments with rho ~ U[0.8,0.99];
    20 % of the non-first frames are exact duplicates of their predecessor; 128 text tokens."""
    rng = np.random.default_rng([2, 0])
    ncut = min(5, max(0, n_frames - 1))
    cuts = np.sort(rng.choice(np.arange(1, n_frames), size=ncut, replace=False)) if ncut else np.array([], int)
    seg_rho = rng.uniform(0.8, 0.99, size=ncut + 1)
    rho = np.empty(n_frames)
    seg = 0
    for t in range(n_frames):
        if seg < ncut and t == cuts[seg]:
            seg += 1
        rho[t] = seg_rho[seg]
    non_cut = np.array([t for t in range(1, n_frames) if t not in set(int(c) for c in cuts)], dtype=int)
    ndup = min(len(non_cut), int(round(0.2 * (n_frames - 1))))
    dups = rng.choice(non_cut, size=ndup, replace=False) if ndup else []
    v = make_video_spec(n_frames, rho, cuts=cuts, duplicates=dups)
    return _new("video_7b", 2, BF16, 13, d, 128, [v], 0.0, num_layers, 4, 128)


def ragged_batch(num_videos: int = 16, d: int = 3584, num_layers: int = 28,
                 frame_choices: Sequence[int] = (8, 16, 32, 64)) -> Workload:
    """16 videos, frame counts uniform from {8,16,32,64}, 196 tokens/frame, bf16;
    per-video rho ~ U[0.7,0.99] and 0-4 cuts; 64 text tokens per video; packed."""
    rng = np.random.default_rng([3, 0])
    videos = []
    for _ in range(num_videos):
        n = int(rng.choice(np.asarray(frame_choices)))
        rho = float(rng.uniform(0.7, 0.99))
        ncut = min(int(rng.integers(0, 5)), n - 1)
        cuts = np.sort(rng.choice(np.arange(1, n), size=ncut, replace=False)) if ncut else []
        videos.append(make_video_spec(n, rho, cuts=cuts))
    return _new("ragged_batch", 3, BF16, 14, d, 64, videos, 0.0, num_layers, 4, 128)


def long_video(n_frames: int = 256, d: int = 3584, num_layers: int = 28) -> Workload:
    """256 frames x 196 tokens, bf16, rho=0.97, 12 cuts, blur sigma=1, 256 text tokens."""
    rng = np.random.default_rng([4, 0])
    ncut = min(12, max(0, n_frames - 1))
    cuts = np.sort(rng.choice(np.arange(1, n_frames), size=ncut, replace=False)) if ncut else []
    v = make_video_spec(n_frames, 0.97, cuts=cuts)
    return _new("long_video", 4, BF16, 14, d, 256, [v], 1.0, num_layers, 4, 128)


def custom(name: str, seed: int, dtype: str, grid: int, d: int, n_text: int,
           videos: List[VideoSpec], blur_sigma: float = 0.0,
           num_layers: int = 1, num_kv_heads: int = 2, head_dim: int = 64) -> Workload:
    return _new(name, seed, dtype, grid, d, n_text, videos, blur_sigma, num_layers, num_kv_heads, head_dim)


PRESETS = {
    "tiny": tiny,
    "onevision_7b": onevision_7b,
    "video_7b": video_7b,
    "ragged_batch": ragged_batch,
    "long_video": long_video,
}
