"""Shared test helpers: moving workloads to the device and the comparison rules.

Tolerances (derived from the arithmetic, measured on the B200):
  scores  |gpu - oracle| <= tol * max(|oracle|, SCORE_FLOOR), SCORE_FLOOR = 1e-3,
     tol = 1e-5 for fp32 inputs, 2e-2 (ceiling) for bf16 inputs; bf16 inputs widen exactly to
     fp32 and every product is accumulated in fp32, so the kernels are also held to TIGHT_TOL.
     One class of rows cannot meet a relative bound in fp32: rows that are parallel without being
     bit-identical (a scaled copy of the previous frame, a token equal to its frame's mean).  Their
     dissimilarity is 0 in exact arithmetic, the oracle's double arithmetic returns 0 to 3e-8, and
     fp32 returns the rounding of the two unit vectors, up to 2.8e-7 (measured worst case).  Where
     the oracle's S or T is below PARALLEL_BELOW the comparison therefore allows PARALLEL_EPS in
     absolute terms (on that term, on I = T + w S, and on the ratio of a frame that holds such rows).
  cosines  |gpu - oracle| <= tol * max(|oracle|, COS_FLOOR): a cosine is a sum of products of unit
     vector components, its fp32 error is a few units of 2^-24 whatever its size.
  integer decisions  exact, except where the oracle's deciding value lies within BOUNDARY_TOL of
     the decision boundary (k-th score of a frame, threshold M, an integer value of ratio*f).
"""
import numpy as np
import torch

SCORE_FLOOR = 1e-3
PARALLEL_BELOW = 1e-6
PARALLEL_EPS = 4e-7
COS_FLOOR = 0.05
TOL = {"f32": 1e-5, "bf16": 2e-2}
TIGHT_TOL = 1e-5
BOUNDARY_TOL = 1e-5
BOUNDARY_FLOOR = 0.05      # scores live in [0, 2 (1 + w)]: the band around a frame's k-th score never shrinks under 5e-7


def to_dev(a: np.ndarray, device="cuda") -> torch.Tensor:
    """numpy -> device tensor; uint16 arrays are bf16 bit patterns."""
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(a).to(device)


def to_host(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def rel_err(g: np.ndarray, o: np.ndarray, floor: float = COS_FLOOR) -> float:
    g = np.asarray(g, dtype=np.float64)
    o = np.asarray(o, dtype=np.float64)
    if g.size == 0:
        return 0.0
    return float(np.max(np.abs(g - o) / np.maximum(np.abs(o), floor)))


def score_errors(g, o, f, keys=("spatial", "temporal", "importance", "ratio")):
    """Worst error of each score array of `g` (host arrays) against the oracle dict `o`, relative to
    max(|oracle|, SCORE_FLOOR), with the absolute allowance PARALLEL_EPS where the oracle says the rows
    are parallel (see the module docstring).  Returns {key: error}."""
    S_o = np.asarray(o["spatial"], np.float64)
    T_o = np.asarray(o["temporal"], np.float64)
    zS, zT = S_o < PARALLEL_BELOW, T_o < PARALLEL_BELOW
    F = S_o.size // f
    masks = {"spatial": zS, "temporal": zT, "importance": zS | zT,
             "ratio": zT.reshape(F, f).any(axis=1) if F else np.zeros(0, bool)}
    out = {}
    for key in keys:
        if key not in g:
            continue
        gg = np.asarray(g[key], np.float64)
        oo = np.asarray(o[key], np.float64)
        if gg.size == 0:
            out[key] = 0.0
            continue
        err = np.maximum(np.abs(gg - oo) - PARALLEL_EPS * masks[key], 0.0)
        out[key] = float(np.max(err / np.maximum(np.abs(oo), SCORE_FLOOR)))
    return out


def assert_scores(g, o, f, tol=TIGHT_TOL, keys=("spatial", "temporal", "importance", "ratio"), what=""):
    """g: dict of device tensors or host arrays."""
    host = {k: (to_host(v) if isinstance(v, torch.Tensor) else v) for k, v in g.items() if k in keys}
    errs = score_errors(host, o, f, keys)
    for key, e in errs.items():
        assert e <= tol, f"{key}: rel err {e:.3e} > {tol} {what}"
    return errs


class DeviceWorkload:
    """Device copies of a workload's arrays and tables."""

    def __init__(self, wl, device="cuda", hidden=True, kv=False):
        self.wl = wl
        self.tokens = to_dev(wl.tokens, device)
        self.video_frame_offsets = torch.from_numpy(wl.video_frame_offsets).to(device)
        self.seq_offsets = torch.from_numpy(wl.seq_offsets).to(device)
        self.vis_begin = torch.from_numpy(wl.vis_begin).to(device)
        self.vis_count = torch.from_numpy(wl.vis_count).to(device)
        self.vis_offsets = torch.from_numpy(wl.vis_offsets).to(device)
        self.hidden = to_dev(wl.hidden, device) if hidden and wl.hidden is not None else None
        self.kv = to_dev(wl.kv, device) if kv and wl.kv is not None else None


def check_budgets(k_gpu, oracle, f, boundary_tol=BOUNDARY_TOL):
    """k may differ from the oracle only on frames whose ratio*f is within boundary_tol*f of an
    integer (there the rounding step is decided by the last bits).  Returns the exempted frames."""
    k_o = oracle["k"]
    diff = np.nonzero(k_gpu != k_o)[0]
    x = oracle["ratio"] * f
    for t in diff:
        assert abs(int(k_gpu[t]) - int(k_o[t])) <= 1, f"frame {t}: k {k_gpu[t]} vs {k_o[t]}"
        assert abs(x[t] - np.round(x[t])) <= boundary_tol * f, f"frame {t}: ratio*f={x[t]} is not at a boundary"
    return diff


def check_kept_sets(idx_gpu, off_gpu, imp_oracle, k_used, f, select_fn, boundary_tol=BOUNDARY_TOL):
    """Kept sets must equal the oracle's selection with the same budgets, except for tokens whose
    oracle importance lies within boundary_tol * max(|I_kth|, BOUNDARY_FLOOR) of the frame's k-th
    score.  Returns the number of exempted tokens."""
    idx_o, off_o = select_fn(imp_oracle, k_used, f)
    np.testing.assert_array_equal(off_gpu, off_o)
    assert idx_gpu.size == idx_o.size
    assert np.all(np.diff(idx_gpu) > 0)
    exempt = 0
    F = len(k_used)
    for t in range(F):
        a = idx_gpu[off_gpu[t]:off_gpu[t + 1]]
        b = idx_o[off_o[t]:off_o[t + 1]]
        assert np.all(a // f == t)
        if np.array_equal(a, b):
            continue
        sym = np.setxor1d(a, b)
        kth = np.sort(imp_oracle[t * f:(t + 1) * f])[::-1][k_used[t] - 1]
        band = boundary_tol * max(abs(kth), BOUNDARY_FLOOR)
        assert np.all(np.abs(imp_oracle[sym] - kth) <= band), f"frame {t}: kept set differs away from the boundary"
        exempt += sym.size
    return exempt


class Guarded:
    """Device buffers with 256 bytes of a known pattern in front of and behind each of them: a kernel that
    writes outside an output leaves a mark that check() finds (stands in for a memory checker on outputs)."""

    PAD, FILL = 256, 0xA5

    def __init__(self, device="cuda"):
        self.device, self.raw = device, []

    def empty(self, shape, dtype):
        shape = (shape,) if isinstance(shape, int) else tuple(shape)
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        body = (n + 255) // 256 * 256
        buf = torch.full((self.PAD + body + self.PAD,), self.FILL, dtype=torch.uint8, device=self.device)
        self.raw.append((buf, n))
        return buf[self.PAD:self.PAD + n].view(dtype).view(shape)

    def check(self, what=""):
        torch.cuda.synchronize()
        for i, (buf, n) in enumerate(self.raw):
            front, back = buf[:self.PAD], buf[self.PAD + n:]
            assert bool((front == self.FILL).all()), f"{what}: bytes in front of output {i} were overwritten"
            assert bool((back == self.FILL).all()), f"{what}: bytes behind output {i} were overwritten"
