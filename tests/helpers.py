"""Shared test helpers: moving workloads to the device and the comparison rules.

Tolerances (derived from the arithmetic):
  scores / cosines   |gpu - oracle| <= tol * max(|oracle|, SCORE_FLOOR)
     tol = 1e-5 for fp32 inputs, 2e-2 (ceiling) for bf16 inputs; bf16 inputs widen exactly to
     fp32 and every product is accumulated in fp32, so the kernels are also held to TIGHT_TOL.
     SCORE_FLOOR: a dissimilarity is the norm of a difference of unit vectors; in fp32 each unit
     vector carries an absolute error of order 2^-24, so the difference has an absolute error
     floor of that order however small the true value is.  Relative error is therefore measured
     against max(|oracle|, 0.05) (scores live in [0, 2]).
  integer decisions  exact, except where the oracle's deciding value lies within BOUNDARY_TOL of
     the decision boundary (k-th score of a frame, threshold M, an integer value of ratio*f).
"""
import numpy as np
import torch

SCORE_FLOOR = 0.05
TOL = {"f32": 1e-5, "bf16": 2e-2}
TIGHT_TOL = 1e-5
BOUNDARY_TOL = 1e-5


def to_dev(a: np.ndarray, device="cuda") -> torch.Tensor:
    """numpy -> device tensor; uint16 arrays are bf16 bit patterns."""
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(a).to(device)


def to_host(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def rel_err(g: np.ndarray, o: np.ndarray, floor: float = SCORE_FLOOR) -> float:
    g = np.asarray(g, dtype=np.float64)
    o = np.asarray(o, dtype=np.float64)
    if g.size == 0:
        return 0.0
    return float(np.max(np.abs(g - o) / np.maximum(np.abs(o), floor)))


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
    oracle importance lies within boundary_tol * max(|I_kth|, SCORE_FLOOR) of the frame's k-th
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
        band = boundary_tol * max(abs(kth), SCORE_FLOOR)
        assert np.all(np.abs(imp_oracle[sym] - kth) <= band), f"frame {t}: kept set differs away from the boundary"
        exempt += sym.size
    return exempt
