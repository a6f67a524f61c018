"""ctypes front end of the SharpV oracle (``sharpv_oracle.c``).

TEST INFRASTRUCTURE, NOT PRODUCT CODE: only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this module.  It never touches the CUDA
library and shares nothing with it.

Array conventions: tokens / hidden / K/V are numpy arrays, ``float32`` for fp32
data and ``uint16`` (raw bf16 bit patterns) for bf16 data.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sharpv_oracle.c")
_LIB = os.path.join(_HERE, "libsharpv_oracle.so")

ROUND_FLOOR, ROUND_NEAREST, ROUND_CEIL = 0, 1, 2
DISSIM, ONE_MINUS_COS = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, OpenMP for the outer loops)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.sharpv_oracle_dissim.restype = C.c_double
        _lib.sharpv_oracle_cosine.restype = C.c_double
        _lib.sharpv_oracle_one_minus_cos.restype = C.c_double
        _lib.sharpv_oracle_select_tokens.restype = C.c_int64
        _lib.sharpv_oracle_select_threshold.restype = C.c_int64
        _lib.sharpv_oracle_kv_calibrate_prune.restype = C.c_int64
        _lib.sharpv_oracle_kv_compact.restype = None
        _lib.sharpv_oracle_gather_rows.restype = None
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return 0
    if a.dtype == np.uint16:
        return 1
    raise TypeError("tokens must be float32 or uint16 (bf16 bits)")


def _row_major(a: np.ndarray) -> int:
    assert a.ndim == 2 and a.strides[1] == a.itemsize, "rows must be contiguous"
    assert a.strides[0] % a.itemsize == 0
    return a.strides[0] // a.itemsize


def dissim(v1, v2) -> float:
    a = np.ascontiguousarray(v1, dtype=np.float64)
    b = np.ascontiguousarray(v2, dtype=np.float64)
    return float(lib().sharpv_oracle_dissim(_ptr(a), _ptr(b), C.c_int(a.size)))


def cosine(v1, v2) -> float:
    a = np.ascontiguousarray(v1, dtype=np.float64)
    b = np.ascontiguousarray(v2, dtype=np.float64)
    return float(lib().sharpv_oracle_cosine(_ptr(a), _ptr(b), C.c_int(a.size)))


def one_minus_cos(v1, v2) -> float:
    a = np.ascontiguousarray(v1, dtype=np.float64)
    b = np.ascontiguousarray(v2, dtype=np.float64)
    return float(lib().sharpv_oracle_one_minus_cos(_ptr(a), _ptr(b), C.c_int(a.size)))


def score_frames(tokens: np.ndarray, video_frame_offsets, f: int, w: float = 1.0,
                 round_mode: int = ROUND_FLOOR, min_keep: int = 0,
                 dissim_kind: int = DISSIM, nthreads: int = 1):
    """Returns dict(spatial, temporal, importance [N_v] f64, ratio [F] f64, k [F] i32)."""
    vfo = np.ascontiguousarray(video_frame_offsets, dtype=np.int32)
    F = int(vfo[-1])
    d = tokens.shape[1]
    ld = _row_major(tokens)
    assert tokens.shape[0] >= F * f
    S = np.empty(F * f, np.float64)
    T = np.empty(F * f, np.float64)
    I = np.empty(F * f, np.float64)
    r = np.empty(F, np.float64)
    k = np.empty(F, np.int32)
    rc = lib().sharpv_oracle_score_frames(
        _ptr(tokens), C.c_int(_dtype_code(tokens)), C.c_int64(ld), C.c_int(len(vfo) - 1), _ptr(vfo),
        C.c_int(f), C.c_int(d), C.c_double(w), C.c_int(round_mode), C.c_int(min_keep),
        C.c_int(dissim_kind), _ptr(S), _ptr(T), _ptr(I), _ptr(r), _ptr(k), C.c_int(nthreads))
    if rc != 0:
        raise RuntimeError("sharpv_oracle_score_frames failed")
    return dict(spatial=S, temporal=T, importance=I, ratio=r, k=k)


def select_tokens(importance, k, f: int) -> Tuple[np.ndarray, np.ndarray]:
    """importance: [F*f] (rounded to fp32 here, the decision precision); k: [F].
    Returns (kept_index ascending int32, kept_offsets [F+1] int32)."""
    imp = np.ascontiguousarray(importance, dtype=np.float32)
    kk = np.ascontiguousarray(k, dtype=np.int32)
    F = kk.size
    assert imp.size == F * f
    idx = np.empty(F * f, np.int32)
    off = np.empty(F + 1, np.int32)
    n = lib().sharpv_oracle_select_tokens(_ptr(imp), _ptr(kk), C.c_int(F), C.c_int(f), _ptr(idx), _ptr(off))
    return idx[:n].copy(), off


def select_threshold(importance, K: float, F: int, f: int):
    imp = np.ascontiguousarray(importance, dtype=np.float32)
    idx = np.empty(F * f, np.int32)
    off = np.empty(F + 1, np.int32)
    n = lib().sharpv_oracle_select_threshold(_ptr(imp), C.c_float(K), C.c_int(F), C.c_int(f), _ptr(idx), _ptr(off))
    return idx[:n].copy(), off


def gather_rows(src: np.ndarray, index) -> np.ndarray:
    idx = np.ascontiguousarray(index, dtype=np.int32)
    ld = _row_major(src)
    out = np.empty((idx.size, src.shape[1]), dtype=src.dtype)
    lib().sharpv_oracle_gather_rows(_ptr(src), C.c_int64(ld * src.itemsize),
                                    C.c_int64(src.shape[1] * src.itemsize), _ptr(idx),
                                    C.c_int64(idx.size), _ptr(out), C.c_int64(out.strides[0]))
    return out


def kv_calibrate_prune(hidden: np.ndarray, visual: np.ndarray, seq_offsets, vis_begin, vis_count,
                       vis_offsets, M: float, nthreads: int = 1):
    """Returns dict(cos [total_visual] f64, kept_pos int32 ascending, kept_seq_offsets [B+1])."""
    so = np.ascontiguousarray(seq_offsets, dtype=np.int32)
    vb = np.ascontiguousarray(vis_begin, dtype=np.int32)
    vc = np.ascontiguousarray(vis_count, dtype=np.int32)
    vo = np.ascontiguousarray(vis_offsets, dtype=np.int32)
    B = so.size - 1
    T = int(so[-1])
    assert hidden.dtype == visual.dtype and hidden.shape[1] == visual.shape[1]
    cos = np.full(visual.shape[0], np.nan, np.float64)
    kept = np.empty(max(T, 1), np.int32)
    kso = np.empty(B + 1, np.int32)
    n = lib().sharpv_oracle_kv_calibrate_prune(
        _ptr(hidden), C.c_int64(_row_major(hidden)), _ptr(visual), C.c_int64(_row_major(visual)),
        C.c_int(_dtype_code(hidden)), C.c_int(hidden.shape[1]), C.c_int(B), _ptr(so), _ptr(vb), _ptr(vc),
        _ptr(vo), C.c_double(M), _ptr(cos), _ptr(kept), _ptr(kso), C.c_int(nthreads))
    if n < 0:
        raise RuntimeError("sharpv_oracle_kv_calibrate_prune failed")
    return dict(cos=cos, kept_pos=kept[:n].copy(), kept_seq_offsets=kso)


def kv_compact(kv_src: np.ndarray, kept_pos, layer_begin: int = 0, layer_end: Optional[int] = None,
               dst: Optional[np.ndarray] = None, nthreads: int = 1) -> np.ndarray:
    """kv_src: [L, 2, H, T, D_h] (any strides with a contiguous last axis).
    Returns dst of the same shape; rows [0, n_kept) of every plane of the layer
    range are written, everything else keeps what dst held (zeros if allocated here)."""
    assert kv_src.ndim == 5 and kv_src.strides[4] == kv_src.itemsize
    kp = np.ascontiguousarray(kept_pos, dtype=np.int32)
    L, _, H, T, Dh = kv_src.shape
    if layer_end is None:
        layer_end = L
    if dst is None:
        dst = np.zeros_like(kv_src)
    assert dst.strides[4] == dst.itemsize
    ss, ds = kv_src.strides, dst.strides
    lib().sharpv_oracle_kv_compact(
        _ptr(kv_src), _ptr(dst), C.c_int(H), C.c_int64(Dh * kv_src.itemsize),
        C.c_int64(ss[0]), C.c_int64(ss[1]), C.c_int64(ss[2]), C.c_int64(ss[3]),
        C.c_int64(ds[0]), C.c_int64(ds[1]), C.c_int64(ds[2]), C.c_int64(ds[3]),
        C.c_int(layer_begin), C.c_int(layer_end), _ptr(kp), C.c_int64(kp.size), C.c_int(nthreads))
    return dst


def kv_compact_inplace(kv: np.ndarray, kept_pos, layer_begin: int = 0, layer_end: Optional[int] = None) -> np.ndarray:
    """In-place compaction of kv [L, 2, H, T, D_h] (modifies and returns kv)."""
    assert kv.ndim == 5 and kv.strides[4] == kv.itemsize
    kp = np.ascontiguousarray(kept_pos, dtype=np.int32)
    L, _, H, T, Dh = kv.shape
    if layer_end is None:
        layer_end = L
    st = kv.strides
    fn = lib().sharpv_oracle_kv_compact_inplace
    fn.restype = C.c_int
    rc = fn(_ptr(kv), C.c_int(H), C.c_int64(Dh * kv.itemsize), C.c_int64(st[0]), C.c_int64(st[1]), C.c_int64(st[2]),
            C.c_int64(st[3]), C.c_int64(T), C.c_int(layer_begin), C.c_int(layer_end), _ptr(kp), C.c_int64(kp.size))
    if rc != 0:
        raise RuntimeError("sharpv_oracle_kv_compact_inplace failed")
    return kv


def kv_prune_layers(hidden_layers, visual: np.ndarray, seq_offsets, vis_begin, vis_count, vis_offsets, M: float,
                    kv: np.ndarray, layer_begin: int = 0, nthreads: int = 0):
    """Section 3.2.3 read layer by layer: Eq. 7 on the hidden state of each layer decides which of that
    layer's K/V rows stay.  hidden_layers[i] is the hidden state of layer layer_begin + i.  Returns the
    per-layer results of kv_calibrate_prune and a copy of kv whose planes of those layers are compacted
    in place (rows at and beyond a layer's kept count keep their old contents)."""
    out = np.array(kv, copy=True)
    results = []
    for i, h in enumerate(hidden_layers):
        o = kv_calibrate_prune(h, visual, seq_offsets, vis_begin, vis_count, vis_offsets, M, nthreads=nthreads)
        kv_compact_inplace(out, o["kept_pos"], layer_begin=layer_begin + i, layer_end=layer_begin + i + 1)
        results.append(o)
    return results, out


def kv_discard_layers(hidden_layers: np.ndarray, visual: np.ndarray, seq_offsets, vis_begin, vis_count,
                      vis_offsets, M: float, nthreads: int = 1):
    """Eq. 7 as printed: one decision per layer (and sequence) on the average cosine between the layer's
    visual hidden states and the original features; the first failing layer and every deeper one lose
    their visual K/V rows.  hidden_layers: [n_layers, T, d].  Returns dict(mean_cos [n, B] f64,
    first_discard [B] int32 (n if none), kept_pos: list of n ascending int32 arrays,
    kept_seq_offsets [n, B+1])."""
    assert hidden_layers.ndim == 3 and hidden_layers.strides[2] == hidden_layers.itemsize
    so = np.ascontiguousarray(seq_offsets, dtype=np.int32)
    vb = np.ascontiguousarray(vis_begin, dtype=np.int32)
    vc = np.ascontiguousarray(vis_count, dtype=np.int32)
    vo = np.ascontiguousarray(vis_offsets, dtype=np.int32)
    n, T, d = hidden_layers.shape
    B = so.size - 1
    assert T == int(so[-1])
    it = hidden_layers.itemsize
    mean = np.zeros((n, B), np.float64)
    first = np.zeros(B, np.int32)
    kept = np.zeros((max(n, 1), max(T, 1)), np.int32)
    kso = np.zeros((max(n, 1), B + 1), np.int32)
    fn = lib().sharpv_oracle_kv_discard_layers
    fn.restype = C.c_int
    rc = fn(_ptr(hidden_layers), C.c_int64(hidden_layers.strides[0] // it), C.c_int64(hidden_layers.strides[1] // it),
            _ptr(visual), C.c_int64(_row_major(visual)), C.c_int(_dtype_code(visual)), C.c_int(d), C.c_int(n),
            C.c_int(B), _ptr(so), _ptr(vb), _ptr(vc), _ptr(vo), C.c_double(M), _ptr(mean), _ptr(first), _ptr(kept),
            _ptr(kso), C.c_int(nthreads))
    if rc != 0:
        raise RuntimeError("sharpv_oracle_kv_discard_layers failed")
    return dict(mean_cos=mean, first_discard=first, kept_pos=[kept[i, :kso[i, -1]].copy() for i in range(n)],
                kept_seq_offsets=kso[:n])


def kv_compact_rope(kv_src: np.ndarray, kept_pos, kept_seq_offsets, seq_offsets, rotary_dim: int, base: float,
                    layer_begin: int = 0, layer_end: Optional[int] = None) -> np.ndarray:
    """Compaction with rotary re-encoding of the keys.  Returns float64 [L', 2, H, n_kept, D_h]."""
    assert kv_src.ndim == 5 and kv_src.strides[4] == kv_src.itemsize
    kp = np.ascontiguousarray(kept_pos, dtype=np.int32)
    kso = np.ascontiguousarray(kept_seq_offsets, dtype=np.int32)
    so = np.ascontiguousarray(seq_offsets, dtype=np.int32)
    L, _, H, T, Dh = kv_src.shape
    if layer_end is None:
        layer_end = L
    n = int(kso[-1])
    out = np.empty((layer_end - layer_begin, 2, H, n, Dh), np.float64)
    it = kv_src.itemsize
    st = [x // it for x in kv_src.strides]
    fn = lib().sharpv_oracle_kv_compact_rope
    fn.restype = C.c_int
    rc = fn(_ptr(kv_src), C.c_int(_dtype_code(kv_src)), C.c_int(H), C.c_int(Dh), C.c_int64(st[0]), C.c_int64(st[1]),
            C.c_int64(st[2]), C.c_int64(st[3]), C.c_int(layer_begin), C.c_int(layer_end), _ptr(kp), _ptr(kso),
            _ptr(so), C.c_int(so.size - 1), C.c_int(rotary_dim), C.c_double(base), _ptr(out))
    if rc != 0:
        raise RuntimeError("sharpv_oracle_kv_compact_rope failed")
    return out
