"""Thin Python binding of ``libsharpv.so`` (declared in ``include/sharpv.h``).

Argument marshalling only: every function here checks tensor placement, allocates the
outputs and workspace the caller did not pass (with torch, which is used for device memory
and streams, nothing else) and calls the C entry point of the same name.  All arithmetic
runs in the CUDA kernels of the library.  There is no fallback: if the shared library is
missing or cannot be loaded, the first call raises.
"""
from __future__ import annotations

import ctypes as C
import enum
import os
from typing import Dict, Optional

import torch

from . import build as _build

# ------------------------------------------------------------------------------- enums
class Status(enum.IntEnum):
    OK = 0
    ERR_INVALID_ARG = 1
    ERR_UNSUPPORTED = 2
    ERR_WORKSPACE = 3
    ERR_CAPACITY = 4
    ERR_CUDA = 5
    ERR_TIMEOUT = 6
    ERR_BOUNDS = 7


F32, BF16, U8 = 0, 1, 2
ROUND_FLOOR, ROUND_NEAREST, ROUND_CEIL = 0, 1, 2
DISSIM, ONE_MINUS_COS = 0, 1
PRUNE_PER_TOKEN, PRUNE_PER_LAYER = 0, 1


class SharpVError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = Status(status)
        msg = lib().sharpv_status_string(int(status)).decode()
        super().__init__(f"{fn}: {self.status.name} ({msg})")


class KVLayout(C.Structure):
    _fields_ = [("num_layers", C.c_int32), ("num_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("dtype", C.c_int32), ("stride_layer", C.c_int64), ("stride_kv", C.c_int64),
                ("stride_head", C.c_int64), ("stride_token", C.c_int64)]


# ------------------------------------------------------------------------------- loading
_lib = None

EXPORTS = (
    "sharpv_version", "sharpv_status_string",
    "sharpv_score_frames_workspace_bytes", "sharpv_score_frames",
    "sharpv_select_tokens_workspace_bytes", "sharpv_select_tokens", "sharpv_select_tokens_threshold",
    "sharpv_prune_frames_workspace_bytes", "sharpv_prune_frames",
    "sharpv_kv_calibrate_prune_workspace_bytes", "sharpv_kv_calibrate_prune",
    "sharpv_kv_calibrate_prune_noalloc",
    "sharpv_kv_prune_layers_workspace_bytes", "sharpv_kv_prune_layers", "sharpv_kv_compact",
    "sharpv_kv_compact_rope_workspace_bytes", "sharpv_kv_compact_rope",
)

NOALLOC_MAX_SEQ_TOKENS = 262144


def lib_path() -> str:
    """The library to load: libsharpv.so next to this file, or the file SHARPV_LIBRARY names (used to run the
    tests against the range-checking debug build, libsharpv_debug.so)."""
    return os.environ.get("SHARPV_LIBRARY") or _build.LIB_PATH


def lib():
    """Loads libsharpv.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_2511_08003_b200.build` "
                           "(there is no CPU or PyTorch fallback)")
    L = C.CDLL(path)
    vp, i32, i64, f32, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_size_t
    L.sharpv_version.restype = C.c_int
    L.sharpv_status_string.restype = C.c_char_p
    L.sharpv_status_string.argtypes = [C.c_int]
    L.sharpv_score_frames_workspace_bytes.restype = sz
    L.sharpv_score_frames_workspace_bytes.argtypes = [i32, i32, i32]
    L.sharpv_score_frames.restype = C.c_int
    L.sharpv_score_frames.argtypes = [vp, C.c_int, i64, i32, vp, i32, i32, i32, f32, C.c_int, C.c_int, i32,
                                      vp, vp, vp, vp, vp, vp, sz, vp, vp]
    L.sharpv_select_tokens_workspace_bytes.restype = sz
    L.sharpv_select_tokens_workspace_bytes.argtypes = [i32, i32]
    L.sharpv_select_tokens.restype = C.c_int
    L.sharpv_select_tokens.argtypes = [vp, vp, i32, i32, vp, C.c_int, i64, i32, vp, vp, vp, i64, vp, vp, sz, vp, vp]
    L.sharpv_select_tokens_threshold.restype = C.c_int
    L.sharpv_select_tokens_threshold.argtypes = [vp, f32, i32, i32, vp, C.c_int, i64, i32, vp, vp, vp, i64, vp,
                                                 vp, sz, vp, vp]
    L.sharpv_prune_frames_workspace_bytes.restype = sz
    L.sharpv_prune_frames_workspace_bytes.argtypes = [i32, i32, i32]
    L.sharpv_prune_frames.restype = C.c_int
    L.sharpv_prune_frames.argtypes = [vp, C.c_int, i64, i32, vp, i32, i32, i32, f32, C.c_int, C.c_int, i32,
                                      vp, vp, vp, vp, vp, vp, vp, vp, i64, vp, vp, sz, vp, vp]
    L.sharpv_kv_calibrate_prune_workspace_bytes.restype = sz
    L.sharpv_kv_calibrate_prune_workspace_bytes.argtypes = [i64, i32]
    L.sharpv_kv_calibrate_prune.restype = C.c_int
    L.sharpv_kv_calibrate_prune.argtypes = [vp, i64, vp, i64, C.c_int, i32, i32, vp, vp, vp, vp, i64, i64, f32,
                                            vp, vp, vp, vp, i64, vp, sz, vp, vp]
    L.sharpv_kv_calibrate_prune_noalloc.restype = C.c_int
    L.sharpv_kv_calibrate_prune_noalloc.argtypes = [vp, i64, vp, i64, C.c_int, i32, i32, vp, vp, vp, vp, i64, i64,
                                                    f32, vp, vp, vp, vp, i64, vp, vp]
    L.sharpv_kv_prune_layers.restype = C.c_int
    L.sharpv_kv_prune_layers_workspace_bytes.restype = sz
    L.sharpv_kv_prune_layers_workspace_bytes.argtypes = [i64, i32, i32]
    L.sharpv_kv_prune_layers.argtypes = [vp, i64, i64, vp, i64, C.c_int, i32, i32, vp, vp, vp, vp, i64, i64, f32,
                                         C.c_int, vp, vp, vp, vp, vp, i64, vp, C.POINTER(KVLayout), vp,
                                         C.POINTER(KVLayout), i32, i32, vp, sz, vp, vp]
    L.sharpv_kv_compact.restype = C.c_int
    L.sharpv_kv_compact.argtypes = [vp, C.POINTER(KVLayout), vp, C.POINTER(KVLayout), i32, i32, vp, vp, i32, i64,
                                    vp, vp]
    L.sharpv_kv_compact_rope_workspace_bytes.restype = sz
    L.sharpv_kv_compact_rope_workspace_bytes.argtypes = [i64, i32]
    L.sharpv_kv_compact_rope.restype = C.c_int
    L.sharpv_kv_compact_rope.argtypes = [vp, C.POINTER(KVLayout), vp, C.POINTER(KVLayout), i32, i32, vp, vp, vp, i32,
                                         i64, i32, C.c_double, vp, sz, vp, vp]
    _lib = L
    return L


# ------------------------------------------------------------------------------- helpers
def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}: float32 or bfloat16 expected")


def _dev(t: Optional[torch.Tensor], name: str, dtype=None):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}")
    return t.data_ptr()


def _rows(t: torch.Tensor, name: str) -> int:
    if t.dim() != 2 or t.stride(1) != 1:
        raise ValueError(f"{name} must be 2-D with a contiguous last axis")
    return t.stride(0)


def _stream(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def _check(fn: str, rc: int):
    if rc != 0:
        raise SharpVError(fn, rc)


def _call(name: str, on: torch.Tensor, *args) -> int:
    """Calls the entry point `name` with the device of `on` current: kernels are launched on the current
    device, and the allocation-free entry point keys its built-in scratch on it."""
    with torch.cuda.device(on.device):
        return getattr(lib(), name)(*args)


def _workspace(ws: Optional[torch.Tensor], nbytes: int, device) -> torch.Tensor:
    if ws is None:
        return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)
    if not ws.is_cuda or ws.dtype != torch.uint8 or not ws.is_contiguous():
        raise ValueError("workspace must be a contiguous CUDA uint8 tensor")
    return ws


def kv_layout(kv: torch.Tensor) -> KVLayout:
    """Layout struct of a 5-D view [L, 2, H, T, D_h] (any strides, contiguous last axis).  One-byte
    caches (uint8 / int8 / fp8 tensors) are described as U8: compaction only copies bits."""
    if kv.dim() != 5 or kv.shape[1] != 2 or kv.stride(4) != 1:
        raise ValueError("K/V cache must be a [L, 2, H, T, D_h] view with a contiguous last axis")
    code = U8 if kv.element_size() == 1 else _dtype_code(kv)
    return KVLayout(kv.shape[0], kv.shape[2], kv.shape[4], code,
                    kv.stride(0), kv.stride(1), kv.stride(2), kv.stride(3))


# ------------------------------------------------------------------------------- entry points
def sharpv_score_frames_workspace_bytes(total_frames: int, f: int, d: int) -> int:
    return int(lib().sharpv_score_frames_workspace_bytes(total_frames, f, d))


def sharpv_score_frames(tokens: torch.Tensor, video_frame_offsets: torch.Tensor, total_frames: int, f: int,
                        w: float = 1.0, dissim_kind: int = DISSIM, round_mode: int = ROUND_FLOOR,
                        min_keep: int = 0, want_spatial: bool = False, want_temporal: bool = False,
                        out: Optional[Dict[str, torch.Tensor]] = None,
                        workspace: Optional[torch.Tensor] = None,
                        status_word: Optional[torch.Tensor] = None, stream=None) -> Dict[str, torch.Tensor]:
    """Scores and budgets of stage one.  Returns dict(importance, ratio, k[, spatial, temporal])."""
    ld = _rows(tokens, "tokens")
    d = tokens.shape[1]
    dev = tokens.device
    out = dict(out) if out else {}
    n = total_frames * f
    if "importance" not in out:
        out["importance"] = torch.empty(n, dtype=torch.float32, device=dev)
    if "ratio" not in out:
        out["ratio"] = torch.empty(total_frames, dtype=torch.float32, device=dev)
    if "k" not in out:
        out["k"] = torch.empty(total_frames, dtype=torch.int32, device=dev)
    if want_spatial and "spatial" not in out:
        out["spatial"] = torch.empty(n, dtype=torch.float32, device=dev)
    if want_temporal and "temporal" not in out:
        out["temporal"] = torch.empty(n, dtype=torch.float32, device=dev)
    nbytes = sharpv_score_frames_workspace_bytes(total_frames, f, d)
    ws = _workspace(workspace, nbytes, dev)
    rc = _call("sharpv_score_frames", tokens,
        _dev(tokens, "tokens"), _dtype_code(tokens), ld, video_frame_offsets.numel() - 1,
        _dev(video_frame_offsets, "video_frame_offsets", torch.int32), total_frames, f, d, float(w),
        int(dissim_kind), int(round_mode), int(min_keep),
        _dev(out["importance"], "importance", torch.float32), _dev(out.get("spatial"), "spatial", torch.float32),
        _dev(out.get("temporal"), "temporal", torch.float32), _dev(out["ratio"], "ratio", torch.float32),
        _dev(out["k"], "k", torch.int32), ws.data_ptr(), ws.numel(),
        _dev(status_word, "status_word", torch.int32), _stream(stream))
    _check("sharpv_score_frames", rc)
    return out


def sharpv_select_tokens_workspace_bytes(total_frames: int, f: int) -> int:
    return int(lib().sharpv_select_tokens_workspace_bytes(total_frames, f))


def _select(fn_name, importance, k, K, total_frames, f, tokens, capacity, gather, out, workspace,
            status_word, stream):
    dev = importance.device
    out = dict(out) if out else {}
    if capacity is None:
        capacity = total_frames * f
    if "kept_index" not in out:
        out["kept_index"] = torch.empty(max(capacity, 1), dtype=torch.int32, device=dev)
    if "kept_offsets" not in out:
        out["kept_offsets"] = torch.empty(total_frames + 1, dtype=torch.int32, device=dev)
    if "num_kept" not in out:
        out["num_kept"] = torch.empty(1, dtype=torch.int32, device=dev)
    tok_ptr, tok_dt, ld, d, out_tok_ptr = None, 0, 0, 0, None
    if gather:
        if tokens is None:
            raise ValueError("gather=True needs tokens")
        ld, d, tok_dt = _rows(tokens, "tokens"), tokens.shape[1], _dtype_code(tokens)
        if "tokens" not in out:
            out["tokens"] = torch.empty((max(capacity, 1), d), dtype=tokens.dtype, device=dev)
        tok_ptr, out_tok_ptr = _dev(tokens, "tokens"), _dev(out["tokens"], "out tokens")
    ws = _workspace(workspace, sharpv_select_tokens_workspace_bytes(total_frames, f), dev)
    common = (total_frames, f, tok_ptr, tok_dt, ld, d, _dev(out["kept_index"], "kept_index", torch.int32),
              _dev(out["kept_offsets"], "kept_offsets", torch.int32), out_tok_ptr, capacity,
              _dev(out["num_kept"], "num_kept", torch.int32), ws.data_ptr(), ws.numel(),
              _dev(status_word, "status_word", torch.int32), _stream(stream))
    if fn_name == "sharpv_select_tokens":
        rc = _call("sharpv_select_tokens", importance, _dev(importance, "importance", torch.float32),
                   _dev(k, "k", torch.int32), *common)
    else:
        rc = _call("sharpv_select_tokens_threshold", importance, _dev(importance, "importance", torch.float32),
                   float(K), *common)
    _check(fn_name, rc)
    return out


def sharpv_select_tokens(importance: torch.Tensor, k: torch.Tensor, total_frames: int, f: int,
                         tokens: Optional[torch.Tensor] = None, capacity: Optional[int] = None,
                         gather: bool = True, out=None, workspace=None, status_word=None, stream=None):
    """Per-frame top-k and gather.  Returns dict(kept_index, kept_offsets, num_kept[, tokens])."""
    return _select("sharpv_select_tokens", importance, k, 0.0, total_frames, f, tokens, capacity,
                   gather and tokens is not None, out, workspace, status_word, stream)


def sharpv_select_tokens_threshold(importance: torch.Tensor, K: float, total_frames: int, f: int,
                                   tokens: Optional[torch.Tensor] = None, capacity: Optional[int] = None,
                                   gather: bool = True, out=None, workspace=None, status_word=None, stream=None):
    """Manual variant: keep importance > K.  Same outputs as sharpv_select_tokens."""
    return _select("sharpv_select_tokens_threshold", importance, None, K, total_frames, f, tokens, capacity,
                   gather and tokens is not None, out, workspace, status_word, stream)


def sharpv_prune_frames_workspace_bytes(total_frames: int, f: int, d: int) -> int:
    return int(lib().sharpv_prune_frames_workspace_bytes(total_frames, f, d))


def sharpv_prune_frames(tokens: torch.Tensor, video_frame_offsets: torch.Tensor, total_frames: int, f: int,
                        w: float = 1.0, dissim_kind: int = DISSIM, round_mode: int = ROUND_FLOOR,
                        min_keep: int = 0, want_spatial: bool = False, want_temporal: bool = False,
                        capacity: Optional[int] = None, gather: bool = True,
                        out: Optional[Dict[str, torch.Tensor]] = None, workspace: Optional[torch.Tensor] = None,
                        status_word: Optional[torch.Tensor] = None, stream=None) -> Dict[str, torch.Tensor]:
    """Stage one in one call: the outputs of sharpv_score_frames and of sharpv_select_tokens run on its
    budgets.  Returns dict(importance, ratio, k, kept_index, kept_offsets, num_kept[, tokens, spatial,
    temporal])."""
    ld = _rows(tokens, "tokens")
    d = tokens.shape[1]
    dev = tokens.device
    out = dict(out) if out else {}
    n = total_frames * f
    if capacity is None:
        capacity = n
    new = lambda shape, dt: torch.empty(shape, dtype=dt, device=dev)
    out.setdefault("importance", new(n, torch.float32))
    out.setdefault("ratio", new(total_frames, torch.float32))
    out.setdefault("k", new(total_frames, torch.int32))
    if want_spatial:
        out.setdefault("spatial", new(n, torch.float32))
    if want_temporal:
        out.setdefault("temporal", new(n, torch.float32))
    out.setdefault("kept_index", new(max(capacity, 1), torch.int32))
    out.setdefault("kept_offsets", new(total_frames + 1, torch.int32))
    out.setdefault("num_kept", new(1, torch.int32))
    if gather:
        out.setdefault("tokens", new((max(capacity, 1), d), tokens.dtype))
    ws = _workspace(workspace, sharpv_prune_frames_workspace_bytes(total_frames, f, d), dev)
    rc = _call("sharpv_prune_frames", tokens,
               _dev(tokens, "tokens"), _dtype_code(tokens), ld, video_frame_offsets.numel() - 1,
               _dev(video_frame_offsets, "video_frame_offsets", torch.int32), total_frames, f, d, float(w),
               int(dissim_kind), int(round_mode), int(min_keep),
               _dev(out["importance"], "importance", torch.float32), _dev(out.get("spatial"), "spatial", torch.float32),
               _dev(out.get("temporal"), "temporal", torch.float32), _dev(out["ratio"], "ratio", torch.float32),
               _dev(out["k"], "k", torch.int32), _dev(out["kept_index"], "kept_index", torch.int32),
               _dev(out["kept_offsets"], "kept_offsets", torch.int32),
               _dev(out.get("tokens"), "out tokens") if gather else None, capacity,
               _dev(out["num_kept"], "num_kept", torch.int32), ws.data_ptr(), ws.numel(),
               _dev(status_word, "status_word", torch.int32), _stream(stream))
    _check("sharpv_prune_frames", rc)
    return out


def sharpv_kv_calibrate_prune_workspace_bytes(total_seq_tokens: int, num_seqs: int) -> int:
    return int(lib().sharpv_kv_calibrate_prune_workspace_bytes(total_seq_tokens, num_seqs))


def _calibrate(fn_name, hidden, visual, seq_offsets, vis_begin, vis_count, vis_offsets, total_seq_tokens, M,
               capacity, want_mean_cos, out, workspace, status_word, stream):
    ldh, ldv = _rows(hidden, "hidden"), _rows(visual, "visual")
    if hidden.dtype != visual.dtype or hidden.shape[1] != visual.shape[1]:
        raise ValueError("hidden and visual must share dtype and feature size")
    dev = hidden.device
    B = seq_offsets.numel() - 1
    total_visual = visual.shape[0]
    out = dict(out) if out else {}
    if capacity is None:
        capacity = total_seq_tokens
    if "cos" not in out:
        out["cos"] = torch.empty(max(total_visual, 1), dtype=torch.float32, device=dev)
    if "kept_pos" not in out:
        out["kept_pos"] = torch.empty(max(capacity, 1), dtype=torch.int32, device=dev)
    if "kept_seq_offsets" not in out:
        out["kept_seq_offsets"] = torch.empty(B + 1, dtype=torch.int32, device=dev)
    if want_mean_cos and "mean_cos" not in out:
        out["mean_cos"] = torch.empty(B, dtype=torch.float32, device=dev)
    head = (_dev(hidden, "hidden"), ldh, _dev(visual, "visual"), ldv, _dtype_code(hidden), hidden.shape[1], B,
            _dev(seq_offsets, "seq_offsets", torch.int32), _dev(vis_begin, "vis_begin", torch.int32),
            _dev(vis_count, "vis_count", torch.int32), _dev(vis_offsets, "vis_offsets", torch.int32),
            total_seq_tokens, total_visual, float(M), _dev(out["cos"], "cos", torch.float32),
            _dev(out.get("mean_cos"), "mean_cos", torch.float32), _dev(out["kept_pos"], "kept_pos", torch.int32),
            _dev(out["kept_seq_offsets"], "kept_seq_offsets", torch.int32), capacity)
    tail = (_dev(status_word, "status_word", torch.int32), _stream(stream))
    if fn_name == "sharpv_kv_calibrate_prune":
        ws = _workspace(workspace, sharpv_kv_calibrate_prune_workspace_bytes(total_seq_tokens, B), dev)
        rc = _call("sharpv_kv_calibrate_prune", hidden, *head, ws.data_ptr(), ws.numel(), *tail)
    else:
        rc = _call("sharpv_kv_calibrate_prune_noalloc", hidden, *head, *tail)
    _check(fn_name, rc)
    return out


def sharpv_kv_calibrate_prune(hidden: torch.Tensor, visual: torch.Tensor, seq_offsets: torch.Tensor,
                              vis_begin: torch.Tensor, vis_count: torch.Tensor, vis_offsets: torch.Tensor,
                              total_seq_tokens: int, M: float = 0.2, capacity: Optional[int] = None,
                              want_mean_cos: bool = False, out=None, workspace=None, status_word=None,
                              stream=None):
    """Self-calibration of stage two.  Returns dict(cos, kept_pos, kept_seq_offsets[, mean_cos])."""
    return _calibrate("sharpv_kv_calibrate_prune", hidden, visual, seq_offsets, vis_begin, vis_count, vis_offsets,
                      total_seq_tokens, M, capacity, want_mean_cos, out, workspace, status_word, stream)


def sharpv_kv_calibrate_prune_noalloc(hidden: torch.Tensor, visual: torch.Tensor, seq_offsets: torch.Tensor,
                                      vis_begin: torch.Tensor, vis_count: torch.Tensor,
                                      vis_offsets: torch.Tensor, total_seq_tokens: int, M: float = 0.2,
                                      capacity: Optional[int] = None, want_mean_cos: bool = False, out=None,
                                      status_word=None, stream=None):
    """Same operation and outputs as sharpv_kv_calibrate_prune for hosts that cannot supply scratch
    memory: the library's built-in scratch array is used (at most NOALLOC_MAX_SEQ_TOKENS packed positions).
    The library call itself allocates nothing; pass every output in `out` if this wrapper must not
    allocate either.  Calls on one device share the scratch and must not overlap on the GPU."""
    return _calibrate("sharpv_kv_calibrate_prune_noalloc", hidden, visual, seq_offsets, vis_begin, vis_count,
                      vis_offsets, total_seq_tokens, M, capacity, want_mean_cos, out, None, status_word, stream)


def sharpv_kv_compact(kv_src: torch.Tensor, kv_dst: torch.Tensor, kept_pos: torch.Tensor,
                      kept_seq_offsets: torch.Tensor, capacity: int, layer_begin: int = 0,
                      layer_end: Optional[int] = None, status_word=None, stream=None) -> torch.Tensor:
    """Compacts every (layer, K|V, head) plane of kv_src [L,2,H,T,D_h] into kv_dst (same view shape,
    its own strides and token capacity).  Returns kv_dst."""
    sl, dl = kv_layout(kv_src), kv_layout(kv_dst)
    if layer_end is None:
        layer_end = kv_src.shape[0]
    rc = _call("sharpv_kv_compact", kv_src,
        _dev(kv_src, "kv_src"), C.byref(sl), _dev(kv_dst, "kv_dst"), C.byref(dl), layer_begin, layer_end,
        _dev(kept_pos, "kept_pos", torch.int32), _dev(kept_seq_offsets, "kept_seq_offsets", torch.int32),
        kept_seq_offsets.numel() - 1, capacity, _dev(status_word, "status_word", torch.int32), _stream(stream))
    _check("sharpv_kv_compact", rc)
    return kv_dst


def sharpv_kv_prune_layers_workspace_bytes(total_seq_tokens: int, num_seqs: int, num_layers: int) -> int:
    return int(lib().sharpv_kv_prune_layers_workspace_bytes(total_seq_tokens, num_seqs, num_layers))


def sharpv_kv_prune_layers(hidden_layers: torch.Tensor, visual: torch.Tensor, seq_offsets: torch.Tensor,
                           vis_begin: torch.Tensor, vis_count: torch.Tensor, vis_offsets: torch.Tensor,
                           total_seq_tokens: int, kv_src: Optional[torch.Tensor], kv_dst: Optional[torch.Tensor],
                           M: float = 0.2, mode: int = PRUNE_PER_TOKEN, layer_begin: int = 0,
                           capacity: Optional[int] = None, want_mean_cos: bool = False, workspace=None,
                           status_word=None, stream=None, kv_layers: Optional[int] = None):
    """Stage two layer by layer.  hidden_layers [n_layers, T, d] holds the hidden states of layers
    layer_begin .. layer_begin + n_layers - 1.  Returns dict(cos [n, total_visual], kept_pos [n, capacity],
    kept_seq_offsets [n, B + 1][, mean_cos [n, B]][, first_discard [B] (per-layer reading)]); kv_dst
    receives the compacted planes.  kv_src = kv_dst = None gives the decisions only (kv_layers then says
    how many layers the model has)."""
    if hidden_layers.dim() != 3 or hidden_layers.stride(2) != 1:
        raise ValueError("hidden_layers must be [layers, tokens, d] with a contiguous last axis")
    n = hidden_layers.shape[0]
    ldv = _rows(visual, "visual")
    if hidden_layers.dtype != visual.dtype or hidden_layers.shape[2] != visual.shape[1]:
        raise ValueError("hidden_layers and visual must share dtype and feature size")
    dev = hidden_layers.device
    B = seq_offsets.numel() - 1
    total_visual = visual.shape[0]
    if capacity is None:
        capacity = total_seq_tokens
    out = {"cos": torch.empty((n, max(total_visual, 1)), dtype=torch.float32, device=dev),
           "kept_pos": torch.empty((n, max(capacity, 1)), dtype=torch.int32, device=dev),
           "kept_seq_offsets": torch.empty((n, B + 1), dtype=torch.int32, device=dev)}
    if want_mean_cos or mode == PRUNE_PER_LAYER:
        out["mean_cos"] = torch.empty((n, B), dtype=torch.float32, device=dev)
    if mode == PRUNE_PER_LAYER:
        out["first_discard"] = torch.empty(B, dtype=torch.int32, device=dev)
    if total_visual == 0 or capacity == 0:
        raise ValueError("sharpv_kv_prune_layers wrapper needs total_visual > 0 and capacity > 0")
    if (kv_src is None) != (kv_dst is None):
        raise ValueError("kv_src and kv_dst: both or none")
    if kv_src is not None:
        sl, dl = kv_layout(kv_src), kv_layout(kv_dst)
    else:
        L = kv_layers if kv_layers is not None else layer_begin + n
        sl = dl = KVLayout(L, 1, 16, _dtype_code(visual), 16, 16, 16, 16)
    ws = _workspace(workspace, sharpv_kv_prune_layers_workspace_bytes(total_seq_tokens, B, n), dev)
    rc = _call("sharpv_kv_prune_layers", hidden_layers,
        _dev(hidden_layers, "hidden_layers"), hidden_layers.stride(0), hidden_layers.stride(1),
        _dev(visual, "visual"), ldv, _dtype_code(visual), visual.shape[1], B,
        _dev(seq_offsets, "seq_offsets", torch.int32), _dev(vis_begin, "vis_begin", torch.int32),
        _dev(vis_count, "vis_count", torch.int32), _dev(vis_offsets, "vis_offsets", torch.int32),
        total_seq_tokens, total_visual, float(M), int(mode), _dev(out["cos"], "cos", torch.float32),
        _dev(out.get("mean_cos"), "mean_cos", torch.float32),
        _dev(out.get("first_discard"), "first_discard", torch.int32), _dev(out["kept_pos"], "kept_pos", torch.int32),
        _dev(out["kept_seq_offsets"], "kept_seq_offsets", torch.int32), capacity,
        _dev(kv_src, "kv_src"), C.byref(sl), _dev(kv_dst, "kv_dst"), C.byref(dl), layer_begin, layer_begin + n,
        ws.data_ptr(), ws.numel(), _dev(status_word, "status_word", torch.int32), _stream(stream))
    _check("sharpv_kv_prune_layers", rc)
    return out


def sharpv_kv_compact_rope_workspace_bytes(capacity: int, rotary_dim: int) -> int:
    return int(lib().sharpv_kv_compact_rope_workspace_bytes(capacity, rotary_dim))


def sharpv_kv_compact_rope(kv_src: torch.Tensor, kv_dst: torch.Tensor, kept_pos: torch.Tensor,
                           kept_seq_offsets: torch.Tensor, seq_offsets: torch.Tensor, capacity: int,
                           rotary_dim: int, rope_base: float, layer_begin: int = 0,
                           layer_end: Optional[int] = None, workspace=None, status_word=None,
                           stream=None) -> torch.Tensor:
    """Compaction with rotary re-encoding of the keys (values are bit copies).  Returns kv_dst."""
    sl, dl = kv_layout(kv_src), kv_layout(kv_dst)
    if layer_end is None:
        layer_end = kv_src.shape[0]
    ws = _workspace(workspace, sharpv_kv_compact_rope_workspace_bytes(capacity, rotary_dim), kv_src.device)
    rc = _call("sharpv_kv_compact_rope", kv_src,
        _dev(kv_src, "kv_src"), C.byref(sl), _dev(kv_dst, "kv_dst"), C.byref(dl), layer_begin, layer_end,
        _dev(kept_pos, "kept_pos", torch.int32), _dev(kept_seq_offsets, "kept_seq_offsets", torch.int32),
        _dev(seq_offsets, "seq_offsets", torch.int32), kept_seq_offsets.numel() - 1, capacity, int(rotary_dim),
        float(rope_base), ws.data_ptr(), ws.numel(), _dev(status_word, "status_word", torch.int32), _stream(stream))
    _check("sharpv_kv_compact_rope", rc)
    return kv_dst
