"""Host-side checks that need no GPU: the shared library builds, loads and exports every symbol
the header declares, and every entry point rejects bad arguments before it touches CUDA."""
import ctypes as C
import os
import re

import pytest

from paper_2511_08003_b200 import binding as sv
from paper_2511_08003_b200 import build as svbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    svbuild.build()
    return sv.lib()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "sharpv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sharpv_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(L):
    names = _declared_functions()
    assert len(names) >= 10
    for n in names:
        assert hasattr(L, n), f"{n} declared in sharpv.h but not exported"
    assert set(names) == set(sv.EXPORTS)
    assert L.sharpv_version() >= 100
    assert L.sharpv_status_string(0) == b"ok"
    for code in range(1, 7):
        assert L.sharpv_status_string(code) not in (b"ok", b"unknown status")


def test_workspace_queries(L):
    assert L.sharpv_score_frames_workspace_bytes(0, 196, 3584) >= 0
    a = L.sharpv_score_frames_workspace_bytes(32, 196, 3584)
    b = L.sharpv_score_frames_workspace_bytes(64, 196, 3584)
    assert 0 < a < b and a % 256 == 0
    assert L.sharpv_select_tokens_workspace_bytes(32, 196) % 256 == 0
    assert L.sharpv_kv_calibrate_prune_workspace_bytes(6336, 1) >= 6336


P = 0x10000  # a fake, 16-byte aligned, non-null address: validation fails before any dereference


def test_score_frames_rejects_bad_arguments(L):
    ok = dict(tokens=P, dtype=1, ld=3584, nv=1, vfo=P, F=4, f=196, d=3584, w=1.0, kind=0, rm=0, mk=0,
              I=P, S=None, T=None, r=P, k=P, ws=P, wsb=1 << 30, st=None, stream=None)

    def call(**kw):
        a = dict(ok, **kw)
        return L.sharpv_score_frames(a["tokens"], a["dtype"], a["ld"], a["nv"], a["vfo"], a["F"], a["f"], a["d"],
                                     a["w"], a["kind"], a["rm"], a["mk"], a["I"], a["S"], a["T"], a["r"], a["k"],
                                     a["ws"], a["wsb"], a["st"], a["stream"])

    S = sv.Status
    assert call(dtype=7) == S.ERR_UNSUPPORTED
    assert call(tokens=None) == S.ERR_INVALID_ARG
    assert call(vfo=None) == S.ERR_INVALID_ARG
    assert call(I=None) == S.ERR_INVALID_ARG
    assert call(f=0) == S.ERR_INVALID_ARG
    assert call(d=0) == S.ERR_INVALID_ARG
    assert call(nv=0) == S.ERR_INVALID_ARG
    assert call(F=-1) == S.ERR_INVALID_ARG
    assert call(ld=100) == S.ERR_INVALID_ARG            # row stride shorter than a row
    assert call(rm=5) == S.ERR_INVALID_ARG
    assert call(kind=2) == S.ERR_INVALID_ARG
    assert call(mk=-1) == S.ERR_INVALID_ARG
    assert call(d=3580, ld=3580) == S.ERR_UNSUPPORTED   # 7160-byte rows: not a multiple of 16
    assert call(tokens=P + 2) == S.ERR_UNSUPPORTED      # misaligned base
    assert call(ld=3585) == S.ERR_UNSUPPORTED           # misaligned stride
    assert call(wsb=16) == S.ERR_WORKSPACE
    assert call(F=0) == S.OK                            # empty input: nothing launched


def test_prune_frames_rejects_bad_arguments(L):
    ok = dict(tokens=P, dtype=1, ld=3584, nv=1, vfo=P, F=4, f=196, d=3584, w=1.0, kind=0, rm=0, mk=0,
              I=P, S=None, T=None, r=P, k=P, ki=P, ko=P, ot=P, cap=784, nk=P, ws=P, wsb=1 << 30, st=None, stream=None)

    def call(**kw):
        a = dict(ok, **kw)
        return L.sharpv_prune_frames(a["tokens"], a["dtype"], a["ld"], a["nv"], a["vfo"], a["F"], a["f"], a["d"],
                                     a["w"], a["kind"], a["rm"], a["mk"], a["I"], a["S"], a["T"], a["r"], a["k"],
                                     a["ki"], a["ko"], a["ot"], a["cap"], a["nk"], a["ws"], a["wsb"], a["st"],
                                     a["stream"])

    S = sv.Status
    assert L.sharpv_prune_frames_workspace_bytes(32, 196, 3584) >= (
        L.sharpv_score_frames_workspace_bytes(32, 196, 3584))
    assert call(dtype=2) == S.ERR_UNSUPPORTED
    assert call(tokens=None) == S.ERR_INVALID_ARG
    assert call(ko=None) == S.ERR_INVALID_ARG
    assert call(ki=None) == S.ERR_INVALID_ARG
    assert call(cap=-1) == S.ERR_INVALID_ARG
    assert call(f=0) == S.ERR_INVALID_ARG
    assert call(ld=100) == S.ERR_INVALID_ARG
    assert call(kind=2) == S.ERR_INVALID_ARG
    assert call(d=3, ld=3) == S.ERR_UNSUPPORTED
    assert call(ot=P + 4) == S.ERR_UNSUPPORTED
    assert call(wsb=1024) == S.ERR_WORKSPACE


def test_select_tokens_rejects_bad_arguments(L):
    def call(imp=P, k=P, F=4, f=196, tok=P, dt=1, ld=3584, d=3584, idx=P, off=P, out=P, cap=100, nk=None, ws=P,
             wsb=1 << 20, st=None):
        return L.sharpv_select_tokens(imp, k, F, f, tok, dt, ld, d, idx, off, out, cap, nk, ws, wsb, st, None)

    S = sv.Status
    assert call(imp=None) == S.ERR_INVALID_ARG
    assert call(k=None) == S.ERR_INVALID_ARG
    assert call(off=None) == S.ERR_INVALID_ARG
    assert call(idx=None) == S.ERR_INVALID_ARG
    assert call(f=0) == S.ERR_INVALID_ARG
    assert call(cap=-1) == S.ERR_INVALID_ARG
    assert call(f=8193) == S.ERR_UNSUPPORTED            # documented limit on tokens per frame
    assert call(dt=9) == S.ERR_UNSUPPORTED
    assert call(tok=None) == S.ERR_INVALID_ARG          # gather requested without a source
    assert call(out=P + 8) == S.ERR_UNSUPPORTED
    assert call(wsb=0) == S.ERR_WORKSPACE
    assert L.sharpv_select_tokens_threshold(None, 1.6, 4, 196, P, 1, 3584, 3584, P, P, P, 100, None, P, 1 << 20,
                                            None, None) == S.ERR_INVALID_ARG


def test_calibrate_rejects_bad_arguments(L):
    def call(h=P, ldh=3584, v=P, ldv=3584, dt=1, d=3584, B=1, so=P, vb=P, vc=P, vo=P, T=1000, NV=900, M=0.2,
             cos=P, mc=None, kp=P, kso=P, cap=1000, ws=P, wsb=1 << 20, st=None):
        return L.sharpv_kv_calibrate_prune(h, ldh, v, ldv, dt, d, B, so, vb, vc, vo, T, NV, M, cos, mc, kp, kso,
                                           cap, ws, wsb, st, None)

    S = sv.Status
    assert call(dt=3) == S.ERR_UNSUPPORTED
    assert call(h=None) == S.ERR_INVALID_ARG
    assert call(v=None) == S.ERR_INVALID_ARG
    assert call(so=None) == S.ERR_INVALID_ARG
    assert call(kso=None) == S.ERR_INVALID_ARG
    assert call(kp=None) == S.ERR_INVALID_ARG
    assert call(B=0) == S.ERR_INVALID_ARG
    assert call(T=-1) == S.ERR_INVALID_ARG
    assert call(ldh=8) == S.ERR_INVALID_ARG
    assert call(d=12, ldh=12, ldv=12) == S.ERR_UNSUPPORTED
    assert call(h=P + 4) == S.ERR_UNSUPPORTED
    assert call(T=1 << 31) == S.ERR_UNSUPPORTED
    assert call(wsb=8) == S.ERR_WORKSPACE


def test_kv_compact_rejects_bad_arguments(L):
    def layout(**kw):
        base = dict(num_layers=28, num_kv_heads=4, head_dim=128, dtype=1, stride_layer=2 * 4 * 1000 * 128,
                    stride_kv=4 * 1000 * 128, stride_head=1000 * 128, stride_token=128)
        base.update(kw)
        return sv.KVLayout(**base)

    FAR = P + (1 << 40)         # far beyond the end of the fake source cache

    def call(src=P, sl=None, dst=FAR, dl=None, lb=0, le=28, kp=P, kso=P, B=1, cap=1000):
        sl = layout() if sl is None else sl
        dl = layout() if dl is None else dl
        return L.sharpv_kv_compact(src, C.byref(sl), dst, C.byref(dl), lb, le, kp, kso, B, cap, None, None)

    S = sv.Status
    assert call(src=None) == S.ERR_INVALID_ARG
    assert call(dst=P, dl=layout(stride_token=256)) == S.ERR_INVALID_ARG   # in place needs identical strides
    assert call(kso=None) == S.ERR_INVALID_ARG
    assert call(kp=None) == S.ERR_INVALID_ARG
    assert call(lb=3, le=2) == S.ERR_INVALID_ARG
    assert call(le=29) == S.ERR_INVALID_ARG
    assert call(B=0) == S.ERR_INVALID_ARG
    assert call(cap=-1) == S.ERR_INVALID_ARG
    assert call(sl=layout(dtype=5)) == S.ERR_UNSUPPORTED
    assert call(sl=layout(head_dim=64)) == S.ERR_INVALID_ARG      # source and destination disagree
    assert call(sl=layout(stride_token=100)) == S.ERR_INVALID_ARG # rows would overlap
    assert call(sl=layout(head_dim=4, stride_token=4), dl=layout(head_dim=4, stride_token=4)) == S.ERR_UNSUPPORTED
    assert call(sl=layout(stride_head=1000 * 128 + 4)) == S.ERR_UNSUPPORTED
    assert call(src=P + 2) == S.ERR_UNSUPPORTED
    assert call(lb=5, le=5) == S.OK                               # empty layer range: nothing to do
    assert call(cap=0, kp=None) == S.OK
    assert L.sharpv_kv_compact(P, None, 2 * P, None, 0, 1, P, P, 1, 10, None, None) == S.ERR_INVALID_ARG
    # a destination that shares bytes with the source without being the source: rejected, nothing launched
    plane = 1000 * 128 * 2                                        # bytes of one (layer, K|V, head) plane
    assert call(dst=P + 256) == S.ERR_INVALID_ARG                 # shifted by one row
    assert call(dst=P + 3 * plane) == S.ERR_INVALID_ARG           # starts inside the source cache
    assert call(src=P + 7 * plane, dst=P, lb=0, le=1) == S.ERR_INVALID_ARG   # source starts in the destination's layer
    assert call(dst=P + 16, lb=3, le=4, cap=1) == S.ERR_INVALID_ARG          # one row, one layer: still shared bytes


def test_kv_compact_rope_rejects_bad_arguments(L):
    def layout(**kw):
        base = dict(num_layers=2, num_kv_heads=4, head_dim=128, dtype=1, stride_layer=2 * 4 * 1000 * 128,
                    stride_kv=4 * 1000 * 128, stride_head=1000 * 128, stride_token=128)
        base.update(kw)
        return sv.KVLayout(**base)

    FAR = P + (1 << 40)

    def call(src=P, sl=None, dst=FAR, dl=None, lb=0, le=2, kp=P, kso=P, so=P, B=1, cap=1000, rd=128, rb=1e6,
             ws=P, wsb=1 << 20):
        sl = layout() if sl is None else sl
        dl = layout() if dl is None else dl
        return L.sharpv_kv_compact_rope(src, C.byref(sl), dst, C.byref(dl), lb, le, kp, kso, so, B, cap, rd, rb, ws,
                                        wsb, None, None)

    S = sv.Status
    assert L.sharpv_kv_compact_rope_workspace_bytes(1000, 128) >= 1000 * 64 * 8
    assert call(so=None) == S.ERR_INVALID_ARG
    assert call(dst=P) == S.ERR_INVALID_ARG                       # out of place only
    assert call(rd=130) == S.ERR_INVALID_ARG
    assert call(rd=63) == S.ERR_INVALID_ARG                       # odd
    assert call(rb=0.0) == S.ERR_INVALID_ARG
    assert call(rd=8) == S.ERR_UNSUPPORTED                        # half a pair narrower than 16 bytes
    assert call(sl=layout(dtype=2), dl=layout(dtype=2)) == S.ERR_UNSUPPORTED     # one-byte caches cannot be rotated
    assert call(wsb=64) == S.ERR_WORKSPACE
    assert call(ws=None) == S.ERR_INVALID_ARG
    assert call(lb=1, le=1) == S.OK
    assert call(dst=P + 4096) == S.ERR_INVALID_ARG                # destination inside the source cache


def test_kv_prune_layers_rejects_bad_arguments(L):
    def layout(**kw):
        base = dict(num_layers=4, num_kv_heads=2, head_dim=64, dtype=1, stride_layer=2 * 2 * 500 * 64,
                    stride_kv=2 * 500 * 64, stride_head=500 * 64, stride_token=64)
        base.update(kw)
        return sv.KVLayout(**base)

    FAR = P + (1 << 40)

    def call(hid=P, hs=500 * 512, dtype=1, sl=None, dl=None, lb=0, le=4, B=1, cap=500, ws=P, wsb=1 << 20, kso=P,
             mode=0, fd=None):
        sl = layout() if sl is None else sl
        dl = layout() if dl is None else dl
        return L.sharpv_kv_prune_layers(hid, hs, 512, P, 512, dtype, 512, B, P, P, P, P, 500, 400, 0.2, mode, P, None,
                                        fd, P, kso, cap, P, C.byref(sl), FAR, C.byref(dl), lb, le, ws, wsb, None, None)

    S = sv.Status
    assert call(lb=2, le=2) == S.OK                               # empty layer range: nothing to do
    assert call(dtype=7) == S.ERR_UNSUPPORTED
    assert call(lb=3, le=2) == S.ERR_INVALID_ARG
    assert call(le=5) == S.ERR_INVALID_ARG                        # beyond the cache's layers
    assert call(hs=-1) == S.ERR_INVALID_ARG
    assert call(hs=500 * 512 + 4) == S.ERR_UNSUPPORTED            # layers of hidden states not 16-byte aligned
    assert call(B=0) == S.ERR_INVALID_ARG
    assert call(wsb=16) == S.ERR_WORKSPACE
    assert call(kso=None) == S.ERR_INVALID_ARG
    assert call(mode=2) == S.ERR_INVALID_ARG
    assert call(mode=0, fd=P) == S.ERR_INVALID_ARG                # the first discarded layer exists per layer only
    assert L.sharpv_kv_prune_layers_workspace_bytes(500, 1, 4) >= 4 * L.sharpv_kv_calibrate_prune_workspace_bytes(500, 1)
    assert L.sharpv_kv_prune_layers(P, 0, 512, P, 512, 1, 512, 1, P, P, P, P, 500, 400, 0.2, 0, P, None, None, P, P,
                                    500, P, None, 2 * P, None, 0, 1, P, 1 << 20, None, None) == S.ERR_INVALID_ARG


def test_binding_fails_loudly_without_library(monkeypatch, tmp_path):
    monkeypatch.setattr(sv, "_lib", None)
    monkeypatch.setattr(sv._build, "LIB_PATH", str(tmp_path / "libsharpv.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        sv.lib()
