"""Host-side behaviour of the C ABI: exported symbols, argument validation,
workspace sizing.  No kernel is launched; runs without a GPU."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import paper_2604_05438_b200 as T
from paper_2604_05438_b200 import binding as B
from paper_2604_05438_b200.build import build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_library()
    return T.load_library()


def test_header_symbols_are_exported(lib):
    text = open(os.path.join(ROOT, "include", "tkphi.h")).read()
    declared = set(re.findall(r"\b(tkphi_[a-z_]+)\s*\(", text))
    declared -= {"tkphi_status"}
    assert declared == set(T.EXPORTED_SYMBOLS), declared ^ set(T.EXPORTED_SYMBOLS)
    for name in declared:
        assert hasattr(lib, name), name
    assert lib.tkphi_version() >= 100


def _desc(cu, n_q=8, n_kv=2, d=64, r=64, n_sink=4, n_tail=8, k=0x1000, v=0x2000, sh=None, st=None):
    cu = np.asarray(cu, np.int64)
    d_ = B._KvDesc(len(cu) - 1, n_q, n_kv, d, r, n_sink, n_tail, cu.ctypes.data, 0x3000, k, v,
                   (int(cu[-1]) * d) if sh is None else sh, d if st is None else st)
    return d_, cu


def _decode(lib, desc, topk, topk_max=None, q=0x4000, y=0x5000, ws=0x10000, ws_bytes=1 << 40):
    topk = np.asarray(topk, np.int32)
    tmax = int(topk.max()) if topk_max is None else topk_max
    return lib.tkphi_topk_decode(C.byref(desc), q, topk.ctypes.data, 0x6000, tmax, None, y, ws, ws_bytes, None)


def test_invalid_arguments_are_rejected_before_any_launch(lib):
    d, cu = _desc([0, 100, 300])
    assert _decode(lib, d, [5, 500]) == -1 and b"topk[1]" in lib.tkphi_last_error()
    assert _decode(lib, d, [5, -1]) == -1
    assert _decode(lib, d, [5, 6], topk_max=5) == -1
    assert _decode(lib, d, [5, 6], q=0) == -1
    assert _decode(lib, d, [5, 6], q=0x4001) == -1
    assert _decode(lib, d, [5, 6], y=0) == -1
    assert _decode(lib, d, [5, 6], ws=0) == -3
    assert _decode(lib, d, [5, 6], ws=0x10010) == -3
    assert _decode(lib, d, [5, 6], ws_bytes=64) == -3 and b"needed" in lib.tkphi_last_error()
    for bad in (dict(d=96), dict(r=32)):
        dd, _c = _desc([0, 100], **bad)
        assert _decode(lib, dd, [1]) == -2
    for bad in (dict(n_q=7), dict(n_sink=-1), dict(k=0), dict(k=0x1008), dict(st=60), dict(st=68)):
        dd, _c = _desc([0, 100], **bad)
        assert _decode(lib, dd, [1]) == -1, bad
    # KV heads that share memory: a zero head stride, a head stride shorter than a head's rows
    # (head-major) with a token stride too short to hold every head (token-major)
    for bad in (dict(sh=0), dict(sh=64 * 50), dict(sh=64, st=64), dict(sh=32, st=128)):
        dd, _c = _desc([0, 100], **bad)
        assert _decode(lib, dd, [1]) == -1 and b"overlap" in lib.tkphi_last_error(), bad
    for good in (dict(sh=64 * 100), dict(sh=64 * 100 + 8), dict(sh=64, st=128), dict(sh=72, st=144)):
        dd, _c = _desc([0, 100], **good)
        assert _decode(lib, dd, [1], ws=0) == -3, good       # passes validation, stops at the NULL workspace
    dd, _c = _desc([0, 100], n_q=4, n_kv=1, sh=0)
    assert _decode(lib, dd, [1], ws=0) == -3                 # one head: its stride is never used
    dd, _c = _desc([0, 100], n_q=18, n_kv=2)
    assert _decode(lib, dd, [1]) == -2                       # group of 9
    dd, _c = _desc([0, 100, 100])
    assert _decode(lib, dd, [1, 0]) == -1                    # empty sequence
    dd, _c = _desc([1, 100])
    assert _decode(lib, dd, [1]) == -1
    dd, _c = _desc([0, 100], n_sink=0, n_tail=0)
    assert _decode(lib, dd, [0]) == -1 and b"empty exact support" in lib.tkphi_last_error()
    dd, _c = _desc([0, 2097152 + 4 + 8 + 1])
    assert _decode(lib, dd, [10]) == -2 and b"2097152" in lib.tkphi_last_error()          # one mid key too many
    dd, _c = _desc([0, 2097152 + 4 + 8])
    assert _decode(lib, dd, [10], ws=0) == -3
    # per-sequence tail counts: both pointers or neither, no negative entry; they replace n_tail in every bound
    tails = np.array([8, 90], np.int32)
    dd, _c = _desc([0, 100, 300])
    dd.n_tail_seq_host = tails.ctypes.data
    assert _decode(lib, dd, [5, 6]) == -1 and b"n_tail_seq" in lib.tkphi_last_error()
    dd.n_tail_seq_dev = 0x7000
    assert _decode(lib, dd, [5, 6], ws=0) == -3
    assert _decode(lib, dd, [89, 6]) == -1 and b"topk[0]" in lib.tkphi_last_error()      # |M_0| = 100 - 4 - 8 = 88
    assert _decode(lib, dd, [88, 107]) == -1 and b"topk[1]" in lib.tkphi_last_error()    # |M_1| = 200 - 4 - 90 = 106
    assert _decode(lib, dd, [88, 106], ws=0) == -3
    tails[1] = -1
    assert _decode(lib, dd, [5, 6]) == -1
    assert lib.tkphi_topk_decode(None, 0x4000, None, None, 0, None, 0x5000, 0x10000, 1 << 30, None) == -1


def test_decode_step_and_build_validation(lib):
    d, cu = _desc([0, 400])
    topk = np.array([3], np.int32)
    ph = B._PhiDesc(0x100, 0x200, 0x300, 0x400, 0.5, 0.5, None)
    args = lambda **kw: (C.byref(d), C.byref(kw.get("ph", ph)), 0x4000, topk.ctypes.data, 0x6000, 3,
                         kw.get("S", 0x7000), 0x8000, None, 0x5000, None, kw.get("flags", 0),
                         kw.get("ws", 0x10000), kw.get("wsb", 1 << 40), None)
    assert lib.tkphi_decode_step(*args(S=0)) == -1
    assert lib.tkphi_decode_step(*args(flags=8)) == -1
    assert lib.tkphi_decode_step(*args(ph=B._PhiDesc(0, 0x200, 0x300, 0x400, 0.5, 0.5, None))) == -1
    assert lib.tkphi_decode_step(*args(ph=B._PhiDesc(0x100, 0x200, 0x300, 0x400, float("nan"), 0.5, None))) == -1
    assert lib.tkphi_decode_step(*args(ph=B._PhiDesc(0x100, 0x200, 0x300, 0x400, 0.5, 0.5, 0x9008))) == -1   # misaligned cache
    assert lib.tkphi_decode_step(*args(wsb=1000)) == -3
    assert lib.tkphi_build_summaries(C.byref(d), C.byref(ph), 0, 0x8000, 0x10000, 1 << 40, None) == -1
    assert lib.tkphi_build_summaries(C.byref(d), None, 0x7000, 0x8000, 0x10000, 1 << 40, None) == -1
    assert lib.tkphi_build_summaries(C.byref(d), C.byref(ph), 0x7000, 0x8000, 0x10000, 16, None) == -3
    assert lib.tkphi_device_status(None, None, None) == -1


def test_mlp_entry_points_validate_their_arguments(lib):
    d, cu = _desc([0, 400])
    topk = np.array([3], np.int32)
    mk = lambda **kw: B._MlpDesc(kw.get("E", 512), kw.get("H", 2), *[kw.get("p%d" % i, 0x100 * (i + 1)) for i in range(9)])
    feats = lambda m, cache=0x9000, ws=0x10000, wsb=1 << 40: lib.tkphi_mlp_key_features(
        C.byref(d), C.byref(m) if m is not None else None, cache, ws, wsb, None)
    assert feats(None) == -1
    assert feats(mk(E=96)) == -2 and feats(mk(E=640)) == -2          # hidden width: 128, 256, 384, 512
    assert feats(mk(H=8)) == -1 and b"n_heads" in lib.tkphi_last_error()   # key side: one map per KV head
    assert feats(mk(p3=0)) == -1 and feats(mk(p7=0x808)) == -1
    assert feats(mk(), cache=0) == -1 and feats(mk(), cache=0x9004) == -1
    assert feats(mk(), ws=0) == -3 and feats(mk(), wsb=4096) == -3
    assert lib.tkphi_workspace_bytes(C.byref(d), None, 0, T.WS_MLP_KEY_FEATURES) > 3 * 2 * 400 * 512 * 2
    # summary build from cached rows
    assert lib.tkphi_build_summaries_cached(C.byref(d), 0, 0x7000, 0x8000, 0x10000, 1 << 40, None) == -1
    assert lib.tkphi_build_summaries_cached(C.byref(d), 0x9004, 0x7000, 0x8000, 0x10000, 1 << 40, None) == -1
    assert lib.tkphi_build_summaries_cached(C.byref(d), 0x9000, 0, 0x8000, 0x10000, 1 << 40, None) == -1
    assert lib.tkphi_build_summaries_cached(C.byref(d), 0x9000, 0x7000, 0x8000, 0x10000, 16, None) == -3
    # decode step with the MLP on the query side: one map per query head; the cache may be NULL only with NOSUB
    step = lambda m, cache=0x9000, flags=0, wsb=1 << 40: lib.tkphi_decode_step_mlp(
        C.byref(d), C.byref(m), cache, 0x4000, topk.ctypes.data, 0x6000, 3, 0x7000, 0x8000, None, 0x5000, None,
        flags, 0x10000, wsb, None)
    assert step(mk(H=2)) == -1
    assert step(mk(H=8), cache=0) == -1 and b"phi_k_cache" in lib.tkphi_last_error()
    assert step(mk(H=8), cache=0, flags=1, wsb=1000) == -3           # passes validation without a cache
    assert step(mk(H=8), wsb=1000) == -3
    assert step(mk(H=8, E=100)) == -2


def test_workspace_sizes_scale_with_the_problem(lib):
    d1, c1 = _desc([0, 4096], n_q=32, n_kv=8)
    d2, c2 = _desc([0, 8192], n_q=32, n_kv=8)
    t = np.array([40], np.int32)
    a = lib.tkphi_workspace_bytes(C.byref(d1), t.ctypes.data, 40, T.WS_DECODE_STEP)
    b = lib.tkphi_workspace_bytes(C.byref(d2), t.ctypes.data, 40, T.WS_DECODE_STEP)
    assert 0 < a < b and a % 256 == 0
    # the fp32 score rows (4 B per query head and token) dominate the growth
    assert abs((b - a) - 4096 * 32 * 4) < 64 * 1024
    assert lib.tkphi_workspace_bytes(C.byref(d1), None, 0, T.WS_BUILD) > 0
    assert lib.tkphi_workspace_bytes(C.byref(d1), None, 40, T.WS_DECODE_STEP) == 0     # topk_host required
    assert lib.tkphi_workspace_bytes(C.byref(d1), t.ctypes.data, 40, 9) == 0
    # the 128K-context layer of the headline workload needs well under 100 MB
    d3, c3 = _desc([0, 131072], n_q=24, n_kv=8, d=128, r=128, n_tail=128)
    t3 = np.array([1309], np.int32)
    assert lib.tkphi_workspace_bytes(C.byref(d3), t3.ctypes.data, 1309, T.WS_DECODE_STEP) < 100e6


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "_LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        B.load_library()
