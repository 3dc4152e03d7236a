"""ctypes binding of libtkphi.so: same names as the C entry points, marshalling only."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libtkphi.so")
_lib = None

WS_BUILD, WS_TOPK_DECODE, WS_DECODE_STEP, WS_MLP_KEY_FEATURES = 0, 1, 2, 3
FLAG_NONE, FLAG_NOSUB = 0, 1

EXPORTED_SYMBOLS = (
    "tkphi_workspace_bytes", "tkphi_build_summaries", "tkphi_topk_decode", "tkphi_decode_step",
    "tkphi_device_status", "tkphi_last_error", "tkphi_version",
    "tkphi_kernel_timing_enable", "tkphi_kernel_timing_read",
    "tkphi_build_summaries_static", "tkphi_static_last_error", "tkphi_static_device_status",
    "tkphi_selftest_timeout",
    "tkphi_mlp_key_features", "tkphi_build_summaries_cached", "tkphi_decode_step_mlp",
)
STATIC_SCRATCH_BYTES = 8 << 20
KERNEL_KINDS = ("score", "select", "exact_residual", "build", "memset", "cached_z", "mlp")
ERR_TIMEOUT = -5


class TkphiError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"tkphi status {status}: {message}")
        self.status = status


class _KvDesc(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("n_feat", C.c_int32), ("n_sink", C.c_int32),
                ("n_tail", C.c_int32), ("cu_seqlens_host", C.c_void_p), ("cu_seqlens_dev", C.c_void_p),
                ("k", C.c_void_p), ("v", C.c_void_p), ("kv_stride_head", C.c_int64),
                ("kv_stride_token", C.c_int64), ("n_tail_seq_host", C.c_void_p), ("n_tail_seq_dev", C.c_void_p)]


class _PhiDesc(C.Structure):
    _fields_ = [("w_q", C.c_void_p), ("b_q", C.c_void_p), ("w_k", C.c_void_p), ("b_k", C.c_void_p),
                ("gamma_q", C.c_float), ("gamma_k", C.c_float), ("phi_k_cache", C.c_void_p)]


class _MlpDesc(C.Structure):
    _fields_ = [("d_emb", C.c_int32), ("n_heads", C.c_int32), ("w_s", C.c_void_p), ("b_s", C.c_void_p),
                ("w_1", C.c_void_p), ("b_1", C.c_void_p), ("w_2", C.c_void_p), ("b_2", C.c_void_p),
                ("alpha", C.c_void_p), ("w_o", C.c_void_p), ("b_o", C.c_void_p)]


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Load libtkphi.so (built in-tree by ``paper_2604_05438_b200.build``); raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} is missing: build it with "
                           "`python -m paper_2604_05438_b200.build` (there is no CPU fallback)")
    lib = C.CDLL(_LIB_PATH)
    lib.tkphi_workspace_bytes.restype = C.c_size_t
    lib.tkphi_workspace_bytes.argtypes = [C.POINTER(_KvDesc), C.c_void_p, C.c_int32, C.c_int]
    lib.tkphi_build_summaries.restype = C.c_int
    lib.tkphi_build_summaries.argtypes = [C.POINTER(_KvDesc), C.POINTER(_PhiDesc), C.c_void_p, C.c_void_p,
                                          C.c_void_p, C.c_size_t, C.c_void_p]
    lib.tkphi_build_summaries_static.restype = C.c_int
    lib.tkphi_build_summaries_static.argtypes = [C.POINTER(_KvDesc), C.POINTER(_PhiDesc), C.c_void_p, C.c_void_p,
                                                 C.c_void_p]
    lib.tkphi_static_last_error.restype = C.c_char_p
    lib.tkphi_static_device_status.restype = C.c_int
    lib.tkphi_static_device_status.argtypes = [C.c_void_p, C.POINTER(C.c_int32)]
    lib.tkphi_selftest_timeout.restype = C.c_int
    lib.tkphi_selftest_timeout.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p]
    lib.tkphi_topk_decode.restype = C.c_int
    lib.tkphi_topk_decode.argtypes = [C.POINTER(_KvDesc), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.tkphi_decode_step.restype = C.c_int
    lib.tkphi_decode_step.argtypes = [C.POINTER(_KvDesc), C.POINTER(_PhiDesc), C.c_void_p, C.c_void_p,
                                      C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                      C.c_void_p, C.c_uint32, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.tkphi_mlp_key_features.restype = C.c_int
    lib.tkphi_mlp_key_features.argtypes = [C.POINTER(_KvDesc), C.POINTER(_MlpDesc), C.c_void_p, C.c_void_p, C.c_size_t,
                                           C.c_void_p]
    lib.tkphi_build_summaries_cached.restype = C.c_int
    lib.tkphi_build_summaries_cached.argtypes = [C.POINTER(_KvDesc), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                                 C.c_size_t, C.c_void_p]
    lib.tkphi_decode_step_mlp.restype = C.c_int
    lib.tkphi_decode_step_mlp.argtypes = [C.POINTER(_KvDesc), C.POINTER(_MlpDesc), C.c_void_p, C.c_void_p, C.c_void_p,
                                          C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                          C.c_void_p, C.c_uint32, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.tkphi_device_status.restype = C.c_int
    lib.tkphi_device_status.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_int32)]
    lib.tkphi_kernel_timing_enable.restype = None
    lib.tkphi_kernel_timing_enable.argtypes = [C.c_int32]
    lib.tkphi_kernel_timing_read.restype = C.c_int
    lib.tkphi_kernel_timing_read.argtypes = [C.POINTER(C.c_float), C.POINTER(C.c_int32)]
    lib.tkphi_last_error.restype = C.c_char_p
    lib.tkphi_version.restype = C.c_int32
    _lib = lib
    return lib


def _check(status: int):
    if status != 0:
        raise TkphiError(status, load_library().tkphi_last_error().decode())


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream or None


@dataclass
class KVCache:
    """One layer's ragged K/V cache as the library sees it (no copies are made).

    k, v: bf16 device tensors addressed as [head, row, dim] through the strides
    (any layout whose innermost dim is contiguous).  cu_seqlens: int64 host array
    [batch+1]; a device copy is kept alongside.
    """
    k: torch.Tensor
    v: torch.Tensor
    cu_seqlens: np.ndarray
    n_q_heads: int
    n_feat: int
    n_sink: int
    n_tail: int
    cu_seqlens_dev: Optional[torch.Tensor] = None
    n_tail_seq: Optional[np.ndarray] = None        # int32 [batch]: per-sequence tail-anchor counts (replace n_tail)
    n_tail_seq_dev: Optional[torch.Tensor] = None

    def __post_init__(self):
        self.cu_seqlens = np.ascontiguousarray(self.cu_seqlens, dtype=np.int64)
        if self.cu_seqlens_dev is None:
            self.cu_seqlens_dev = torch.from_numpy(self.cu_seqlens).to(self.k.device)
        if self.n_tail_seq is not None:
            self.n_tail_seq = np.ascontiguousarray(self.n_tail_seq, dtype=np.int32)
            assert self.n_tail_seq.shape == (len(self.cu_seqlens) - 1,)
            if self.n_tail_seq_dev is None:
                self.n_tail_seq_dev = torch.from_numpy(self.n_tail_seq).to(self.k.device)

    @property
    def batch(self) -> int:
        return len(self.cu_seqlens) - 1

    def desc(self) -> _KvDesc:
        k, v = self.k, self.v
        assert k.dtype == torch.bfloat16 and v.dtype == torch.bfloat16 and k.dim() == 3
        assert k.stride() == v.stride() and k.stride(2) == 1
        return _KvDesc(self.batch, self.n_q_heads, k.shape[0], k.shape[2], self.n_feat, self.n_sink,
                       self.n_tail, self.cu_seqlens.ctypes.data, self.cu_seqlens_dev.data_ptr(),
                       k.data_ptr(), v.data_ptr(), k.stride(0), k.stride(1),
                       None if self.n_tail_seq is None else self.n_tail_seq.ctypes.data,
                       None if self.n_tail_seq is None else self.n_tail_seq_dev.data_ptr())


@dataclass
class PhiMaps:
    """fp32 device parameters of phi(x) = exp(W x + b - gamma |x|^2)."""
    w_q: torch.Tensor
    b_q: torch.Tensor
    w_k: torch.Tensor
    b_k: torch.Tensor
    gamma_q: float
    gamma_k: float
    phi_k_cache: Optional[torch.Tensor] = None   # optional fp32 [n_kv_heads][T_total][n_feat]: written by the build, read by decode_step

    def desc(self) -> _PhiDesc:
        for t in (self.w_q, self.b_q, self.w_k, self.b_k):
            assert t.dtype == torch.float32 and t.is_contiguous()
        cache = None
        if self.phi_k_cache is not None:
            assert self.phi_k_cache.dtype == torch.float32 and self.phi_k_cache.is_contiguous()
            cache = self.phi_k_cache.data_ptr()
        return _PhiDesc(self.w_q.data_ptr(), self.b_q.data_ptr(), self.w_k.data_ptr(), self.b_k.data_ptr(),
                        float(self.gamma_q), float(self.gamma_k), cache)


@dataclass
class MlpMaps:
    """fp32 device parameters of one side's ReZero-MLP feature maps (App. C.2): phi(x) =
    exp(W_o (g0 + alpha (W_2 GeLU(W_1 g0 + b_1) + b_2)) + b_o), g0 = W_s x + b_s; leading dim = heads."""
    w_s: torch.Tensor
    b_s: torch.Tensor
    w_1: torch.Tensor
    b_1: torch.Tensor
    w_2: torch.Tensor
    b_2: torch.Tensor
    alpha: torch.Tensor
    w_o: torch.Tensor
    b_o: torch.Tensor

    def desc(self) -> _MlpDesc:
        ts = (self.w_s, self.b_s, self.w_1, self.b_1, self.w_2, self.b_2, self.alpha, self.w_o, self.b_o)
        for t in ts:
            assert t.dtype == torch.float32 and t.is_contiguous()
        return _MlpDesc(self.w_1.shape[1], self.w_s.shape[0], *[t.data_ptr() for t in ts])


def _topk_host(topk) -> np.ndarray:
    return np.ascontiguousarray(topk, dtype=np.int32)


def workspace_bytes(kv: KVCache, topk_host, topk_max: int, which: int) -> int:
    lib = load_library()
    d = kv.desc()
    th = None if topk_host is None else _topk_host(topk_host)
    n = lib.tkphi_workspace_bytes(C.byref(d), None if th is None else th.ctypes.data, int(topk_max), which)
    if n == 0:
        raise TkphiError(-1, lib.tkphi_last_error().decode())
    return int(n)


def build_summaries(kv: KVCache, phi: PhiMaps, S: torch.Tensor, u: torch.Tensor,
                    workspace: torch.Tensor, stream=None) -> None:
    lib = load_library()
    d, ph = kv.desc(), phi.desc()
    _check(lib.tkphi_build_summaries(C.byref(d), C.byref(ph), S.data_ptr(), u.data_ptr(),
                                     workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                     _stream_ptr(stream)))


def build_summaries_static(kv: KVCache, phi: PhiMaps, S: torch.Tensor, u: torch.Tensor, stream=None) -> None:
    """Summary build on the library's built-in scratch: for callers that may not
    allocate device memory.  Problems needing more than STATIC_SCRATCH_BYTES of
    scratch raise TkphiError (status -3).  Calls that overlap on the GPU race."""
    lib = load_library()
    d, ph = kv.desc(), phi.desc()
    st = lib.tkphi_build_summaries_static(C.byref(d), C.byref(ph), S.data_ptr(), u.data_ptr(), _stream_ptr(stream))
    if st != 0:
        raise TkphiError(st, lib.tkphi_static_last_error().decode())


def static_device_status(stream=None) -> int:
    """Status word of the last build_summaries_static call on the current device (0 = fine)."""
    lib = load_library()
    out = C.c_int32(0)
    st = lib.tkphi_static_device_status(_stream_ptr(stream), C.byref(out))
    if st != 0:
        raise TkphiError(st, lib.tkphi_static_last_error().decode())
    return int(out.value)


def selftest_timeout(workspace: torch.Tensor, stream=None) -> None:
    """Runs the library's bounded-wait self-test kernel; device_status(workspace) then reads ERR_TIMEOUT."""
    lib = load_library()
    _check(lib.tkphi_selftest_timeout(workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                      _stream_ptr(stream)))


def mlp_key_features(kv: KVCache, mlp_k: MlpMaps, phi_k_cache: torch.Tensor, workspace: torch.Tensor, stream=None) -> None:
    lib = load_library()
    d, m = kv.desc(), mlp_k.desc()
    _check(lib.tkphi_mlp_key_features(C.byref(d), C.byref(m), phi_k_cache.data_ptr(), workspace.data_ptr(),
                                      workspace.numel() * workspace.element_size(), _stream_ptr(stream)))


def build_summaries_cached(kv: KVCache, phi_k_cache: torch.Tensor, S: torch.Tensor, u: torch.Tensor,
                           workspace: torch.Tensor, stream=None) -> None:
    lib = load_library()
    d = kv.desc()
    _check(lib.tkphi_build_summaries_cached(C.byref(d), phi_k_cache.data_ptr(), S.data_ptr(), u.data_ptr(),
                                            workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                            _stream_ptr(stream)))


def decode_step_mlp(kv: KVCache, mlp_q: MlpMaps, phi_k_cache: Optional[torch.Tensor], q: torch.Tensor, topk_host,
                    topk_dev: torch.Tensor, topk_max: int, S: torch.Tensor, u: torch.Tensor,
                    idx_out: Optional[torch.Tensor], y_out: torch.Tensor, dbg_out: Optional[torch.Tensor], flags: int,
                    workspace: torch.Tensor, stream=None) -> None:
    lib = load_library()
    d, m = kv.desc(), mlp_q.desc()
    th = _topk_host(topk_host)
    _check(lib.tkphi_decode_step_mlp(C.byref(d), C.byref(m), _ptr(phi_k_cache), q.data_ptr(), th.ctypes.data,
                                     topk_dev.data_ptr(), int(topk_max), S.data_ptr(), u.data_ptr(), _ptr(idx_out),
                                     y_out.data_ptr(), _ptr(dbg_out), int(flags), workspace.data_ptr(),
                                     workspace.numel() * workspace.element_size(), _stream_ptr(stream)))


def topk_decode(kv: KVCache, q: torch.Tensor, topk_host, topk_dev: torch.Tensor, topk_max: int,
                idx_out: Optional[torch.Tensor], y_out: torch.Tensor, workspace: torch.Tensor,
                stream=None) -> None:
    lib = load_library()
    d = kv.desc()
    th = _topk_host(topk_host)
    _check(lib.tkphi_topk_decode(C.byref(d), q.data_ptr(), th.ctypes.data, topk_dev.data_ptr(), int(topk_max),
                                 _ptr(idx_out), y_out.data_ptr(), workspace.data_ptr(),
                                 workspace.numel() * workspace.element_size(), _stream_ptr(stream)))


def decode_step(kv: KVCache, phi: PhiMaps, q: torch.Tensor, topk_host, topk_dev: torch.Tensor,
                topk_max: int, S: torch.Tensor, u: torch.Tensor, idx_out: Optional[torch.Tensor],
                y_out: torch.Tensor, dbg_out: Optional[torch.Tensor], flags: int,
                workspace: torch.Tensor, stream=None) -> None:
    lib = load_library()
    d, ph = kv.desc(), phi.desc()
    th = _topk_host(topk_host)
    _check(lib.tkphi_decode_step(C.byref(d), C.byref(ph), q.data_ptr(), th.ctypes.data, topk_dev.data_ptr(),
                                 int(topk_max), S.data_ptr(), u.data_ptr(), _ptr(idx_out), y_out.data_ptr(),
                                 _ptr(dbg_out), int(flags), workspace.data_ptr(),
                                 workspace.numel() * workspace.element_size(), _stream_ptr(stream)))


def device_status(workspace: torch.Tensor, stream=None) -> int:
    lib = load_library()
    out = C.c_int32(0)
    _check(lib.tkphi_device_status(workspace.data_ptr(), _stream_ptr(stream), C.byref(out)))
    return int(out.value)


def kernel_timing(fn) -> dict:
    """Run ``fn()`` with the library's per-kernel event timing on; returns
    {kind: {"ms": total, "launches": n, "avg_ms": ms/n}} for the kinds that ran."""
    lib = load_library()
    lib.tkphi_kernel_timing_enable(1)
    try:
        fn()
        torch.cuda.synchronize()
        ms = (C.c_float * len(KERNEL_KINDS))()
        cnt = (C.c_int32 * len(KERNEL_KINDS))()
        _check(lib.tkphi_kernel_timing_read(ms, cnt))
    finally:
        lib.tkphi_kernel_timing_enable(0)
    return {k: {"ms": float(ms[i]), "launches": int(cnt[i]), "avg_ms": float(ms[i]) / cnt[i]}
            for i, k in enumerate(KERNEL_KINDS) if cnt[i] > 0}
