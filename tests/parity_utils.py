"""Shared helpers of the GPU parity tests: run the CUDA path through the binding,
run the float64 oracle on the same tensors, compare under the stated tolerances."""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

from oracle import tkphi_oracle as O
from workloads import LayerInputs, PhiParams, WorkloadConfig

# Tolerances (bf16 inputs, fp32 accumulation):
Y_TOL = 2e-3          # max_j |y_hat - y| / max_j |y| per output vector
SU_TOL = 1e-3         # max |S_hat - S| / max |S| per head (same for u)
TIE_TOL = 1e-5        # index sets may differ only where |s_i - tau| <= TIE_TOL * max(|tau|, 1)
RESID_TOL = 2e-4      # residual terms, relative to the unsubtracted feature mass phi_q.u_M (see check_residual)
DIR_MIN_LEFT = 0.005  # the residual direction is compared whenever more than this share of the mass is left
ME_TOL = 1e-4         # absolute, on the exact-branch max score
FP32_TINY = 1.2e-38   # below the smallest normal fp32 a summary entry is not representable

# Worst errors seen by the helpers below since the last reset, by name; the GPU test modules print
# them as one JSON line per test (conftest.py).
STATS: dict = {}


def note(name: str, value: float) -> float:
    value = float(value)
    if not (STATS.get(name, -math.inf) >= value):
        STATS[name] = value
    return value


def max_rel(a, b) -> float:
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    den = np.abs(b).max()
    return float(np.abs(a - b).max() / (den if den > 0 else 1.0))


@dataclass
class GpuLayer:
    """Device-resident copy of one layer's inputs plus the binding's descriptors."""
    cfg: WorkloadConfig
    inp: LayerInputs
    phi: PhiParams
    kv: object
    maps: object
    dev: torch.device


def to_gpu(cfg, inp: LayerInputs, phi: PhiParams, token_major: bool = False) -> GpuLayer:
    import paper_2604_05438_b200 as T
    dev = torch.device("cuda:0")
    if token_major:   # [row][head][dim] storage, viewed as [head][row][dim]
        k = inp.k.permute(1, 0, 2).contiguous().to(dev).permute(1, 0, 2)
        v = inp.v.permute(1, 0, 2).contiguous().to(dev).permute(1, 0, 2)
    else:
        k, v = inp.k.to(dev), inp.v.to(dev)
    kv = T.KVCache(k, v, inp.cu_seqlens, cfg.n_q_heads, cfg.n_feat, inp.n_sink, inp.n_tail)
    p = phi.to(dev)
    maps = T.PhiMaps(p.w_q, p.b_q, p.w_k, p.b_k, p.gamma_q, p.gamma_k)
    return GpuLayer(cfg, inp, phi, kv, maps, dev)


def gpu_build(gl: GpuLayer):
    import paper_2604_05438_b200 as T
    B, Hkv, d, r = gl.kv.batch, gl.cfg.n_kv_heads, gl.cfg.head_dim, gl.cfg.n_feat
    S = torch.full((B, Hkv, d, r), float("nan"), device=gl.dev)
    u = torch.full((B, Hkv, r), float("nan"), device=gl.dev)
    ws = torch.empty(T.workspace_bytes(gl.kv, None, 0, T.WS_BUILD), dtype=torch.uint8, device=gl.dev)
    T.build_summaries(gl.kv, gl.maps, S, u, ws)
    torch.cuda.synchronize()
    assert T.device_status(ws) == 0
    return S, u


def gpu_decode(gl: GpuLayer, q: torch.Tensor, topk: np.ndarray, S=None, u=None, with_phi=True,
               flags=0, topk_max: Optional[int] = None, want_idx=True):
    """q: bf16 [B, H_q, d] (host or device).  Returns dict of host arrays."""
    import paper_2604_05438_b200 as T
    B, Hq, d = gl.kv.batch, gl.cfg.n_q_heads, gl.cfg.head_dim
    topk = np.ascontiguousarray(topk, np.int32)
    tmax = int(topk.max()) if topk_max is None else topk_max
    qd = q.to(gl.dev).contiguous()
    topk_dev = torch.from_numpy(topk).to(gl.dev)
    which = T.WS_DECODE_STEP if with_phi else T.WS_TOPK_DECODE
    ws = torch.empty(T.workspace_bytes(gl.kv, topk, tmax, which), dtype=torch.uint8, device=gl.dev)
    ws.fill_(0xA5)        # the library must not rely on workspace contents
    idx = torch.full((B, Hq, max(tmax, 1)), -7, dtype=torch.int32, device=gl.dev) if want_idx else None
    y = torch.full((B, Hq, d), float("nan"), device=gl.dev)
    dbg = None
    if with_phi:
        dbg = torch.full((B, Hq, 4 + d), float("nan"), device=gl.dev)
        T.decode_step(gl.kv, gl.maps, qd, topk, topk_dev, tmax, S, u, idx if tmax > 0 else None, y, dbg,
                      flags, ws)
    else:
        T.topk_decode(gl.kv, qd, topk, topk_dev, tmax, idx if tmax > 0 else None, y, ws)
    torch.cuda.synchronize()
    assert T.device_status(ws) == 0
    return dict(y=y.cpu().numpy(), idx=None if idx is None else idx.cpu().numpy(),
                dbg=None if dbg is None else dbg.cpu().numpy())


def seq_arrays(inp: LayerInputs, b: int, kvh: int):
    lo, hi = int(inp.cu_seqlens[b]), int(inp.cu_seqlens[b + 1])
    K = inp.k[kvh, lo:hi].cpu().double().numpy()
    V = inp.v[kvh, lo:hi].cpu().double().numpy()
    return K, V


def check_residual(dbg_row, res, res_nosub, where) -> None:
    """Residual terms of one query head against the oracle.

    dbg_row: the library's debug row ([2] log Z_hat_R, [4:] nu_hat_R / Z_hat_R); res: the oracle's
    result; res_nosub: the oracle's result with the subtraction skipped, whose log_Zhat_R is the
    unsubtracted feature mass log(phi_q . u_M).

    Z_hat_R = phi_q.u_M - sum_i z_i and nu_hat_R = S_M phi_q - sum_i z_i v_i are differences (Eq.
    subtraction): rounding errors of the two sides do not shrink with the difference, so every
    error is bounded relative to the unsubtracted mass phi_q.u_M.  With `left` the share of that
    mass the subtraction leaves, the share itself is held to RESID_TOL, log Z_hat_R to
    RESID_TOL / left, and the direction nu_hat_R / Z_hat_R to RESID_TOL / left of its largest entry
    (both whenever left > DIR_MIN_LEFT; below that nothing but the share is meaningful).
    """
    log_ZM = res_nosub.log_Zhat_R
    if not math.isfinite(log_ZM):
        return                                   # no feature mass at all (zero summaries)
    left = 0.0 if res.clamped else math.exp(res.log_Zhat_R - log_ZM)
    got = math.exp(dbg_row[2] - log_ZM) if math.isfinite(dbg_row[2]) else 0.0   # -inf: clamped away
    e_share = note("resid_share_abs_err", abs(got - left))
    assert e_share <= RESID_TOL, (where, dbg_row[2], res.log_Zhat_R, left)
    if left > DIR_MIN_LEFT:
        e_log = note("resid_logz_err_x_left", abs(dbg_row[2] - res.log_Zhat_R) * left)
        e_dir = note("resid_dir_err_x_left", max_rel(dbg_row[4:], res.y_R_hat) * left)
        note("resid_min_left_checked", -left)
        assert e_log <= RESID_TOL, (where, dbg_row[2], res.log_Zhat_R, left)
        assert e_dir <= RESID_TOL, (where, e_dir, left)


def check_selection(q64, K, n_sink, n_tail, topk, got_idx_row) -> np.ndarray:
    """Index-set parity under the tie rule; returns the GPU's retrieved set."""
    got = got_idx_row[:topk].astype(np.int64)
    pad = got_idx_row[topk:]
    assert (pad == -1).all(), "idx_out must be padded with -1"
    assert (np.diff(got) > 0).all(), "retrieved indices must be strictly ascending"
    L = K.shape[0]
    if topk:
        assert got.min() >= n_sink and got.max() < L - n_tail
    want = O.select_topk(q64, K, n_sink, n_tail, topk, score_dtype=np.float64)
    diff = np.setxor1d(got, want)
    if diff.size:
        tau = O.kth_score(q64, K, n_sink, n_tail, topk)
        s = O.scores(q64, K[diff])
        bad = np.abs(s - tau) > TIE_TOL * max(abs(tau), 1.0)
        assert not bad.any(), f"index sets differ away from the threshold: {diff[bad]} tau={tau} s={s[bad]}"
    return got


def calibrate_visible_shift(cfg, inp: LayerInputs, phi: PhiParams, frac: float, n_probe: int = 4,
                            kv_heads=None, b: int = 0) -> torch.Tensor:
    """Per-KV-head shift of b_k that puts median(log Z_hat_R - log Z_R) at zero
    (computed with the oracle on a few queries of sequence b; heads not in `kv_heads` keep 0)."""
    Hkv, G = cfg.n_kv_heads, cfg.group
    shifts = torch.zeros(Hkv)
    topk = int(inp.topk(frac)[b])
    phi = phi.to("cpu")
    for kvh in (range(Hkv) if kv_heads is None else kv_heads):
        K, V = seq_arrays(inp, b, kvh)
        S, u = O.build_summaries(K, V, phi.w_k[kvh].double().numpy(), phi.b_k[kvh].double().numpy(),
                                 phi.gamma_k, inp.n_sink, inp.n_tail)
        errs = []
        for n in range(n_probe):
            hq = kvh * G + (n % G)
            step = n // G % inp.q.shape[0]
            q64 = inp.q[step, b, hq].cpu().double().numpy()
            res = O.topkphi_attention(q64, K, V, inp.n_sink, inp.n_tail, topk,
                                      phi.w_q[hq].double().numpy(), phi.b_q[hq].double().numpy(), phi.gamma_q,
                                      phi.w_k[kvh].double().numpy(), phi.b_k[kvh].double().numpy(), phi.gamma_k,
                                      S=S, u=u)
            lz = O.residual_log_z(q64, K, inp.n_sink, inp.n_tail, res.retrieved)
            if math.isfinite(res.log_Zhat_R) and math.isfinite(lz):
                errs.append(res.log_Zhat_R - lz)
        shifts[kvh] = -float(np.median(errs)) if errs else 0.0
    return shifts
