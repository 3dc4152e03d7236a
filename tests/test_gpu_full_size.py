"""Parity at the full sizes of the workload table, on sampled heads.

Inputs are drawn on the GPU at the sizes and in the launch configuration that
``bench.py`` times (one call per layer, all heads); the float64 oracle is then run on
a few sampled (sequence, head) pairs, whose K/V rows are copied back to the host.
"""
import math

import numpy as np
import pytest
import torch

from oracle import tkphi_oracle as O
from workloads import CONFIGS, make_layer_inputs, make_phi_params

import parity_utils as PU

pytestmark = pytest.mark.gpu


def _run_full(cfg_name, frac, samples, seed=0, build_heads=None):
    """samples: list of (sequence, query head).  Returns the worst y error seen."""
    import paper_2604_05438_b200 as T
    cfg = CONFIGS[cfg_name]
    dev = torch.device("cuda:0")
    inp = make_layer_inputs(cfg, seed, device=dev, n_steps=1)
    phi = make_phi_params(cfg, seed, device=dev)
    kv = T.KVCache(inp.k, inp.v, inp.cu_seqlens, cfg.n_q_heads, cfg.n_feat, cfg.n_sink, cfg.n_tail)
    maps = T.PhiMaps(phi.w_q, phi.b_q, phi.w_k, phi.b_k, phi.gamma_q, phi.gamma_k)
    B, Hq, Hkv, d, r = kv.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_feat
    topk = inp.topk(frac)
    tmax = int(topk.max())
    S = torch.full((B, Hkv, d, r), float("nan"), device=dev)
    u = torch.full((B, Hkv, r), float("nan"), device=dev)
    wsb = torch.empty(T.workspace_bytes(kv, None, 0, T.WS_BUILD), dtype=torch.uint8, device=dev)
    T.build_summaries(kv, maps, S, u, wsb)
    ws = torch.empty(T.workspace_bytes(kv, topk, tmax, T.WS_DECODE_STEP), dtype=torch.uint8, device=dev)
    idx = torch.full((B, Hq, tmax), -7, dtype=torch.int32, device=dev)
    y = torch.full((B, Hq, d), float("nan"), device=dev)
    dbg = torch.full((B, Hq, 4 + d), float("nan"), device=dev)
    q = inp.q[0].contiguous()
    T.decode_step(kv, maps, q, topk, torch.from_numpy(topk).to(dev), tmax, S, u, idx, y, dbg, 0, ws)
    y_top = torch.full((B, Hq, d), float("nan"), device=dev)
    T.topk_decode(kv, q, topk, torch.from_numpy(topk).to(dev), tmax, None, y_top, ws)
    torch.cuda.synchronize()
    assert T.device_status(ws) == 0 and T.device_status(wsb) == 0
    assert torch.isfinite(y).all() and torch.isfinite(S).all() and torch.isfinite(u).all()
    yh, yth, ih, dh = y.cpu().numpy(), y_top.cpu().numpy(), idx.cpu().numpy(), dbg.cpu().numpy()
    phic = phi.to("cpu")
    G = cfg.group
    worst = 0.0
    built = {}
    for b, hq in samples:
        kvh = hq // G
        lo, hi = int(inp.cu_seqlens[b]), int(inp.cu_seqlens[b + 1])
        if (b, kvh) not in built:
            K = inp.k[kvh, lo:hi].cpu().double().numpy()
            V = inp.v[kvh, lo:hi].cpu().double().numpy()
            S0, u0 = O.build_summaries(K, V, phic.w_k[kvh].double().numpy(), phic.b_k[kvh].double().numpy(),
                                       phic.gamma_k, cfg.n_sink, cfg.n_tail)
            Sg, ug = S[b, kvh].cpu().double().numpy(), u[b, kvh].cpu().double().numpy()
            if np.abs(S0).max() >= PU.FP32_TINY:
                assert PU.max_rel(Sg, S0) <= PU.SU_TOL and PU.max_rel(ug, u0) <= PU.SU_TOL, (b, kvh)
            built[(b, kvh)] = (K, V, Sg, ug)
        K, V, Sg, ug = built[(b, kvh)]
        q64 = q[b, hq].cpu().double().numpy()
        kk = int(topk[b])
        ret = PU.check_selection(q64, K, cfg.n_sink, cfg.n_tail, kk, ih[b, hq])
        res = O.topkphi_attention(q64, K, V, cfg.n_sink, cfg.n_tail, kk,
                                  phic.w_q[hq].double().numpy(), phic.b_q[hq].double().numpy(), phic.gamma_q,
                                  phic.w_k[kvh].double().numpy(), phic.b_k[kvh].double().numpy(), phic.gamma_k,
                                  S=Sg, u=ug, retrieved=ret)
        e = PU.max_rel(yh[b, hq], res.y)
        assert e <= PU.Y_TOL, (b, hq, e)
        assert abs(dh[b, hq, 0] - res.m_E) <= PU.ME_TOL * max(1.0, abs(res.m_E))
        if not res.clamped and math.isfinite(dh[b, hq, 2]):
            assert abs(dh[b, hq, 2] - res.log_Zhat_R) <= PU.LOGZ_TOL, (b, hq, dh[b, hq, 2], res.log_Zhat_R)
        y0, _ = O.topk_attention(q64, K, V, cfg.n_sink, cfg.n_tail, kk, retrieved=ret)
        e2 = PU.max_rel(yth[b, hq], y0)
        assert e2 <= PU.Y_TOL, (b, hq, e2)
        worst = max(worst, e, e2)
    return worst


def test_c2_32k_full_layer_all_heads():
    _run_full("c2_1b_32k", 0.01, [(0, h) for h in range(32)])


@pytest.mark.parametrize("frac", [0.005, 0.01, 0.04])
def test_c3_128k_full_layer_sampled_heads(frac):
    _run_full("c3_3b_128k", frac, [(0, 0), (0, 4), (0, 11), (0, 23)])


def test_c4_ragged_32_sequences_sampled():
    _run_full("c4_1b_ragged", 0.01, [(0, 0), (7, 13), (19, 31), (31, 5)], seed=1)


def test_c5_four_sequences_of_one_million_tokens_sampled():
    _run_full("c5_3b_1m", 0.01, [(0, 7), (3, 20)])
