"""Parity at the full sizes of the workload table, on sampled heads.

Inputs are drawn on the GPU at the sizes and in the launch configuration that
``bench.py`` times (one call per layer, all heads); the float64 oracle is then run on
sampled (sequence, head) pairs, whose K/V rows are copied back to the host.  Every
workload runs twice: with the workload's own feature map, under which the residual is a
vanishing share of the mass, and with the visible-residual map (shared random features,
oracle-calibrated bias shift) under which the residual branch carries an O(1) share, so
that the subtraction, the residual estimate and the merge are seen by the comparison.
"""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import tkphi_oracle as O
from workloads import CONFIGS, draw_seq_lens, make_layer_inputs, make_phi_params

import parity_utils as PU

pytestmark = pytest.mark.gpu


def _phi_for(cfg, inp, seed, kind, frac, samples, dev):
    if kind == "baseline":
        return make_phi_params(cfg, seed, device=dev)
    phi0 = make_phi_params(cfg, seed, kind="visible")
    shift = torch.zeros(cfg.n_kv_heads)
    done = set()
    for b, hq in samples:                       # calibrate the KV heads that are compared, on their sequence
        kvh = hq // cfg.group
        if kvh not in done:
            done.add(kvh)
            shift[kvh] = PU.calibrate_visible_shift(cfg, inp, phi0, frac, n_probe=2, kv_heads=[kvh], b=b)[kvh]
    return make_phi_params(cfg, seed, kind="visible", device=dev, bk_shift=shift)


def _run_full(cfg_name, frac, samples, seed=0, kind="baseline"):
    """samples: list of (sequence, query head); cfg_name: a key of CONFIGS or a WorkloadConfig."""
    import paper_2604_05438_b200 as T
    cfg = CONFIGS[cfg_name] if isinstance(cfg_name, str) else cfg_name
    dev = torch.device("cuda:0")
    inp = make_layer_inputs(cfg, seed, device=dev, n_steps=1)
    phi = _phi_for(cfg, inp, seed, kind, frac, samples, dev)
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
    built = {}
    for b, hq in samples:
        kvh = hq // G
        if (b, kvh) not in built:
            if len(built) >= 2:                 # million-token heads take gigabytes in float64: keep two
                built.pop(next(iter(built)))
            K, V = PU.seq_arrays(inp, b, kvh)
            S0, u0 = O.build_summaries(K, V, phic.w_k[kvh].double().numpy(), phic.b_k[kvh].double().numpy(),
                                       phic.gamma_k, cfg.n_sink, cfg.n_tail)
            Sg, ug = S[b, kvh].cpu().double().numpy(), u[b, kvh].cpu().double().numpy()
            if np.abs(S0).max() >= PU.FP32_TINY:
                assert PU.note("S_rel_err", PU.max_rel(Sg, S0)) <= PU.SU_TOL, (b, kvh)
                assert PU.note("u_rel_err", PU.max_rel(ug, u0)) <= PU.SU_TOL, (b, kvh)
            built[(b, kvh)] = (K, V, Sg, ug)
        K, V, Sg, ug = built[(b, kvh)]
        q64 = q[b, hq].cpu().double().numpy()
        kk = int(topk[b])
        ret = PU.check_selection(q64, K, cfg.n_sink, cfg.n_tail, kk, ih[b, hq])
        pa = (phic.w_q[hq].double().numpy(), phic.b_q[hq].double().numpy(), phic.gamma_q,
              phic.w_k[kvh].double().numpy(), phic.b_k[kvh].double().numpy(), phic.gamma_k)
        res = O.topkphi_attention(q64, K, V, cfg.n_sink, cfg.n_tail, kk, *pa, S=Sg, u=ug, retrieved=ret)
        nosub = O.topkphi_attention(q64, K, V, cfg.n_sink, cfg.n_tail, kk, *pa, S=Sg, u=ug, retrieved=ret,
                                    subtract=False)
        e = PU.note("y_rel_err", PU.max_rel(yh[b, hq], res.y))
        assert e <= PU.Y_TOL, (b, hq, e)
        assert PU.note("m_E_abs_err", abs(dh[b, hq, 0] - res.m_E)) <= PU.ME_TOL * max(1.0, abs(res.m_E))
        PU.check_residual(dh[b, hq], res, nosub, (b, hq))
        y0, _ = O.topk_attention(q64, K, V, cfg.n_sink, cfg.n_tail, kk, retrieved=ret)
        e2 = PU.note("y_topk_rel_err", PU.max_rel(yth[b, hq], y0))
        assert e2 <= PU.Y_TOL, (b, hq, e2)
        if kind == "visible":                   # the residual branch must matter in this setting
            PU.note("visible_y_minus_ytopk", PU.max_rel(res.y, y0))


KINDS = ["baseline", "visible"]


@pytest.mark.parametrize("kind", KINDS)
def test_c2_32k_full_layer_all_heads(kind):
    _run_full("c2_1b_32k", 0.01, [(0, h) for h in range(32)], kind=kind)


@pytest.mark.parametrize("kind", KINDS)
def test_c3_128k_full_layer_all_heads(kind):
    _run_full("c3_3b_128k", 0.01, [(0, h) for h in range(24)], seed=0, kind=kind)


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("seed", [1, 2])
def test_c3_128k_other_seeds_sampled_heads(seed, kind):
    _run_full("c3_3b_128k", 0.01, [(0, 0), (0, 4), (0, 11), (0, 23)], seed=seed, kind=kind)


@pytest.mark.parametrize("frac,kind", [(0.005, "baseline"), (0.04, "baseline"), (0.02, "visible"), (0.04, "visible")])
def test_c3_128k_other_budgets_sampled_heads(frac, kind):
    _run_full("c3_3b_128k", frac, [(0, 2), (0, 9), (0, 13), (0, 22)], kind=kind)


@pytest.mark.parametrize("kind", KINDS)
def test_c4_ragged_32_sequences_sampled(kind):
    # the two shortest and the two longest sequences of the draw, and twelve others
    cfg = CONFIGS["c4_1b_ragged"]
    order = [int(b) for b in np.argsort(draw_seq_lens(cfg, 1), kind="stable")]      # shortest first
    picks = [order[0], order[1], order[-1], order[-2]] + [int(b) for b in order[3:27:2]]
    samples = [(b, (5 * i + 3) % cfg.n_q_heads) for i, b in enumerate(picks)]
    assert len(samples) >= 16
    _run_full("c4_1b_ragged", 0.01, samples, seed=1, kind=kind)


@pytest.mark.parametrize("kind", KINDS)
def test_c5_four_sequences_of_one_million_tokens_sampled(kind):
    # eight rows over three (sequence, KV head) pairs
    _run_full("c5_3b_1m", 0.01, [(0, 6), (0, 7), (0, 8), (3, 18), (3, 19), (3, 20), (1, 0), (1, 1)], kind=kind)


def test_longest_supported_sequence_2097152_mid_keys():
    # the documented limit of the selection kernel (16 rounds per CTA of an 8-CTA cluster); two KV heads
    cfg = dataclasses.replace(CONFIGS["c1_1b_4k"], n_q_heads=4, n_kv_heads=2, seq_len=2097152 + 4 + 64, needles_per_head=8)
    _run_full(cfg, 0.001, [(0, 1), (0, 2)], seed=3, kind="baseline")
