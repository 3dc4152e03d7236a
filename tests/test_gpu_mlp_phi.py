"""The paper's one-block ReZero-MLP feature map (App. C.2) through the C ABI: key features into the
cache, the summary build from the cache, and the decode step whose query features come from the MLP
and whose retrieved key features come from the cache.  Against the float64 oracle."""
import dataclasses
import math

import numpy as np
import pytest
import torch

from oracle import tkphi_oracle as O
from workloads import CONFIGS, make_layer_inputs, make_mlp_phi_params

import parity_utils as PU

pytestmark = pytest.mark.gpu

# Key-side MLP: weights and the three stored activations are bf16 (2^-9 relative each), accumulation
# fp32.  One rounding source moves the exponent a_j = (W_o g1 + b_o)_j by about
# 2^-9 * |w_o row| * |g1| / sqrt(d_emb) ~ 2^-9 * 0.5 * 1.5 ~ 1.5e-3 (random signs over d_emb = 512
# terms); seven sources (four weight matrices, g0, the GeLU output, g1) add in quadrature to ~4e-3 rms,
# and the maximum over 10^5..10^7 entries sits five to six sigma out (~2.5e-2).
MLP_LOG_TOL = 4e-2
# Query-side MLP: fp32 weights, fp32 FMA chains of length <= 512.
MLP_Q_LOG_TOL = 1e-4


def _maps(T, p):
    return T.MlpMaps(p.w_s, p.b_s, p.w_1, p.b_1, p.w_2, p.b_2, p.alpha, p.w_o, p.b_o)


def _log_features(X, params, chunk=16384):
    """Oracle log phi(x) of the rows of X, a block of rows at a time (bounds the float64 intermediates)."""
    return np.concatenate([O.phi_mlp_log(X[i:i + chunk], **params) for i in range(0, X.shape[0], chunk)], axis=0)


def _calibrate_bo_shift(cfg, inp, pk, pq, frac, kv_heads, n_probe=2):
    """Per-KV-head shift of the key side's b_o that puts median(log Z_hat_R - log Z_R) at zero, so that
    the residual branch carries a visible share of the mass (oracle only, sequence 0)."""
    shift = torch.zeros(cfg.n_kv_heads)
    topk = int(inp.topk(frac)[0])
    for kvh in kv_heads:
        K, V = PU.seq_arrays(inp, 0, kvh)
        Phi = np.exp(_log_features(K, pk.head(kvh)))
        S, u = O.build_summaries_from_features(V, Phi, inp.n_sink, inp.n_tail)
        errs = []
        for n in range(n_probe):
            hq = kvh * cfg.group + n % cfg.group
            q64 = inp.q[0, 0, hq].cpu().double().numpy()
            ret = O.select_topk(q64, K, inp.n_sink, inp.n_tail, topk)
            res = O.merge_from_features(q64, K, V, inp.n_sink, inp.n_tail, ret, S, u,
                                        O.phi_mlp_log(q64, **pq.head(hq)), Phi[ret])
            lz = O.residual_log_z(q64, K, inp.n_sink, inp.n_tail, ret)
            if math.isfinite(res.log_Zhat_R) and math.isfinite(lz):
                errs.append(res.log_Zhat_R - lz)
        shift[kvh] = -float(np.median(errs)) if errs else 0.0
    return shift


def _check_mlp(cfg, seed, seq_lens, frac, heads, d_emb=512, on_device=False, token_major=False):
    """heads: the query heads compared; the oracle runs on their KV heads only."""
    import paper_2604_05438_b200 as T
    dev = torch.device("cuda:0")
    inp = make_layer_inputs(cfg, seed, seq_lens=seq_lens, n_steps=1, device=dev if on_device else "cpu")
    heads = list(heads)
    kv_heads = sorted({hq // cfg.group for hq in heads})
    pq = make_mlp_phi_params(cfg, seed, "q", d_emb)
    pk = make_mlp_phi_params(cfg, seed, "k", d_emb)
    pk = make_mlp_phi_params(cfg, seed, "k", d_emb, bo_shift=_calibrate_bo_shift(cfg, inp, pk, pq, frac, kv_heads))
    if token_major:   # [row][head][dim] storage, viewed as [head][row][dim]
        kd = inp.k.permute(1, 0, 2).contiguous().to(dev).permute(1, 0, 2)
        vd = inp.v.permute(1, 0, 2).contiguous().to(dev).permute(1, 0, 2)
    else:
        kd, vd = inp.k.to(dev), inp.v.to(dev)
    kv = T.KVCache(kd, vd, inp.cu_seqlens, cfg.n_q_heads, cfg.n_feat, inp.n_sink, inp.n_tail)
    Hq, Hkv, d, r, B = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_feat, inp.batch
    T_total = int(inp.cu_seqlens[-1])

    # (1) key features of every token into the cache
    cache = torch.full((Hkv, T_total, r), float("nan"), device=dev)
    ws = torch.empty(T.workspace_bytes(kv, None, 0, T.WS_MLP_KEY_FEATURES), dtype=torch.uint8, device=dev)
    ws.fill_(0xA5)
    T.mlp_key_features(kv, _maps(T, pk.to(dev)), cache, ws)
    torch.cuda.synchronize()
    assert T.device_status(ws) == 0
    assert bool(torch.isfinite(cache).all()) and bool((cache > 0).all())
    ch = {kvh: cache[kvh].cpu().double().numpy() for kvh in kv_heads}
    Phi_o = {}
    for kvh in kv_heads:
        a = _log_features(inp.k[kvh].cpu().double().numpy(), pk.head(kvh))
        Phi_o[kvh] = a
        e = np.abs(np.log(ch[kvh]) - a).max()
        assert PU.note("mlp_key_log_feature_abs_err", e) <= MLP_LOG_TOL, (kvh, e)

    # (2) the summary build from the cached rows, against the oracle fed the same rows
    S = torch.full((B, Hkv, d, r), float("nan"), device=dev)
    u = torch.full((B, Hkv, r), float("nan"), device=dev)
    wsb = torch.empty(T.workspace_bytes(kv, None, 0, T.WS_BUILD), dtype=torch.uint8, device=dev)
    T.build_summaries_cached(kv, cache, S, u, wsb)
    torch.cuda.synchronize()
    assert T.device_status(wsb) == 0
    Sh, uh = S.cpu().double().numpy(), u.cpu().double().numpy()
    for b in range(B):
        lo, hi = int(inp.cu_seqlens[b]), int(inp.cu_seqlens[b + 1])
        for kvh in kv_heads:
            K, V = PU.seq_arrays(inp, b, kvh)
            S0, u0 = O.build_summaries_from_features(V, ch[kvh][lo:hi], inp.n_sink, inp.n_tail)
            if np.abs(S0).max() >= PU.FP32_TINY:
                assert PU.note("S_rel_err", PU.max_rel(Sh[b, kvh], S0)) <= PU.SU_TOL, (b, kvh)
                assert PU.note("u_rel_err", PU.max_rel(uh[b, kvh], u0)) <= PU.SU_TOL, (b, kvh)
            else:
                assert np.abs(Sh[b, kvh]).max() == 0 and np.abs(uh[b, kvh]).max() == 0
            # how far the bf16 MLP moves the summaries from those of the float64 feature map (reported only)
            S1, u1 = O.build_summaries_from_features(V, np.exp(Phi_o[kvh][lo:hi]), inp.n_sink, inp.n_tail)
            if np.abs(u1).max() > 0:
                PU.note("u_rel_err_vs_f64_mlp", PU.max_rel(uh[b, kvh], u1))

    # (3) the decode step: MLP query features, cached key features
    topk = inp.topk(frac)
    tmax = int(topk.max())
    wsd = torch.empty(T.workspace_bytes(kv, topk, tmax, T.WS_DECODE_STEP), dtype=torch.uint8, device=dev)
    wsd.fill_(0xA5)
    idx = torch.full((B, Hq, max(tmax, 1)), -7, dtype=torch.int32, device=dev)
    y = torch.full((B, Hq, d), float("nan"), device=dev)
    dbg = torch.full((B, Hq, 4 + d), float("nan"), device=dev)
    y_ns = torch.full((B, Hq, d), float("nan"), device=dev)
    dbg_ns = torch.full((B, Hq, 4 + d), float("nan"), device=dev)
    qd = inp.q[0].to(dev).contiguous()
    td = torch.from_numpy(topk).to(dev)
    mq = _maps(T, pq.to(dev))
    T.decode_step_mlp(kv, mq, cache, qd, topk, td, tmax, S, u, idx if tmax > 0 else None, y, dbg, 0, wsd)
    T.decode_step_mlp(kv, mq, None, qd, topk, td, tmax, S, u, None, y_ns, dbg_ns, T.FLAG_NOSUB, wsd)
    torch.cuda.synchronize()
    assert T.device_status(wsd) == 0
    yh, ih, dh = y.cpu().numpy(), idx.cpu().numpy(), dbg.cpu().numpy()
    ynh, dnh = y_ns.cpu().numpy(), dbg_ns.cpu().numpy()
    for b in range(B):
        lo, hi = int(inp.cu_seqlens[b]), int(inp.cu_seqlens[b + 1])
        for hq in heads:
            kvh = hq // cfg.group
            K, V = PU.seq_arrays(inp, b, kvh)
            q64 = inp.q[0, b, hq].cpu().double().numpy()
            kk = int(topk[b])
            ret = PU.check_selection(q64, K, inp.n_sink, inp.n_tail, kk, ih[b, hq])
            a_q = O.phi_mlp_log(q64, **pq.head(hq))
            Phi_ret = ch[kvh][lo:hi][ret]
            res = O.merge_from_features(q64, K, V, inp.n_sink, inp.n_tail, ret, Sh[b, kvh], uh[b, kvh], a_q, Phi_ret)
            nosub = O.merge_from_features(q64, K, V, inp.n_sink, inp.n_tail, ret, Sh[b, kvh], uh[b, kvh], a_q, Phi_ret,
                                          subtract=False)
            e = PU.note("y_rel_err", PU.max_rel(yh[b, hq], res.y))
            assert e <= PU.Y_TOL, (b, hq, e)
            e = PU.note("y_nosub_rel_err", PU.max_rel(ynh[b, hq], nosub.y))
            assert e <= PU.Y_TOL, (b, hq, e)
            assert PU.note("m_E_abs_err", abs(dh[b, hq, 0] - res.m_E)) <= PU.ME_TOL * max(1.0, abs(res.m_E))
            # the unsubtracted mass log(phi_q . u_M) checks the query-side MLP by itself
            if math.isfinite(nosub.log_Zhat_R):
                e = PU.note("mlp_q_log_mass_abs_err", abs(dnh[b, hq, 2] - nosub.log_Zhat_R))
                assert e <= MLP_Q_LOG_TOL * max(1.0, abs(nosub.log_Zhat_R)), (b, hq, e)
            PU.check_residual(dh[b, hq], res, nosub, (b, hq))
            y0, _ = O.topk_attention(q64, K, V, inp.n_sink, inp.n_tail, kk, retrieved=ret)
            PU.note("visible_y_minus_ytopk", PU.max_rel(res.y, y0))


def test_mlp_phi_1b_geometry_two_sequences():
    cfg = dataclasses.replace(CONFIGS["c1_1b_4k"], n_tail=16)
    _check_mlp(cfg, 3, [1500, 333], 0.02, heads=range(cfg.n_q_heads))


def test_mlp_phi_3b_geometry():
    cfg = dataclasses.replace(CONFIGS["c3_3b_128k"], n_tail=32)
    _check_mlp(cfg, 4, [2100], 0.02, heads=range(0, cfg.n_q_heads, 2))


def test_mlp_phi_smaller_hidden_width_and_short_sequences():
    # d_emb = 256; a sequence with an empty mid-region contributes zero summaries
    cfg = dataclasses.replace(CONFIGS["c1_1b_4k"], n_tail=16)
    _check_mlp(cfg, 5, [700, 18, 129], 0.05, heads=range(0, cfg.n_q_heads, 3), d_emb=256)


def test_mlp_phi_one_full_size_128k_layer_sampled_heads():
    # one layer of the 128K workload in its own geometry and anchors; the oracle runs on two KV heads
    cfg = CONFIGS["c3_3b_128k"]
    _check_mlp(cfg, 0, None, 0.01, heads=[3, 4, 5, 21], on_device=True)


def test_mlp_phi_hidden_width_384_token_major_cache():
    # 128-wide GEMM tiles (384 is not a multiple of 256), keys read through a token-major cache layout
    cfg = dataclasses.replace(CONFIGS["c3_3b_128k"], n_tail=32, n_q_heads=6, n_kv_heads=2)
    _check_mlp(cfg, 6, [900, 517], 0.03, heads=range(cfg.n_q_heads), d_emb=384, token_major=True)
