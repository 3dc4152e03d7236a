"""Cached key features (Sec. 4.2 mentions a cached implementation): the summary build also stores
every mid-region phi_k row; the decode step takes the retrieved tokens' rows from that cache instead
of recomputing them.  Against the float64 oracle, element by element, through the C ABI."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import tkphi_oracle as O
from workloads import CONFIGS, make_layer_inputs, make_phi_params

import parity_utils as PU

pytestmark = pytest.mark.gpu

CACHE_TOL = 1e-4      # fp32 features: an exponent of magnitude up to ~60 keeps 60 x 2^-23 = 7e-6 per rounding (a few roundings), W_k hi+lo 2e-6, exp2.approx 2^-22


def _cached_layer(cfg, seed, seq_lens, frac):
    import paper_2604_05438_b200 as T
    inp = make_layer_inputs(cfg, seed, seq_lens=seq_lens, n_steps=1)
    phi0 = make_phi_params(cfg, seed, kind="visible")
    phi = make_phi_params(cfg, seed, kind="visible", bk_shift=PU.calibrate_visible_shift(cfg, inp, phi0, frac))
    gl = PU.to_gpu(cfg, inp, phi)
    T_total = int(inp.cu_seqlens[-1])
    cache = torch.full((cfg.n_kv_heads, T_total, cfg.n_feat), float("nan"), device=gl.dev)
    gl_c = dataclasses.replace(gl, maps=dataclasses.replace(gl.maps, phi_k_cache=cache))
    return inp, phi, gl, gl_c, cache


def _check_cached(cfg, seed, seq_lens, frac, heads=None):
    inp, phi, gl, gl_c, cache = _cached_layer(cfg, seed, seq_lens, frac)
    S_plain, u_plain = PU.gpu_build(gl)
    S, u = PU.gpu_build(gl_c)
    assert torch.equal(S, S_plain) and torch.equal(u, u_plain)        # the cache is a by-product of the same build
    ch = cache.cpu().double().numpy()
    G = cfg.group
    topk = inp.topk(frac)
    out = PU.gpu_decode(gl_c, inp.q[0], topk, S, u)
    out_re = PU.gpu_decode(gl, inp.q[0], topk, S, u)                  # recompute path on the same summaries
    Sh, uh = S.cpu().double().numpy(), u.cpu().double().numpy()
    for b in range(inp.batch):
        lo, hi = int(inp.cu_seqlens[b]), int(inp.cu_seqlens[b + 1])
        L = hi - lo
        for kvh in range(cfg.n_kv_heads):
            K, V = PU.seq_arrays(inp, b, kvh)
            Phi = O.phi(K, phi.w_k[kvh].double().numpy(), phi.b_k[kvh].double().numpy(), phi.gamma_k)
            mid = slice(min(inp.n_sink, L), max(min(inp.n_sink, L), L - inp.n_tail))
            got = ch[kvh, lo:hi]
            if mid.stop > mid.start:
                err = np.abs(got[mid] - Phi[mid]).max() / np.abs(Phi[mid]).max()
                assert PU.note("phi_cache_rel_err", err) <= CACHE_TOL, (b, kvh, err)
            assert np.isnan(got[:mid.start]).all() and np.isnan(got[mid.stop:]).all()   # anchor rows untouched
        for hq in (range(cfg.n_q_heads) if heads is None else heads):
            kvh = hq // G
            K, V = PU.seq_arrays(inp, b, kvh)
            q64 = inp.q[0, b, hq].double().numpy()
            kk = int(topk[b])
            ret = PU.check_selection(q64, K, inp.n_sink, inp.n_tail, kk, out["idx"][b, hq])
            Phi_c = np.nan_to_num(ch[kvh, lo:hi])
            pa = (phi.w_q[hq].double().numpy(), phi.b_q[hq].double().numpy(), phi.gamma_q)
            res = O.topkphi_attention_cached(q64, K, V, inp.n_sink, inp.n_tail, kk, *pa, Phi_c, Sh[b, kvh], uh[b, kvh],
                                             retrieved=ret)
            nosub = O.topkphi_attention_cached(q64, K, V, inp.n_sink, inp.n_tail, kk, *pa, Phi_c, Sh[b, kvh], uh[b, kvh],
                                               retrieved=ret, subtract=False)
            assert PU.note("y_rel_err", PU.max_rel(out["y"][b, hq], res.y)) <= PU.Y_TOL, (b, hq)
            PU.check_residual(out["dbg"][b, hq], res, nosub, (b, hq))
            # and the method does not change: the same output as with recomputed features
            exact = O.topkphi_attention(q64, K, V, inp.n_sink, inp.n_tail, kk, *pa,
                                        phi.w_k[kvh].double().numpy(), phi.b_k[kvh].double().numpy(), phi.gamma_k,
                                        S=Sh[b, kvh], u=uh[b, kvh], retrieved=ret)
            assert PU.max_rel(out["y"][b, hq], exact.y) <= PU.Y_TOL
            assert PU.note("y_cached_vs_recomputed", PU.max_rel(out["y"][b, hq], out_re["y"][b, hq])) <= PU.Y_TOL


def test_cached_features_c1_geometry():
    _check_cached(CONFIGS["c1_1b_4k"], 41, [3000, 500], 0.02)


def test_cached_features_c3_geometry_one_shot_kernel():
    cfg = dataclasses.replace(CONFIGS["c3_3b_128k"], needle_every=512)
    _check_cached(cfg, 42, [5000], 0.03)


def test_cached_features_streaming_kernel():
    # more slice pairs than SMs at head_dim 128: the persistent exact/residual kernel takes the cached z
    cfg = dataclasses.replace(CONFIGS["c3_3b_128k"], batch=8, needle_every=256)
    _check_cached(cfg, 43, [900, 300, 133, 1500, 700, 2049, 132, 1100], 0.2, heads=range(0, 24, 5))


def test_cached_features_mixed_dims():
    for d, r in ((64, 128), (128, 64)):
        cfg = dataclasses.replace(CONFIGS["c1_1b_4k"], head_dim=d, n_feat=r, n_q_heads=6, n_kv_heads=2)
        _check_cached(cfg, 44, [900], 0.03)
