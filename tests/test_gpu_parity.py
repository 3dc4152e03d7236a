"""CUDA path vs float64 oracle, element by element, through the C ABI.  Needs a GPU."""
import dataclasses
import math

import numpy as np
import pytest
import torch

from oracle import tkphi_oracle as O
from workloads import CONFIGS, make_layer_inputs, make_phi_params

import parity_utils as PU

pytestmark = pytest.mark.gpu


def _cfg(name, **kw):
    return dataclasses.replace(CONFIGS[name], **kw)


def _phi_arrays(phi, hq, kvh):
    return (phi.w_q[hq].double().numpy(), phi.b_q[hq].double().numpy(), phi.gamma_q,
            phi.w_k[kvh].double().numpy(), phi.b_k[kvh].double().numpy(), phi.gamma_k)


def _check_build(gl, S, u, heads=None):
    cfg, inp, phi = gl.cfg, gl.inp, gl.phi
    Sh, uh = S.cpu().numpy(), u.cpu().numpy()
    assert np.isfinite(Sh).all() and np.isfinite(uh).all()
    worst = 0.0
    for b in range(inp.batch):
        for kvh in (range(cfg.n_kv_heads) if heads is None else heads):
            K, V = PU.seq_arrays(inp, b, kvh)
            S0, u0 = O.build_summaries(K, V, phi.w_k[kvh].double().numpy(), phi.b_k[kvh].double().numpy(),
                                       phi.gamma_k, inp.n_sink, inp.n_tail)
            if np.abs(S0).max() == 0:
                assert np.abs(Sh[b, kvh]).max() == 0 and np.abs(uh[b, kvh]).max() == 0
                continue
            if np.abs(S0).max() < PU.FP32_TINY and np.abs(u0).max() < PU.FP32_TINY:
                # every feature underflows fp32 (the summaries are plain fp32 sums)
                assert np.abs(Sh[b, kvh]).max() < PU.FP32_TINY and np.abs(uh[b, kvh]).max() < PU.FP32_TINY
                continue
            eS, eu = PU.note("S_rel_err", PU.max_rel(Sh[b, kvh], S0)), PU.note("u_rel_err", PU.max_rel(uh[b, kvh], u0))
            worst = max(worst, eS, eu)
            assert eS <= PU.SU_TOL and eu <= PU.SU_TOL, (b, kvh, eS, eu)
    return worst


def _check_decode(gl, step, frac, S, u, with_phi=True, flags=0, heads=None, topk=None, topk_max=None,
                  check_resid=True):
    cfg, inp, phi = gl.cfg, gl.inp, gl.phi
    topk = inp.topk(frac) if topk is None else np.asarray(topk, np.int32)
    q = inp.q[step]
    out = PU.gpu_decode(gl, q, topk, S, u, with_phi=with_phi, flags=flags, topk_max=topk_max)
    Sh = None if S is None else S.cpu().double().numpy()
    uh = None if u is None else u.cpu().double().numpy()
    G = cfg.group
    worst = 0.0
    for b in range(inp.batch):
        for hq in (range(cfg.n_q_heads) if heads is None else heads):
            kvh = hq // G
            K, V = PU.seq_arrays(inp, b, kvh)
            q64 = q[b, hq].double().numpy()
            kk = int(topk[b])
            if out["idx"] is not None and (topk_max or topk.max()) > 0:
                ret = PU.check_selection(q64, K, inp.n_sink, inp.n_tail, kk, out["idx"][b, hq])
            else:
                ret = O.select_topk(q64, K, inp.n_sink, inp.n_tail, kk)
            if with_phi:
                res = O.topkphi_attention(q64, K, V, inp.n_sink, inp.n_tail, kk, *_phi_arrays(phi, hq, kvh),
                                          S=Sh[b, kvh], u=uh[b, kvh], retrieved=ret,
                                          subtract=not (flags & 1))
                y0 = res.y
                dbg = out["dbg"][b, hq]
                if math.isfinite(res.m_E):
                    assert PU.note("m_E_abs_err", abs(dbg[0] - res.m_E)) <= PU.ME_TOL * max(1.0, abs(res.m_E)), \
                        (b, hq, dbg[0], res.m_E)
                    assert PU.note("Z_E_rel_err", abs(dbg[1] - res.Z_E) / res.Z_E) <= 1e-4
                if check_resid:
                    nosub = res if (flags & 1) else O.topkphi_attention(
                        q64, K, V, inp.n_sink, inp.n_tail, kk, *_phi_arrays(phi, hq, kvh),
                        S=Sh[b, kvh], u=uh[b, kvh], retrieved=ret, subtract=False)
                    PU.check_residual(dbg, res, nosub, (b, hq))
            else:
                y0, _ = O.topk_attention(q64, K, V, inp.n_sink, inp.n_tail, kk, retrieved=ret)
            e = PU.note("y_rel_err" if with_phi else "y_topk_rel_err", PU.max_rel(out["y"][b, hq], y0))
            worst = max(worst, e)
            assert e <= PU.Y_TOL, (b, hq, e)
    return worst


# ------------------------------------------------------------------ config 1, full size
@pytest.mark.parametrize("seed", [0, 1])
def test_c1_full_size_topk_and_topkphi(seed):
    cfg = CONFIGS["c1_1b_4k"]
    inp = make_layer_inputs(cfg, seed, n_steps=3)
    phi = make_phi_params(cfg, seed)
    gl = PU.to_gpu(cfg, inp, phi)
    S, u = PU.gpu_build(gl)
    _check_build(gl, S, u)
    for step in range(3):
        _check_decode(gl, step, 0.01, None, None, with_phi=False)
        _check_decode(gl, step, 0.01, S, u, with_phi=True)


def test_c1_visible_residual_phi():
    cfg = CONFIGS["c1_1b_4k"]
    inp = make_layer_inputs(cfg, 2, n_steps=2)
    phi0 = make_phi_params(cfg, 2, kind="visible")
    shift = PU.calibrate_visible_shift(cfg, inp, phi0, 0.01)
    phi = make_phi_params(cfg, 2, kind="visible", bk_shift=shift)
    gl = PU.to_gpu(cfg, inp, phi)
    S, u = PU.gpu_build(gl)
    _check_build(gl, S, u)
    for step in range(2):
        _check_decode(gl, step, 0.01, S, u)
        _check_decode(gl, step, 0.01, S, u, flags=1)          # NoSub ablation
    # the residual must actually matter here: Top-K+phi differs visibly from Top-K
    out_phi = PU.gpu_decode(gl, inp.q[0], inp.topk(0.01), S, u)
    out_top = PU.gpu_decode(gl, inp.q[0], inp.topk(0.01), with_phi=False)
    assert np.abs(out_phi["y"] - out_top["y"]).max() > 1e-2


# ------------------------------------------------------------------ 3B geometry, several tiles + ragged tail
@pytest.mark.parametrize("kind", ["baseline", "visible"])
def test_c3_geometry_reduced_length(kind):
    cfg = _cfg("c3_3b_128k", needle_every=512)
    inp = make_layer_inputs(cfg, 0, seq_lens=[5000], n_steps=2)
    phi = make_phi_params(cfg, 0, kind=kind)
    if kind == "visible":
        phi = make_phi_params(cfg, 0, kind=kind, bk_shift=PU.calibrate_visible_shift(cfg, inp, phi, 0.02))
    gl = PU.to_gpu(cfg, inp, phi)
    S, u = PU.gpu_build(gl)
    _check_build(gl, S, u)
    for frac in (0.005, 0.04):
        _check_decode(gl, 0, frac, S, u)
    _check_decode(gl, 1, 0.02, None, None, with_phi=False)


# ------------------------------------------------------------------ ragged batch (config 4 shape, small lengths)
def test_c4_ragged_batch():
    cfg = _cfg("c4_1b_ragged", batch=5)
    inp = make_layer_inputs(cfg, 3, seq_lens=[700, 69, 2049, 68, 1300], n_steps=1)
    phi = make_phi_params(cfg, 3)
    gl = PU.to_gpu(cfg, inp, phi)
    S, u = PU.gpu_build(gl)
    _check_build(gl, S, u)
    topk = inp.topk(0.05)
    assert topk.tolist()[1] == 0 and topk.tolist()[3] == 0
    _check_decode(gl, 0, 0.05, S, u, topk=topk, topk_max=int(topk.max()) + 5)
    _check_decode(gl, 0, 0.05, None, None, with_phi=False, topk=topk)


@pytest.mark.parametrize("n_feat", [128, 64])
def test_many_rows_take_the_streaming_exact_kernel(n_feat):
    # 8 sequences x 24 query heads = 192 rows, each at least one slice pair: more pairs than SMs at
    # head_dim 128, so the persistent, software-pipelined exact/residual kernel runs (items of
    # different length, KV head changes and sequence boundaries inside a CTA's range)
    cfg = _cfg("c3_3b_128k", batch=8, needle_every=256, n_feat=n_feat)
    inp = make_layer_inputs(cfg, 7, seq_lens=[900, 300, 133, 1500, 700, 2049, 132, 1100], n_steps=1)
    phi0 = make_phi_params(cfg, 7, kind="visible")
    phi = make_phi_params(cfg, 7, kind="visible", bk_shift=PU.calibrate_visible_shift(cfg, inp, phi0, 0.2))
    gl = PU.to_gpu(cfg, inp, phi)
    S, u = PU.gpu_build(gl)
    topk = inp.topk(0.2)
    assert int(topk.max()) > 256 and int(topk.min()) == 0      # several slice pairs for some heads, none retrieved for others
    _check_decode(gl, 0, 0.2, S, u, topk=topk, heads=range(0, 24, 5))
    _check_decode(gl, 0, 0.2, S, u, topk=topk, flags=1, heads=[1, 22])
    _check_decode(gl, 0, 0.2, None, None, with_phi=False, topk=topk, heads=[2, 17])


@pytest.mark.parametrize("layout", ["token_major", "padded_heads"])
def test_streaming_exact_kernel_other_cache_layouts(layout):
    # token-major caches gather rows as token * H + head; a cache whose head stride is not a multiple of
    # its token stride has no 2-D row view: the call then runs the one-shot kernel with 16-byte copies
    import paper_2604_05438_b200 as T
    cfg = _cfg("c3_3b_128k", batch=8, needle_every=256)
    inp = make_layer_inputs(cfg, 8, seq_lens=[900, 300, 133, 1500, 700, 2049, 132, 1100], n_steps=1)
    phi = make_phi_params(cfg, 8)
    gl = PU.to_gpu(cfg, inp, phi, token_major=(layout == "token_major"))
    if layout == "padded_heads":
        H, Tn, d = inp.k.shape
        def padded(x):
            store = torch.zeros(H, Tn * d + 8, dtype=x.dtype, device=gl.dev)
            view = store[:, : Tn * d].view(H, Tn, d)
            view.copy_(x.to(gl.dev))
            return view
        k, v = padded(inp.k), padded(inp.v)
        assert k.stride(0) == Tn * d + 8
        gl.kv = T.KVCache(k, v, inp.cu_seqlens, cfg.n_q_heads, cfg.n_feat, inp.n_sink, inp.n_tail)
    S, u = PU.gpu_build(gl)
    topk = inp.topk(0.2)
    _check_decode(gl, 0, 0.2, S, u, topk=topk, heads=[0, 7, 23])


def test_one_cta_row_budgets_from_one_key_to_half_the_row():
    # a row of 8192..16384 mid keys is selected by a single CTA; budgets from one key to half of the
    # row, needles give exact ties at the threshold
    cfg = _cfg("c1_1b_4k", needle_every=300)
    inp = make_layer_inputs(cfg, 9, seq_lens=[12000], n_steps=1)
    gl = PU.to_gpu(cfg, inp, make_phi_params(cfg, 9))
    n_mid = 12000 - inp.n_sink - inp.n_tail
    for k in (1, 119, n_mid // 8, n_mid // 8 + 1, n_mid // 2):
        _check_decode(gl, 0, 0.0, None, None, with_phi=False, topk=[k], heads=[0, 5, 31])


def test_c5_zipf_norms_reduced_length():
    cfg = _cfg("c5_3b_1m", batch=2)
    inp = make_layer_inputs(cfg, 1, seq_lens=[6000, 3001], n_steps=1)
    phi = make_phi_params(cfg, 1)
    gl = PU.to_gpu(cfg, inp, phi)
    S, u = PU.gpu_build(gl)
    _check_build(gl, S, u)
    _check_decode(gl, 0, 0.01, S, u, heads=range(0, 24, 5))


# ------------------------------------------------------------------ layouts and head groupings
def test_token_major_layout_and_group_of_eight():
    cfg = _cfg("c1_1b_4k", n_q_heads=16, n_kv_heads=2)        # G = 8: two scoring passes
    inp = make_layer_inputs(cfg, 5, seq_lens=[1500], n_steps=1)
    phi = make_phi_params(cfg, 5)
    gl = PU.to_gpu(cfg, inp, phi, token_major=True)
    S, u = PU.gpu_build(gl)
    _check_build(gl, S, u)
    _check_decode(gl, 0, 0.03, S, u)


def test_mixed_dims_d64_r128_and_d128_r64():
    for d, r in ((64, 128), (128, 64)):
        cfg = _cfg("c1_1b_4k", head_dim=d, n_feat=r, n_q_heads=6, n_kv_heads=2)   # G = 3
        inp = make_layer_inputs(cfg, 6, seq_lens=[900], n_steps=1)
        phi = make_phi_params(cfg, 6)
        gl = PU.to_gpu(cfg, inp, phi)
        S, u = PU.gpu_build(gl)
        _check_build(gl, S, u)
        _check_decode(gl, 0, 0.02, S, u)


# ------------------------------------------------------------------ degenerate cases
def test_budget_edges_zero_and_full():
    cfg = _cfg("c1_1b_4k", n_q_heads=8, n_kv_heads=2)
    inp = make_layer_inputs(cfg, 7, seq_lens=[600], n_steps=1)
    phi0 = make_phi_params(cfg, 7, kind="visible")
    phi = make_phi_params(cfg, 7, kind="visible", bk_shift=PU.calibrate_visible_shift(cfg, inp, phi0, 0.05))
    gl = PU.to_gpu(cfg, inp, phi)
    S, u = PU.gpu_build(gl)
    n_mid = 600 - 68
    # K = 0: anchors plus the whole-mid residual
    _check_decode(gl, 0, 0.0, S, u, topk=[0])
    _check_decode(gl, 0, 0.0, None, None, with_phi=False, topk=[0])
    # K = 1 and K = |M| - 1
    _check_decode(gl, 0, 0.0, S, u, topk=[1])
    _check_decode(gl, 0, 0.0, S, u, topk=[n_mid - 1])
    # K = |M|: residual summaries cancel -> full attention (invariant of the method)
    out = PU.gpu_decode(gl, inp.q[0], np.array([n_mid], np.int32), S, u)
    assert (out["idx"][0, :, :n_mid] == np.arange(4, 600 - 64)).all()
    for hq in range(cfg.n_q_heads):
        K, V = PU.seq_arrays(inp, 0, hq // cfg.group)
        y_full = O.full_attention(inp.q[0, 0, hq].double().numpy(), K, V)
        assert PU.max_rel(out["y"][0, hq], y_full) <= PU.Y_TOL


def test_no_anchors_and_tiny_sequences():
    cfg = _cfg("c1_1b_4k", n_q_heads=4, n_kv_heads=1, n_sink=0, n_tail=0)
    inp = make_layer_inputs(cfg, 8, seq_lens=[1, 257, 33], n_steps=1)
    phi = make_phi_params(cfg, 8)
    gl = PU.to_gpu(cfg, inp, phi)
    S, u = PU.gpu_build(gl)
    _check_build(gl, S, u)
    _check_decode(gl, 0, 0.0, S, u, topk=[1, 30, 33])
    _check_decode(gl, 0, 0.0, None, None, with_phi=False, topk=[1, 256, 2])
    # anchors longer than the sequence: everything is an anchor
    cfg2 = _cfg("c1_1b_4k", n_q_heads=4, n_kv_heads=1)
    inp2 = make_layer_inputs(cfg2, 9, seq_lens=[3, 68, 70], n_steps=1)
    gl2 = PU.to_gpu(cfg2, inp2, make_phi_params(cfg2, 9))
    S2, u2 = PU.gpu_build(gl2)
    _check_build(gl2, S2, u2)
    _check_decode(gl2, 0, 0.0, S2, u2, topk=[0, 0, 2])
    _check_decode(gl2, 0, 0.0, None, None, with_phi=False, topk=[0, 0, 1])


def test_exact_ties_break_towards_lower_index():
    cfg = _cfg("c1_1b_4k", n_q_heads=4, n_kv_heads=1, needles_per_head=0)
    inp = make_layer_inputs(cfg, 10, seq_lens=[1000], n_steps=1)
    # every mid key identical -> every score ties exactly; then plant blocks of duplicates
    inp.k[0, 4:936] = inp.k[0, 4].clone()
    gl = PU.to_gpu(cfg, inp, make_phi_params(cfg, 10))
    out = PU.gpu_decode(gl, inp.q[0], np.array([37], np.int32), with_phi=False)
    assert (out["idx"][0, :, :37] == np.arange(4, 41)).all()
    inp2 = make_layer_inputs(cfg, 11, seq_lens=[3000], n_steps=1)
    src = inp2.k[0, 100:110].clone()
    for rep in range(40):                       # 40 copies of 10 distinct rows, spread out
        inp2.k[0, 200 + rep * 60: 210 + rep * 60] = src
    gl2 = PU.to_gpu(cfg, inp2, make_phi_params(cfg, 11))
    for kk in (5, 57, 203, 411):
        _check_decode(gl2, 0, 0.0, None, None, with_phi=False, topk=[kk])


def test_generated_tokens_stay_exact():
    """Decode after n_gen generated tokens (Eq. implemented_decode): summaries from the prefill,
    then a decode call whose tail-anchor count is n_tail + n_gen over the grown cache."""
    import paper_2604_05438_b200 as T
    cfg = _cfg("c1_1b_4k", n_q_heads=8, n_kv_heads=2)
    L, n_gen = 2000, 37
    inp = make_layer_inputs(cfg, 13, seq_lens=[L + n_gen], n_steps=1)
    phi0 = make_phi_params(cfg, 13, kind="visible")
    pre = dataclasses.replace(inp, cu_seqlens=np.array([0, L], np.int64), k=inp.k[:, :L].contiguous(),
                              v=inp.v[:, :L].contiguous())
    phi = make_phi_params(cfg, 13, kind="visible", bk_shift=PU.calibrate_visible_shift(cfg, pre, phi0, 0.02))
    gl_pre = PU.to_gpu(cfg, pre, phi)
    S, u = PU.gpu_build(gl_pre)                              # prefill state
    grown = dataclasses.replace(inp, n_tail=cfg.n_tail + n_gen)
    gl = PU.to_gpu(cfg, grown, phi)                          # cache with the generated rows appended
    topk = np.array([39], np.int32)
    out = PU.gpu_decode(gl, inp.q[0], topk, S, u)
    Sh, uh = S.cpu().double().numpy(), u.cpu().double().numpy()
    for hq in range(cfg.n_q_heads):
        kvh = hq // cfg.group
        K, V = PU.seq_arrays(inp, 0, kvh)
        q64 = inp.q[0, 0, hq].double().numpy()
        ret = PU.check_selection(q64, K[:L], cfg.n_sink, cfg.n_tail, 39, out["idx"][0, hq])
        y0, _ = O.topkphi_attention_generated(q64, K, V, L, cfg.n_sink, cfg.n_tail, 39, *_phi_arrays(phi, hq, kvh),
                                              S=Sh[0, kvh], u=uh[0, kvh], retrieved=ret)
        assert PU.max_rel(out["y"][0, hq], y0) <= PU.Y_TOL, hq


def test_sequences_with_different_tail_counts_share_a_call():
    """Per-sequence tail-anchor counts (n_tail_seq): the build takes a different n_tail per sequence, and
    the decode call n_tail_b + n_gen_b over caches that have grown by different numbers of generated tokens."""
    import paper_2604_05438_b200 as T
    cfg = _cfg("c1_1b_4k", n_q_heads=8, n_kv_heads=2)
    dev = torch.device("cuda:0")
    L = [1500, 700, 300]
    tails = np.array([16, 40, 3], np.int32)
    n_gen = np.array([37, 0, 5], np.int32)
    inp = make_layer_inputs(cfg, 17, seq_lens=[l + int(g) for l, g in zip(L, n_gen)], n_steps=1)
    phi = make_phi_params(cfg, 17, kind="visible", bk_shift=torch.full((cfg.n_kv_heads,), 2.0))
    # prefill cache: the first L_b rows of every sequence
    rows = np.concatenate([np.arange(int(inp.cu_seqlens[b]), int(inp.cu_seqlens[b]) + L[b]) for b in range(3)])
    cu_pre = np.concatenate([[0], np.cumsum(L)]).astype(np.int64)
    kp, vp = inp.k[:, rows].contiguous().to(dev), inp.v[:, rows].contiguous().to(dev)
    kv_pre = T.KVCache(kp, vp, cu_pre, cfg.n_q_heads, cfg.n_feat, cfg.n_sink, 999, n_tail_seq=tails)   # n_tail itself is ignored
    pd = phi.to(dev)
    maps = T.PhiMaps(pd.w_q, pd.b_q, pd.w_k, pd.b_k, pd.gamma_q, pd.gamma_k)
    B, Hq, Hkv, d, r = 3, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_feat
    S = torch.full((B, Hkv, d, r), float("nan"), device=dev)
    u = torch.full((B, Hkv, r), float("nan"), device=dev)
    wsb = torch.empty(T.workspace_bytes(kv_pre, None, 0, T.WS_BUILD), dtype=torch.uint8, device=dev)
    T.build_summaries(kv_pre, maps, S, u, wsb)
    # decode over the grown caches
    kv = T.KVCache(inp.k.to(dev), inp.v.to(dev), inp.cu_seqlens, cfg.n_q_heads, cfg.n_feat, cfg.n_sink, 0,
                   n_tail_seq=tails + n_gen)
    topk = np.array([29, 13, 6], np.int32)
    tmax = int(topk.max())
    ws = torch.empty(T.workspace_bytes(kv, topk, tmax, T.WS_DECODE_STEP), dtype=torch.uint8, device=dev)
    idx = torch.full((B, Hq, tmax), -7, dtype=torch.int32, device=dev)
    y = torch.full((B, Hq, d), float("nan"), device=dev)
    T.decode_step(kv, maps, inp.q[0].to(dev).contiguous(), topk, torch.from_numpy(topk).to(dev), tmax, S, u, idx, y,
                  None, 0, ws)
    torch.cuda.synchronize()
    assert T.device_status(ws) == 0 and T.device_status(wsb) == 0
    Sh, uh, yh, ih = S.cpu().double().numpy(), u.cpu().double().numpy(), y.cpu().numpy(), idx.cpu().numpy()
    for b in range(B):
        for kvh in range(Hkv):
            K, V = PU.seq_arrays(inp, b, kvh)
            S0, u0 = O.build_summaries(K[:L[b]], V[:L[b]], phi.w_k[kvh].double().numpy(), phi.b_k[kvh].double().numpy(),
                                       phi.gamma_k, cfg.n_sink, int(tails[b]))
            assert PU.note("S_rel_err", PU.max_rel(Sh[b, kvh], S0)) <= PU.SU_TOL, (b, kvh)
            assert PU.note("u_rel_err", PU.max_rel(uh[b, kvh], u0)) <= PU.SU_TOL, (b, kvh)
        for hq in range(Hq):
            kvh = hq // cfg.group
            K, V = PU.seq_arrays(inp, b, kvh)
            q64 = inp.q[0, b, hq].double().numpy()
            kk = int(topk[b])
            ret = PU.check_selection(q64, K[:L[b]], cfg.n_sink, int(tails[b]), kk, ih[b, hq])
            y0, _ = O.topkphi_attention_generated(q64, K, V, L[b], cfg.n_sink, int(tails[b]), kk, *_phi_arrays(phi, hq, kvh),
                                                  S=Sh[b, kvh], u=uh[b, kvh], retrieved=ret)
            assert PU.note("y_rel_err", PU.max_rel(yh[b, hq], y0)) <= PU.Y_TOL, (b, hq)


def test_results_are_run_to_run_identical():
    cfg = CONFIGS["c1_1b_4k"]
    inp = make_layer_inputs(cfg, 12, seq_lens=[2500], n_steps=1)
    gl = PU.to_gpu(cfg, inp, make_phi_params(cfg, 12))
    S, u = PU.gpu_build(gl)
    S2, u2 = PU.gpu_build(gl)
    assert torch.equal(S, S2) and torch.equal(u, u2)
    a = PU.gpu_decode(gl, inp.q[0], inp.topk(0.02), S, u)
    b = PU.gpu_decode(gl, inp.q[0], inp.topk(0.02), S, u)
    assert np.array_equal(a["y"], b["y"]) and np.array_equal(a["idx"], b["idx"])


def test_decode_step_is_capturable_in_a_cuda_graph():
    """The library allocates nothing and synchronises nothing, so a decode step (three launches chained as
    programmatic dependents) can be captured once and replayed; the replay gives the eager result bit for bit."""
    import paper_2604_05438_b200 as T
    cfg = CONFIGS["c1_1b_4k"]
    inp = make_layer_inputs(cfg, 21, seq_lens=[3000, 1200], n_steps=2)
    gl = PU.to_gpu(cfg, inp, make_phi_params(cfg, 21))
    S, u = PU.gpu_build(gl)
    dev = gl.dev
    topk = inp.topk(0.02)
    tmax = int(topk.max())
    B, Hq, d = gl.kv.batch, cfg.n_q_heads, cfg.head_dim
    ws = torch.empty(T.workspace_bytes(gl.kv, topk, tmax, T.WS_DECODE_STEP), dtype=torch.uint8, device=dev)
    td = torch.from_numpy(topk).to(dev)
    q = inp.q[0].to(dev).contiguous()
    y = torch.zeros(B, Hq, d, device=dev)
    idx = torch.zeros(B, Hq, tmax, dtype=torch.int32, device=dev)
    T.decode_step(gl.kv, gl.maps, q, topk, td, tmax, S, u, idx, y, None, 0, ws)        # eager (also warms up)
    torch.cuda.synchronize()
    y_eager, idx_eager = y.clone(), idx.clone()
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            T.decode_step(gl.kv, gl.maps, q, topk, td, tmax, S, u, idx, y, None, 0, ws, stream=stream)
    y.zero_()
    idx.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert T.device_status(ws) == 0
    assert torch.equal(y, y_eager) and torch.equal(idx, idx_eager)
    q.copy_(inp.q[1].to(dev))                                                           # new query, same graph
    graph.replay()
    torch.cuda.synchronize()
    y_replay = y.clone()
    T.decode_step(gl.kv, gl.maps, q, topk, td, tmax, S, u, idx, y, None, 0, ws)
    torch.cuda.synchronize()
    assert torch.equal(y, y_replay)


def test_per_sequence_tails_in_the_streaming_exact_kernel():
    """Per-sequence tail-anchor counts on a call large enough for the persistent exact/residual kernel
    (head_dim 128, more slice pairs than SMs): every item of that kernel takes its sequence's own tail."""
    import paper_2604_05438_b200 as T
    cfg = _cfg("c3_3b_128k", batch=8, needle_every=256)
    dev = torch.device("cuda:0")
    lens = [900, 300, 133, 1500, 700, 2049, 132, 1100]
    tails = np.array([128, 7, 0, 300, 64, 512, 200, 1], np.int32)
    inp = make_layer_inputs(cfg, 23, seq_lens=lens, n_steps=1)
    phi = make_phi_params(cfg, 23, kind="visible", bk_shift=torch.full((cfg.n_kv_heads,), 3.0))
    kv = T.KVCache(inp.k.to(dev), inp.v.to(dev), inp.cu_seqlens, cfg.n_q_heads, cfg.n_feat, cfg.n_sink, 5, n_tail_seq=tails)
    pd = phi.to(dev)
    maps = T.PhiMaps(pd.w_q, pd.b_q, pd.w_k, pd.b_k, pd.gamma_q, pd.gamma_k)
    B, Hq, Hkv, d, r = 8, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_feat
    S = torch.full((B, Hkv, d, r), float("nan"), device=dev)
    u = torch.full((B, Hkv, r), float("nan"), device=dev)
    wsb = torch.empty(T.workspace_bytes(kv, None, 0, T.WS_BUILD), dtype=torch.uint8, device=dev)
    T.build_summaries(kv, maps, S, u, wsb)
    n_mid = np.maximum(0, np.array(lens) - cfg.n_sink - tails)
    topk = np.floor(0.2 * n_mid).astype(np.int32)
    tmax = int(topk.max())
    assert tmax > 256 and int(topk.min()) == 0
    ws = torch.empty(T.workspace_bytes(kv, topk, tmax, T.WS_DECODE_STEP), dtype=torch.uint8, device=dev)
    idx = torch.full((B, Hq, tmax), -7, dtype=torch.int32, device=dev)
    y = torch.full((B, Hq, d), float("nan"), device=dev)
    dbg = torch.full((B, Hq, 4 + d), float("nan"), device=dev)
    T.decode_step(kv, maps, inp.q[0].to(dev).contiguous(), topk, torch.from_numpy(topk).to(dev), tmax, S, u, idx, y,
                  dbg, 0, ws)
    torch.cuda.synchronize()
    assert T.device_status(ws) == 0 and T.device_status(wsb) == 0
    Sh, uh, yh, ih, dh = S.cpu().double().numpy(), u.cpu().double().numpy(), y.cpu().numpy(), idx.cpu().numpy(), dbg.cpu().numpy()
    for b in range(B):
        nt = int(tails[b])
        for hq in range(0, Hq, 5):
            kvh = hq // cfg.group
            K, V = PU.seq_arrays(inp, b, kvh)
            if hq == 0 and n_mid[b] > 0:
                S0, u0 = O.build_summaries(K, V, phi.w_k[kvh].double().numpy(), phi.b_k[kvh].double().numpy(),
                                           phi.gamma_k, cfg.n_sink, nt)
                assert PU.note("S_rel_err", PU.max_rel(Sh[b, kvh], S0)) <= PU.SU_TOL, b
            q64 = inp.q[0, b, hq].double().numpy()
            kk = int(topk[b])
            ret = PU.check_selection(q64, K, cfg.n_sink, nt, kk, ih[b, hq])
            pa = _phi_arrays(phi, hq, kvh)
            res = O.topkphi_attention(q64, K, V, cfg.n_sink, nt, kk, *pa, S=Sh[b, kvh], u=uh[b, kvh], retrieved=ret)
            nosub = O.topkphi_attention(q64, K, V, cfg.n_sink, nt, kk, *pa, S=Sh[b, kvh], u=uh[b, kvh], retrieved=ret,
                                        subtract=False)
            assert PU.note("y_rel_err", PU.max_rel(yh[b, hq], res.y)) <= PU.Y_TOL, (b, hq)
            PU.check_residual(dh[b, hq], res, nosub, (b, hq))
