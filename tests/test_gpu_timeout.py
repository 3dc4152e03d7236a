"""The error path of the bounded device-side waits, seen to run: a wait that nothing ends gives
up after its poll limit, the other warp of the CTA is released through the abort flag, the kernel
returns and the status word reads TKPHI_ERR_TIMEOUT; the next ordinary call clears it."""
import dataclasses

import pytest
import torch

from workloads import CONFIGS, make_layer_inputs, make_phi_params

import parity_utils as PU

pytestmark = pytest.mark.gpu


def test_bounded_wait_runs_out_and_reports():
    import paper_2604_05438_b200 as T
    cfg = dataclasses.replace(CONFIGS["c1_1b_4k"], n_q_heads=8, n_kv_heads=2)
    inp = make_layer_inputs(cfg, 31, seq_lens=[1200], n_steps=1)
    gl = PU.to_gpu(cfg, inp, make_phi_params(cfg, 31))
    topk = inp.topk(0.02)
    tmax = int(topk.max())
    ws = torch.zeros(T.workspace_bytes(gl.kv, topk, tmax, T.WS_DECODE_STEP), dtype=torch.uint8, device=gl.dev)
    assert T.device_status(ws) == 0
    T.selftest_timeout(ws)
    torch.cuda.synchronize()                                  # the kernel ends by itself
    assert T.device_status(ws) == T.ERR_TIMEOUT == -5
    # the context is intact and an ordinary call on the same workspace resets the word
    y = torch.empty(1, cfg.n_q_heads, cfg.head_dim, device=gl.dev)
    T.topk_decode(gl.kv, inp.q[0].to(gl.dev), topk, torch.from_numpy(topk).to(gl.dev), tmax, None, y, ws)
    torch.cuda.synchronize()
    assert T.device_status(ws) == 0 and torch.isfinite(y).all()
    # a build workspace likewise
    wsb = torch.zeros(T.workspace_bytes(gl.kv, None, 0, T.WS_BUILD), dtype=torch.uint8, device=gl.dev)
    T.selftest_timeout(wsb)
    assert T.device_status(wsb) == T.ERR_TIMEOUT
    S, u = PU.gpu_build(gl)                                   # (its own workspace; asserts status 0)
    B, Hkv, d, r = 1, cfg.n_kv_heads, cfg.head_dim, cfg.n_feat
    S2 = torch.empty(B, Hkv, d, r, device=gl.dev)
    u2 = torch.empty(B, Hkv, r, device=gl.dev)
    T.build_summaries(gl.kv, gl.maps, S2, u2, wsb)
    torch.cuda.synchronize()
    assert T.device_status(wsb) == 0 and torch.equal(S, S2) and torch.equal(u, u2)


def test_selftest_rejects_bad_workspaces():
    import paper_2604_05438_b200 as T
    ws = torch.zeros(512, dtype=torch.uint8, device="cuda:0")
    with pytest.raises(T.TkphiError):
        T.selftest_timeout(ws[:128])
    with pytest.raises(T.TkphiError):
        T.selftest_timeout(ws[16:400])
