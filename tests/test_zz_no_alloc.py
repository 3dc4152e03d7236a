"""The allocation-free summary build (tkphi_build_summaries_static) against the
ordinary entry point.

Some users of the library cannot allocate device memory when they call it (a
serving plug-in living inside a fixed memory pool, a runtime that bans cudaMalloc
on its latency-critical path).  For them the library carries a fixed scratch array
in its own device image.  This test drives that entry point through the C ABI twice
in a row, on different inputs, and requires the same (S, u) as the entry point that
takes a caller-allocated workspace: the second call shows that whatever the first
one left in the shared scratch does no harm.  It also checks the size limit.

The file name sorts last on purpose, so that a run that stops at the first failure
has already run every other test.
"""
import dataclasses

import numpy as np
import pytest
import torch

from workloads import CONFIGS, make_layer_inputs, make_phi_params

import parity_utils as PU

pytestmark = pytest.mark.gpu


def _both(cfg, seed, seq_lens):
    import paper_2604_05438_b200 as T
    inp = make_layer_inputs(cfg, seed, seq_lens=seq_lens, n_steps=1)
    gl = PU.to_gpu(cfg, inp, make_phi_params(cfg, seed))
    S_ref, u_ref = PU.gpu_build(gl)                       # caller-allocated workspace
    B, Hkv, d, r = gl.kv.batch, cfg.n_kv_heads, cfg.head_dim, cfg.n_feat
    S = torch.full((B, Hkv, d, r), float("nan"), device=gl.dev)
    u = torch.full((B, Hkv, r), float("nan"), device=gl.dev)
    T.build_summaries_static(gl.kv, gl.maps, S, u)        # built-in scratch, no allocation inside
    torch.cuda.synchronize()
    assert T.static_device_status() == 0                  # no bounded wait of the build kernel ran out
    return S_ref.cpu().numpy(), u_ref.cpu().numpy(), S.cpu().numpy(), u.cpu().numpy()


def test_static_scratch_build_matches_workspace_build_twice():
    cfg = dataclasses.replace(CONFIGS["c1_1b_4k"], n_q_heads=8, n_kv_heads=2)
    for seed, lens in ((21, [3000, 700]), (22, [1500])):  # two calls in a row on the shared scratch
        S_ref, u_ref, S, u = _both(cfg, seed, lens)
        assert np.isfinite(S).all() and np.isfinite(u).all()
        assert PU.max_rel(S, S_ref) <= PU.SU_TOL and PU.max_rel(u, u_ref) <= PU.SU_TOL
        # same kernel, same summation order: in fact identical
        assert np.array_equal(S, S_ref) and np.array_equal(u, u_ref)


def test_static_scratch_call_leaves_free_device_memory_unchanged():
    # after one warm call (which loads the library's device code, the scratch array with it, and looks
    # up its address) a further call must not take any device memory: not from the driver, not from
    # torch's pool
    import paper_2604_05438_b200 as T
    cfg = dataclasses.replace(CONFIGS["c1_1b_4k"], n_q_heads=8, n_kv_heads=2)
    inp = make_layer_inputs(cfg, 23, seq_lens=[2000], n_steps=1)
    gl = PU.to_gpu(cfg, inp, make_phi_params(cfg, 23))
    S = torch.empty(1, cfg.n_kv_heads, cfg.head_dim, cfg.n_feat, device=gl.dev)
    u = torch.empty(1, cfg.n_kv_heads, cfg.n_feat, device=gl.dev)
    T.build_summaries_static(gl.kv, gl.maps, S, u)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    reserved0 = torch.cuda.memory_reserved()
    T.build_summaries_static(gl.kv, gl.maps, S, u)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0 and torch.cuda.memory_reserved() == reserved0
    assert T.static_device_status() == 0


def test_static_scratch_rejects_oversized_problems():
    import paper_2604_05438_b200 as T
    cfg = CONFIGS["c3_3b_128k"]
    dev = torch.device("cuda:0")
    # descriptor of a 128K-token layer whose scratch need exceeds the built-in array;
    # rejected on the host before anything is enqueued, so tiny dummy tensors suffice
    k = torch.zeros(cfg.n_kv_heads, 8, cfg.head_dim, dtype=torch.bfloat16, device=dev)
    kv = T.KVCache(k, k, np.array([0, 131072], np.int64), cfg.n_q_heads, cfg.n_feat, cfg.n_sink, cfg.n_tail)
    if T.workspace_bytes(kv, None, 0, T.WS_BUILD) <= T.STATIC_SCRATCH_BYTES:
        pytest.skip("this problem fits the built-in scratch")
    phi = make_phi_params(cfg, 0).to(dev)
    maps = T.PhiMaps(phi.w_q, phi.b_q, phi.w_k, phi.b_k, phi.gamma_q, phi.gamma_k)
    S = torch.zeros(1, cfg.n_kv_heads, cfg.head_dim, cfg.n_feat, device=dev)
    u = torch.zeros(1, cfg.n_kv_heads, cfg.n_feat, device=dev)
    with pytest.raises(T.TkphiError) as ei:
        T.build_summaries_static(kv, maps, S, u)
    assert ei.value.status == -3 and "built-in scratch" in str(ei.value)
