"""Seeded input generators: determinism, shapes and planted structure.  CPU only."""
import dataclasses

import numpy as np
import torch

from workloads import CONFIGS, budget_to_topk, make_layer_inputs, make_phi_params


def _small(name, **kw):
    return dataclasses.replace(CONFIGS[name], **kw)


def test_budgets_match_workload_table():
    assert budget_to_topk(4096, 4, 64, 0.01) == 40
    assert budget_to_topk(32768, 4, 64, 0.01) == 327
    assert [budget_to_topk(131072, 4, 128, f) for f in (0.005, 0.01, 0.02, 0.04)] == [654, 1309, 2618, 5237]
    assert budget_to_topk(1048576, 4, 256, 0.01) == 10483
    assert budget_to_topk(10, 4, 64, 0.5) == 0


def test_deterministic_and_shapes():
    cfg = CONFIGS["c1_1b_4k"]
    a = make_layer_inputs(cfg, 3, seq_lens=[512])
    b = make_layer_inputs(cfg, 3, seq_lens=[512])
    c = make_layer_inputs(cfg, 4, seq_lens=[512])
    assert torch.equal(a.k, b.k) and torch.equal(a.v, b.v) and torch.equal(a.q, b.q)
    assert not torch.equal(a.k, c.k)
    assert a.k.shape == (8, 512, 64) and a.k.dtype == torch.bfloat16
    assert a.q.shape == (16, 1, 32, 64)
    assert a.cu_seqlens.tolist() == [0, 512]


def test_needles_are_identical_rows_in_the_mid_region():
    cfg = CONFIGS["c1_1b_4k"]
    x = make_layer_inputs(cfg, 0, seq_lens=[1024])
    for h in range(cfg.n_kv_heads):
        pos = x.needle_pos[0][h]
        assert len(pos) == 8 and pos.min() >= 4 and pos.max() < 1024 - 64
        rows = x.k[h, torch.from_numpy(pos)]
        assert torch.equal(rows, rows[:1].expand_as(rows))


def test_ragged_lengths_and_zipf_scaling():
    cfg = _small("c4_1b_ragged", batch=4, seq_len=600, seq_len_min=200)
    x = make_layer_inputs(cfg, 1)
    lens = np.diff(x.cu_seqlens)
    assert len(lens) == 4 and lens.min() >= 200 and lens.max() <= 600
    assert x.k.shape[1] == lens.sum()
    cfg5 = _small("c5_3b_1m", batch=1)
    z = make_layer_inputs(cfg5, 0, seq_lens=[3000])
    norms = z.k[0, 4:3000 - 256].float().norm(dim=1)
    assert norms.max() > 20 and norms.median() < 8          # a few large rows, a flat tail


def test_phi_param_kinds():
    cfg = CONFIGS["c3_3b_128k"]
    p = make_phi_params(cfg, 0)
    assert p.w_q.shape == (24, 128, 128) and p.w_k.shape == (8, 128, 128) and p.gamma_k == 0.5
    assert abs(p.w_k.std().item() - 128 ** -0.5) < 0.01
    v = make_phi_params(cfg, 0, kind="visible", bk_shift=torch.arange(8.0))
    assert torch.equal(v.w_q[4], v.w_k[1]) and torch.equal(v.w_q[5], v.w_k[1])
    assert abs(v.b_k[3, 0].item() - (3.0 - 0.5 * np.log(128))) < 1e-5
