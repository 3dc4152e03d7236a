"""Seeded synthetic tensors shaped like the paper's decode setting.

The paper evaluates frozen Llama-3.2-1B/3B-Instruct backbones on long-context
suites (Sec. 5.1); neither the checkpoints nor the suites are available here,
so random tensors with the same head geometry, context lengths, anchor counts
and exact-support budgets stand in for them.  Everything is drawn from a
seeded ``torch.Generator`` so that the CPU oracle and the CUDA kernels read the
same bits.  No attention arithmetic lives in this file.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np
import torch


@dataclass(frozen=True)
class WorkloadConfig:
    """Shape of one synthetic workload (one row of the workload table)."""

    name: str
    batch: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_feat: int
    seq_len: int                 # prefill length N (upper bound when ragged)
    n_sink: int
    n_tail: int
    budgets: tuple               # fractions of the mid-region retrieved exactly
    n_steps: int
    seq_len_min: Optional[int] = None   # ragged: lengths uniform in [min, seq_len]
    needles_per_head: Optional[int] = None   # fixed count, or
    needle_every: Optional[int] = None       # one needle per this many tokens
    zipf_key_norms: bool = False
    topic_queries: bool = True   # queries correlated with the planted needles

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads


CONFIGS: Dict[str, WorkloadConfig] = {
    # Single layer, Llama-3.2-1B head geometry, N=4096.
    "c1_1b_4k": WorkloadConfig("c1_1b_4k", 1, 1, 32, 8, 64, 64, 4096, 4, 64,
                               (0.01,), 16, needles_per_head=8),
    # 16 layers, 1B geometry, N=32768.
    "c2_1b_32k": WorkloadConfig("c2_1b_32k", 1, 16, 32, 8, 64, 64, 32768, 4, 64,
                                (0.01,), 64, needle_every=1024),
    # 28 layers, Llama-3.2-3B geometry, N=131072, budget sweep.
    "c3_3b_128k": WorkloadConfig("c3_3b_128k", 1, 28, 24, 8, 128, 128, 131072, 4, 128,
                                 (0.005, 0.01, 0.02, 0.04), 32, needle_every=4096),
    # 32 ragged sequences, 1B geometry.
    "c4_1b_ragged": WorkloadConfig("c4_1b_ragged", 32, 16, 32, 8, 64, 64, 65536, 4, 64,
                                   (0.01,), 16, seq_len_min=8192, topic_queries=False),
    # one 3B-geometry layer, 4 x 1M tokens, Zipf-scaled key norms.
    "c5_3b_1m": WorkloadConfig("c5_3b_1m", 4, 1, 24, 8, 128, 128, 1048576, 4, 256,
                               (0.01,), 8, zipf_key_norms=True, topic_queries=False),
}


def budget_to_topk(n_tokens: int, n_sink: int, n_tail: int, frac: float) -> int:
    """Retrieved-token count for a budget given as a fraction of the mid-region."""
    n_mid = max(0, n_tokens - n_sink - n_tail)
    return int(math.floor(frac * n_mid + 1e-9))


def bf16_round(x: torch.Tensor) -> torch.Tensor:
    """Round an fp32 tensor to bf16 (round-to-nearest-even)."""
    return x.to(torch.bfloat16)


@dataclass
class PhiParams:
    """Parameters of phi(x) = exp(W x + b - gamma * ||x||^2), fp32."""

    w_q: torch.Tensor   # [H_q, r, d]
    b_q: torch.Tensor   # [H_q, r]
    w_k: torch.Tensor   # [H_kv, r, d]
    b_k: torch.Tensor   # [H_kv, r]
    gamma_q: float
    gamma_k: float
    kind: str = "baseline"

    def to(self, device) -> "PhiParams":
        return PhiParams(self.w_q.to(device), self.b_q.to(device), self.w_k.to(device),
                         self.b_k.to(device), self.gamma_q, self.gamma_k, self.kind)


@dataclass
class LayerInputs:
    """One attention layer of a workload: ragged K/V cache plus decode queries."""

    cu_seqlens: np.ndarray            # int64 [B+1], token offsets into the cache
    k: torch.Tensor                   # bf16 [H_kv, T_total, d]
    v: torch.Tensor                   # bf16 [H_kv, T_total, d]
    q: torch.Tensor                   # bf16 [n_steps, B, H_q, d]
    n_sink: int
    n_tail: int
    needle_pos: List[List[np.ndarray]] = field(default_factory=list)  # [B][H_kv] positions

    @property
    def batch(self) -> int:
        return len(self.cu_seqlens) - 1

    def seq_len(self, b: int) -> int:
        return int(self.cu_seqlens[b + 1] - self.cu_seqlens[b])

    def topk(self, frac: float) -> np.ndarray:
        return np.array([budget_to_topk(self.seq_len(b), self.n_sink, self.n_tail, frac)
                         for b in range(self.batch)], dtype=np.int32)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def make_phi_params(cfg: WorkloadConfig, seed: int, kind: str = "baseline",
                    device="cpu", bk_shift: Optional[torch.Tensor] = None) -> PhiParams:
    """Random-init feature-map parameters.

    kind="baseline": separate maps, W entries ~ N(0, 1/d), b ~ N(0, 0.1^2),
        gamma = 1/2 for both sides.
    kind="visible": every query head shares its KV head's projection, rows
        ~ N(0, I) / d^(1/4), gamma = 1/(2 sqrt d), b = -ln(r)/2; an optional
        per-KV-head shift is added to b_k (callers use it to put the residual
        branch on the same scale as the exact branch).
    """
    d, r = cfg.head_dim, cfg.n_feat
    g = _gen(seed * 7919 + 17, device)
    if kind == "baseline":
        w_q = torch.randn(cfg.n_q_heads, r, d, generator=g, device=device) / math.sqrt(d)
        w_k = torch.randn(cfg.n_kv_heads, r, d, generator=g, device=device) / math.sqrt(d)
        b_q = 0.1 * torch.randn(cfg.n_q_heads, r, generator=g, device=device)
        b_k = 0.1 * torch.randn(cfg.n_kv_heads, r, generator=g, device=device)
        gq = gk = 0.5
    elif kind == "visible":
        w_k = torch.randn(cfg.n_kv_heads, r, d, generator=g, device=device) / d ** 0.25
        w_q = w_k.repeat_interleave(cfg.group, dim=0).clone()
        b_q = torch.full((cfg.n_q_heads, r), -0.5 * math.log(r), device=device)
        b_k = torch.full((cfg.n_kv_heads, r), -0.5 * math.log(r), device=device)
        if bk_shift is not None:
            b_k = b_k + bk_shift.to(device=device, dtype=torch.float32).reshape(-1, 1)
        gq = gk = 1.0 / (2.0 * math.sqrt(d))
    else:
        raise ValueError(f"unknown phi kind {kind!r}")
    return PhiParams(w_q.float().contiguous(), b_q.float().contiguous(),
                     w_k.float().contiguous(), b_k.float().contiguous(), gq, gk, kind)


@dataclass
class MlpPhiParams:
    """Parameters of one side's one-block ReZero-MLP feature maps (hidden width d_emb), fp32;
    the leading dimension runs over the heads of that side."""

    w_s: torch.Tensor   # [H, d_emb, d]
    b_s: torch.Tensor   # [H, d_emb]
    w_1: torch.Tensor   # [H, d_emb, d_emb]
    b_1: torch.Tensor   # [H, d_emb]
    w_2: torch.Tensor   # [H, d_emb, d_emb]
    b_2: torch.Tensor   # [H, d_emb]
    alpha: torch.Tensor  # [H]
    w_o: torch.Tensor   # [H, r, d_emb]
    b_o: torch.Tensor   # [H, r]

    def to(self, device) -> "MlpPhiParams":
        return MlpPhiParams(*[getattr(self, f).to(device) for f in
                              ("w_s", "b_s", "w_1", "b_1", "w_2", "b_2", "alpha", "w_o", "b_o")])

    def head(self, h: int) -> dict:
        """float64 numpy arrays of head h, keyed like the feature map's symbols."""
        return dict(W_s=self.w_s[h].double().numpy(), b_s=self.b_s[h].double().numpy(),
                    W_1=self.w_1[h].double().numpy(), b_1=self.b_1[h].double().numpy(),
                    W_2=self.w_2[h].double().numpy(), b_2=self.b_2[h].double().numpy(),
                    alpha=float(self.alpha[h]), W_o=self.w_o[h].double().numpy(), b_o=self.b_o[h].double().numpy())


def make_mlp_phi_params(cfg: WorkloadConfig, seed: int, side: str, d_emb: int = 512, device="cpu",
                        bo_shift: Optional[torch.Tensor] = None) -> MlpPhiParams:
    """Random-init ReZero-MLP feature maps for the query side (one per query head) or the key side
    (one per KV head): weights ~ N(0, 1/fan_in), biases ~ N(0, 0.1^2), alpha ~ U(0.3, 0.7) (a trained
    gate is not zero), output rows scaled by 1/2 so that the exponents stay within a few units.
    An optional per-head shift is added to b_o."""
    H = cfg.n_q_heads if side == "q" else cfg.n_kv_heads
    d, r = cfg.head_dim, cfg.n_feat
    g = _gen(seed * 104729 + (1 if side == "q" else 2), device)
    rn = lambda *shape: torch.randn(*shape, generator=g, device=device)
    w_s = rn(H, d_emb, d) / math.sqrt(d)
    b_s = 0.1 * rn(H, d_emb)
    w_1 = rn(H, d_emb, d_emb) / math.sqrt(d_emb)
    b_1 = 0.1 * rn(H, d_emb)
    w_2 = rn(H, d_emb, d_emb) / math.sqrt(d_emb)
    b_2 = 0.1 * rn(H, d_emb)
    alpha = 0.3 + 0.4 * torch.rand(H, generator=g, device=device)
    w_o = 0.5 * rn(H, r, d_emb) / math.sqrt(d_emb)
    b_o = 0.1 * rn(H, r)
    if bo_shift is not None:
        b_o = b_o + bo_shift.to(device=device, dtype=torch.float32).reshape(-1, 1)
    return MlpPhiParams(*[t.float().contiguous() for t in (w_s, b_s, w_1, b_1, w_2, b_2, alpha, w_o, b_o)])


def draw_seq_lens(cfg: WorkloadConfig, seed: int) -> List[int]:
    """Prefill lengths of the workload's sequences: uniform in [seq_len_min, seq_len] for ragged
    workloads (the same for every layer of a seed), else seq_len for all."""
    if cfg.seq_len_min is None:
        return [cfg.seq_len] * cfg.batch
    gl = np.random.default_rng(seed * 7 + 3)
    return [int(x) for x in gl.integers(cfg.seq_len_min, cfg.seq_len + 1, size=cfg.batch)]


def make_layer_inputs(cfg: WorkloadConfig, seed: int, layer: int = 0, device="cpu",
                      seq_lens: Optional[List[int]] = None,
                      n_steps: Optional[int] = None) -> LayerInputs:
    """Draw one layer's K/V cache and decode queries for ``cfg``.

    K and V are iid N(0,1) rounded to bf16.  Per (sequence, KV head) a topic
    vector g ~ N(0, I) is drawn; needle keys are bf16(3 g) at distinct random
    mid-region positions (bit-identical, so their scores tie exactly), and,
    when ``cfg.topic_queries``, the queries of that head group are
    bf16(0.25 g + sqrt(1 - 0.25^2) eps).  With ``cfg.zipf_key_norms`` each key
    row i of a (sequence, KV head) is scaled by 3 * rank_i^(-1.1/4) for a random
    ranking of the rows.  ``seq_lens`` overrides the lengths (tests use small
    ones); ragged configs draw lengths uniformly in [seq_len_min, seq_len].
    """
    g = _gen(seed * 1000003 + layer * 101 + 1, device)
    B, Hq, Hkv, d = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    if seq_lens is None:
        seq_lens = draw_seq_lens(cfg, seed)
    B = len(seq_lens)
    steps = cfg.n_steps if n_steps is None else n_steps
    cu = np.zeros(B + 1, dtype=np.int64)
    cu[1:] = np.cumsum(seq_lens)
    T = int(cu[-1])
    k = torch.empty(Hkv, T, d, dtype=torch.bfloat16, device=device)
    v = torch.empty(Hkv, T, d, dtype=torch.bfloat16, device=device)
    # fill in slabs so that the fp32 temporaries stay small at 1M-token sizes
    slab = max(1, (1 << 24) // d)
    for h in range(Hkv):
        for t0 in range(0, T, slab):
            t1 = min(T, t0 + slab)
            k[h, t0:t1] = torch.randn(t1 - t0, d, generator=g, device=device).to(torch.bfloat16)
            v[h, t0:t1] = torch.randn(t1 - t0, d, generator=g, device=device).to(torch.bfloat16)
    topic = torch.randn(B, Hkv, d, generator=g, device=device)
    eps = torch.randn(steps, B, Hq, d, generator=g, device=device)
    if cfg.topic_queries:
        t = topic.repeat_interleave(cfg.group, dim=1).unsqueeze(0)      # [1,B,Hq,d]
        q = 0.25 * t + math.sqrt(1.0 - 0.25 ** 2) * eps
    else:
        q = eps
    q = q.to(torch.bfloat16).contiguous()
    needle_pos: List[List[np.ndarray]] = []
    rs = np.random.default_rng(seed * 31 + layer * 5 + 11)
    for b in range(B):
        n_b = seq_lens[b]
        lo, hi = cfg.n_sink, n_b - cfg.n_tail
        row: List[np.ndarray] = []
        for h in range(Hkv):
            n_mid = max(0, hi - lo)
            if cfg.needles_per_head is not None:
                n_needle = min(cfg.needles_per_head, n_mid)
            elif cfg.needle_every is not None:
                n_needle = min(n_b // cfg.needle_every, n_mid)
            else:
                n_needle = 0
            if cfg.zipf_key_norms and n_mid > 0:
                perm = torch.from_numpy(rs.permutation(n_mid) + 1).to(device=device,
                                                                        dtype=torch.float32)
                scale = 3.0 * perm.pow(-1.1 / 4.0)
                seg = k[h, cu[b] + lo: cu[b] + hi].float() * scale.unsqueeze(1)
                k[h, cu[b] + lo: cu[b] + hi] = seg.to(torch.bfloat16)
            if n_needle > 0:
                pos = np.sort(rs.choice(n_mid, size=n_needle, replace=False)) + lo
                k[h, torch.from_numpy(cu[b] + pos).to(device)] = \
                    (3.0 * topic[b, h]).to(torch.bfloat16)
                row.append(pos.astype(np.int64))
            else:
                row.append(np.zeros(0, dtype=np.int64))
        needle_pos.append(row)
    return LayerInputs(cu, k, v, q, cfg.n_sink, cfg.n_tail, needle_pos)
