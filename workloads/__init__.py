"""Seeded synthetic inputs for the Top-K+phi decode path.

This package holds tensor generators and workload shapes only.  It contains
none of the method's arithmetic (no scores, no softmax, no feature maps):
both the CPU oracle's tests and the CUDA path's tests and benchmark draw their
inputs from here so that the two sides see identical bits.
"""
from .synthetic import (  # noqa: F401
    CONFIGS,
    WorkloadConfig,
    LayerInputs,
    PhiParams,
    draw_seq_lens,
    make_layer_inputs,
    make_phi_params,
    MlpPhiParams,
    make_mlp_phi_params,
    budget_to_topk,
    bf16_round,
)
