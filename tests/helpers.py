"""Shared test plumbing: conversions between the seeded input tensors and the oracle's numpy view."""
import numpy as np
import torch

import oracle
from paper_2404_19124_b200 import synth


def to_oracle_weights(sw: synth.SpecWeights, round_state_bf16: bool = True) -> oracle.Weights:
    cfg = sw.cfg
    return oracle.Weights(
        V=cfg.V, d_base=cfg.d_base, d_inner=cfg.d_inner,
        emb=[synth.bf16_bits(t) for t in sw.emb],
        proj=[synth.bf16_bits(t) for t in sw.proj],
        ln_gamma=[t.detach().cpu().numpy().astype(np.float32) for t in sw.ln_gamma],
        ln_beta=[t.detach().cpu().numpy().astype(np.float32) for t in sw.ln_beta],
        head=[synth.bf16_bits(t) for t in sw.head],
        state_weight=sw.state_weight, emb_weight=sw.emb_weight, ln_eps=sw.ln_eps,
        round_state_bf16=round_state_bf16)


def small_cfg(name="small", d_base=48, d_inner=32, V=40, topk=(3, 2, 2), K=5, B=2, seed=7, std=None):
    return synth.SpecConfig(name, d_base, d_inner, V, tuple(topk), K, B, std, 1.0, "none", seed)


def f64(t: torch.Tensor) -> torch.Tensor:
    return t.detach().cpu().to(torch.float64)
