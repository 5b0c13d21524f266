"""Seeded synthetic inputs for the draft + verify path.

This module only draws random tensors of the right shapes, dtypes and distributions; it
holds none of the method's arithmetic and imports neither the CUDA binding nor the CPU
oracle, so both can be fed identical bytes from it.

The presets mirror the shapes the paper works with (Sec. 4: vocabulary of 32k, latent
width 4096, base widths 4096 / 5120, 3 heads for language models and more for code
models, branching such as 6/3/2 pruned to k candidates, weights initialised with standard
deviation d^-1/2) and stand in for its real workloads (trained speculators driven by
Llama2 / Codellama / Granite on web documents), which are not available here.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch


@dataclass(frozen=True)
class SpecConfig:
    name: str
    d_base: int
    d_inner: int
    V: int
    topk: Tuple[int, ...]
    K: int
    B: int
    weight_std: Optional[float]   # None: N(0, 1/sqrt(fan_in)) per matrix; float: fixed std
    logits_std: float
    plant: str                    # "none" | "bernoulli40" | "prefix"
    seed: int

    @property
    def n(self) -> int:
        return len(self.topk)

    @property
    def leaves(self) -> int:
        return int(np.prod(self.topk))

    def nodes(self, level: int) -> int:
        """Nodes entering head `level` (rows of that head's vocabulary GEMM)."""
        return self.B * int(np.prod(self.topk[:level]))

    def d_in(self, level: int) -> int:
        return self.d_base if level == 0 else self.d_inner


CONFIGS: Dict[str, SpecConfig] = {c.name: c for c in [
    SpecConfig("tiny", 256, 256, 1024, (4, 3, 2), 8, 1, 0.02, 1.0, "none", 0),
    SpecConfig("llama2-7b", 4096, 3072, 32000, (4, 3, 2), 16, 8, None, 2.0, "none", 1),
    SpecConfig("llama2-13b", 5120, 4096, 32000, (6, 4, 3), 32, 16, None, 2.0, "bernoulli40", 2),
    SpecConfig("codellama-34b", 8192, 4096, 32000, (4, 3, 2, 2), 16, 32, None, 2.0, "prefix", 3),
    SpecConfig("llama3-8b", 4096, 3072, 128256, (8, 4, 3, 2), 64, 64, None, 2.0, "none", 4),
]}


def mix_weights(n_heads: int, emb_std: float) -> Tuple[float, float]:
    """Scalars (a, b) of the state/embedding mix.

    Sec. 4 asks that the base model's state account for half of the variance of the state
    at the last head.  Treating the projected state and the scaled embedding as
    independent and unit-variance, the base share after n stages is a^(2n) = 1/2, and b
    scales an embedding of per-element std `emb_std` to the remaining variance 1 - a^2.
    """
    a = 2.0 ** (-1.0 / (2.0 * n_heads))
    b = math.sqrt(1.0 - a * a) / emb_std
    return float(a), float(b)


def _gen(seed: int, device: str) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _normal_bf16(shape: Sequence[int], std: float, g: torch.Generator, device: str) -> torch.Tensor:
    # draw in fp32 in slabs (keeps the fp32 temporary small), scale, round to bf16
    out = torch.empty(tuple(shape), dtype=torch.bfloat16, device=device)
    flat = out.view(-1)
    step = 1 << 26
    for s in range(0, flat.numel(), step):
        e = min(flat.numel(), s + step)
        flat[s:e] = (torch.randn(e - s, generator=g, device=device, dtype=torch.float32) * std).to(torch.bfloat16)
    return out


@dataclass
class SpecWeights:
    cfg: SpecConfig
    emb: List[torch.Tensor]       # bf16 [V, d_inner]
    proj: List[torch.Tensor]      # bf16 [d_inner, d_in]
    ln_gamma: List[torch.Tensor]  # fp32 [d_inner]
    ln_beta: List[torch.Tensor]   # fp32 [d_inner]
    head: List[torch.Tensor]      # bf16 [V, d_inner]
    state_weight: float
    emb_weight: float
    ln_eps: float = 1e-5


def make_weights(cfg: SpecConfig, device: str = "cpu") -> SpecWeights:
    g = _gen(1000 + cfg.seed, device)
    emb, proj, gam, bet, head = [], [], [], [], []
    emb_std = cfg.weight_std if cfg.weight_std is not None else cfg.d_inner ** -0.5
    for l in range(cfg.n):
        d_in = cfg.d_in(l)
        std_p = cfg.weight_std if cfg.weight_std is not None else d_in ** -0.5
        std_h = cfg.weight_std if cfg.weight_std is not None else cfg.d_inner ** -0.5
        emb.append(_normal_bf16((cfg.V, cfg.d_inner), emb_std, g, device))
        proj.append(_normal_bf16((cfg.d_inner, d_in), std_p, g, device))
        gam.append(1.0 + 0.02 * torch.randn(cfg.d_inner, generator=g, device=device, dtype=torch.float32))
        bet.append(0.02 * torch.randn(cfg.d_inner, generator=g, device=device, dtype=torch.float32))
        head.append(_normal_bf16((cfg.V, cfg.d_inner), std_h, g, device))
    a, b = mix_weights(cfg.n, emb_std)
    return SpecWeights(cfg, emb, proj, gam, bet, head, a, b)


def make_draft_inputs(cfg: SpecConfig, device: str = "cpu", B: Optional[int] = None):
    """ctx_state bf16 [B, d_base] ~ N(0,1); last_tok int32 [B] uniform in [0, V)."""
    B = cfg.B if B is None else B
    g = _gen(2000 + cfg.seed, device)
    ctx = _normal_bf16((B, cfg.d_base), 1.0, g, device)
    tok = torch.randint(0, cfg.V, (B,), generator=g, device=device, dtype=torch.int64).to(torch.int32)
    return ctx, tok


def random_cand_tok(cfg: SpecConfig, device: str = "cpu", B: Optional[int] = None, K: Optional[int] = None):
    B = cfg.B if B is None else B
    K = cfg.K if K is None else K
    g = _gen(4000 + cfg.seed, device)
    return torch.randint(0, cfg.V, (B, K, cfg.n), generator=g, device=device, dtype=torch.int64).to(torch.int32)


def make_base_logits(cfg: SpecConfig, cand_tok: torch.Tensor, device: str = "cpu",
                     dtype: torch.dtype = torch.bfloat16, B: Optional[int] = None, K: Optional[int] = None):
    """base_logits [B, K, n+1, V] ~ N(0, logits_std), optionally with planted matches.

    plant == "bernoulli40": each (b,k,j<n) row independently, with probability 0.4, gets
      +40 at the candidate's token (so that row's argmax equals the candidate).
    plant == "prefix": per (b,k) a match length m uniform in 0..n is drawn; rows j<m get
      +40 at the candidate token and row m (when m<n) gets +40 at a different token.
    `cand_tok` only selects where the planted values go.
    """
    B = cfg.B if B is None else B
    K = cfg.K if K is None else K
    n, V = cfg.n, cfg.V
    g = _gen(3000 + cfg.seed, device)
    out = torch.empty((B, K, n + 1, V), dtype=dtype, device=device)
    flat = out.view(-1)
    step = 1 << 26
    for s in range(0, flat.numel(), step):
        e = min(flat.numel(), s + step)
        flat[s:e] = (torch.randn(e - s, generator=g, device=device, dtype=torch.float32) * cfg.logits_std).to(dtype)
    ct = cand_tok.to(device=device, dtype=torch.int64)
    assert ct.shape == (B, K, n)
    if cfg.plant == "bernoulli40":
        mask = torch.rand((B, K, n), generator=g, device=device) < 0.4
        b, k, j = torch.nonzero(mask, as_tuple=True)
        out[b, k, j, ct[b, k, j]] = 40.0
    elif cfg.plant == "prefix":
        m = torch.randint(0, n + 1, (B, K), generator=g, device=device)
        jj = torch.arange(n, device=device).view(1, 1, n)
        match = jj < m.unsqueeze(-1)
        b, k, j = torch.nonzero(match, as_tuple=True)
        out[b, k, j, ct[b, k, j]] = 40.0
        b, k = torch.nonzero(m < n, as_tuple=True)
        mm = m[b, k]
        out[b, k, mm, (ct[b, k, mm] + 1) % V] = 40.0
    return out


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 bit patterns (host copy)."""
    assert t.dtype == torch.bfloat16
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
