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


# ------------------------------------------------------------------ GPU-side plumbing (tests only)
def weights_to_cuda(sw: synth.SpecWeights) -> synth.SpecWeights:
    mv = lambda lst: [t.cuda().contiguous() for t in lst]
    return synth.SpecWeights(sw.cfg, mv(sw.emb), mv(sw.proj), mv(sw.ln_gamma), mv(sw.ln_beta), mv(sw.head),
                             sw.state_weight, sw.emb_weight, sw.ln_eps)


def ws_view(ws: torch.Tensor, offset: int, count: int, dtype: torch.dtype) -> torch.Tensor:
    nbytes = count * torch.empty((), dtype=dtype).element_size()
    return ws[offset:offset + nbytes].view(dtype)


LOGIT_TOL = 2e-2      # max-abs tolerance on head logits (bf16 operands, fp32 accumulation)
TIE_TOL = 1e-3        # logits closer than this may be ordered either way


class DraftChecker:
    """Compares one sequence of a GPU draft with the oracle.

    Exact comparison first; where the candidate lists differ, a teacher-forced check: the
    oracle re-scores every GPU path along the GPU's own tokens and accepts it iff each chosen
    token is in the oracle's top-k at that node or within TIE_TOL (logit) of the oracle's
    k-th value, the path score agrees within n * LOGIT_TOL, and no oracle leaf that the GPU
    left out beats the GPU's K-th score by more than that tolerance."""

    def __init__(self, ow: oracle.Weights, topk, K):
        self.ow, self.topk, self.K, self.n = ow, tuple(topk), K, len(topk)
        self.tolerated = 0
        self.exact = 0

    def _node(self, cache, level, parent_state, prefix):
        key = (level, prefix)
        if key not in cache:
            s = oracle.stage_state(self.ow, level, parent_state, prefix[-1])
            lg = oracle.stage_logits(self.ow, level, s[None])[0]
            cache[key] = (s, lg, oracle.logsumexp(lg))
        return cache[key]

    def check(self, ctx_bits_row: np.ndarray, last_tok: int, gpu_tok: np.ndarray, gpu_logp: np.ndarray):
        n, K = self.n, self.K
        tol = n * LOGIT_TOL
        o_tok, o_lp = oracle.draft(self.ow, ctx_bits_row[None], np.array([last_tok], np.int32), self.topk, K)
        o_tok, o_lp = o_tok[0], o_lp[0]
        assert (np.diff(gpu_logp) <= 0).all(), "GPU candidates are not sorted by score"
        assert len({tuple(r) for r in gpu_tok}) == K, "GPU candidates are not distinct"
        if np.array_equal(o_tok, gpu_tok):
            assert np.abs(o_lp - gpu_logp).max() <= tol, (o_lp, gpu_logp)
            self.exact += 1
            return
        self.tolerated += 1
        cache = {}
        ctx = oracle.bf16_bits_to_f32(ctx_bits_row)
        for k in range(K):
            state, prefix, score = ctx, (int(last_tok),), 0.0
            for l in range(n):
                s, lg, lse = self._node(cache, l, state, prefix)
                t = int(gpu_tok[k, l])
                kth = np.sort(lg)[-self.topk[l]]
                assert lg[t] >= kth - TIE_TOL, f"cand {k} level {l}: token {t} is not a top-{self.topk[l]} token"
                score += float(lg[t] - lse)
                state, prefix = s, prefix + (t,)
            assert abs(score - gpu_logp[k]) <= tol, (k, score, gpu_logp[k])
        gpu_set = {tuple(r) for r in gpu_tok}
        for k in range(K):
            if tuple(o_tok[k]) not in gpu_set:
                assert o_lp[k] <= gpu_logp[K - 1] + tol, f"oracle leaf {k} was dropped although it scores higher"
