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

    Exact comparison of the candidate list first.  A bf16 state element that lands on the
    other side of a rounding boundary moves a logit by up to ~1e-3, so near-ties can resolve
    differently and change a whole subtree; where the lists differ the check is therefore
    teacher-forced level by level on the GPU's own intermediates (read from the workspace):
      * every state of level l must equal, within one bf16 ulp, the oracle's stage applied to
        the GPU's parent state and token;
      * the oracle's logits of the GPU's state decide the branches: the GPU's children must be
        the oracle's top-k, or differ only where logits tie within TIE_TOL, with
        child score = parent score + logit - logsumexp within LOGIT_TOL;
      * the returned candidates must be exactly the K best of the GPU's own leaf scores
        (score descending, leaf index ascending) with the tokens on their paths."""

    def __init__(self, ow: oracle.Weights, topk, K):
        self.ow, self.topk, self.K, self.n = ow, tuple(topk), K, len(topk)
        self.tolerated = 0
        self.exact = 0
        self.max_unshared = 0     # most candidates of one tolerated sequence that the oracle's list does not hold

    def check(self, ctx_bits_row: np.ndarray, last_tok: int, gpu_tok: np.ndarray, gpu_logp: np.ndarray,
              levels=None, force_levels: bool = False):
        """levels: dict with lists `state` (fp32 [N_l, d], level l), `tok` and `score` (level l + 1),
        restricted to this sequence."""
        n, K = self.n, self.K
        tol = n * LOGIT_TOL
        o_tok, o_lp = oracle.draft(self.ow, ctx_bits_row[None], np.array([last_tok], np.int32), self.topk, K)
        o_tok, o_lp = o_tok[0], o_lp[0]
        assert (np.diff(gpu_logp) <= 0).all(), "GPU candidates are not sorted by score"
        assert len({tuple(r) for r in gpu_tok}) == K, "GPU candidates are not distinct"
        same = np.array_equal(o_tok, gpu_tok)
        if same:
            assert np.abs(o_lp - gpu_logp).max() <= tol, (o_lp, gpu_logp)
            self.exact += 1
            if not force_levels:
                return
        else:
            self.tolerated += 1
            assert levels is not None, "candidate lists differ and no intermediates were given"
            # what a near-tie can change is the order of neighbours and, at the K-th place, one membership:
            # candidates both lists hold must carry the same score within the tolerance
            theirs = {tuple(r): s for r, s in zip(o_tok.tolist(), o_lp.tolist())}
            ours = {tuple(r): s for r, s in zip(gpu_tok.tolist(), gpu_logp.tolist())}
            shared = set(theirs) & set(ours)
            self.max_unshared = max(self.max_unshared, K - len(shared))
            assert all(abs(theirs[c] - ours[c]) <= tol for c in shared), "shared candidates' scores differ"
        self._check_levels(ctx_bits_row, last_tok, gpu_tok, gpu_logp, levels)

    def _check_levels(self, ctx_bits_row, last_tok, gpu_tok, gpu_logp, lv):
        n, K, topk = self.n, self.K, self.topk
        parent_states = oracle.bf16_bits_to_f32(ctx_bits_row)[None]
        toks_in = np.array([last_tok], np.int32)
        score_in = np.zeros(1, np.float32)
        for l in range(n):
            S = lv["state"][l]
            N = S.shape[0]
            assert N == toks_in.shape[0]
            div = 1 if l == 0 else topk[l - 1]
            for r in range(N):
                s_or = oracle.stage_state(self.ow, l, parent_states[r // div], int(toks_in[r]))
                assert np.allclose(S[r], s_or, rtol=0.008, atol=2e-4), f"level {l} node {r}: state differs"
            logits = oracle.stage_logits(self.ow, l, S)
            k = topk[l]
            ctok, cscore = lv["tok"][l].reshape(N, k), lv["score"][l].reshape(N, k)
            for r in range(N):
                ids, vals = oracle.topk(logits[r], k)
                lse = oracle.logsumexp(logits[r])
                got = logits[r, ctok[r]]
                if not np.array_equal(ids, ctok[r]):
                    assert len(set(ctok[r].tolist())) == k
                    assert (got >= vals[-1] - TIE_TOL).all(), f"level {l} node {r}: not a top-{k} token"
                    assert (np.diff(got) <= TIE_TOL).all(), f"level {l} node {r}: children out of order"
                want = score_in[r] + (got - lse)
                assert np.abs(want - cscore[r]).max() <= LOGIT_TOL, f"level {l} node {r}: child scores"
            parent_states, toks_in, score_in = S, lv["tok"][l], lv["score"][l]
        leaf = lv["score"][n - 1]
        order = np.lexsort((np.arange(leaf.size), -leaf.astype(np.float64)))[:K]
        assert np.array_equal(leaf[order], gpu_logp), "returned scores are not the K best leaf scores"
        for kk, idx in enumerate(order):
            for l in range(n - 1, -1, -1):
                assert gpu_tok[kk, l] == lv["tok"][l][idx], "back-trace of the candidate tokens"
                idx //= topk[l]
