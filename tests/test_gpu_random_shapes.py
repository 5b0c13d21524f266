"""Seeded random shapes through the C ABI against the oracle: ragged vocabularies and widths, row counts
around the 128-row tile, every number of heads, branching factors up to the limit, both logits dtypes and
both verify forms.  Small sizes, so the oracle recomputes everything."""
import numpy as np
import pytest
import torch

import oracle
from paper_2404_19124_b200 import synth
from helpers import DraftChecker, small_cfg, to_oracle_weights, weights_to_cuda, ws_view

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2404_19124_b200 import build
    build.build()
    from paper_2404_19124_b200 import binding
    return binding


def _draft_case(rng):
    n = int(rng.integers(1, 5))
    topk = tuple(int(rng.integers(1, 9 if n <= 2 else 4)) for _ in range(n))
    L = int(np.prod(topk))
    K = int(rng.integers(1, L + 1))
    Bn = int(rng.choice([1, 2, 3, 5, 17, 40]))
    V = int(rng.choice([8, 24, 40, 264, 1000, 1096, 3000])) if max(topk) <= 8 else 1000
    V = max(V, max(topk))
    d_base = int(rng.choice([16, 48, 72, 128, 200]))
    d = int(rng.choice([16, 32, 64, 136, 256]))
    return topk, K, Bn, V, d_base, d


@pytest.mark.parametrize("case", range(14))
def test_draft_random_shapes(B, case):
    rng = np.random.default_rng(1000 + case)
    topk, K, Bn, V, d_base, d = _draft_case(rng)
    cfg = small_cfg(d_base=d_base, d_inner=d, V=V, topk=topk, K=K, B=Bn, seed=200 + case)
    sw = synth.make_weights(cfg)
    ow, gw = to_oracle_weights(sw), weights_to_cuda(sw)
    ctx, tok = synth.make_draft_inputs(cfg)
    h = B.spec_create(gw)
    if case % 3 == 2 and d % 16 == 0:
        B.spec_attach_fp8_heads(h)          # every third case through the e4m3 heads
    elif case % 3 == 1:
        B.spec_set_option(h, B.SPEC_OPT_HEAD_SWAP_MAX_ROWS, 128)   # every third case: nodes as MMA columns
        B.spec_set_option(h, B.SPEC_OPT_HEAD_PAIR, 1)              # ... up to 128 nodes, CTA pairs above
    cand_tok, cand_logp, ws = B.spec_draft(h, ctx.cuda(), tok.cuda(), cfg.topk, cfg.K)
    assert B.spec_poll_error(ws) == 0
    ct, lp = cand_tok.cpu().numpy(), cand_logp.cpu().numpy()
    lay = B.spec_draft_layout(h, cfg.B, cfg.topk, cfg.K)
    chk = DraftChecker(ow, cfg.topk, cfg.K)
    ctx_bits = synth.bf16_bits(ctx)
    for b in range(cfg.B):
        st, tk, sc = [], [], []
        for l in range(cfg.n):
            per, N = cfg.nodes(l) // cfg.B, cfg.nodes(l)
            S = ws_view(ws, lay.state[l], N * cfg.d_inner, torch.bfloat16).view(N, cfg.d_inner)
            st.append(S[b * per:(b + 1) * per].to(torch.float32).cpu().numpy())
            N1 = cfg.nodes(l + 1)
            per1 = N1 // cfg.B
            tk.append(ws_view(ws, lay.tok[l + 1], N1, torch.int32)[b * per1:(b + 1) * per1].cpu().numpy())
            sc.append(ws_view(ws, lay.score[l + 1], N1, torch.float32)[b * per1:(b + 1) * per1].cpu().numpy())
        chk.check(ctx_bits[b], int(tok[b]), ct[b], lp[b], levels={"state": st, "tok": tk, "score": sc},
                  force_levels=(b == 0))
    assert chk.exact + chk.tolerated == cfg.B
    B.spec_destroy(h)


@pytest.mark.parametrize("case", range(24))
def test_verify_random_shapes(B, case):
    rng = np.random.default_rng(5000 + case)
    Bn, K, n = int(rng.integers(1, 9)), int(rng.integers(1, 33)), int(rng.integers(1, 8))
    V = int(rng.choice([1, 5, 8, 64, 1000, 1021, 4096, 32000, 50264]))
    dtype = torch.bfloat16 if case % 2 == 0 else torch.float32
    g = torch.Generator().manual_seed(case)
    logits = (torch.randn(Bn, K, n + 1, V, generator=g) * 2).to(dtype)
    if case % 5 == 0:
        logits[..., : max(1, V // 3)] = logits[..., :1]                 # long runs of equal values
    cand = torch.randint(0, V, (Bn, K, n), generator=g, dtype=torch.int64).to(torch.int32)
    am = logits.to(torch.float32).argmax(-1)
    for b in range(Bn):
        for k in range(K):
            m = int(rng.integers(0, n + 1))
            cand[b, k, :m] = am[b, k, :m].to(torch.int32)
    ln = synth.bf16_bits(logits) if dtype == torch.bfloat16 else logits.numpy()
    want = oracle.verify(cand.numpy(), ln, oracle.BF16 if dtype == torch.bfloat16 else oracle.F32)
    for early in (False, True):
        acc, best, nxt, ws = B.spec_verify(cand.cuda(), logits.cuda(), early_exit=early)
        got = (acc.cpu().numpy(), best.cpu().numpy(), nxt.cpu().numpy())
        for a, w in zip(got, want):
            assert np.array_equal(a, w), (early, Bn, K, n, V, dtype)
