"""Vocabulary-parallel heads on one GPU: the ranks are handles holding disjoint row ranges of every head
matrix, run one after the other on the same stream; the exchange is a copy between their workspaces.
No kernel waits for another.  Every emulated rank must return what the oracle (and spec_draft on the
unsplit weights) returns."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2404_19124_b200 import shard, synth
from helpers import DraftChecker, small_cfg, to_oracle_weights, weights_to_cuda

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2404_19124_b200 import build
    build.build()
    from paper_2404_19124_b200 import binding
    return binding


def _run_ranks(B, gw, cfg, world, ctx, tok):
    """Emulates `world` ranks; returns their (cand_tok, cand_logp) and the handles' workspaces."""
    parts = shard.split_vocab(cfg.V, world)
    hs = []
    for r, (lo, cnt) in enumerate(parts):
        w = dataclasses.replace(gw, head=[t[lo:lo + cnt].contiguous() for t in gw.head])
        hs.append(B.spec_create(w, vocab_shard=(r, world, lo)))
    wss = [torch.empty(B.spec_draft_workspace_bytes(h, cfg.B, cfg.topk, cfg.K), dtype=torch.uint8, device="cuda")
           for h in hs]
    cands = [torch.empty((cfg.B, cfg.K, cfg.n), dtype=torch.int32, device="cuda") for _ in hs]
    logps = [torch.empty((cfg.B, cfg.K), dtype=torch.float32, device="cuda") for _ in hs]
    for level in range(cfg.n):
        for h, ws in zip(hs, wss):
            B.spec_draft_vp_local(h, level, ctx, tok, cfg.topk, cfg.K, ws)
        off, slot = B.spec_draft_vp_exchange(hs[0], cfg.B, cfg.topk, cfg.K, level)
        for r, ws in enumerate(wss):                      # "all-gather": everyone copies everyone's slot
            for g, src in enumerate(wss):
                if g != r:
                    ws[off + g * slot: off + (g + 1) * slot].copy_(src[off + g * slot: off + (g + 1) * slot])
        last = level == cfg.n - 1
        for h, ws, c, lp in zip(hs, wss, cands, logps):
            B.spec_draft_vp_merge(h, level, cfg.B, cfg.topk, cfg.K, ws, c if last else None, lp if last else None)
    torch.cuda.synchronize()
    for ws in wss:
        assert B.spec_poll_error(ws) == 0
    out = [(c.cpu().numpy(), lp.cpu().numpy()) for c, lp in zip(cands, logps)]
    for h in hs:
        B.spec_destroy(h)
    return out


@pytest.mark.parametrize("world", [2, 3, 8])
@pytest.mark.parametrize("topk,K,Bn,V,d_base,d", [((3, 2, 2), 5, 2, 1000, 72, 64), ((4, 3), 12, 5, 520, 64, 128),
                                                   ((8, 8), 64, 2, 2048, 128, 192), ((1, 1, 1), 1, 3, 512, 64, 64)])
def test_vocab_parallel_draft_matches_oracle(B, world, topk, K, Bn, V, d_base, d):
    cfg = small_cfg(d_base=d_base, d_inner=d, V=V, topk=topk, K=K, B=Bn, seed=world * 10 + len(topk))
    sw = synth.make_weights(cfg)
    ow, gw = to_oracle_weights(sw), weights_to_cuda(sw)
    ctx, tok = synth.make_draft_inputs(cfg)
    results = _run_ranks(B, gw, cfg, world, ctx.cuda(), tok.cuda())
    # every rank holds the same answer
    for ct, lp in results[1:]:
        assert np.array_equal(ct, results[0][0]) and np.array_equal(lp, results[0][1])
    # and it is the oracle's
    chk = DraftChecker(ow, cfg.topk, cfg.K)
    ctx_bits = synth.bf16_bits(ctx)
    ct, lp = results[0]
    for b in range(cfg.B):
        chk.check(ctx_bits[b], int(tok[b]), ct[b], lp[b])
    assert chk.exact + chk.tolerated == cfg.B
    # the unsplit library path gives the same tokens and, up to the two-stage log-sum-exp, the same scores
    h = B.spec_create(gw)
    c1, l1, _ = B.spec_draft(h, ctx.cuda(), tok.cuda(), cfg.topk, cfg.K)
    if chk.tolerated == 0:
        assert np.array_equal(c1.cpu().numpy(), ct)
    assert np.abs(np.sort(l1.cpu().numpy(), axis=1) - np.sort(lp, axis=1)).max() < 1e-4
    B.spec_destroy(h)


def test_vocab_parallel_full_width_two_ranks(B):
    """Llama2-7B-shaped widths and vocabulary, two ranks, three sequences against the oracle."""
    cfg = dataclasses.replace(synth.CONFIGS["llama2-7b"], B=3)
    sw = synth.make_weights(cfg)
    ow, gw = to_oracle_weights(sw), weights_to_cuda(sw)
    ctx, tok = synth.make_draft_inputs(cfg)
    results = _run_ranks(B, gw, cfg, 2, ctx.cuda(), tok.cuda())
    assert np.array_equal(results[0][0], results[1][0]) and np.array_equal(results[0][1], results[1][1])
    chk = DraftChecker(ow, cfg.topk, cfg.K)
    ctx_bits = synth.bf16_bits(ctx)
    for b in range(cfg.B):
        chk.check(ctx_bits[b], int(tok[b]), results[0][0][b], results[0][1][b])
    assert chk.exact + chk.tolerated == cfg.B


def test_sharded_handle_refuses_the_unsplit_calls(B):
    cfg = small_cfg(d_base=64, d_inner=64, V=512, topk=(2, 2), K=3, B=2, seed=3)
    sw = synth.make_weights(cfg)
    gw = weights_to_cuda(sw)
    w = dataclasses.replace(gw, head=[t[:256].contiguous() for t in gw.head])
    h = B.spec_create(w, vocab_shard=(0, 2, 0))
    ctx, tok = synth.make_draft_inputs(cfg)
    ws = torch.empty(B.spec_draft_workspace_bytes(h, cfg.B, cfg.topk, cfg.K), dtype=torch.uint8, device="cuda")
    with pytest.raises(B.SpecError):
        B.spec_draft(h, ctx.cuda(), tok.cuda(), cfg.topk, cfg.K, workspace=ws)
    assert B.spec_head_workspace_bytes(h, 4, 2) == 0
    with pytest.raises(B.SpecError):                            # rows past the end of the vocabulary
        B.spec_set_vocab_shard(h, 1, 2, 300, 256)
    with pytest.raises(B.SpecError):
        B.spec_set_vocab_shard(h, 2, 2, 0, 256)
    B.spec_destroy(h)
