"""Exact ties of leaf scores through spec_draft: the prune (Sec. 4.1: keep the K most confident leaves of
the product tree) must order equal scores by ascending leaf index, in its ranked form (up to 256 leaves per
sequence) and its sorted form (more), with bf16 and with e4m3 heads."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2404_19124_b200 import synth
from helpers import small_cfg, to_oracle_weights, weights_to_cuda, ws_view

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2404_19124_b200 import build
    build.build()
    from paper_2404_19124_b200 import binding
    return binding


def _leaf_digits(leaf, topk):
    digits = []
    for k in reversed(topk):
        digits.append(leaf % k)
        leaf //= k
    return digits[::-1]


@pytest.mark.parametrize("fp8", [False, True])
@pytest.mark.parametrize("topk,K", [((3, 2, 2), 5), ((2, 2), 1), ((6, 4, 3), 32), ((4, 4, 4, 5), 300), ((8, 8, 8), 511)])
def test_all_scores_equal_returns_the_lowest_leaves_in_order(B, topk, K, fp8):
    """All-zero output matrices: every logit is exactly 0, every top-k list is tokens 0..k-1, every leaf of a
    sequence scores -n ln V.  The candidates must be leaves 0..K-1 in index order (leaf i spells i in the
    mixed radix topk) - written out here, and equal to the oracle's output."""
    cfg = small_cfg(d_base=64, d_inner=128, V=1096, topk=topk, K=K, B=3, seed=17)
    sw = synth.make_weights(cfg)
    for l in range(cfg.n):
        sw.head[l].zero_()
    gw = weights_to_cuda(sw)
    ctx, tok = synth.make_draft_inputs(cfg)
    h = B.spec_create(gw)
    if fp8:
        B.spec_attach_fp8_heads(h)
        B.spec_set_option(h, B.SPEC_OPT_FP8_MAX_ROWS, 4096)
    else:   # the levels of up to 128 nodes in the form with the nodes as MMA columns
        B.spec_set_option(h, B.SPEC_OPT_HEAD_SWAP_MAX_ROWS, 128 if K % 2 else 0)
        B.spec_set_option(h, B.SPEC_OPT_HEAD_PAIR, 1 if K % 2 else 0)      # and CTA pairs above 128 nodes
    ct, lp, ws = B.spec_draft(h, ctx.cuda(), tok.cuda(), cfg.topk, K)
    assert B.spec_poll_error(ws) == 0
    want = [_leaf_digits(i, topk) for i in range(K)]
    for b in range(cfg.B):
        assert ct[b].cpu().tolist() == want
    assert (lp.cpu().numpy() + cfg.n * math.log(cfg.V)).__abs__().max() < 1e-4
    o_tok, o_lp = oracle.draft(to_oracle_weights(sw), synth.bf16_bits(ctx), tok.numpy(), topk, K)
    assert np.array_equal(o_tok, ct.cpu().numpy())
    B.spec_destroy(h)


@pytest.mark.parametrize("fp8", [False, True])
@pytest.mark.parametrize("topk,K,Bn,V,d", [((3, 2, 2), 7, 4, 8000, 512), ((6, 4, 2), 33, 16, 32000, 1024),
                                          ((8, 8, 3, 2), 101, 2, 2048, 256)])
def test_tie_across_the_K_boundary_keeps_the_lower_leaf(B, topk, K, Bn, V, d, fp8):
    """Two tokens x < y whose rows of the last head are the same positive constant vector: post-GELU
    states have a positive mean, so at every node of the last level x and y are the two largest logits and
    exactly equal.  With a last branching factor of 2 the leaves 2i (token x) and 2i + 1 (token y) tie
    pairwise, and an odd K cuts through a pair: the candidate that stays must be the one ending in x."""
    assert topk[-1] == 2 and K % 2 == 1
    cfg = small_cfg(d_base=128, d_inner=d, V=V, topk=topk, K=K, B=Bn, seed=V % 89 + Bn)
    sw = synth.make_weights(cfg)
    x, y = 37, V - 5                                     # far apart: different vocabulary tiles
    sw.head[-1][x] = 0.25
    sw.head[-1][y] = 0.25
    ow, gw = to_oracle_weights(sw), weights_to_cuda(sw)
    ctx, tok = synth.make_draft_inputs(cfg)
    h = B.spec_create(gw)
    if fp8:
        B.spec_attach_fp8_heads(h)
        B.spec_set_option(h, B.SPEC_OPT_FP8_MAX_ROWS, 4096)
    else:
        B.spec_set_option(h, B.SPEC_OPT_HEAD_SWAP_MAX_ROWS, 128 if Bn % 4 == 0 else 0)
        B.spec_set_option(h, B.SPEC_OPT_HEAD_PAIR, 1 if Bn % 4 == 0 else 0)
    ct, lp, ws = B.spec_draft(h, ctx.cuda(), tok.cuda(), cfg.topk, K)
    assert B.spec_poll_error(ws) == 0
    ct, lp = ct.cpu().numpy(), lp.cpu().numpy()
    lay = B.spec_draft_layout(h, cfg.B, cfg.topk, K)
    L = cfg.leaves
    leaf = ws_view(ws, lay.score[cfg.n], cfg.B * L, torch.float32).view(cfg.B, L).cpu().numpy()
    leaf_tok = ws_view(ws, lay.tok[cfg.n], cfg.B * L, torch.int32).view(cfg.B, L).cpu().numpy()
    assert (leaf_tok[:, 0::2] == x).all() and (leaf_tok[:, 1::2] == y).all()
    assert np.array_equal(leaf[:, 0::2], leaf[:, 1::2]), "duplicate rows must give bit-identical scores"
    for b in range(cfg.B):
        order = np.lexsort((np.arange(L), -leaf[b].astype(np.float64)))[:K]
        assert np.array_equal(leaf[b][order], lp[b])
        assert ct[b, K - 1, -1] == x, "K cuts a tied pair: the lower leaf (token x) stays"
        for k in range(0, K - 1, 2):                     # pairs come out adjacent, x first
            assert ct[b, k, -1] == x and ct[b, k + 1, -1] == y
            assert np.array_equal(ct[b, k, :-1], ct[b, k + 1, :-1]) and lp[b, k] == lp[b, k + 1]
    # and against the oracle on a sample of sequences (exact unless an unrelated near-tie flips a branch)
    same = 0
    for b in range(min(cfg.B, 3)):
        o_tok, o_lp = oracle.draft(ow, synth.bf16_bits(ctx)[b:b + 1], tok.numpy()[b:b + 1], topk, K)
        assert o_tok[0, K - 1, -1] == x
        same += int(np.array_equal(o_tok[0], ct[b]))
    if not fp8:
        assert same >= min(cfg.B, 3) - 1
    B.spec_destroy(h)
