"""Pins for the CPU oracle: it is checked against float64 library routines, closed forms,
brute force and hand-built cases, never against itself or the CUDA path.

Paper passages: the stage formula and the candidate tree are Sec. 3.1; branching and
pruning by confidence are Sec. 4.1; the n+1 tokens-per-step cap is Sec. 5.
"""
import itertools
import json
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from paper_2404_19124_b200 import synth
from helpers import f64, small_cfg, to_oracle_weights

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- bf16 helpers
def test_bf16_rounding_matches_library_cast():
    g = torch.Generator().manual_seed(3)
    x = torch.randn(20000, generator=g) * torch.exp(torch.randn(20000, generator=g) * 4)
    # exact ties between two bf16 neighbours and special values
    ties = torch.tensor([1.00390625, 1.01171875, -1.00390625, 0.0, -0.0, 3.3895314e38, 1e-40, float("inf")])
    x = torch.cat([x, ties])
    want = x.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([oracle.f32_to_bf16_bits(v) for v in x.numpy()], dtype=np.uint16)
    assert np.array_equal(got, want)
    back = oracle.bf16_bits_to_f32(want)
    assert np.array_equal(back, x.to(torch.bfloat16).to(torch.float32).numpy())


# ----------------------------------------------------------------------------- one stage
def _torch_stage(sw, level, s_parent64, tok):
    """Stage written with float64 library routines only (embedding, linear, layer_norm, gelu)."""
    z = F.embedding(torch.tensor([tok]), f64(sw.emb[level]))[0]
    p = F.linear(s_parent64, f64(sw.proj[level]))
    h = sw.state_weight * p.to(torch.float32).to(torch.float64) + sw.emb_weight * z
    y = F.layer_norm(h, (h.numel(),), f64(sw.ln_gamma[level]), f64(sw.ln_beta[level]), sw.ln_eps)
    s = F.gelu(y, approximate="none")
    return p, h, y, s


@pytest.mark.parametrize("level", [0, 1, 2])
def test_stage_against_float64_library_routines(level):
    cfg = small_cfg(d_base=48, d_inner=32, V=40)
    sw = synth.make_weights(cfg)
    ow = to_oracle_weights(sw, round_state_bf16=False)
    g = torch.Generator().manual_seed(11 + level)
    d_in = cfg.d_in(level)
    s_parent = torch.randn(d_in, generator=g).to(torch.bfloat16).to(torch.float32)
    tok = 17
    s, p, h, y = oracle.stage_state(ow, level, s_parent.numpy(), tok, intermediates=True)
    p64, h64, y64, s64 = _torch_stage(sw, level, s_parent.to(torch.float64), tok)
    assert np.allclose(p, p64.numpy(), rtol=1e-6, atol=1e-6)
    assert np.allclose(h, h64.numpy(), rtol=1e-5, atol=1e-6)
    assert np.allclose(y, y64.numpy(), rtol=1e-5, atol=2e-6)
    assert np.allclose(s, s64.numpy(), rtol=1e-5, atol=2e-6)
    # the embedding term must matter (a dropped b*z would pass none of the above, but make it explicit)
    s_other = oracle.stage_state(ow, level, s_parent.numpy(), tok + 1)
    assert np.abs(s_other - s).max() > 1e-3


def test_stage_state_rounding_is_library_bf16_cast():
    cfg = small_cfg()
    sw = synth.make_weights(cfg)
    g = torch.Generator().manual_seed(5)
    s_parent = torch.randn(cfg.d_base, generator=g).numpy()
    s_full = oracle.stage_state(to_oracle_weights(sw, False), 0, s_parent, 3)
    s_rnd = oracle.stage_state(to_oracle_weights(sw, True), 0, s_parent, 3)
    want = torch.from_numpy(s_full).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(s_rnd, want)


def test_layernorm_invariants_without_affine():
    cfg = small_cfg(d_inner=64)
    sw = synth.make_weights(cfg)
    for l in range(cfg.n):
        sw.ln_gamma[l] = torch.ones(cfg.d_inner)
        sw.ln_beta[l] = torch.zeros(cfg.d_inner)
    ow = to_oracle_weights(sw, False)
    g = torch.Generator().manual_seed(2)
    s_parent = torch.randn(cfg.d_base, generator=g).numpy()
    _, _, h, y = oracle.stage_state(ow, 0, s_parent, 9, intermediates=True)
    var_h = np.var(h.astype(np.float64))
    assert abs(y.astype(np.float64).mean()) < 1e-6
    assert abs(np.var(y.astype(np.float64)) - var_h / (var_h + sw.ln_eps)) < 1e-5


def test_token_range_is_an_error():
    cfg = small_cfg()
    ow = to_oracle_weights(synth.make_weights(cfg))
    with pytest.raises(oracle.OracleError) as e:
        oracle.stage_state(ow, 0, np.zeros(cfg.d_base, np.float32), cfg.V)
    assert e.value.code == oracle.ERR_TOKEN
    ctx, tok = synth.make_draft_inputs(cfg)
    bad = tok.numpy().copy()
    bad[0] = -1
    with pytest.raises(oracle.OracleError):
        oracle.draft(ow, synth.bf16_bits(ctx), bad, cfg.topk, cfg.K)


# ----------------------------------------------------------------------------- logits / lse / top-k
def test_logits_are_a_float64_linear_layer():
    cfg = small_cfg(d_inner=40, V=56)   # V != d_inner: a transposed operand cannot pass
    sw = synth.make_weights(cfg)
    ow = to_oracle_weights(sw)
    g = torch.Generator().manual_seed(4)
    S = torch.randn(5, cfg.d_inner, generator=g)
    got = oracle.stage_logits(ow, 1, S.numpy())
    want = F.linear(S.to(torch.float64), f64(sw.head[1]))
    assert got.shape == (5, cfg.V)
    assert np.allclose(got, want.numpy(), rtol=1e-6, atol=1e-6)


def test_logsumexp_and_topk_against_library():
    g = torch.Generator().manual_seed(8)
    x = (torch.randn(1000, generator=g) * 3 + 50.0).to(torch.float32)   # large offset: needs max-subtraction
    lse = oracle.logsumexp(x.numpy())
    assert abs(lse - torch.logsumexp(x.to(torch.float64), 0).item()) < 1e-5
    assert abs(np.exp(x.numpy().astype(np.float64) - lse).sum() - 1.0) < 1e-5
    ids, vals = oracle.topk(x.numpy(), 7)
    tv, ti = torch.topk(x, 7)
    assert np.array_equal(ids, ti.numpy()) and np.array_equal(vals, tv.numpy())


def test_topk_ties_prefer_lower_index():
    x = np.array([1.0, 5.0, 5.0, 2.0, 5.0, 0.0], np.float32)
    ids, vals = oracle.topk(x, 4)
    assert ids.tolist() == [1, 2, 4, 3] and vals.tolist() == [5.0, 5.0, 5.0, 2.0]


# ----------------------------------------------------------------------------- whole tree
def _brute_force_paths(sw, ctx_bits, last_tok, topk, b):
    """Independent enumeration: recursive walk with float64 library routines for each node.

    Returns [(score, leaf_index, tokens)] for every root-to-leaf path of sequence b."""
    n = len(topk)
    out = []

    def rec(level, s_parent64, tok, score, leaf, toks):
        if level == n:
            out.append((score, leaf, tuple(toks)))
            return
        _, _, _, s = _torch_stage(sw, level, s_parent64, tok)
        s = s.to(torch.float32).to(torch.bfloat16).to(torch.float64)      # carried state is bf16
        logits = F.linear(s, f64(sw.head[level])).to(torch.float32).to(torch.float64)
        logp = F.log_softmax(logits, dim=0)
        order = sorted(range(logits.numel()), key=lambda v: (-logits[v].item(), v))[: topk[level]]
        for j, v in enumerate(order):
            rec(level + 1, s, v, score + logp[v].item(), leaf * topk[level] + j, toks + [v])

    ctx = torch.from_numpy(oracle.bf16_bits_to_f32(ctx_bits[b])).to(torch.float64)
    rec(0, ctx, int(last_tok[b]), 0.0, 0, [])
    return out


@pytest.mark.parametrize("topk", [(3, 2, 2), (2, 3), (4, 1, 2, 2)])
def test_pruned_tree_equals_brute_force_for_every_K(topk):
    cfg = small_cfg(topk=topk, K=1, B=2, V=24, d_inner=16, d_base=24, std=0.3)
    sw = synth.make_weights(cfg)
    ow = to_oracle_weights(sw)
    ctx, tok = synth.make_draft_inputs(cfg)
    ctx_bits, tok_np = synth.bf16_bits(ctx), tok.numpy()
    L = cfg.leaves
    full_tok, full_lp = oracle.draft(ow, ctx_bits, tok_np, topk, L)
    for b in range(cfg.B):
        paths = _brute_force_paths(sw, ctx_bits, tok_np, topk, b)
        assert len(paths) == L
        paths.sort(key=lambda t: (-t[0], t[1]))
        for k, (score, _, toks) in enumerate(paths):
            assert tuple(full_tok[b, k]) == toks
            assert abs(full_lp[b, k] - score) < 1e-4
    for K in range(1, L):   # prefix property: the K best are the first K rows of the full ordering
        ct, lp = oracle.draft(ow, ctx_bits, tok_np, topk, K)
        assert np.array_equal(ct, full_tok[:, :K]) and np.array_equal(lp, full_lp[:, :K])


@pytest.mark.parametrize("n", [2, 3])
def test_full_tree_enumerates_a_probability_distribution(n):
    V = 4
    cfg = small_cfg(topk=(V,) * n, K=V ** n, B=3, V=V, d_inner=16, d_base=8, std=0.5)
    sw = synth.make_weights(cfg)
    ctx, tok = synth.make_draft_inputs(cfg)
    ct, lp = oracle.draft(to_oracle_weights(sw), synth.bf16_bits(ctx), tok.numpy(), cfg.topk, cfg.K)
    mass = np.exp(lp.astype(np.float64)).sum(axis=1)
    assert np.allclose(mass, 1.0, atol=1e-5)
    for b in range(cfg.B):   # every V^n n-gram appears exactly once
        assert {tuple(r) for r in ct[b]} == set(itertools.product(range(V), repeat=n))


def test_structure_of_the_candidate_list():
    cfg = small_cfg(topk=(3, 2, 2), K=7, B=3, V=50)
    sw = synth.make_weights(cfg)
    ow = to_oracle_weights(sw)
    ctx, tok = synth.make_draft_inputs(cfg)
    ct, lp, dd = oracle.draft(ow, synth.bf16_bits(ctx), tok.numpy(), cfg.topk, cfg.K, dump=True)
    assert ct.shape == (3, 7, 3) and lp.shape == (3, 7)
    assert (lp <= 0).all() and (np.diff(lp, axis=1) <= 0).all()
    for b in range(cfg.B):
        assert len({tuple(r) for r in ct[b]}) == cfg.K
    # level sizes follow the product tree of Sec. 4.1 (3, 3*2, 3*2*2 children per sequence)
    assert [t.size for t in dd.tok] == [3 * 3, 3 * 6, 3 * 12]
    # every first token is one of its sequence's head-0 top-k tokens
    for b in range(cfg.B):
        assert set(ct[b, :, 0]) <= set(dd.tok[0][b * 3:(b + 1) * 3])


def test_single_branch_is_the_greedy_chain():
    cfg = small_cfg(topk=(1, 1, 1), K=1, B=2, V=30)
    sw = synth.make_weights(cfg)
    ow = to_oracle_weights(sw)
    ctx, tok = synth.make_draft_inputs(cfg)
    ctx_bits = synth.bf16_bits(ctx)
    ct, lp = oracle.draft(ow, ctx_bits, tok.numpy(), cfg.topk, 1)
    for b in range(cfg.B):
        s = oracle.bf16_bits_to_f32(ctx_bits[b])
        t, score = int(tok[b]), 0.0
        for l in range(cfg.n):
            s = oracle.stage_state(ow, l, s, t)
            logits = torch.from_numpy(oracle.stage_logits(ow, l, s[None])[0]).to(torch.float64)
            t = int(torch.argmax(logits))
            score += F.log_softmax(logits, 0)[t].item()
            assert ct[b, 0, l] == t
        assert abs(lp[b, 0] - score) < 1e-4


def test_without_embedding_weight_the_tree_is_a_cartesian_product():
    """b = 0 removes the token conditioning: every node of a level sees the same state
    chain, so candidates are products of per-level top-k lists (the parallel-head
    structure the paper starts from, Sec. 3.1)."""
    cfg = small_cfg(topk=(3, 2, 2), K=12, B=2, V=30)
    sw = synth.make_weights(cfg)
    sw.emb_weight = 0.0
    ow = to_oracle_weights(sw)
    ctx, tok = synth.make_draft_inputs(cfg)
    ct, lp, dd = oracle.draft(ow, synth.bf16_bits(ctx), tok.numpy(), cfg.topk, cfg.K, dump=True)
    for b in range(cfg.B):
        per_level = []
        for l in range(cfg.n):
            N_b = int(np.prod(cfg.topk[:l]))
            kids = dd.tok[l].reshape(cfg.B, N_b, cfg.topk[l])[b]
            assert (kids == kids[0]).all()          # all nodes of the level agree
            lg = dd.logits[l].reshape(cfg.B, N_b, cfg.V)[b, 0].astype(np.float64)
            logp = lg - oracle.logsumexp(lg.astype(np.float32))
            per_level.append({int(t): logp[t] for t in kids[0]})
        scores = {toks: sum(per_level[l][toks[l]] for l in range(cfg.n))
                  for toks in itertools.product(*[list(d) for d in per_level])}
        assert {tuple(r) for r in ct[b]} == set(scores)
        for k in range(cfg.K):
            assert abs(lp[b, k] - scores[tuple(ct[b, k])]) < 1e-4


def test_children_depend_on_the_sampled_token():
    """Hand-built weights: the embedding of token A steers head 1 to token X and that of
    token B to token Y, while the state projection is silent - the conditioning that the
    paper adds over parallel heads (Sec. 3.1, the "Step Step Step" discussion)."""
    V, d = 6, 8
    cfg = synth.SpecConfig("hand", 4, d, V, (2, 1), 2, 1, 0.0, 1.0, "none", 0)
    z = lambda *s: torch.zeros(*s)
    emb0, emb1 = z(V, d), z(V, d)
    head0, head1 = z(V, d), z(V, d)
    # head 0: last_tok = 0 lights unit 0 -> logits favour token 1 (A) then token 2 (B)
    emb0[0, 0] = 4.0
    head0[1, 0], head0[2, 0] = 3.0, 2.0
    # head 1: embedding of A lights unit 1, of B lights unit 2; unit 1 -> token 4 (X), unit 2 -> token 5 (Y)
    emb1[1, 1] = 4.0
    emb1[2, 2] = 4.0
    head1[4, 1] = 3.0
    head1[5, 2] = 3.0
    ow = oracle.Weights(
        V=V, d_base=4, d_inner=d,
        emb=[synth.bf16_bits(t.to(torch.bfloat16)) for t in (emb0, emb1)],
        proj=[synth.bf16_bits(z(d, 4).to(torch.bfloat16)), synth.bf16_bits(z(d, d).to(torch.bfloat16))],
        ln_gamma=[np.ones(d, np.float32)] * 2, ln_beta=[np.zeros(d, np.float32)] * 2,
        head=[synth.bf16_bits(t.to(torch.bfloat16)) for t in (head0, head1)],
        state_weight=1.0, emb_weight=1.0)
    ctx = synth.bf16_bits(torch.ones(1, 4, dtype=torch.bfloat16))
    ct, lp = oracle.draft(ow, ctx, np.array([0], np.int32), cfg.topk, 2)
    assert ct[0].tolist() == [[1, 4], [2, 5]]
    assert lp[0, 0] > lp[0, 1]


def _tie_weights(V, d, n, heads, embs, d_base=4):
    """Hand-built speculator: zero projections (the state carries nothing), identity LayerNorm affine."""
    z = lambda *s: torch.zeros(*s)
    bits = lambda t: synth.bf16_bits(t.to(torch.bfloat16))
    return oracle.Weights(
        V=V, d_base=d_base, d_inner=d, emb=[bits(t) for t in embs],
        proj=[bits(z(d, d_base if l == 0 else d)) for l in range(n)],
        ln_gamma=[np.ones(d, np.float32)] * n, ln_beta=[np.zeros(d, np.float32)] * n,
        head=[bits(t) for t in heads], state_weight=1.0, emb_weight=1.0)


@pytest.mark.parametrize("topk,K", [((3, 2, 2), 5), ((2, 2), 1), ((2, 3), 6), ((4, 4, 4, 4), 200)])
def test_prune_with_all_scores_equal_keeps_the_lowest_leaf_indices(topk, K):
    """All-zero output matrices: every logit is 0, so every top-k list is tokens 0..k-1 in id order with
    log-probability -ln V each, every leaf scores -n ln V, and pruning by confidence (Sec. 4.1) with
    equal scores must return leaves 0..K-1 in index order.  Leaf i spells i in the mixed radix topk."""
    V, d, n = 11, 8, len(topk)
    g = torch.Generator().manual_seed(21)
    embs = [torch.randn(V, d, generator=g) for _ in range(n)]          # states differ per token; logits do not
    ow = _tie_weights(V, d, n, [torch.zeros(V, d)] * n, embs)
    ctx = synth.bf16_bits(torch.ones(2, 4, dtype=torch.bfloat16))
    ct, lp = oracle.draft(ow, ctx, np.array([3, 7], np.int32), topk, K)
    want = []
    for leaf in range(K):
        digits, rest = [], leaf
        for k in reversed(topk):
            digits.append(rest % k)
            rest //= k
        want.append(digits[::-1])
    for b in range(2):
        assert ct[b].tolist() == want
    assert np.abs(lp + n * math.log(V)).max() < 1e-5


def test_prune_tie_across_the_K_boundary_prefers_the_lower_leaf():
    """Two head-0 tokens (5 and 9) with identical output rows and identical level-1 embeddings: their
    subtrees score exactly alike.  Leaves in index order: 0 = (5, X), 1 = (5, Y), 2 = (9, X), 3 = (9, Y)
    with score(0) == score(2) > score(1) == score(3); the order by (score desc, leaf asc) is 0, 2, 1, 3,
    so K = 1 must keep leaf 0 and K = 3 must keep leaves 0, 2, 1 (Sec. 4.1 prune; ties to the lower leaf)."""
    V, d = 12, 8
    z = lambda *s: torch.zeros(*s)
    emb0, emb1, head0, head1 = z(V, d), z(V, d), z(V, d), z(V, d)
    emb0[0, 0] = 4.0                       # last_tok = 0 lights unit 0
    head0[5, 0] = head0[9, 0] = 3.0        # ... which favours tokens 5 and 9 equally
    emb1[5, 1] = emb1[9, 1] = 4.0          # both light unit 1 at the next stage
    head1[2, 1], head1[7, 1] = 3.0, 2.0    # X = 2 then Y = 7
    ow = _tie_weights(V, d, 2, [head0, head1], [emb0, emb1])
    ctx = synth.bf16_bits(torch.ones(1, 4, dtype=torch.bfloat16))
    tok = np.array([0], np.int32)
    full_tok, full_lp = oracle.draft(ow, ctx, tok, (2, 2), 4)
    assert full_tok[0].tolist() == [[5, 2], [9, 2], [5, 7], [9, 7]]
    assert full_lp[0, 0] == full_lp[0, 1] and full_lp[0, 2] == full_lp[0, 3] and full_lp[0, 1] > full_lp[0, 2]
    ct1, _ = oracle.draft(ow, ctx, tok, (2, 2), 1)
    assert ct1[0].tolist() == [[5, 2]]
    ct3, _ = oracle.draft(ow, ctx, tok, (2, 2), 3)
    assert ct3[0].tolist() == [[5, 2], [9, 2], [5, 7]]


# ----------------------------------------------------------------------------- verification
def _logits_from_argmax(g, V, dtype=np.float32):
    g = np.asarray(g)
    x = np.zeros(g.shape + (V,), dtype)
    np.put_along_axis(x, g[..., None], 10.0, axis=-1)
    return x


def test_verify_worked_example_from_fixture():
    with open(os.path.join(GOLDEN, "verify_worked_example.json")) as f:
        ex = json.load(f)
    for case in ex["cases"]:
        V = ex["V"]
        x = _logits_from_argmax([case["g"]], V)
        for (k, j, v) in case.get("extra_max", []):
            x[0, k, j, v] = 10.0
        ct = np.array([case["cand_tok"]], np.int32)
        acc, best, nxt, g = oracle.verify(ct, x, oracle.F32, want_g=True)
        assert (int(acc[0]), int(best[0]), int(nxt[0])) == (case["accept_len"], case["best_cand"], case["next_tok"])
        # same through the bf16 route
        xb = synth.bf16_bits(torch.from_numpy(x).to(torch.bfloat16))
        acc2, best2, nxt2 = oracle.verify(ct, xb, oracle.BF16)
        assert (acc2[0], best2[0], nxt2[0]) == (acc[0], best[0], nxt[0])


def test_verify_argmax_is_library_argmax_and_first_max_wins():
    g = torch.Generator().manual_seed(1)
    x = (torch.randn(2, 3, 4, 500, generator=g) * 2).to(torch.bfloat16)      # bf16: many exact ties
    ct = np.zeros((2, 3, 3), np.int32)
    _, _, _, got = oracle.verify(ct, synth.bf16_bits(x), oracle.BF16, want_g=True)
    xf = x.to(torch.float32).numpy()
    want = np.argmax(xf, axis=-1)            # numpy: first occurrence of the maximum
    assert np.array_equal(got, want)
    ties = (xf == xf.max(-1, keepdims=True)).sum(-1)
    assert (ties > 1).any(), "fixture should contain tied maxima"


def test_verify_nan_never_wins():
    x = np.zeros((1, 1, 2, 6), np.float32)
    x[0, 0, 0] = [np.nan, 1.0, np.nan, 3.0, 3.0, -1.0]
    x[0, 0, 1] = np.nan
    _, _, _, g = oracle.verify(np.zeros((1, 1, 1), np.int32), x, oracle.F32, want_g=True)
    assert g[0, 0].tolist() == [3, 0]


def test_verify_planted_prefix_lengths_and_invariants():
    rng = np.random.default_rng(0)
    B, K, n, V = 4, 5, 3, 64
    ct = rng.integers(0, V, (B, K, n)).astype(np.int32)
    m_plant = rng.integers(0, n + 1, (B, K))
    x = rng.normal(0, 1, (B, K, n + 1, V)).astype(np.float32)
    for b in range(B):
        for k in range(K):
            for j in range(n):
                if j < m_plant[b, k]:
                    x[b, k, j, ct[b, k, j]] = 30.0
                elif j == m_plant[b, k]:
                    x[b, k, j, (ct[b, k, j] + 1) % V] = 30.0
    acc, best, nxt, g = oracle.verify(ct, x, oracle.F32, want_g=True)
    assert np.array_equal(acc, m_plant.max(1))
    assert np.array_equal(best, m_plant.argmax(1))             # numpy argmax: lowest k among ties
    assert ((0 <= acc) & (acc <= n)).all()
    for b in range(B):
        assert nxt[b] == g[b, best[b], acc[b]]
        full = acc[b] == n
        assert full == bool((ct[b, best[b]] == g[b, best[b], :n]).all())
    # permuting the non-best candidates does not change accept_len
    for b in range(B):
        perm = [k for k in range(K) if k != best[b]]
        rng.shuffle(perm)
        order = [best[b]] + perm
        a2, b2, n2 = oracle.verify(ct[b:b + 1, order], x[b:b + 1, order], oracle.F32)
        assert a2[0] == acc[b] and n2[0] == nxt[b]


def test_candidate_equal_to_argmax_chain_is_fully_accepted():
    rng = np.random.default_rng(5)
    B, K, n, V = 2, 3, 4, 32
    x = rng.normal(0, 1, (B, K, n + 1, V)).astype(np.float32)
    g = x.argmax(-1)
    ct = rng.integers(0, V, (B, K, n)).astype(np.int32)
    ct[:, 1] = g[:, 1, :n]
    acc, best, nxt = oracle.verify(ct, x, oracle.F32)
    assert (acc == n).all() and (best == 1).all() and np.array_equal(nxt, g[:, 1, n])


def test_mix_weights_follow_the_variance_rule():
    # Sec. 4: base state = half the variance at the last head  <=>  a^(2n) = 1/2, a^2 + (b sigma_E)^2 = 1
    for n in (3, 5, 7):
        a, b = synth.mix_weights(n, 4096 ** -0.5)
        assert abs(a ** (2 * n) - 0.5) < 1e-12
        assert abs(a * a + (b * 4096 ** -0.5) ** 2 - 1.0) < 1e-12


def test_next_ctx_hand_built_example():
    """Sec. 3.1: the next draft starts from the base model's state at the last accepted position of the
    best candidate.  Entry (b, k, j, i) of the tensor is the number b k j i read in base 10, so every
    expected value below can be checked by eye."""
    B, K, n, d = 2, 3, 2, 4
    base = np.empty((B, K, n + 1, d), np.int64)
    for b in range(B):
        for k in range(K):
            for j in range(n + 1):
                for i in range(d):
                    base[b, k, j, i] = 1000 * b + 100 * k + 10 * j + i
    out = oracle.next_ctx(base, best_cand=np.array([2, 0]), accept_len=np.array([1, 2]))
    assert out.tolist() == [[210, 211, 212, 213], [1020, 1021, 1022, 1023]]
    # nothing accepted: the state at position 0 (the one that produced the bonus token)
    assert oracle.next_ctx(base, np.array([1, 1]), np.array([0, 0])).tolist() == [[100, 101, 102, 103],
                                                                                 [1100, 1101, 1102, 1103]]
    with pytest.raises(oracle.OracleError):
        oracle.next_ctx(base, np.array([3, 0]), np.array([0, 0]))
    with pytest.raises(oracle.OracleError):
        oracle.next_ctx(base, np.array([0, 0]), np.array([0, 3]))
