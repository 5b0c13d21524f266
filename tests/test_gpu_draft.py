"""GPU parity of the draft path against the oracle: head logits (tensor-core main loop),
fused top-k / log-prob epilogue, per-level states and tokens, and whole spec_draft calls."""
import numpy as np
import pytest
import torch

import oracle
from paper_2404_19124_b200 import synth
from helpers import LOGIT_TOL, TIE_TOL, DraftChecker, small_cfg, to_oracle_weights, weights_to_cuda, ws_view

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2404_19124_b200 import build
    build.build()
    from paper_2404_19124_b200 import binding
    return binding


def _states(rows, d, seed):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(rows, d, generator=g) * 0.5).to(torch.bfloat16)


def _setup(cfg):
    sw = synth.make_weights(cfg)
    return sw, to_oracle_weights(sw), weights_to_cuda(sw)


# rows: 1 / 4 / 12 are the tiny config's levels; 130 spans two 128-row tiles with a ragged tail;
# V = 1000 / 1096 leave a ragged last vocabulary tile; d = 200 is not a multiple of the 64-wide K block.
@pytest.mark.parametrize("impl", [0, 1])
@pytest.mark.parametrize("rows,V,d", [(1, 1024, 256), (4, 1024, 256), (12, 1024, 256), (130, 1024, 256),
                                      (33, 1000, 200), (257, 1096, 64), (96, 8000, 512)])
def test_head_logits_match_oracle(B, impl, rows, V, d):
    cfg = small_cfg(d_base=d, d_inner=d, V=V, topk=(2, 2), std=None, seed=rows + V)
    sw, ow, gw = _setup(cfg)
    h = B.spec_create(gw)
    B.spec_set_option(h, B.SPEC_OPT_GEMM_IMPL, impl)
    S = _states(rows, d, 3)
    got = B.spec_head_logits(h, 1, S.cuda())
    torch.cuda.synchronize()
    want = oracle.stage_logits(ow, 1, S.to(torch.float32).numpy())
    err = np.abs(got.cpu().numpy() - want).max()
    assert err <= LOGIT_TOL, err
    assert err <= 2e-3, f"fp32-accumulated logits should be far inside the tolerance, got {err}"
    B.spec_destroy(h)


@pytest.mark.parametrize("block_n", [32, 96, 224, 256])
def test_head_logits_every_tile_width(B, block_n):
    cfg = small_cfg(d_base=128, d_inner=320, V=2000, topk=(2, 2), seed=block_n)
    sw, ow, gw = _setup(cfg)
    h = B.spec_create(gw)
    B.spec_set_option(h, B.SPEC_OPT_HEAD_BLOCK_N, block_n)
    S = _states(140, cfg.d_inner, 9)
    got = B.spec_head_logits(h, 0, S.cuda())
    want = oracle.stage_logits(ow, 0, S.to(torch.float32).numpy())
    assert np.abs(got.cpu().numpy() - want).max() <= 2e-3
    B.spec_destroy(h)


def _check_topk_rows(tok, logp, logits, k):
    """tok/logp [rows, k] against oracle logits [rows, V] with the tie rule."""
    tolerated = 0
    for r in range(logits.shape[0]):
        ids, vals = oracle.topk(logits[r], k)
        lse = oracle.logsumexp(logits[r])
        if np.array_equal(ids, tok[r]):
            assert np.abs((vals - lse) - logp[r]).max() <= LOGIT_TOL
            continue
        tolerated += 1
        kth = vals[-1]
        for j in range(k):
            assert logits[r, tok[r, j]] >= kth - TIE_TOL
            assert abs((logits[r, tok[r, j]] - lse) - logp[r, j]) <= LOGIT_TOL
        assert len(set(tok[r].tolist())) == k
    return tolerated


# impl 0: tensor cores, nodes as columns of the MMA for up to 128 rows (the weight-stream form); 1: CUDA-core
# debug GEMM; 2: tensor cores with one thread per node row at every size; 3: CTA pairs above 128 rows
@pytest.mark.parametrize("impl", [0, 1, 2, 3])
@pytest.mark.parametrize("rows,V,d,k", [(1, 1024, 256, 4), (12, 1024, 256, 2), (130, 1000, 128, 8),
                                        (40, 8000, 512, 6), (5, 64, 64, 8), (3, 40, 64, 1), (16, 32000, 256, 6),
                                        (96, 20040, 192, 3), (128, 5000, 64, 5), (33, 1000, 200, 8), (64, 129, 72, 7),
                                        (384, 2048, 256, 3), (257, 1096, 64, 6), (700, 3000, 192, 2)])
def test_head_topk_matches_oracle(B, impl, rows, V, d, k):
    if impl == 3 and rows <= 128:
        pytest.skip("pairs serve levels of more than 128 rows")
    cfg = small_cfg(d_base=d, d_inner=d, V=V, topk=(2, 2), seed=rows * 7 + k)
    sw, ow, gw = _setup(cfg)
    h = B.spec_create(gw)
    B.spec_set_option(h, B.SPEC_OPT_GEMM_IMPL, impl & 1 if impl < 3 else 0)
    B.spec_set_option(h, B.SPEC_OPT_HEAD_SWAP_MAX_ROWS, 0 if impl == 2 else 128)
    B.spec_set_option(h, B.SPEC_OPT_HEAD_PAIR, 1 if impl == 3 else 0)
    S = _states(rows, d, 4)
    tok, logp, ws = B.spec_head_topk(h, 0, S.cuda(), k)
    assert B.spec_poll_error(ws) == 0
    logits = oracle.stage_logits(ow, 0, S.to(torch.float32).numpy())
    tolerated = _check_topk_rows(tok.cpu().numpy(), logp.cpu().numpy(), logits, k)
    assert tolerated <= max(1, rows // 20)
    B.spec_destroy(h)


@pytest.mark.parametrize("swapped", [False, True])
def test_head_topk_exact_ties_prefer_lower_token_id(B, swapped):
    """Duplicate output rows give exactly equal logits: the lower token id must come first,
    also when the two copies sit in different vocabulary tiles (and, in the weight-stream form, in
    different segments of one tile)."""
    cfg = small_cfg(d_base=64, d_inner=64, V=1024, topk=(2, 2), seed=21)
    sw = synth.make_weights(cfg)
    for l in range(cfg.n):
        sw.head[l][700] = sw.head[l][3]
        sw.head[l][4] = sw.head[l][3]
    ow, gw = to_oracle_weights(sw), weights_to_cuda(sw)
    h = B.spec_create(gw)
    if swapped:
        B.spec_set_option(h, B.SPEC_OPT_HEAD_SWAP_MAX_ROWS, 128)
    else:
        B.spec_set_option(h, B.SPEC_OPT_HEAD_BLOCK_N, 32)
    # a state aligned with row 3 makes tokens 3, 4 and 700 the tied maximum
    S = (sw.head[0][3].to(torch.float32) * 40).to(torch.bfloat16)[None].contiguous()
    tok, logp, _ = B.spec_head_topk(h, 0, S.cuda(), 4)
    logits = oracle.stage_logits(ow, 0, S.to(torch.float32).numpy())
    ids, _ = oracle.topk(logits[0], 4)
    assert ids[:3].tolist() == [3, 4, 700]
    assert tok.cpu().numpy()[0].tolist() == ids.tolist()
    B.spec_destroy(h)


def _draft_and_check(B, cfg, seqs=None, impl=0, check_levels=False, tie_weights=False, fp8=False, fp8_rows=None,
                     swap=None):
    """Runs spec_draft at the config's full batch and compares the sequences in `seqs`
    (default: all) with the oracle, one sequence at a time (sequences are independent).
    tie_weights: every head after the first aliases the second head's tensors (the weight-tied
    variant the paper mentions in Sec. 3.1 / Sec. 5: same computation, shared parameters)."""
    if tie_weights:
        sw = synth.make_weights(cfg)
        for l in range(2, cfg.n):
            for lst in (sw.emb, sw.proj, sw.ln_gamma, sw.ln_beta, sw.head):
                lst[l] = lst[1]
        ow, gw = to_oracle_weights(sw), weights_to_cuda(sw)
        for l in range(2, cfg.n):       # on the device too the heads share one copy, not equal copies
            for lst in (gw.emb, gw.proj, gw.ln_gamma, gw.ln_beta, gw.head):
                lst[l] = lst[1]
    else:
        sw, ow, gw = _setup(cfg)
    ctx, tok = synth.make_draft_inputs(cfg)
    h = B.spec_create(gw)
    B.spec_set_option(h, B.SPEC_OPT_GEMM_IMPL, impl)
    if swap is not None:   # levels of up to `swap` nodes run the head with the nodes as MMA columns (0: none)
        B.spec_set_option(h, B.SPEC_OPT_HEAD_SWAP_MAX_ROWS, swap)
        B.spec_set_option(h, B.SPEC_OPT_HEAD_PAIR, 1 if swap else 0)   # and levels of > 128 nodes on CTA pairs / not
    if fp8:      # levels of up to 128 nodes multiply in e4m3 and re-score a short list exactly
        B.spec_attach_fp8_heads(h)
        if fp8_rows is not None:   # also levels with more than the default 128 nodes
            B.spec_set_option(h, B.SPEC_OPT_FP8_MAX_ROWS, fp8_rows)
    cand_tok, cand_logp, ws = B.spec_draft(h, ctx.cuda(), tok.cuda(), cfg.topk, cfg.K)
    assert B.spec_poll_error(ws) == 0
    ct, lp = cand_tok.cpu().numpy(), cand_logp.cpu().numpy()
    ctx_bits = synth.bf16_bits(ctx)
    chk = DraftChecker(ow, cfg.topk, cfg.K)
    lay = B.spec_draft_layout(h, cfg.B, cfg.topk, cfg.K)

    def levels_of(b):
        st, tk, sc = [], [], []
        for l in range(cfg.n):
            per, N = cfg.nodes(l) // cfg.B, cfg.nodes(l)
            S = ws_view(ws, lay.state[l], N * cfg.d_inner, torch.bfloat16).view(N, cfg.d_inner)
            st.append(S[b * per:(b + 1) * per].to(torch.float32).cpu().numpy())
            N1 = cfg.nodes(l + 1)
            per1 = N1 // cfg.B
            tk.append(ws_view(ws, lay.tok[l + 1], N1, torch.int32)[b * per1:(b + 1) * per1].cpu().numpy())
            sc.append(ws_view(ws, lay.score[l + 1], N1, torch.float32)[b * per1:(b + 1) * per1].cpu().numpy())
        return {"state": st, "tok": tk, "score": sc}

    for i, b in enumerate(range(cfg.B) if seqs is None else seqs):
        chk.check(ctx_bits[b], int(tok[b]), ct[b], lp[b], levels=levels_of(b), force_levels=(i == 0))
    # the K rows returned are the best K of the library's own leaf scores (property, any size)
    leaf = ws_view(ws, lay.score[cfg.n], cfg.B * cfg.leaves, torch.float32).view(cfg.B, cfg.leaves)
    top = torch.sort(leaf, dim=1, descending=True, stable=True).values[:, :cfg.K]
    assert torch.equal(top.cpu(), cand_logp.cpu())
    if check_levels:
        o_tok, o_lp, dd = oracle.draft(ow, ctx_bits, tok.numpy(), cfg.topk, cfg.K, dump=True, dump_logits=False)
        N = cfg.B
        for l in range(cfg.n if chk.tolerated == 0 else 1):
            S = ws_view(ws, lay.state[l], N * cfg.d_inner, torch.bfloat16).view(N, cfg.d_inner)
            S = S.to(torch.float32).cpu().numpy()
            # not teacher-forced: a one-ulp bf16 difference at one level perturbs the next level's input,
            # so the allowance grows with the depth (the per-level check in DraftChecker is the strict one)
            assert np.allclose(S, dd.states[l], rtol=0.008 * (1 + l), atol=2e-4 * (1 + l)), f"level {l} states"
            N *= cfg.topk[l]
            if chk.tolerated == 0:
                t = ws_view(ws, lay.tok[l + 1], N, torch.int32).cpu().numpy()
                sc = ws_view(ws, lay.score[l + 1], N, torch.float32).cpu().numpy()
                assert np.array_equal(t, dd.tok[l]), f"level {l} tokens"
                assert np.abs(sc - dd.score[l]).max() <= (l + 1) * LOGIT_TOL
    B.spec_destroy(h)
    return chk


@pytest.mark.parametrize("impl", [0, 1])
def test_draft_tiny_config(B, impl):
    chk = _draft_and_check(B, synth.CONFIGS["tiny"], impl=impl, check_levels=True)
    assert chk.tolerated == 0


@pytest.mark.parametrize("topk,K,Bn,V,d_base,d", [((3, 2, 2), 5, 2, 1000, 72, 64), ((1, 1, 1), 1, 3, 512, 64, 64),
                                                   ((8, 8), 64, 2, 2048, 128, 192), ((2, 2, 2, 2, 2), 7, 5, 640, 64, 128),
                                                   ((4, 3), 12, 150, 512, 64, 64)])
@pytest.mark.parametrize("swap", [0, 128])
def test_draft_odd_shapes(B, topk, K, Bn, V, d_base, d, swap):
    cfg = small_cfg(d_base=d_base, d_inner=d, V=V, topk=topk, K=K, B=Bn, seed=len(topk) + Bn)
    chk = _draft_and_check(B, cfg, check_levels=True, swap=swap)
    assert chk.tolerated <= max(1, Bn // 5)


@pytest.mark.parametrize("d", [2040, 2056, 4088, 4104])
@pytest.mark.parametrize("topk,K", [((3, 2), 5), ((2, 1, 1), 2)])
def test_draft_row_widths_round_the_thread_counts(B, topk, K, d):
    """State rows just below and above 2048 and 4096 elements: the row steps change their thread count and the
    number of element groups per thread there (256 threads, 512 threads, the wider kernels), in the separate mix
    kernel (three children per node) and in the fused merge + mix kernel (one or two children per node)."""
    cfg = small_cfg(d_base=72, d_inner=d, V=1000, topk=topk, K=K, B=3, seed=d % 97 + len(topk))
    chk = _draft_and_check(B, cfg, check_levels=True)
    assert chk.tolerated <= 1


@pytest.mark.parametrize("topk,K", [((3, 2, 2, 1, 1), 9), ((2, 2, 2, 1, 1, 1, 1), 8), ((2, 1, 2, 1, 2, 1, 2, 1), 16)])
def test_draft_code_model_head_counts(B, topk, K):
    """5, 7 (the code models of Sec. 4.3 / 4.4) and the maximum of 8 heads."""
    cfg = small_cfg(d_base=96, d_inner=128, V=3000, topk=topk, K=K, B=3, seed=40 + len(topk))
    chk = _draft_and_check(B, cfg, check_levels=True)
    assert chk.tolerated <= 1


def test_draft_weight_tied_heads(B):
    cfg = small_cfg(d_base=128, d_inner=128, V=2048, topk=(3, 2, 2, 2), K=10, B=4, seed=77)
    chk = _draft_and_check(B, cfg, check_levels=True, tie_weights=True)
    assert chk.tolerated <= 1


@pytest.mark.parametrize("name,Bn", [("llama2-7b", 1), ("llama2-7b", 16), ("llama2-7b", 64), ("llama2-13b", 1),
                                     ("llama2-13b", 16), ("llama2-13b", 64)])
def test_draft_single_candidate_at_production_width(B, name, Bn):
    """k = 1 (Sec. 4.2 / Sec. 5: the setting the paper recommends under load): topk = 1 at every head, one
    candidate per sequence, at the Llama2-7B- and 13B-shaped widths.  This is the chain of eight launches
    (the merge of a level also writes the one child's state): the candidate is the greedy chain."""
    import dataclasses
    cfg = dataclasses.replace(synth.CONFIGS[name], topk=(1, 1, 1), K=1, B=Bn)
    chk = _draft_and_check(B, cfg, seqs=range(0, Bn, max(1, Bn // 4)), check_levels=False)
    assert chk.tolerated <= 1


@pytest.mark.parametrize("topk,K", [((2, 2, 2), 5), ((2, 1, 2, 1), 3), ((1, 2, 1), 2)])
def test_draft_one_or_two_children_per_node(B, topk, K):
    """Branching factors of one and two: the merge of a level writes the children's states in the same launch."""
    cfg = small_cfg(d_base=96, d_inner=160, V=3000, topk=topk, K=K, B=5, seed=11 + len(topk))
    chk = _draft_and_check(B, cfg, check_levels=True)
    assert chk.tolerated <= 1


def test_quantize_head_is_rowwise_e4m3(B):
    """spec_quantize_head against the format's definition written with library casts: one scale per
    vocabulary row, max|row| / 448, and round-to-nearest-even e4m3 of row / scale."""
    cfg = small_cfg(d_base=64, d_inner=160, V=777, topk=(2, 2), seed=5)
    sw, ow, gw = _setup(cfg)
    gw.head[1][5].zero_()                                # an all-zero row keeps scale 1
    h = B.spec_create(gw)
    B.spec_attach_fp8_heads(h, levels=[1])
    q, sc = h._fp8[1]
    w = gw.head[1].to(torch.float32)
    amax = w.abs().amax(dim=1)
    want_sc = torch.where(amax > 0, torch.div(amax, torch.full_like(amax, 448.0)), torch.ones_like(amax))   # true division
    assert torch.equal(sc, want_sc)
    want_q = (w * torch.div(torch.ones_like(want_sc), want_sc)[:, None]).to(torch.float8_e4m3fn).view(torch.uint8)
    assert torch.equal(q, want_q)
    B.spec_destroy(h)


@pytest.mark.parametrize("topk,K,Bn,V,d_base,d", [((4, 3, 2), 8, 1, 1024, 256, 256), ((3, 2, 2), 5, 7, 1000, 80, 64),
                                                   ((8, 8), 64, 2, 2048, 128, 192), ((6, 4, 3), 32, 4, 8000, 96, 512)])
def test_draft_fp8_heads_small_shapes(B, topk, K, Bn, V, d_base, d):
    """e4m3 head + exact re-scoring of the short list: same protocol and tolerances as the bf16 path."""
    cfg = small_cfg(d_base=d_base, d_inner=d, V=V, topk=topk, K=K, B=Bn, seed=3 * len(topk) + Bn)
    # the normaliser comes from approximate logits (error ~1e-3), so leaves with nearly equal scores may
    # swap places against the oracle; every such list goes through the level-by-level check in DraftChecker
    chk = _draft_and_check(B, cfg, check_levels=False, fp8=True)
    assert chk.exact + chk.tolerated == Bn


@pytest.mark.parametrize("topk,K,Bn", [((4, 3), 12, 60), ((2, 3, 2), 6, 90)])
def test_draft_fp8_heads_on_levels_of_several_row_tiles(B, topk, K, Bn):
    """SPEC_OPT_FP8_MAX_ROWS raised: levels of 240 and 540 nodes (two and five 128-row tiles) in e4m3 too."""
    cfg = small_cfg(d_base=64, d_inner=128, V=1096, topk=topk, K=K, B=Bn, seed=Bn)
    chk = _draft_and_check(B, cfg, seqs=range(0, Bn, 7), fp8=True, fp8_rows=4096)
    assert chk.exact + chk.tolerated == len(range(0, Bn, 7))


@pytest.mark.parametrize("name,seqs", [("llama2-7b", (0, 3, 7)), ("llama2-13b", (1, 9))])
def test_draft_fp8_heads_full_size(B, name, seqs):
    """Full batch at the benchmark shapes with the e4m3 heads on the weight-bound levels; the oracle
    re-computes whole trees for a sample of sequences, and the candidates agree with the bf16 path's."""
    cfg = synth.CONFIGS[name]
    _draft_and_check(B, cfg, seqs=seqs, fp8=True)
    sw, ow, gw = _setup(cfg)
    ctx, tok = synth.make_draft_inputs(cfg)
    h = B.spec_create(gw)
    ref_tok, ref_lp, _ = B.spec_draft(h, ctx.cuda(), tok.cuda(), cfg.topk, cfg.K)
    B.spec_attach_fp8_heads(h)
    got_tok, got_lp, ws = B.spec_draft(h, ctx.cuda(), tok.cuda(), cfg.topk, cfg.K)
    assert B.spec_poll_error(ws) == 0
    # The normaliser of an e4m3 level comes from approximate logits (error ~1e-3 per level), so candidates
    # whose scores nearly coincide may swap places or, at the K-th place, be exchanged: compare what is
    # stable - the best candidate, the candidate SET of most sequences, and the scores of shared candidates.
    rt, gt = ref_tok.cpu().numpy(), got_tok.cpu().numpy()
    rl, gl = ref_lp.cpu().numpy(), got_lp.cpu().numpy()
    assert (rt[:, 0] == gt[:, 0]).all(), "the most confident candidate must not change"
    same_set = 0
    for b in range(cfg.B):
        ref = {tuple(c): s for c, s in zip(rt[b].tolist(), rl[b].tolist())}
        got = {tuple(c): s for c, s in zip(gt[b].tolist(), gl[b].tolist())}
        shared = set(ref) & set(got)
        assert len(shared) >= cfg.K - 2
        assert max(abs(ref[c] - got[c]) for c in shared) <= cfg.n * 5e-3
        same_set += len(shared) == cfg.K
    assert same_set >= 0.8 * cfg.B
    B.spec_destroy(h)


def _report_tolerated(record_property, name, chk, checked):
    """The number of sequences whose candidate list differs from the oracle's at a near-tie (each of them
    verified level by level on the GPU's own intermediates) is part of the result: print and record it."""
    print(f"[tolerated] {name}: {chk.tolerated} of {checked} checked sequences teacher-forced, {chk.exact} exact; "
          f"at most {chk.max_unshared} of {chk.K} candidates of such a sequence not in the oracle's list")
    record_property("tolerated", chk.tolerated)
    record_property("max_unshared", chk.max_unshared)
    record_property("checked", checked)


@pytest.mark.parametrize("swap", [None, 128])
def test_draft_llama2_7b_shape(B, record_property, swap):
    cfg = synth.CONFIGS["llama2-7b"]
    chk = _draft_and_check(B, cfg, swap=swap)
    _report_tolerated(record_property, cfg.name, chk, cfg.B)
    assert chk.exact + chk.tolerated == cfg.B
    # near-ties after a bf16 rounding flip (the synthetic heads give nearly flat distributions, so leaf scores
    # crowd together); each such sequence is checked level by level, and differs by neighbours changing places
    assert chk.tolerated <= cfg.B // 2 and chk.max_unshared <= 2


# one sequence of the first, a middle and the last 128-row tile of the last level at least
@pytest.mark.parametrize("name,seqs", [("llama2-13b", (0, 3, 7, 11, 15)), ("codellama-34b", (0, 9, 15, 22, 31)),
                                       ("llama3-8b", (0, 31, 63))])
def test_draft_full_size_sampled_sequences(B, record_property, name, seqs):
    """Full batch on the GPU in the benchmark's launch configuration; the oracle re-computes
    whole trees for a sample of sequences (the full batch would take it minutes to hours)."""
    chk = _draft_and_check(B, synth.CONFIGS[name], seqs=seqs)
    _report_tolerated(record_property, name, chk, len(seqs))
    assert chk.exact + chk.tolerated == len(seqs)
    # the more candidates are kept, the likelier two of them score within the rounding of a bf16 state and come
    # out in the other order (64 of 192 leaves on the largest shape: every sequence); what is bounded is how far a
    # tolerated list may be from the oracle's: neighbours changing places, and at most two memberships at the K-th place
    assert chk.max_unshared <= 2


def test_draft_is_deterministic_and_stream_ordered(B):
    cfg = synth.CONFIGS["tiny"]
    sw, ow, gw = _setup(cfg)
    ctx, tok = synth.make_draft_inputs(cfg)
    h = B.spec_create(gw)
    a = B.spec_draft(h, ctx.cuda(), tok.cuda(), cfg.topk, cfg.K)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        b = B.spec_draft(h, ctx.cuda(), tok.cuda(), cfg.topk, cfg.K, stream=s)
    s.synchronize()
    torch.cuda.synchronize()
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    B.spec_destroy(h)


def test_draft_token_out_of_range_sets_error_word_without_trapping(B):
    cfg = synth.CONFIGS["tiny"]
    sw, ow, gw = _setup(cfg)
    ctx, tok = synth.make_draft_inputs(cfg)
    bad = tok.clone()
    bad[0] = cfg.V + 5
    h = B.spec_create(gw)
    _, _, ws = B.spec_draft(h, ctx.cuda(), bad.cuda(), cfg.topk, cfg.K)
    assert B.spec_poll_error(ws) == B.SPEC_ERR_TOKEN_RANGE
    assert B.spec_poll_error(ws) == 0                       # cleared by the poll
    ct, lp, ws = B.spec_draft(h, ctx.cuda(), tok.cuda(), cfg.topk, cfg.K)   # the context is still usable
    assert B.spec_poll_error(ws) == 0
    B.spec_destroy(h)


def test_draft_argument_errors(B):
    cfg = synth.CONFIGS["tiny"]
    sw, ow, gw = _setup(cfg)
    ctx, tok = synth.make_draft_inputs(cfg)
    h = B.spec_create(gw)
    with pytest.raises(B.SpecError) as e:
        B.spec_draft(h, ctx.cuda(), tok.cuda(), cfg.topk, cfg.leaves + 1)
    assert e.value.status == B.SPEC_ERR_SHAPE
    with pytest.raises(B.SpecError) as e:
        B.spec_draft(h, ctx.cuda(), tok.cuda(), (9, 1, 1), 2)
    assert e.value.status == B.SPEC_ERR_SHAPE
    with pytest.raises(B.SpecError) as e:
        B.spec_draft(h, ctx.cuda(), tok.cuda(), cfg.topk, cfg.K, workspace=torch.empty(512, dtype=torch.uint8, device="cuda"))
    assert e.value.status == B.SPEC_ERR_WORKSPACE
    B.spec_destroy(h)


def test_draft_then_verify_chain_and_graph_replay(B):
    """Draft feeds verify on one stream; a CUDA graph of both replays to the same answer."""
    cfg = synth.CONFIGS["tiny"]
    sw, ow, gw = _setup(cfg)
    ctx, tok = synth.make_draft_inputs(cfg)
    ctx_d, tok_d = ctx.cuda(), tok.cuda()
    h = B.spec_create(gw)
    cand, logp, ws = B.spec_draft(h, ctx_d, tok_d, cfg.topk, cfg.K)
    logits = synth.make_base_logits(cfg, cand.cpu()).cuda()
    logits[0, 3, 0, cand[0, 3, 0]] = 30.0
    logits[0, 3, 1, cand[0, 3, 1]] = 30.0
    acc, best, nxt, vws = B.spec_verify(cand, logits)
    torch.cuda.synchronize()
    o = oracle.verify(cand.cpu().numpy(), synth.bf16_bits(logits), oracle.BF16)
    assert (acc.item(), best.item(), nxt.item()) == (o[0][0], o[1][0], o[2][0]) and acc.item() >= 2
    ref = (cand.clone(), logp.clone(), acc.clone(), best.clone(), nxt.clone())
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        with torch.cuda.graph(graph, stream=s):
            B.spec_draft(h, ctx_d, tok_d, cfg.topk, cfg.K, cand_tok=cand, cand_logp=logp, workspace=ws, stream=s)
            B.spec_verify(cand, logits, accept_len=acc, best_cand=best, next_tok=nxt, workspace=vws, stream=s)
    for t in (cand, logp, acc, best, nxt):
        t.zero_()
    graph.replay()
    torch.cuda.synchronize()
    for got, want in zip((cand, logp, acc, best, nxt), ref):
        assert torch.equal(got, want)
    B.spec_destroy(h)


@pytest.mark.parametrize("topk,K,fp8", [((8, 8, 8), 100, False), ((8, 8, 8), 512, False), ((8, 8, 8, 8), 300, False),
                                        ((8, 8, 8, 8), 4096, False), ((4, 4, 4, 5), 320, True)])
def test_draft_many_leaves_up_to_the_limit(B, topk, K, fp8):
    """More than 256 leaves per sequence (the sorted prune instead of the ranked one), up to
    SPEC_MAX_LEAVES = 4096 with K = every leaf."""
    cfg = small_cfg(d_base=48, d_inner=64, V=96, topk=topk, K=K, B=2, seed=sum(topk) + K)
    chk = _draft_and_check(B, cfg, fp8=fp8)
    assert chk.exact + chk.tolerated == cfg.B


def test_draft_refuses_more_leaves_than_the_limit(B):
    cfg = small_cfg(d_base=48, d_inner=64, V=96, topk=(8, 8, 8, 8, 2), K=4, B=1, seed=1)   # 8192 leaves
    sw, ow, gw = _setup(cfg)
    h = B.spec_create(gw)
    ctx, tok = synth.make_draft_inputs(cfg)
    assert B.spec_draft_workspace_bytes(h, 1, cfg.topk, 4) == 0
    with pytest.raises(B.SpecError) as e:
        B.spec_draft(h, ctx.cuda(), tok.cuda(), cfg.topk, 4)
    assert e.value.status == B.SPEC_ERR_SHAPE
    assert B.spec_draft_workspace_bytes(h, 1, (8, 8, 8, 8, 1), 4096) > 0       # exactly at the limit
    with pytest.raises(B.SpecError) as e:                                       # K beyond the leaves
        B.spec_draft(h, ctx.cuda(), tok.cuda(), (8, 8, 8, 8, 1), 4097)
    assert e.value.status == B.SPEC_ERR_SHAPE
    B.spec_destroy(h)


@pytest.mark.parametrize("d,fp8", [(4104, False), (5120, False), (16384, False), (16448, False),
                                   (5120, True), (16384, True), (16448, True)])
def test_draft_wide_states(B, d, fp8):
    """State widths beyond the benchmark shapes: each range of d_inner has its own mix + LayerNorm + GELU
    kernel (rows kept in registers up to 16384 elements, in shared memory beyond)."""
    cfg = small_cfg(d_base=64, d_inner=d, V=264, topk=(2, 2), K=3, B=2, seed=d % 97)
    chk = _draft_and_check(B, cfg, check_levels=not fp8, fp8=fp8)
    assert chk.exact + chk.tolerated == cfg.B


@pytest.mark.parametrize("name,fp8", [("llama2-13b", False), ("codellama-34b", False), ("llama2-7b", True)])
def test_draft_repeats_are_bit_identical_at_full_size(B, name, fp8):
    """200 back-to-back drafts of the same input into rotating output buffers: the CTA that happens to finish a
    sequence's last level also prunes it, so which CTA that is varies from run to run; the result must not."""
    cfg = synth.CONFIGS[name]
    sw = synth.make_weights(cfg, device="cuda")
    h = B.spec_create(sw)
    if fp8:
        B.spec_attach_fp8_heads(h)
    ctx, tok = synth.make_draft_inputs(cfg, device="cuda")
    ws = torch.empty(B.spec_draft_workspace_bytes(h, cfg.B, cfg.topk, cfg.K), dtype=torch.uint8, device="cuda")
    reps = 200
    cands = torch.full((reps, cfg.B, cfg.K, cfg.n), -1, dtype=torch.int32, device="cuda")
    logps = torch.full((reps, cfg.B, cfg.K), float("nan"), dtype=torch.float32, device="cuda")
    for i in range(reps):
        B.spec_draft(h, ctx, tok, cfg.topk, cfg.K, cand_tok=cands[i], cand_logp=logps[i], workspace=ws)
    torch.cuda.synchronize()
    assert B.spec_poll_error(ws) == 0
    assert bool((cands == cands[0]).all()) and bool((logps == logps[0]).all())
    assert int(cands.min()) >= 0
    B.spec_destroy(h)
