"""GPU parity of spec_verify against the oracle: bit-exact g, accept_len, best_cand, next_tok."""
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


def _np_logits(x: torch.Tensor):
    if x.dtype == torch.bfloat16:
        return synth.bf16_bits(x), oracle.BF16
    return x.detach().cpu().numpy(), oracle.F32


def _check_g(g_gpu, o_g, cand_np, early):
    """Streaming form: every row's arg-max.  Early-exit form: rows up to and including a candidate's
    first mismatch (all n + 1 rows when everything matches) equal the oracle's, the rest hold -1."""
    if not early:
        assert np.array_equal(g_gpu, o_g)
        return
    Bn, K, n = cand_np.shape
    m = np.zeros((Bn, K), np.int64)
    for j in range(n - 1, -1, -1):
        m = np.where(cand_np[:, :, j] == o_g[:, :, j], m + 1, 0)     # matched prefix length
    read = np.arange(n + 1)[None, None, :] <= m[:, :, None]
    assert np.array_equal(g_gpu[read], o_g[read])
    assert (g_gpu[~read] == -1).all()


def _run_and_compare(B, cand: torch.Tensor, logits: torch.Tensor, forms=(False, True)):
    Bn, K, n = cand.shape
    ln, dt = _np_logits(logits)
    o_acc, o_best, o_nxt, o_g = oracle.verify(cand.cpu().numpy(), ln, dt, want_g=True)
    for early in forms:
        acc, best, nxt, ws = B.spec_verify(cand.cuda(), logits.cuda(), early_exit=early)
        assert B.spec_poll_error(ws) == 0
        g_gpu = ws_view(ws, 256, Bn * K * (n + 1), torch.int32).cpu().numpy().reshape(Bn, K, n + 1)
        V = logits.shape[-1]
        vectors = V % (8 if logits.dtype == torch.bfloat16 else 4) == 0     # else the early form falls back
        _check_g(g_gpu, o_g, cand.cpu().numpy(), early and vectors)
        assert np.array_equal(acc.cpu().numpy(), o_acc)
        assert np.array_equal(best.cpu().numpy(), o_best)
        assert np.array_equal(nxt.cpu().numpy(), o_nxt)
    return o_acc


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("shape", [(1, 8, 3, 1024), (3, 5, 2, 1000), (2, 3, 4, 1021), (2, 7, 1, 8), (1, 1, 1, 1),
                                   (4, 2, 7, 4100), (2, 64, 4, 50264), (2, 20, 12, 96), (1, 300, 9, 64)])
def test_verify_small_shapes(B, dtype, shape):
    Bn, K, n, V = shape
    g = torch.Generator().manual_seed(sum(shape))
    logits = (torch.randn(Bn, K, n + 1, V, generator=g) * 2).to(dtype)
    cand = torch.randint(0, V, (Bn, K, n), generator=g, dtype=torch.int64).to(torch.int32)
    # plant prefixes of varying length so that accept_len is not always 0
    am = logits.to(torch.float32).argmax(-1)
    for b in range(Bn):
        for k in range(K):
            m = (b + 2 * k) % (n + 1)
            cand[b, k, :m] = am[b, k, :m].to(torch.int32)
    acc = _run_and_compare(B, cand, logits)
    if K > 1 and n > 1:
        assert acc.max() > 0


def test_verify_unaligned_base_pointer(B):
    g = torch.Generator().manual_seed(5)
    V = 1000
    buf = (torch.randn(2 * 3 * 4 * V + 3, generator=g) * 2).to(torch.bfloat16).cuda()
    logits = buf[3:].view(2, 3, 4, V)          # 6-byte offset: takes the scalar path
    assert logits.data_ptr() % 16 != 0
    cand = torch.randint(0, V, (2, 3, 3), generator=g, dtype=torch.int64).to(torch.int32)
    acc, best, nxt, ws = B.spec_verify(cand.cuda(), logits)
    ln = synth.bf16_bits(logits.cpu().contiguous())
    o = oracle.verify(cand.numpy(), ln, oracle.BF16)
    assert np.array_equal(acc.cpu().numpy(), o[0]) and np.array_equal(best.cpu().numpy(), o[1])
    assert np.array_equal(nxt.cpu().numpy(), o[2])


def test_verify_ties_nan_and_infinities(B):
    V = 2048
    x = torch.zeros(1, 3, 4, V)                           # n = 3; the last row of every candidate is all zeros
    x[0, 0, 0, [7, 900, 2047]] = 5.0                      # tie: first wins
    x[0, 0, 1] = float("nan")                             # all NaN -> 0
    x[0, 0, 2] = float("-inf")                            # all -inf -> 0
    x[0, 1, 0, 5] = float("nan"); x[0, 1, 0, 1500] = 1.0  # NaN never wins
    x[0, 1, 1, 100] = float("inf"); x[0, 1, 1, 101] = float("inf")
    x[0, 1, 2] = -1.0; x[0, 1, 2, 2040] = -0.0            # -0.0 is the maximum
    x[0, 2, 0] = -3.0; x[0, 2, 0, 1024] = -2.5
    x[0, 2, 1, 0] = 1.0
    x[0, 2, 2, V - 1] = 1.0
    cand = torch.tensor([[[7, 0, 0], [1500, 100, 9], [1024, 0, 5]]], dtype=torch.int32)
    for dt in (torch.bfloat16, torch.float32):
        acc = _run_and_compare(B, cand, x.to(dt))
        assert acc[0] == 3


def test_verify_worked_example(B):
    g = [[2, 3, 0, 4], [2, 3, 1, 0], [2, 0, 0, 3]]
    x = torch.zeros(1, 3, 4, 5)
    for k in range(3):
        for j in range(4):
            x[0, k, j, g[k][j]] = 10.0
    cand = torch.tensor([[[2, 4, 1], [2, 3, 0], [1, 0, 0]]], dtype=torch.int32)
    acc, best, nxt, _ = B.spec_verify(cand.cuda(), x.cuda())
    assert (acc.item(), best.item(), nxt.item()) == (2, 1, 1)
    x[0, 1, 1, 1] = 10.0
    acc, best, nxt, _ = B.spec_verify(cand.cuda(), x.cuda())
    assert (acc.item(), best.item(), nxt.item()) == (1, 0, 3)


@pytest.mark.parametrize("name", ["tiny", "llama2-7b", "llama2-13b", "codellama-34b", "llama3-8b"])
def test_verify_full_size_configs(B, name):
    """Full benchmark shapes in the launch configuration the benchmark times, streaming and early-exit
    forms; the oracle checks every row (the CPU arg-max over the whole tensor takes seconds)."""
    cfg = synth.CONFIGS[name]
    cand = synth.random_cand_tok(cfg, device="cuda")
    logits = synth.make_base_logits(cfg, cand, device="cuda")
    rows = cfg.B * cfg.K * (cfg.n + 1)
    got = []
    for early in (False, True):
        acc, best, nxt, ws = B.spec_verify(cand, logits, early_exit=early)
        torch.cuda.synchronize()
        g_gpu = ws_view(ws, 256, rows, torch.int32).cpu().numpy().reshape(cfg.B, cfg.K, cfg.n + 1)
        got.append((g_gpu, acc.cpu().numpy(), best.cpu().numpy(), nxt.cpu().numpy()))
    bits = synth.bf16_bits(logits)
    del logits
    o_acc, o_best, o_nxt, o_g = oracle.verify(cand.cpu().numpy(), bits, oracle.BF16, want_g=True)
    for early, (g_gpu, acc, best, nxt) in zip((False, True), got):
        _check_g(g_gpu, o_g, cand.cpu().numpy(), early)
        assert np.array_equal(acc, o_acc)
        assert np.array_equal(best, o_best)
        assert np.array_equal(nxt, o_nxt)
    if cfg.plant != "none":
        assert o_acc.max() >= 1


def test_verify_argument_errors(B):
    cand = torch.zeros((1, 2, 2), dtype=torch.int32, device="cuda")
    logits = torch.zeros((1, 2, 3, 64), dtype=torch.bfloat16, device="cuda")
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.SpecError) as e:
        B.spec_verify(cand, logits, workspace=small)
    assert e.value.status == B.SPEC_ERR_WORKSPACE


@pytest.mark.parametrize("B_,K,n,d", [(1, 1, 1, 8), (3, 5, 3, 40), (16, 8, 3, 5120), (4, 7, 2, 13), (64, 16, 4, 4096)])
def test_next_ctx_matches_the_oracle(B, B_, K, n, d):
    g = torch.Generator().manual_seed(B_ * 131 + d)
    base = torch.randn(B_, K, n + 1, d, generator=g).to(torch.bfloat16)
    best = torch.randint(0, K, (B_,), generator=g, dtype=torch.int64).to(torch.int32)
    acc = torch.randint(0, n + 1, (B_,), generator=g, dtype=torch.int64).to(torch.int32)
    want = oracle.next_ctx(synth.bf16_bits(base), best.numpy(), acc.numpy())
    err = torch.zeros(64, dtype=torch.int32, device="cuda")
    got = B.spec_next_ctx(base.cuda(), best.cuda(), acc.cuda(), err_workspace=err)
    assert np.array_equal(synth.bf16_bits(got.cpu()), want)
    assert int(err[0]) == 0
    # an unaligned view of the same data takes the element-wise path
    if d % 8 == 0:
        flat = torch.empty(base.numel() + 1, dtype=torch.bfloat16, device="cuda")
        flat[1:] = base.cuda().flatten()
        got2 = B.spec_next_ctx(flat[1:].view(B_, K, n + 1, d), best.cuda(), acc.cuda())
        assert np.array_equal(synth.bf16_bits(got2.cpu()), want)


def test_next_ctx_reports_bad_indices_and_writes_zeros(B):
    B_, K, n, d = 3, 4, 2, 16
    base = torch.ones(B_, K, n + 1, d, dtype=torch.bfloat16, device="cuda")
    best = torch.tensor([0, K, 1], dtype=torch.int32, device="cuda")       # K is one past the end
    acc = torch.tensor([n, 0, n + 1], dtype=torch.int32, device="cuda")    # n + 1 too
    err = torch.zeros(64, dtype=torch.int32, device="cuda")
    out = B.spec_next_ctx(base, best, acc, err_workspace=err)
    assert int(err[0]) == B.SPEC_ERR_INDEX_RANGE
    assert out.float().cpu().tolist() == [[1.0] * d, [0.0] * d, [0.0] * d]


def test_draft_verify_next_ctx_close_the_loop(B):
    """Three decode steps chained on the device: draft -> verify -> next_ctx -> draft, no host round trip
    between the calls; each step's results equal the oracle's run on the same inputs."""
    cfg = small_cfg(d_base=64, d_inner=64, V=520, topk=(3, 2, 2), K=5, B=4, seed=77)
    sw = synth.make_weights(cfg)
    ow, gw = to_oracle_weights(sw), weights_to_cuda(sw)
    ctx, tok = synth.make_draft_inputs(cfg)
    h = B.spec_create(gw)
    ctx_d, tok_d = ctx.cuda(), tok.cuda()
    gen = torch.Generator().manual_seed(5)
    for step in range(3):
        cand, logp, dws = B.spec_draft(h, ctx_d, tok_d, cfg.topk, cfg.K)
        logits = torch.randn(cfg.B, cfg.K, cfg.n + 1, cfg.V, generator=gen).to(torch.bfloat16)
        hidden = torch.randn(cfg.B, cfg.K, cfg.n + 1, cfg.d_base, generator=gen).to(torch.bfloat16)
        c = cand.cpu()
        for b in range(cfg.B):                       # make some candidates partly right
            for k in range(cfg.K):
                for j in range((b + k + step) % (cfg.n + 1)):
                    logits[b, k, j, int(c[b, k, j])] = 30.0
        acc, best, nxt, vws = B.spec_verify(cand, logits.cuda())
        nctx = B.spec_next_ctx(hidden.cuda(), best, acc, err_workspace=vws)
        assert B.spec_poll_error(dws) == 0 and B.spec_poll_error(vws) == 0
        # oracle on the same inputs
        o_cand, o_logp = oracle.draft(ow, synth.bf16_bits(ctx_d.cpu()), tok_d.cpu().numpy(), cfg.topk, cfg.K)[:2]
        assert np.array_equal(c.numpy(), o_cand)
        o_acc, o_best, o_nxt = oracle.verify(o_cand, synth.bf16_bits(logits), oracle.BF16)
        assert np.array_equal(acc.cpu().numpy(), o_acc) and np.array_equal(best.cpu().numpy(), o_best)
        assert np.array_equal(nxt.cpu().numpy(), o_nxt)
        o_ctx = oracle.next_ctx(synth.bf16_bits(hidden), o_best, o_acc)
        assert np.array_equal(synth.bf16_bits(nctx.cpu()), o_ctx)
        assert int(acc.max()) > 0
        ctx_d, tok_d = nctx, nxt
    B.spec_destroy(h)


@pytest.mark.parametrize("K,n", [(4096, 2), (1536, 7), (12288 // 33, 32)])
def test_verify_at_the_row_limit(B, K, n):
    """K (n + 1) = 12288 rows per sequence (or the largest K below it) is the documented limit."""
    Bn, V = 2, 40
    g = torch.Generator().manual_seed(K + n)
    logits = torch.randn(Bn, K, n + 1, V, generator=g).to(torch.bfloat16)
    cand = torch.randint(0, V, (Bn, K, n), generator=g, dtype=torch.int64).to(torch.int32)
    am = logits.to(torch.float32).argmax(-1)
    cand[0, K - 1] = am[0, K - 1, :n].to(torch.int32)        # the last candidate of sequence 0 is fully right
    cand[1, K // 2, : n // 2 + 1] = am[1, K // 2, : n // 2 + 1].to(torch.int32)
    want = oracle.verify(cand.numpy(), synth.bf16_bits(logits), oracle.BF16)
    for early in (False, True):
        acc, best, nxt, _ = B.spec_verify(cand.cuda(), logits.cuda(), early_exit=early)
        for a, w in zip((acc, best, nxt), want):
            assert np.array_equal(a.cpu().numpy(), w)
    assert int(want[0][0]) == n


def test_verify_refuses_more_rows_than_the_limit(B):
    K, n, V = 4097, 2, 8                                       # 12291 rows per sequence
    logits = torch.zeros(1, K, n + 1, V, dtype=torch.bfloat16, device="cuda")
    cand = torch.zeros(1, K, n, dtype=torch.int32, device="cuda")
    ws = torch.empty(1 << 22, dtype=torch.uint8, device="cuda")
    outs = [torch.empty(1, dtype=torch.int32, device="cuda") for _ in range(3)]
    with pytest.raises(B.SpecError) as e:
        B.spec_verify(cand, logits, accept_len=outs[0], best_cand=outs[1], next_tok=outs[2], workspace=ws)
    assert e.value.status == B.SPEC_ERR_SHAPE
