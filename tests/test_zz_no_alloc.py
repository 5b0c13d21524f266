"""spec_verify_static (the verify entry point for callers that cannot supply scratch memory: the
partial maxima and the arg-max table live in an array built into the library) must give exactly what
spec_verify gives, call after call, although every call reuses the same array and finds the previous
call's leftovers in it.  Collected last on purpose: a run that stops at the first failure has then
already been through every other test."""
import pytest
import torch

from paper_2404_19124_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2404_19124_b200 import build
    build.build()
    from paper_2404_19124_b200 import binding
    return binding


def _case(shape, seed, dtype):
    Bn, K, n, V = shape
    g = torch.Generator().manual_seed(seed)
    logits = (torch.randn(Bn, K, n + 1, V, generator=g) * 2).to(dtype)
    cand = torch.randint(0, V, (Bn, K, n), generator=g, dtype=torch.int64).to(torch.int32)
    am = logits.to(torch.float32).argmax(-1)
    for b in range(Bn):
        for k in range(K):
            m = (b + 3 * k + seed) % (n + 1)       # planted prefixes: accept_len is not all zero
            cand[b, k, :m] = am[b, k, :m].to(torch.int32)
    return cand.cuda(), logits.cuda()


def _both(B, cand, logits):
    want = B.spec_verify(cand, logits)[:3]
    got = [torch.full((cand.shape[0],), -7, dtype=torch.int32, device="cuda") for _ in range(3)]
    B.spec_verify_static(cand, logits, *got)
    torch.cuda.synchronize()
    for g, w in zip(got, want):
        assert torch.equal(g, w)       # integer results: bit-exact, as for spec_verify itself
    return want[0]


def test_two_calls_in_a_row_match_the_workspace_entry_point(B):
    # first call: many rows, several partial slots per row; it leaves the array full of its own partials
    acc1 = _both(B, *_case((3, 16, 3, 8000), 1, torch.bfloat16))
    assert acc1.max().item() > 0
    # second call straight after, other shape and dtype, same array, nothing cleared in between
    acc2 = _both(B, *_case((2, 5, 4, 50264), 2, torch.float32))
    assert acc2.max().item() > 0
    # and the first problem again: the leftovers of the second call must not leak into it
    _both(B, *_case((3, 16, 3, 8000), 1, torch.bfloat16))


def test_benchmark_shape_fits_and_oversized_problem_is_refused(B):
    cfg = synth.CONFIGS["llama2-13b"]
    assert B.spec_verify_workspace_bytes(cfg.B, cfg.K, cfg.n, cfg.V, B.SPEC_BF16) <= B.SPEC_VERIFY_STATIC_SCRATCH_BYTES
    cand = synth.random_cand_tok(cfg, device="cuda")
    logits = synth.make_base_logits(cfg, cand, device="cuda")
    _both(B, cand, logits)
    # rows * slots beyond the array: refused on the host, nothing runs
    Bn, K, n, V = 4096, 16, 3, 8
    assert B.spec_verify_workspace_bytes(Bn, K, n, V, B.SPEC_BF16) > B.SPEC_VERIFY_STATIC_SCRATCH_BYTES
    cand = torch.zeros((Bn, K, n), dtype=torch.int32, device="cuda")
    logits = torch.zeros((Bn, K, n + 1, V), dtype=torch.bfloat16, device="cuda")
    outs = [torch.empty(Bn, dtype=torch.int32, device="cuda") for _ in range(3)]
    with pytest.raises(B.SpecError) as e:
        B.spec_verify_static(cand, logits, *outs)
    assert e.value.status == B.SPEC_ERR_STATIC_SCRATCH
