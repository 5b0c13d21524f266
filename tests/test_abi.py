"""The C-ABI library loads without a GPU and exports every entry point the header declares;
host-side argument checks answer without touching a device."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2404_19124_b200 import build
    build.build()
    from paper_2404_19124_b200 import binding as b
    return b


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "spec_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(spec_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(binding):
    names = _declared_functions()
    assert "spec_draft" in names and "spec_verify" in names and len(names) >= 12
    lib = C.CDLL(binding.LIB_PATH)
    for name in names:
        assert hasattr(lib, name), f"{name} declared in include/spec_b200.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_version_and_status_strings(binding):
    assert binding.spec_version() >= 1
    seen = {binding.spec_status_str(s) for s in range(8)}
    assert len(seen) == 8 and "ok" in seen
    assert binding.spec_status_str(99) == "unknown status"


def test_verify_host_side_validation(binding):
    lib = C.CDLL(binding.LIB_PATH)
    lib.spec_verify_workspace_bytes.restype = C.c_size_t
    assert lib.spec_verify_workspace_bytes(0, 4, 3, 100, 0) == 0
    assert lib.spec_verify_workspace_bytes(2, 4, 3, 100, 7) == 0
    need = lib.spec_verify_workspace_bytes(2, 4, 3, 1000, 0)
    assert need >= 256 + 4 * 2 * 4 * 4 and need % 256 == 0
    # null pointers and bad shapes are rejected before anything is enqueued
    assert lib.spec_verify(None, None, 0, 1, 1, 1, 8, None, None, None, None, C.c_size_t(0), None) == binding.SPEC_ERR_INVALID_ARG
    one = C.c_void_p(256)
    args = lambda K, n: (one, one, 0, 1, K, n, 8, one, one, one, one, C.c_size_t(1 << 30), None)
    lib.spec_verify.argtypes = binding._lib.spec_verify.argtypes
    assert lib.spec_verify(*args(70000, 1)) == binding.SPEC_ERR_SHAPE
    assert lib.spec_verify(one, one, 0, 1, 2, 2, 8, one, one, one, None, C.c_size_t(0), None) == binding.SPEC_ERR_WORKSPACE
    assert lib.spec_verify(one, one, 0, 1, 2, 2, 8, one, one, one, C.c_void_p(257), C.c_size_t(1 << 20), None) == binding.SPEC_ERR_WORKSPACE


def test_create_rejects_bad_weights_and_missing_device(binding):
    import torch
    w = binding.SpecWeightsC()
    h = C.c_void_p()
    assert binding._lib.spec_create(C.byref(h), None) == binding.SPEC_ERR_INVALID_ARG
    w.n_heads, w.V, w.d_base, w.d_inner = 0, 10, 16, 16
    assert binding._lib.spec_create(C.byref(h), C.byref(w)) == binding.SPEC_ERR_SHAPE
    w.n_heads, w.d_inner = 1, 12       # not a multiple of 8
    assert binding._lib.spec_create(C.byref(h), C.byref(w)) == binding.SPEC_ERR_SHAPE
    w.d_inner = 16                      # null weight pointers
    assert binding._lib.spec_create(C.byref(h), C.byref(w)) == binding.SPEC_ERR_INVALID_ARG
    if not torch.cuda.is_available():
        for arr in (w.emb, w.proj, w.ln_gamma, w.ln_beta, w.head):
            arr[0] = 4096
        w.ln_eps = 1e-5
        # the product path refuses to run without a device instead of falling back to anything
        assert binding._lib.spec_create(C.byref(h), C.byref(w)) == binding.SPEC_ERR_NO_DEVICE
        assert not h.value


def test_choose_k_follows_the_callers_batch_table(binding):
    """Sec. 4.2 / Sec. 5: several candidates at batch size 1 (the paper quotes k = 5 with 6/3/2 branching pruned
    to k, Sec. 4.1), one candidate under load, speculation off beyond a batch size.  The thresholds are the
    caller's; the call only looks the batch size up.  Runs on the host, no device needed."""
    rules = [(1, 5, (6, 3, 2)), (8, 2, (2, 1, 1)), (32, 1, (1, 1, 1)), (64, 0, ())]
    want = {1: (5, (6, 3, 2)), 2: (2, (2, 1, 1)), 8: (2, (2, 1, 1)), 9: (1, (1, 1, 1)), 32: (1, (1, 1, 1)),
            33: (0, ()), 64: (0, ()), 65: (0, ()), 10 ** 6: (0, ())}
    for b, w in want.items():
        assert binding.spec_choose_k(b, 3, rules) == w
    bad = [
        [(4, 1, (1, 1, 1)), (4, 0, ())],            # max_batch not strictly ascending
        [(4, 5, (2, 2, 1))],                        # K beyond the leaves
        [(4, 1, (1, 0, 1))],                        # a branching factor of zero
        [(4, 1, (9, 1, 1))],                        # beyond SPEC_MAX_TOPK
        [(0, 1, (1, 1, 1))],                        # a batch limit below one
        [(4, -1, (1, 1, 1))],
    ]
    for table in bad:
        with pytest.raises(binding.SpecError) as e:
            binding.spec_choose_k(2, 3, table)
        assert e.value.status == binding.SPEC_ERR_INVALID_ARG
    with pytest.raises(binding.SpecError):
        binding.spec_choose_k(0, 3, rules)
