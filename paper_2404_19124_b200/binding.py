"""Thin ctypes binding of libspec_b200.so (the C ABI declared in include/spec_b200.h).

Argument marshalling only: every step of the draft / verify path runs inside the CUDA
library.  PyTorch supplies device memory and streams.  There is no fallback: if the
compiled library is missing, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Tuple, List, Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libspec_b200.so")

MAX_HEADS, MAX_TOPK, MAX_LEAVES = 8, 8, 4096
(SPEC_OK, SPEC_ERR_INVALID_ARG, SPEC_ERR_SHAPE, SPEC_ERR_WORKSPACE, SPEC_ERR_CUDA, SPEC_ERR_TOKEN_RANGE,
 SPEC_ERR_TIMEOUT, SPEC_ERR_NO_DEVICE, SPEC_ERR_STATIC_SCRATCH, SPEC_ERR_INDEX_RANGE) = range(10)
SPEC_VERIFY_STATIC_SCRATCH_BYTES = 1 << 20
SPEC_BF16, SPEC_F32 = 0, 1
SPEC_OPT_GEMM_IMPL, SPEC_OPT_HEAD_BLOCK_N, SPEC_OPT_PROJ_BLOCK_N, SPEC_OPT_PROFILE, SPEC_OPT_FP8_MAX_ROWS = 0, 1, 2, 3, 4
SPEC_OPT_HEAD_SWAP_MAX_ROWS = 5
SPEC_OPT_GEMM_PRODUCERS = 6
SPEC_OPT_HEAD_PAIR = 7

EXPORTS = [
    "spec_version", "spec_status_str", "spec_last_cuda_error", "spec_create", "spec_destroy", "spec_set_option",
    "spec_draft_workspace_bytes", "spec_draft_layout", "spec_draft", "spec_verify_workspace_bytes", "spec_verify",
    "spec_profile_read", "spec_poll_error", "spec_head_workspace_bytes", "spec_head_logits", "spec_head_topk",
    "spec_verify_static", "spec_verify_early", "spec_quantize_head", "spec_set_head_fp8",
    "spec_head_partials", "spec_next_ctx", "spec_choose_k",
    "spec_set_vocab_shard", "spec_draft_vp_exchange", "spec_draft_vp_local", "spec_draft_vp_merge",
]

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2404_19124_b200.build` "
        "(nvcc, sm_100a). There is no CPU or PyTorch fallback for the draft / verify path.")

_lib = C.CDLL(LIB_PATH)


class SpecWeightsC(C.Structure):
    _fields_ = [
        ("n_heads", C.c_int32), ("V", C.c_int32), ("d_base", C.c_int32), ("d_inner", C.c_int32),
        ("emb", C.c_void_p * MAX_HEADS), ("proj", C.c_void_p * MAX_HEADS),
        ("ln_gamma", C.c_void_p * MAX_HEADS), ("ln_beta", C.c_void_p * MAX_HEADS),
        ("head", C.c_void_p * MAX_HEADS),
        ("state_weight", C.c_float), ("emb_weight", C.c_float), ("ln_eps", C.c_float),
    ]


class SpecDraftLayoutC(C.Structure):
    _fields_ = [
        ("total_bytes", C.c_uint64), ("error_word", C.c_uint64),
        ("tok", C.c_uint64 * (MAX_HEADS + 1)), ("score", C.c_uint64 * (MAX_HEADS + 1)),
        ("state", C.c_uint64 * MAX_HEADS), ("proj", C.c_uint64), ("state8", C.c_uint64), ("state8_scale", C.c_uint64),
        ("part_val", C.c_uint64), ("part_idx", C.c_uint64), ("part_ms", C.c_uint64), ("logits", C.c_uint64),
        ("block_n", C.c_int32 * MAX_HEADS), ("n_tiles", C.c_int32 * MAX_HEADS),
    ]


_lib.spec_version.restype = C.c_int
_lib.spec_status_str.restype = C.c_char_p
_lib.spec_status_str.argtypes = [C.c_int]
_lib.spec_last_cuda_error.restype = C.c_int
_lib.spec_create.argtypes = [C.POINTER(C.c_void_p), C.POINTER(SpecWeightsC)]
_lib.spec_destroy.argtypes = [C.c_void_p]
_lib.spec_set_option.argtypes = [C.c_void_p, C.c_int, C.c_int]
_lib.spec_draft_workspace_bytes.restype = C.c_size_t
_lib.spec_draft_workspace_bytes.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_int32), C.c_int]
_lib.spec_draft_layout.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_int32), C.c_int, C.POINTER(SpecDraftLayoutC)]
_lib.spec_draft.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.POINTER(C.c_int32), C.c_int,
                            C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
_lib.spec_verify_workspace_bytes.restype = C.c_size_t
_lib.spec_verify_workspace_bytes.argtypes = [C.c_int] * 5
_lib.spec_verify.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                             C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
_lib.spec_choose_k.argtypes = [C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
_lib.spec_verify_static.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                    C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
_lib.spec_verify_early.argtypes = _lib.spec_verify.argtypes
_lib.spec_set_vocab_shard.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int]
_lib.spec_draft_vp_exchange.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_int32), C.c_int, C.c_int,
                                        C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
_lib.spec_draft_vp_local.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int, C.POINTER(C.c_int32), C.c_int,
                                     C.c_void_p, C.c_size_t, C.c_void_p]
_lib.spec_draft_vp_merge.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_int32), C.c_int, C.c_void_p, C.c_void_p,
                                     C.c_void_p, C.c_size_t, C.c_void_p]
_lib.spec_next_ctx.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p,
                                C.c_void_p, C.c_void_p]
_lib.spec_quantize_head.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
_lib.spec_set_head_fp8.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
_lib.spec_poll_error.argtypes = [C.c_void_p, C.c_void_p]
_lib.spec_profile_read.argtypes = [C.c_void_p, C.POINTER(C.c_float), C.c_int, C.POINTER(C.c_int)]
_lib.spec_head_workspace_bytes.restype = C.c_size_t
_lib.spec_head_workspace_bytes.argtypes = [C.c_void_p, C.c_int, C.c_int]
_lib.spec_head_logits.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
_lib.spec_head_partials.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_size_t, C.c_void_p]
_lib.spec_head_topk.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                C.c_void_p, C.c_size_t, C.c_void_p]


class SpecError(RuntimeError):
    def __init__(self, status: int, where: str):
        msg = _lib.spec_status_str(status).decode()
        extra = f" (cuda error {_lib.spec_last_cuda_error()})" if status == SPEC_ERR_CUDA else ""
        super().__init__(f"{where}: {msg}{extra}")
        self.status = status


def _check(status: int, where: str) -> None:
    if status != SPEC_OK:
        raise SpecError(status, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream_ptr(stream: Optional[torch.cuda.Stream]):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _dev(t: torch.Tensor, dtype: torch.dtype, shape=None, name: str = "tensor") -> torch.Tensor:
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CUDA tensor of {dtype}")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} must have shape {tuple(shape)}, got {tuple(t.shape)}")
    return t


def _topk_arr(topk: Sequence[int]):
    return (C.c_int32 * len(topk))(*[int(x) for x in topk])


def spec_version() -> int:
    return int(_lib.spec_version())


def spec_status_str(status: int) -> str:
    return _lib.spec_status_str(int(status)).decode()


class SpecHandle:
    """Owns a spec_handle_t and keeps the weight tensors alive."""

    def __init__(self, emb: List[torch.Tensor], proj: List[torch.Tensor], ln_gamma: List[torch.Tensor],
                 ln_beta: List[torch.Tensor], head: List[torch.Tensor], state_weight: float, emb_weight: float,
                 ln_eps: float = 1e-5, vocab_shard: Optional[Tuple[int, int, int]] = None):
        """vocab_shard = (rank, n_ranks, vocab_offset): the head tensors hold only the vocabulary rows
        [vocab_offset, vocab_offset + head[l].shape[0]) (spec_set_vocab_shard); emb keeps all V rows."""
        n = len(head)
        if not (1 <= n <= MAX_HEADS) or not all(len(x) == n for x in (emb, proj, ln_gamma, ln_beta)):
            raise ValueError("need the same number (1..8) of emb / proj / ln_gamma / ln_beta / head tensors")
        head_rows, d_inner = head[0].shape
        V = emb[0].shape[0]
        if head_rows != V and vocab_shard is None:
            raise ValueError("head tensors with fewer rows than the embeddings need vocab_shard=(rank, n_ranks, offset)")
        d_base = proj[0].shape[1]
        w = SpecWeightsC()
        w.n_heads, w.V, w.d_base, w.d_inner = n, V, d_base, d_inner
        for l in range(n):
            d_in = d_base if l == 0 else d_inner
            w.emb[l] = _dev(emb[l], torch.bfloat16, (V, d_inner), f"emb[{l}]").data_ptr()
            w.proj[l] = _dev(proj[l], torch.bfloat16, (d_inner, d_in), f"proj[{l}]").data_ptr()
            w.ln_gamma[l] = _dev(ln_gamma[l], torch.float32, (d_inner,), f"ln_gamma[{l}]").data_ptr()
            w.ln_beta[l] = _dev(ln_beta[l], torch.float32, (d_inner,), f"ln_beta[{l}]").data_ptr()
            w.head[l] = _dev(head[l], torch.bfloat16, (head_rows, d_inner), f"head[{l}]").data_ptr()
        w.state_weight, w.emb_weight, w.ln_eps = state_weight, emb_weight, ln_eps
        self._keep = (emb, proj, ln_gamma, ln_beta, head)
        self.n_heads, self.V, self.d_base, self.d_inner = n, V, d_base, d_inner
        self.device = head[0].device
        self._h = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(_lib.spec_create(C.byref(self._h), C.byref(w)), "spec_create")
        self.vp_rank, self.vp_ranks = 0, 1
        if vocab_shard is not None:
            rank, n_ranks, offset = (int(x) for x in vocab_shard)
            _check(_lib.spec_set_vocab_shard(self._h, rank, n_ranks, offset, int(head_rows)), "spec_set_vocab_shard")
            self.vp_rank, self.vp_ranks = rank, n_ranks

    def close(self) -> None:
        if getattr(self, "_h", None) and self._h.value:
            _lib.spec_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def ptr(self):
        return self._h


def spec_create(weights, vocab_shard: Optional[Tuple[int, int, int]] = None) -> SpecHandle:
    """`weights`: an object with emb / proj / ln_gamma / ln_beta / head tensor lists (CUDA) and the scalars
    state_weight, emb_weight, ln_eps (e.g. synth.SpecWeights moved to the GPU).  vocab_shard: see SpecHandle."""
    return SpecHandle(weights.emb, weights.proj, weights.ln_gamma, weights.ln_beta, weights.head,
                      weights.state_weight, weights.emb_weight, weights.ln_eps, vocab_shard=vocab_shard)


def spec_destroy(h: SpecHandle) -> None:
    h.close()


def spec_set_option(h: SpecHandle, option: int, value: int) -> None:
    _check(_lib.spec_set_option(h.ptr, int(option), int(value)), "spec_set_option")


def spec_draft_workspace_bytes(h: SpecHandle, B: int, topk: Sequence[int], K: int) -> int:
    return int(_lib.spec_draft_workspace_bytes(h.ptr, int(B), _topk_arr(topk), int(K)))


def spec_draft_layout(h: SpecHandle, B: int, topk: Sequence[int], K: int) -> SpecDraftLayoutC:
    lay = SpecDraftLayoutC()
    _check(_lib.spec_draft_layout(h.ptr, int(B), _topk_arr(topk), int(K), C.byref(lay)), "spec_draft_layout")
    return lay


def spec_draft(h: SpecHandle, ctx_state: torch.Tensor, last_tok: torch.Tensor, topk: Sequence[int], K: int,
               cand_tok: Optional[torch.Tensor] = None, cand_logp: Optional[torch.Tensor] = None,
               workspace: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """Enqueues one draft; returns (cand_tok [B,K,n] int32, cand_logp [B,K] fp32, workspace)."""
    B = ctx_state.shape[0]
    _dev(ctx_state, torch.bfloat16, (B, h.d_base), "ctx_state")
    _dev(last_tok, torch.int32, (B,), "last_tok")
    if len(topk) != h.n_heads:
        raise SpecError(SPEC_ERR_SHAPE, "spec_draft: len(topk) != n_heads")
    if cand_tok is None:
        cand_tok = torch.empty((B, K, h.n_heads), dtype=torch.int32, device=h.device)
    if cand_logp is None:
        cand_logp = torch.empty((B, K), dtype=torch.float32, device=h.device)
    _dev(cand_tok, torch.int32, (B, K, h.n_heads), "cand_tok")
    _dev(cand_logp, torch.float32, (B, K), "cand_logp")
    if workspace is None:
        need = spec_draft_workspace_bytes(h, B, topk, K)
        if need == 0:
            raise SpecError(SPEC_ERR_SHAPE, "spec_draft_workspace_bytes")
        workspace = torch.empty(need, dtype=torch.uint8, device=h.device)
    _check(_lib.spec_draft(h.ptr, _ptr(ctx_state), _ptr(last_tok), B, _topk_arr(topk), int(K), _ptr(cand_tok),
                           _ptr(cand_logp), _ptr(workspace), workspace.numel(), _stream_ptr(stream)), "spec_draft")
    return cand_tok, cand_logp, workspace


def spec_set_vocab_shard(h: SpecHandle, rank: int, n_ranks: int, vocab_offset: int, head_rows: int) -> None:
    _check(_lib.spec_set_vocab_shard(h.ptr, int(rank), int(n_ranks), int(vocab_offset), int(head_rows)),
           "spec_set_vocab_shard")
    h.vp_rank, h.vp_ranks = int(rank), int(n_ranks)


def spec_draft_vp_exchange(h: SpecHandle, B: int, topk: Sequence[int], K: int, level: int) -> Tuple[int, int]:
    """(byte offset of slot 0 in the draft workspace, bytes of one rank's slot) at `level`."""
    off, sz = C.c_uint64(), C.c_uint64()
    _check(_lib.spec_draft_vp_exchange(h.ptr, int(B), _topk_arr(topk), int(K), int(level), C.byref(off), C.byref(sz)),
           "spec_draft_vp_exchange")
    return int(off.value), int(sz.value)


def spec_draft_vp_local(h: SpecHandle, level: int, ctx_state: torch.Tensor, last_tok: torch.Tensor,
                        topk: Sequence[int], K: int, workspace: torch.Tensor,
                        stream: Optional[torch.cuda.Stream] = None) -> None:
    B = ctx_state.shape[0]
    _dev(ctx_state, torch.bfloat16, (B, h.d_base), "ctx_state")
    _dev(last_tok, torch.int32, (B,), "last_tok")
    _check(_lib.spec_draft_vp_local(h.ptr, int(level), _ptr(ctx_state), _ptr(last_tok), B, _topk_arr(topk), int(K),
                                    _ptr(workspace), workspace.numel(), _stream_ptr(stream)), "spec_draft_vp_local")


def spec_draft_vp_merge(h: SpecHandle, level: int, B: int, topk: Sequence[int], K: int, workspace: torch.Tensor,
                        cand_tok: Optional[torch.Tensor] = None, cand_logp: Optional[torch.Tensor] = None,
                        stream: Optional[torch.cuda.Stream] = None) -> None:
    if cand_tok is not None:
        _dev(cand_tok, torch.int32, (B, K, h.n_heads), "cand_tok")
        _dev(cand_logp, torch.float32, (B, K), "cand_logp")
    _check(_lib.spec_draft_vp_merge(h.ptr, int(level), int(B), _topk_arr(topk), int(K),
                                    _ptr(cand_tok) if cand_tok is not None else None,
                                    _ptr(cand_logp) if cand_logp is not None else None,
                                    _ptr(workspace), workspace.numel(), _stream_ptr(stream)), "spec_draft_vp_merge")


def spec_verify_workspace_bytes(B: int, K: int, n: int, V: int, logits_dtype: int) -> int:
    return int(_lib.spec_verify_workspace_bytes(B, K, n, V, logits_dtype))


class SpecKRuleC(C.Structure):
    _fields_ = [("max_batch", C.c_int32), ("K", C.c_int32), ("topk", C.c_int32 * MAX_HEADS)]


def spec_choose_k(B: int, n_heads: int, rules: Sequence[Tuple[int, int, Sequence[int]]]) -> Tuple[int, Tuple[int, ...]]:
    """rules: (max_batch, K, topk) entries by ascending max_batch; returns (K, topk) for a batch of B sequences,
    (0, ()) when speculation is off at that batch size.  Host-only."""
    arr = (SpecKRuleC * len(rules))()
    for i, (mb, K, topk) in enumerate(rules):
        arr[i].max_batch, arr[i].K = int(mb), int(K)
        for l, t in enumerate(topk):
            arr[i].topk[l] = int(t)
    K_out = C.c_int32(0)
    tk = (C.c_int32 * MAX_HEADS)()
    _check(_lib.spec_choose_k(int(B), int(n_heads), arr, len(rules), C.byref(K_out), tk), "spec_choose_k")
    return int(K_out.value), (tuple(int(tk[l]) for l in range(n_heads)) if K_out.value > 0 else ())


def spec_verify(cand_tok: torch.Tensor, base_logits: torch.Tensor, accept_len: Optional[torch.Tensor] = None,
                best_cand: Optional[torch.Tensor] = None, next_tok: Optional[torch.Tensor] = None,
                workspace: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None,
                early_exit: bool = False):
    """Enqueues one verification; returns (accept_len, best_cand, next_tok, workspace), int32 [B] each.
    early_exit: the form that stops reading a candidate's rows at its first mismatch (spec_verify_early)."""
    B, K, n = cand_tok.shape
    _dev(cand_tok, torch.int32, name="cand_tok")
    if base_logits.dtype == torch.bfloat16:
        dt = SPEC_BF16
    elif base_logits.dtype == torch.float32:
        dt = SPEC_F32
    else:
        raise ValueError("base_logits must be bf16 or fp32")
    V = base_logits.shape[-1]
    _dev(base_logits, base_logits.dtype, (B, K, n + 1, V), "base_logits")
    dev = cand_tok.device
    outs = []
    for t, name in ((accept_len, "accept_len"), (best_cand, "best_cand"), (next_tok, "next_tok")):
        if t is None:
            t = torch.empty(B, dtype=torch.int32, device=dev)
        outs.append(_dev(t, torch.int32, (B,), name))
    if workspace is None:
        need = spec_verify_workspace_bytes(B, K, n, V, dt)
        if need == 0:
            raise SpecError(SPEC_ERR_SHAPE, "spec_verify_workspace_bytes")
        workspace = torch.empty(need, dtype=torch.uint8, device=dev)
    fn = _lib.spec_verify_early if early_exit else _lib.spec_verify
    _check(fn(_ptr(cand_tok), _ptr(base_logits), dt, B, K, n, V, _ptr(outs[0]), _ptr(outs[1]),
              _ptr(outs[2]), _ptr(workspace), workspace.numel(), _stream_ptr(stream)), "spec_verify")
    return outs[0], outs[1], outs[2], workspace


def spec_verify_static(cand_tok: torch.Tensor, base_logits: torch.Tensor, accept_len: torch.Tensor,
                       best_cand: torch.Tensor, next_tok: torch.Tensor,
                       stream: Optional[torch.cuda.Stream] = None) -> None:
    """spec_verify for callers that cannot provide a workspace: the scratch is an array inside the
    library (SPEC_VERIFY_STATIC_SCRATCH_BYTES).  All three outputs must be passed in (int32 [B], CUDA);
    this wrapper creates no tensor.  Raises SpecError(SPEC_ERR_STATIC_SCRATCH) when the problem is too
    large for the array.  Make the first call on a device outside of stream capture; calls that may
    overlap on the GPU must be ordered by the caller, they share the array."""
    B, K, n = cand_tok.shape
    _dev(cand_tok, torch.int32, name="cand_tok")
    if base_logits.dtype == torch.bfloat16:
        dt = SPEC_BF16
    elif base_logits.dtype == torch.float32:
        dt = SPEC_F32
    else:
        raise ValueError("base_logits must be bf16 or fp32")
    V = base_logits.shape[-1]
    _dev(base_logits, base_logits.dtype, (B, K, n + 1, V), "base_logits")
    for t, name in ((accept_len, "accept_len"), (best_cand, "best_cand"), (next_tok, "next_tok")):
        _dev(t, torch.int32, (B,), name)
    with torch.cuda.device(cand_tok.device):
        _check(_lib.spec_verify_static(_ptr(cand_tok), _ptr(base_logits), dt, B, K, n, V, _ptr(accept_len),
                                       _ptr(best_cand), _ptr(next_tok), _stream_ptr(stream)), "spec_verify_static")


def spec_next_ctx(base_state: torch.Tensor, best_cand: torch.Tensor, accept_len: torch.Tensor,
                  ctx_state: Optional[torch.Tensor] = None, err_workspace: Optional[torch.Tensor] = None,
                  stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """ctx_state[b] = base_state[b, best_cand[b], accept_len[b]]: the state the next spec_draft starts from.
    `err_workspace` (e.g. the verify workspace) receives SPEC_ERR_INDEX_RANGE at offset 0 on a bad index."""
    B, K, n1, d = base_state.shape
    _dev(base_state, torch.bfloat16, name="base_state")
    _dev(best_cand, torch.int32, (B,), "best_cand")
    _dev(accept_len, torch.int32, (B,), "accept_len")
    if ctx_state is None:
        ctx_state = torch.empty((B, d), dtype=torch.bfloat16, device=base_state.device)
    _dev(ctx_state, torch.bfloat16, (B, d), "ctx_state")
    with torch.cuda.device(base_state.device):
        _check(_lib.spec_next_ctx(_ptr(base_state), _ptr(best_cand), _ptr(accept_len), B, K, n1 - 1, d, _ptr(ctx_state),
                                  _ptr(err_workspace) if err_workspace is not None else None, _stream_ptr(stream)),
               "spec_next_ctx")
    return ctx_state


def spec_attach_fp8_heads(h: SpecHandle, levels: Optional[Sequence[int]] = None,
                          stream: Optional[torch.cuda.Stream] = None) -> None:
    """Quantises the heads of `levels` (default: all) to e4m3 (spec_quantize_head) into tensors the handle
    keeps alive and attaches them (spec_set_head_fp8).  Allocation happens here, in the caller's framework,
    not in the library."""
    if not hasattr(h, "_fp8"):
        h._fp8 = {}
    for l in (range(h.n_heads) if levels is None else levels):
        q = torch.empty((h.V, h.d_inner), dtype=torch.uint8, device=h.device)
        sc = torch.empty(h.V, dtype=torch.float32, device=h.device)
        _check(_lib.spec_quantize_head(h.ptr, int(l), _ptr(q), _ptr(sc), _stream_ptr(stream)), "spec_quantize_head")
        _check(_lib.spec_set_head_fp8(h.ptr, int(l), _ptr(q), _ptr(sc)), "spec_set_head_fp8")
        h._fp8[int(l)] = (q, sc)


def spec_detach_fp8_heads(h: SpecHandle) -> None:
    for l in range(h.n_heads):
        _check(_lib.spec_set_head_fp8(h.ptr, int(l), None, None), "spec_set_head_fp8")
    h._fp8 = {}


def spec_profile_read(h: SpecHandle) -> List[float]:
    """Per-kernel milliseconds of the last profiled spec_draft (see SPEC_OPT_PROFILE)."""
    buf = (C.c_float * 64)()
    cnt = C.c_int(0)
    _check(_lib.spec_profile_read(h.ptr, buf, 64, C.byref(cnt)), "spec_profile_read")
    return [float(buf[i]) for i in range(cnt.value)]


def spec_poll_error(workspace: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> int:
    return int(_lib.spec_poll_error(_ptr(workspace), _stream_ptr(stream)))


def spec_head_workspace_bytes(h: SpecHandle, rows: int, topk: int) -> int:
    return int(_lib.spec_head_workspace_bytes(h.ptr, int(rows), int(topk)))


def spec_head_logits(h: SpecHandle, level: int, states: torch.Tensor, logits: Optional[torch.Tensor] = None,
                     stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    rows = states.shape[0]
    _dev(states, torch.bfloat16, (rows, h.d_inner), "states")
    if logits is None:
        logits = torch.empty((rows, h.V), dtype=torch.float32, device=h.device)
    _dev(logits, torch.float32, (rows, h.V), "logits")
    _check(_lib.spec_head_logits(h.ptr, int(level), _ptr(states), rows, _ptr(logits), _stream_ptr(stream)),
           "spec_head_logits")
    return logits


def spec_head_partials(h: SpecHandle, level: int, states: torch.Tensor, topk: int, workspace: torch.Tensor,
                       stream: Optional[torch.cuda.Stream] = None) -> None:
    """The head GEMM with its fused epilogue alone (first kernel of spec_head_topk); for timing."""
    rows = states.shape[0]
    _dev(states, torch.bfloat16, (rows, h.d_inner), "states")
    _check(_lib.spec_head_partials(h.ptr, int(level), _ptr(states), rows, int(topk), _ptr(workspace),
                                   workspace.numel(), _stream_ptr(stream)), "spec_head_partials")


def spec_head_topk(h: SpecHandle, level: int, states: torch.Tensor, topk: int, tok: Optional[torch.Tensor] = None,
                   logp: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                   stream: Optional[torch.cuda.Stream] = None):
    rows = states.shape[0]
    _dev(states, torch.bfloat16, (rows, h.d_inner), "states")
    if tok is None:
        tok = torch.empty((rows, topk), dtype=torch.int32, device=h.device)
    if logp is None:
        logp = torch.empty((rows, topk), dtype=torch.float32, device=h.device)
    if workspace is None:
        workspace = torch.empty(spec_head_workspace_bytes(h, rows, topk), dtype=torch.uint8, device=h.device)
    _check(_lib.spec_head_topk(h.ptr, int(level), _ptr(states), rows, int(topk), _ptr(tok), _ptr(logp),
                               _ptr(workspace), workspace.numel(), _stream_ptr(stream)), "spec_head_topk")
    return tok, logp, workspace
