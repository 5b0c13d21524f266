"""ctypes front-end of the CPU oracle (``spec_oracle.c``).

TEST INFRASTRUCTURE ONLY: the test-suite, the smoke check and the CPU-baseline leg of the
benchmark load this; the CUDA library and its Python binding never do, and this package
imports nothing from them.  All arrays are numpy; bf16 tensors travel as ``uint16`` bit
patterns so both sides read identical bytes.

Paper passages restated by each routine are cited in ``spec_oracle.c``.
``next_ctx`` (the one routine written here, in numpy) is pinned by a hand-built example in the tests.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "spec_oracle.c")


def _cpu_tag() -> str:
    """Short hash of this host's CPU feature flags: the library is compiled with -march=native, so a
    copy built on another machine must not be loaded here."""
    import hashlib
    flags = ""
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    flags = line
                    break
    except OSError:
        pass
    return hashlib.sha1(flags.encode()).hexdigest()[:10]


_LIB = os.path.join(_HERE, f"libspec_oracle.{_cpu_tag()}.so")

MAX_HEADS = 8
BF16, F32 = 0, 1
OK, ERR_ARG, ERR_SHAPE, ERR_TOKEN, ERR_NOMEM = 0, 1, 2, 3, 4


class OracleError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"oracle {where} failed with status {code}")
        self.code = code


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C11 + OpenMP); returns the library path."""
    if force or (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O3", "-march=native", "-fopenmp", "-std=c11", "-Wall", "-shared", "-fPIC",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _CWeights(C.Structure):
    _fields_ = [
        ("n_heads", C.c_int32), ("V", C.c_int32), ("d_base", C.c_int32), ("d_inner", C.c_int32),
        ("emb", C.c_void_p * MAX_HEADS),
        ("proj", C.c_void_p * MAX_HEADS),
        ("ln_gamma", C.c_void_p * MAX_HEADS),
        ("ln_beta", C.c_void_p * MAX_HEADS),
        ("head", C.c_void_p * MAX_HEADS),
        ("state_weight", C.c_float), ("emb_weight", C.c_float), ("ln_eps", C.c_float),
        ("round_state_bf16", C.c_int32),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_logsumexp.restype = C.c_float
        _lib.oracle_bf16_to_f32.restype = C.c_float
        _lib.oracle_bf16_to_f32.argtypes = [C.c_uint16]
        _lib.oracle_f32_to_bf16.restype = C.c_uint16
        _lib.oracle_f32_to_bf16.argtypes = [C.c_float]
        _lib.oracle_row_argmax.restype = C.c_int32
        _lib.oracle_row_argmax.argtypes = [C.c_void_p, C.c_int, C.c_size_t, C.c_int]
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, "bf16 data must be passed as uint16 bit patterns"
    return a


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


@dataclass
class Weights:
    """Speculator parameters: one (emb, proj, ln_gamma, ln_beta, head) set per head."""
    V: int
    d_base: int
    d_inner: int
    emb: List[np.ndarray]        # uint16 (bf16 bits) [V, d_inner]
    proj: List[np.ndarray]       # uint16 [d_inner, d_in]
    ln_gamma: List[np.ndarray]   # float32 [d_inner]
    ln_beta: List[np.ndarray]    # float32 [d_inner]
    head: List[np.ndarray]       # uint16 [V, d_inner]
    state_weight: float
    emb_weight: float
    ln_eps: float = 1e-5
    round_state_bf16: bool = True
    _keep: list = field(default_factory=list, repr=False)

    @property
    def n_heads(self) -> int:
        return len(self.head)

    def d_in(self, level: int) -> int:
        return self.d_base if level == 0 else self.d_inner

    def c_struct(self) -> _CWeights:
        n = self.n_heads
        assert 1 <= n <= MAX_HEADS
        cw = _CWeights()
        cw.n_heads, cw.V, cw.d_base, cw.d_inner = n, self.V, self.d_base, self.d_inner
        self._keep = []
        for l in range(n):
            e, p, h = _u16(self.emb[l]), _u16(self.proj[l]), _u16(self.head[l])
            g, b = _f32(self.ln_gamma[l]), _f32(self.ln_beta[l])
            assert e.shape == (self.V, self.d_inner) and h.shape == (self.V, self.d_inner)
            assert p.shape == (self.d_inner, self.d_in(l))
            assert g.shape == (self.d_inner,) and b.shape == (self.d_inner,)
            self._keep += [e, p, h, g, b]
            cw.emb[l], cw.proj[l], cw.head[l] = e.ctypes.data, p.ctypes.data, h.ctypes.data
            cw.ln_gamma[l], cw.ln_beta[l] = g.ctypes.data, b.ctypes.data
        cw.state_weight, cw.emb_weight, cw.ln_eps = self.state_weight, self.emb_weight, self.ln_eps
        cw.round_state_bf16 = 1 if self.round_state_bf16 else 0
        return cw


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (numpy only; used to feed float inputs)."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def f32_to_bf16_bits(x) -> int:
    return int(lib().oracle_f32_to_bf16(C.c_float(float(x))))


def stage_state(w: Weights, level: int, s_parent: np.ndarray, tok: int, intermediates: bool = False):
    """One node of one stage: returns the post-GELU state (and p, h, y when asked)."""
    cw = w.c_struct()
    sp = _f32(s_parent)
    assert sp.shape == (w.d_in(level),)
    s = np.empty(w.d_inner, np.float32)
    p = np.empty(w.d_inner, np.float32) if intermediates else None
    h = np.empty(w.d_inner, np.float32) if intermediates else None
    y = np.empty(w.d_inner, np.float32) if intermediates else None
    rc = lib().oracle_stage_state(C.byref(cw), C.c_int(level), _ptr(sp), C.c_int32(int(tok)), _ptr(s),
                                  _ptr(p), _ptr(h), _ptr(y))
    if rc != OK:
        raise OracleError(rc, "stage_state")
    return (s, p, h, y) if intermediates else s


def stage_logits(w: Weights, level: int, S: np.ndarray) -> np.ndarray:
    """logits[r, :] = Wout_level . S[r] for a batch of states."""
    cw = w.c_struct()
    S = _f32(S)
    assert S.ndim == 2 and S.shape[1] == w.d_inner
    out = np.empty((S.shape[0], w.V), np.float32)
    rc = lib().oracle_stage_logits(C.byref(cw), C.c_int(level), _ptr(S), C.c_int(S.shape[0]), _ptr(out))
    if rc != OK:
        raise OracleError(rc, "stage_logits")
    return out


def logsumexp(x: np.ndarray) -> float:
    x = _f32(x)
    return float(lib().oracle_logsumexp(_ptr(x), C.c_int(x.size)))


def topk(x: np.ndarray, k: int):
    x = _f32(x)
    ids = np.empty(k, np.int32)
    vals = np.empty(k, np.float32)
    rc = lib().oracle_topk(_ptr(x), C.c_int(x.size), C.c_int(k), _ptr(ids), _ptr(vals))
    if rc != OK:
        raise OracleError(rc, "topk")
    return ids, vals


@dataclass
class DraftDump:
    states: List[np.ndarray]
    logits: List[np.ndarray]
    tok: List[np.ndarray]
    score: List[np.ndarray]


def draft(w: Weights, ctx_state_bits: np.ndarray, last_tok: np.ndarray, topk_per_head: Sequence[int], K: int,
          dump: bool = False, dump_logits: bool = True):
    """Draft tree for a batch; returns (cand_tok [B,K,n] int32, cand_logp [B,K] float32[, DraftDump])."""
    cw = w.c_struct()
    ctx = _u16(ctx_state_bits)
    lt = _i32(last_tok)
    B = lt.shape[0]
    assert ctx.shape == (B, w.d_base)
    n = w.n_heads
    tk = _i32(list(topk_per_head))
    assert tk.shape == (n,)
    cand_tok = np.empty((B, K, n), np.int32)
    cand_logp = np.empty((B, K), np.float32)
    dd = None
    arrs = [None] * 4
    if dump:
        N = B
        st, lg, tt, sc = [], [], [], []
        for l in range(n):
            st.append(np.empty((N, w.d_inner), np.float32))
            lg.append(np.empty((N, w.V), np.float32) if dump_logits else None)
            tt.append(np.empty(N * int(tk[l]), np.int32))
            sc.append(np.empty(N * int(tk[l]), np.float32))
            N *= int(tk[l])
        dd = DraftDump(st, lg, tt, sc)

        def parr(lst):
            a = (C.c_void_p * MAX_HEADS)()
            for i, x in enumerate(lst):
                a[i] = None if x is None else x.ctypes.data
            return a
        arrs = [parr(st), parr(lg), parr(tt), parr(sc)]
    rc = lib().oracle_draft(C.byref(cw), _ptr(ctx), _ptr(lt), C.c_int(B), _ptr(tk), C.c_int(int(K)),
                            _ptr(cand_tok), _ptr(cand_logp), arrs[0], arrs[1], arrs[2], arrs[3])
    if rc != OK:
        raise OracleError(rc, "draft")
    return (cand_tok, cand_logp, dd) if dump else (cand_tok, cand_logp)


def row_argmax(base_logits: np.ndarray, dtype: int, row: int, V: int) -> int:
    """First index of the maximum of one row (rows are V contiguous elements)."""
    a = np.ascontiguousarray(base_logits)
    return int(lib().oracle_row_argmax(_ptr(a), C.c_int(dtype), C.c_size_t(int(row) * V), C.c_int(V)))


def verify(cand_tok: np.ndarray, base_logits: np.ndarray, dtype: int, want_g: bool = False):
    """Greedy verification.  base_logits: [B,K,n+1,V] (uint16 bf16 bits when dtype == BF16, else float32)."""
    ct = _i32(cand_tok)
    B, K, n = ct.shape
    bl = np.ascontiguousarray(base_logits)
    assert bl.shape[:3] == (B, K, n + 1)
    V = bl.shape[3]
    assert bl.dtype == (np.uint16 if dtype == BF16 else np.float32)
    acc = np.empty(B, np.int32)
    best = np.empty(B, np.int32)
    nxt = np.empty(B, np.int32)
    g = np.empty((B, K, n + 1), np.int32) if want_g else None
    rc = lib().oracle_verify(_ptr(ct), _ptr(bl), C.c_int(dtype), C.c_int(B), C.c_int(K), C.c_int(n), C.c_int(V),
                             _ptr(acc), _ptr(best), _ptr(nxt), _ptr(g))
    if rc != OK:
        raise OracleError(rc, "verify")
    return (acc, best, nxt, g) if want_g else (acc, best, nxt)


def next_ctx(base_state: np.ndarray, best_cand: np.ndarray, accept_len: np.ndarray) -> np.ndarray:
    """State vector the next draft starts from (Sec. 3.1: the speculator is fed the base model's latest
    state; after a verified step that is the one at the last accepted position of the best candidate).
    base_state [B, K, n+1, d] of any dtype -> [B, d].  Written as the loop it is, one sequence at a time."""
    B, K, n1, d = base_state.shape
    out = np.empty((B, d), base_state.dtype)
    for b in range(B):
        k, m = int(best_cand[b]), int(accept_len[b])
        if not (0 <= k < K and 0 <= m < n1):
            raise OracleError(1, "next_ctx: index out of range")
        for i in range(d):
            out[b, i] = base_state[b, k, m, i]
    return out


def num_threads() -> int:
    return int(lib().oracle_num_threads())
