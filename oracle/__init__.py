"""CPU oracle for the BlockFFN chunk-verify FFN forward (ctypes front end).

TEST INFRASTRUCTURE, NOT PRODUCT: only the tests, the smoke check and the
benchmark's CPU-baseline leg import this package. It loads the plain C file
``blockffn_oracle.c`` (compiled with gcc on first use) and exposes each routine
with numpy arrays in and out. It imports nothing from the CUDA package.

Every function names the passage of the paper it follows; the arithmetic lives
in the C file, in double precision, sequential and unblocked.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "blockffn_oracle.c")
_LIB = os.path.join(_HERE, "libblockffn_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle's C file into a shared object next to it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fvisibility=hidden",
             "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_tls.restype = ctypes.c_double
        _lib.oracle_cls.restype = ctypes.c_double
    return _lib


def _p(a, ctype):
    if a is None:
        return None
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def mask_words(E: int) -> int:
    return (E + 31) // 32


def router(x, W_r, gain, bias=None, eps=1e-6):
    """Eq. 3: scores = RMSNorm(ReLU(W_router^T x)) with per-expert gain.

    x: uint16 bf16 bits [L][d]; W_r: [E][d]. Returns (a0, scores), float64 [L][E].
    """
    x, W_r, gain, bias = _u16(x), _u16(W_r), _f32(gain), _f32(bias)
    L, d = x.shape
    E = W_r.shape[0]
    assert W_r.shape == (E, d) and gain.shape == (E,)
    a0 = np.empty((L, E), np.float64)
    s = np.empty((L, E), np.float64)
    _load().oracle_router(_p(x, ctypes.c_uint16), _p(W_r, ctypes.c_uint16), _p(gain, ctypes.c_float),
                          _p(bias, ctypes.c_float), L, d, E, ctypes.c_double(eps),
                          _p(a0, ctypes.c_double), _p(s, ctypes.c_double))
    return a0, s


def router_relu_only(x, W_r, bias=None):
    """Sec. 4.2.3 ablation: the router without RMSNorm, scores = ReLU(W_router^T x).

    Returns (a0, scores), float64 [L][E]."""
    x, W_r, bias = _u16(x), _u16(W_r), _f32(bias)
    L, d = x.shape
    E = W_r.shape[0]
    assert W_r.shape == (E, d)
    a0 = np.empty((L, E), np.float64)
    s = np.empty((L, E), np.float64)
    _load().oracle_router_relu_only(_p(x, ctypes.c_uint16), _p(W_r, ctypes.c_uint16),
                                    _p(bias, ctypes.c_float), L, d, E, _p(a0, ctypes.c_double),
                                    _p(s, ctypes.c_double))
    return a0, s


def reuse_ratio(scores, acc=None):
    """Sec. 4.1.2: adds the sum of |S_i n S_{i+1}| / |S_i| over the successive token pairs of one
    sequence to acc[0] and the number of pairs counted to acc[1] (float64[2], created when None).
    The sequence's reuse ratio is acc[0] / acc[1]."""
    scores = np.ascontiguousarray(scores, dtype=np.float64)
    L, E = scores.shape
    if acc is None:
        acc = np.zeros(2, np.float64)
    assert acc.dtype == np.float64 and acc.shape == (2,)
    _load().oracle_reuse_ratio(_p(scores, ctypes.c_double), L, E, _p(acc, ctypes.c_double))
    return acc


def token_masks(scores):
    """Sec. 3.3 sparse pattern of A(x): bit i of row t set iff scores[t, i] != 0."""
    scores = np.ascontiguousarray(scores, dtype=np.float64)
    L, E = scores.shape
    m = np.empty((L, mask_words(E)), np.uint32)
    _load().oracle_token_masks(_p(scores, ctypes.c_double), L, E, _p(m, ctypes.c_uint32))
    return m


def chunk_union(tok_mask, E, stats=None):
    """Sec. 3.3 Union(x) + the Sec. 2.1 counters. Returns (union_mask, ids[E], n_union).

    stats: optional uint64[4] accumulated in place (tokens, active, chunks, union).
    """
    tok_mask = np.ascontiguousarray(tok_mask, dtype=np.uint32)
    L = tok_mask.shape[0]
    um = np.empty(mask_words(E), np.uint32)
    ids = np.empty(E, np.int32)
    n = ctypes.c_int32(0)
    if stats is not None:
        assert stats.dtype == np.uint64 and stats.shape == (4,)
    _load().oracle_chunk_union(_p(tok_mask, ctypes.c_uint32), L, E, _p(um, ctypes.c_uint32),
                               _p(ids, ctypes.c_int32), ctypes.byref(n), _p(stats, ctypes.c_uint64))
    return um, ids, int(n.value)


def tls(stats, E):
    """Sec. 2.1 token-level sparsity from the counters."""
    stats = np.ascontiguousarray(stats, dtype=np.uint64)
    return float(_load().oracle_tls(_p(stats, ctypes.c_uint64), E))


def cls(stats, E):
    """Sec. 2.1 chunk-level sparsity CLS_L from the counters (one call = one chunk)."""
    stats = np.ascontiguousarray(stats, dtype=np.uint64)
    return float(_load().oracle_cls(_p(stats, ctypes.c_uint64), E))


def expert_ffn(x, scores, U, D, expert_ids=None):
    """Eq. 1 + Eq. 2. expert_ids=None sums over all experts (the definition);
    a list restricts the sum to those experts (Sec. 3.3). Returns float64 [L][d]."""
    x, U, D = _u16(x), _u16(U), _u16(D)
    scores = np.ascontiguousarray(scores, dtype=np.float64)
    L, d = x.shape
    E, d_e, d2 = U.shape
    assert d2 == d and D.shape == (E, d, d_e) and scores.shape == (L, E)
    out = np.empty((L, d), np.float64)
    ids = None if expert_ids is None else np.ascontiguousarray(expert_ids, dtype=np.int32)
    n = 0 if ids is None else int(ids.shape[0])
    _load().oracle_expert_ffn(_p(x, ctypes.c_uint16), _p(scores, ctypes.c_double),
                              _p(U, ctypes.c_uint16), _p(D, ctypes.c_uint16), L, d, E, d_e,
                              _p(ids, ctypes.c_int32), n, _p(out, ctypes.c_double))
    return out


@dataclass
class LayerResult:
    a0: np.ndarray | None      # float64 [L][E] pre-ReLU router logits (router path only)
    scores: np.ndarray         # float64 [L][E]
    tok_mask: np.ndarray       # uint32 [L][W]
    union_mask: np.ndarray     # uint32 [W]
    union_ids: np.ndarray      # int32 [E], ascending, tail -1
    n_union: int
    out: np.ndarray            # float64 [L][d]


def layer_forward_scores(x, scores_f32, U, D, union_only=False, stats=None) -> LayerResult:
    """Scores-in layer: masks -> Union(x) -> counters -> Eq. 1/2."""
    x, U, D = _u16(x), _u16(U), _u16(D)
    sf = _f32(scores_f32)
    L, d = x.shape
    E, d_e, _ = U.shape
    assert sf.shape == (L, E)
    W = mask_words(E)
    s = np.empty((L, E), np.float64)
    tm = np.empty((L, W), np.uint32)
    um = np.empty(W, np.uint32)
    ids = np.empty(E, np.int32)
    n = ctypes.c_int32(0)
    out = np.empty((L, d), np.float64)
    _load().oracle_layer_forward_scores(
        _p(x, ctypes.c_uint16), _p(sf, ctypes.c_float), _p(U, ctypes.c_uint16),
        _p(D, ctypes.c_uint16), L, d, E, d_e, int(bool(union_only)), _p(s, ctypes.c_double),
        _p(tm, ctypes.c_uint32), _p(um, ctypes.c_uint32), _p(ids, ctypes.c_int32),
        ctypes.byref(n), _p(stats, ctypes.c_uint64), _p(out, ctypes.c_double))
    return LayerResult(None, s, tm, um, ids, int(n.value), out)


def layer_forward(x, W_r, gain, U, D, bias=None, eps=1e-6, union_only=False,
                  stats=None, rmsnorm=True) -> LayerResult:
    """Full layer: Eq. 3 router -> Union(x) -> Eq. 1/2. rmsnorm=False takes the router of the
    Sec. 4.2.3 ablation instead (gain and eps unused), step by step through the same routines."""
    if not rmsnorm:
        a0, s = router_relu_only(x, W_r, bias)
        tm = token_masks(s)
        um, ids, n = chunk_union(tm, W_r.shape[0], stats)
        out = expert_ffn(x, s, U, D, expert_ids=ids[:n] if union_only else None)
        return LayerResult(a0, s, tm, um, ids, n, out)
    x, W_r, U, D = _u16(x), _u16(W_r), _u16(U), _u16(D)
    gain, bias = _f32(gain), _f32(bias)
    L, d = x.shape
    E, d_e, _ = U.shape
    W = mask_words(E)
    a0 = np.empty((L, E), np.float64)
    s = np.empty((L, E), np.float64)
    tm = np.empty((L, W), np.uint32)
    um = np.empty(W, np.uint32)
    ids = np.empty(E, np.int32)
    n = ctypes.c_int32(0)
    out = np.empty((L, d), np.float64)
    _load().oracle_layer_forward(
        _p(x, ctypes.c_uint16), _p(W_r, ctypes.c_uint16), _p(gain, ctypes.c_float),
        _p(bias, ctypes.c_float), _p(U, ctypes.c_uint16), _p(D, ctypes.c_uint16), L, d, E, d_e,
        ctypes.c_double(eps), int(bool(union_only)), _p(a0, ctypes.c_double),
        _p(s, ctypes.c_double), _p(tm, ctypes.c_uint32), _p(um, ctypes.c_uint32),
        _p(ids, ctypes.c_int32), ctypes.byref(n), _p(stats, ctypes.c_uint64),
        _p(out, ctypes.c_double))
    return LayerResult(a0, s, tm, um, ids, int(n.value), out)


def residual_step(res, out):
    """Stacked decode: res += out (in place, float64); returns bf16 bits of f32(res)."""
    assert res.dtype == np.float64 and res.flags.c_contiguous
    out = np.ascontiguousarray(out, dtype=np.float64)
    nxt = np.empty(res.shape, np.uint16)
    _load().oracle_residual_step(_p(res, ctypes.c_double), _p(out, ctypes.c_double),
                                 int(res.size), _p(nxt, ctypes.c_uint16))
    return nxt


def round_to_bf16(a):
    """float32 -> bf16 bits (round to nearest even), the oracle's own rounding."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    o = np.empty(a.shape, np.uint16)
    _load().oracle_round_to_bf16(_p(a, ctypes.c_float), int(a.size), _p(o, ctypes.c_uint16))
    return o
