"""ctypes front end of the CPU oracle (``ilre_oracle.c``).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the bench's CPU-baseline leg may import this package.
It builds the C file with gcc on first use and never touches the CUDA library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ilre_oracle.c")
_LIB = os.path.join(_HERE, "_build", "libilre_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (gcc, -O2, OpenMP).  Returns the path of the shared object."""
    os.makedirs(os.path.dirname(_LIB), exist_ok=True)
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        c_i32p = ctypes.POINTER(ctypes.c_int32)
        c_i64p = ctypes.POINTER(ctypes.c_int64)
        c_u16p = ctypes.POINTER(ctypes.c_uint16)
        c_f64p = ctypes.POINTER(ctypes.c_double)
        lib.ilre_oracle_row_stats.argtypes = [c_u16p, ctypes.c_int64, ctypes.c_int, c_u16p,
                                              ctypes.c_int, ctypes.c_int, ctypes.c_int, c_i32p,
                                              ctypes.c_int, c_f64p, c_f64p]
        lib.ilre_oracle_scores_at.argtypes = [c_u16p, ctypes.c_int64, ctypes.c_int, c_u16p,
                                              ctypes.c_int, ctypes.c_int, ctypes.c_int, c_f64p,
                                              c_f64p, c_i64p, ctypes.c_int64, c_f64p]
        lib.ilre_oracle_scores.argtypes = [c_u16p, ctypes.c_int64, ctypes.c_int, c_u16p,
                                           ctypes.c_int, ctypes.c_int, ctypes.c_int, c_f64p,
                                           c_f64p, c_f64p]
        lib.ilre_oracle_maxpool.argtypes = [c_f64p, ctypes.c_int64, ctypes.c_int, c_f64p]
        lib.ilre_oracle_maxpool.restype = ctypes.c_int64
        lib.ilre_oracle_winpool.argtypes = [c_f64p, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                            c_f64p]
        lib.ilre_oracle_winpool.restype = None
        lib.ilre_oracle_avg_precision.argtypes = [ctypes.c_int]
        lib.ilre_oracle_avg_precision.restype = None
        lib.ilre_oracle_allocate.argtypes = [c_f64p, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                             c_i32p, ctypes.c_int, c_i32p, ctypes.c_int,
                                             ctypes.c_int, c_i32p, c_i32p, c_i32p, c_f64p, c_f64p,
                                             c_i32p]
        lib.ilre_oracle_dca_rerope.argtypes = [c_u16p, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                               ctypes.c_int, ctypes.c_int, ctypes.c_double, c_f64p]
        _lib = lib
    return _lib


def _u16(x) -> np.ndarray:
    """bf16 torch tensor (CPU) or uint16 array -> contiguous uint16 numpy array."""
    if isinstance(x, np.ndarray):
        assert x.dtype == np.uint16
        return np.ascontiguousarray(x)
    import torch
    assert x.dtype == torch.bfloat16 and x.device.type == "cpu"
    return x.contiguous().view(torch.int16).numpy().view(np.uint16)


def _p(a: np.ndarray, ty):
    return a.ctypes.data_as(ctypes.POINTER(ty))


def row_stats(K, Q, rows: Sequence[int]):
    """(row_max, row_sum) of Eq. 4's softmax for rows given as i * n_q_heads + h."""
    k, q = _u16(K), _u16(Q)
    L, n_kv, d = k.shape
    q_len, n_q, _ = q.shape
    r = np.ascontiguousarray(np.asarray(rows, dtype=np.int32))
    m = np.empty(len(r), dtype=np.float64)
    z = np.empty(len(r), dtype=np.float64)
    rc = _load().ilre_oracle_row_stats(_p(k, ctypes.c_uint16), L, n_kv, _p(q, ctypes.c_uint16),
                                       q_len, n_q, d, _p(r, ctypes.c_int32), len(r),
                                       _p(m, ctypes.c_double), _p(z, ctypes.c_double))
    if rc != 0:
        raise RuntimeError(f"ilre_oracle_row_stats failed: {rc}")
    return m, z


def scores_at(K, Q, row_max: np.ndarray, row_sum: np.ndarray, positions: Sequence[int]):
    """Eq. 5 at chosen positions, given the statistics of all q_len * n_q_heads rows."""
    k, q = _u16(K), _u16(Q)
    L, n_kv, d = k.shape
    q_len, n_q, _ = q.shape
    pos = np.ascontiguousarray(np.asarray(positions, dtype=np.int64))
    m = np.ascontiguousarray(row_max, dtype=np.float64)
    z = np.ascontiguousarray(row_sum, dtype=np.float64)
    assert m.size == q_len * n_q and z.size == q_len * n_q
    a = np.empty(len(pos), dtype=np.float64)
    rc = _load().ilre_oracle_scores_at(_p(k, ctypes.c_uint16), L, n_kv, _p(q, ctypes.c_uint16),
                                       q_len, n_q, d, _p(m, ctypes.c_double),
                                       _p(z, ctypes.c_double), _p(pos, ctypes.c_int64), len(pos),
                                       _p(a, ctypes.c_double))
    if rc != 0:
        raise RuntimeError(f"ilre_oracle_scores_at failed: {rc}")
    return a


def scores(K, Q, with_stats: bool = False):
    """A^C [L] of Eq. 4 + Eq. 5 (fp64); optionally also (row_max, row_sum)."""
    k, q = _u16(K), _u16(Q)
    L, n_kv, d = k.shape
    q_len, n_q, _ = q.shape
    a = np.empty(L, dtype=np.float64)
    m = np.empty(q_len * n_q, dtype=np.float64)
    z = np.empty(q_len * n_q, dtype=np.float64)
    rc = _load().ilre_oracle_scores(_p(k, ctypes.c_uint16), L, n_kv, _p(q, ctypes.c_uint16),
                                    q_len, n_q, d, _p(a, ctypes.c_double),
                                    _p(m, ctypes.c_double), _p(z, ctypes.c_double))
    if rc != 0:
        raise RuntimeError(f"ilre_oracle_scores failed: {rc}")
    return (a, m, z) if with_stats else a


def maxpool(a: np.ndarray, m: int) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float64)
    out = np.empty((len(a) + m - 1) // m, dtype=np.float64)
    n = _load().ilre_oracle_maxpool(_p(a, ctypes.c_double), len(a), m, _p(out, ctypes.c_double))
    assert n == len(out)
    return out


def winpool(p: np.ndarray, n: int, op: int, avg_single: bool = False) -> np.ndarray:
    """Stride-1 window pooling.  ``avg_single``: add and divide the averaging window in single
    precision, left to right (see ``allocate``)."""
    p = np.ascontiguousarray(p, dtype=np.float64)
    out = np.empty(len(p), dtype=np.float64)
    lib = _load()
    lib.ilre_oracle_avg_precision(int(avg_single))
    try:
        lib.ilre_oracle_winpool(_p(p, ctypes.c_double), len(p), n, op, _p(out, ctypes.c_double))
    finally:
        lib.ilre_oracle_avg_precision(0)
    return out


def allocate(A: np.ndarray, budget: int, max_sizes: Sequence[int], win_sizes: Sequence[int],
             win_op: int, n_sink: int = 0, diagnostics: bool = False, avg_single: bool = False):
    """Algorithm 1 on a score array: ascending positions [n_sink + budget] (int32).

    ``avg_single``: the averaging window is added left to right and divided in single precision
    instead of double.  Which cells rank first is an integer decision taken from those sums; to
    check such a decision of an implementation that averages in single precision (on scores
    that are exact floats), both sides have to round alike.  ``diagnostics`` adds per
    combination the quota, the tokens taken, the pooled value of the last contributing and of
    the K_m-th cell, and per position the combination that allocated it (-1 = none)."""
    a = np.ascontiguousarray(A, dtype=np.float64)
    ms = np.ascontiguousarray(np.asarray(max_sizes, dtype=np.int32))
    ws = np.ascontiguousarray(np.asarray(win_sizes, dtype=np.int32))
    nc = len(ms) * len(ws)
    out = np.empty(max(n_sink + budget, 1), dtype=np.int32)
    quota = np.zeros(nc, dtype=np.int32)
    taken = np.zeros(nc, dtype=np.int32)
    last_v = np.zeros(nc, dtype=np.float64)
    kth_v = np.zeros(nc, dtype=np.float64)
    comb_of = np.empty(len(a), dtype=np.int32) if diagnostics else None
    lib = _load()
    lib.ilre_oracle_avg_precision(int(avg_single))
    try:
        rc = lib.ilre_oracle_allocate(_p(a, ctypes.c_double), len(a), n_sink, budget,
                                      _p(ms, ctypes.c_int32), len(ms), _p(ws, ctypes.c_int32),
                                      len(ws), win_op, _p(out, ctypes.c_int32),
                                      _p(quota, ctypes.c_int32), _p(taken, ctypes.c_int32),
                                      _p(last_v, ctypes.c_double), _p(kth_v, ctypes.c_double),
                                      _p(comb_of, ctypes.c_int32) if diagnostics else None)
    finally:
        lib.ilre_oracle_avg_precision(0)
    if rc != 0:
        raise RuntimeError(f"ilre_oracle_allocate failed: {rc}")
    out = out[: n_sink + budget]
    if diagnostics:
        return out, dict(quota=quota, taken=taken, last_value=last_v, kth_value=kth_v,
                         combination_of=comb_of)
    return out


def recall(K, Q, budget: int, max_sizes: Sequence[int], win_sizes: Sequence[int], win_op: int,
           n_sink: int = 0):
    """The whole path: (ascending indices, A^C)."""
    a = scores(K, Q)
    return allocate(a, budget, max_sizes, win_sizes, win_op, n_sink), a


def dca_rerope(K, chunk: int, n_sink: int = 0, theta: float = 500000.0) -> np.ndarray:
    """Eq. 7: the cached keys re-rotated chunk by chunk (fp64, not rounded)."""
    k = _u16(K)
    L, n_kv, d = k.shape
    out = np.empty((L, n_kv, d), dtype=np.float64)
    rc = _load().ilre_oracle_dca_rerope(_p(k, ctypes.c_uint16), L, n_kv, d, chunk, n_sink,
                                        float(theta), _p(out, ctypes.c_double))
    if rc != 0:
        raise RuntimeError(f"ilre_oracle_dca_rerope failed: {rc}")
    return out


def dca_rerope_sinks(K_sink, chunk_index: int, chunk: int, theta: float = 500000.0) -> np.ndarray:
    """Eq. 6: the sink keys of a layer before the retrieval layer as the i-th chunk sees them,
    K^{S,i} = R^{i-2}(D_C) K^S for i > 2 (1-based chunk index; the first two chunks see the
    sinks as cached).  Written as the equation states it: the rotation by the chunk size D_C
    applied i - 2 times to the cached sink keys, fp64, not rounded.  R(D) turns the channel
    pair (c, c + d/2) by the angle D * theta^(-2c/d) (rotate-half layout, as in Eq. 7).

    K_sink: bf16 [n_sink, n_kv, d].  Returns fp64 [n_sink, n_kv, d]."""
    import torch
    k = K_sink.to(torch.float64).numpy().copy()
    d = k.shape[-1]
    half = d // 2
    c = np.arange(half, dtype=np.float64)
    ang = float(chunk) * theta ** (-2.0 * c / d)
    cs, sn = np.cos(ang), np.sin(ang)
    for _ in range(max(0, int(chunk_index) - 2)):
        lo, hi = k[..., :half].copy(), k[..., half:].copy()
        k[..., :half] = lo * cs - hi * sn
        k[..., half:] = lo * sn + hi * cs
    return k


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp64 values to the nearest bf16 (ties to even); returns the uint16 patterns."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float64)).to(torch.bfloat16)
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def key_fill(X, W, pos0: int, theta: float = 500000.0, bias=None) -> np.ndarray:
    """Eq. 1 + Eq. 3 for the keys of the retrieval layer: K = PE(X W_K^T (+ b)), fp64.

    X: bf16 [n_tok, d_model] hidden states of the tokens at positions pos0 .. pos0 + n_tok - 1;
    W: bf16 [n_kv * d_h, d_model] (one row per output channel); bias: optional bf16
    [n_kv * d_h].  PE is RoPE in the rotate-half layout of the cache (pair (c, c + d_h/2) of
    every head turns by pos * theta^(-2c/d_h)), d_h = 128.  Returns fp64 [n_tok, n_kv, 128],
    not rounded.  The matrix product is numpy's fp64 matmul (a library step)."""
    import torch
    x = X.to(torch.float64).numpy() if hasattr(X, "numpy") else np.asarray(X, dtype=np.float64)
    w = W.to(torch.float64).numpy() if hasattr(W, "numpy") else np.asarray(W, dtype=np.float64)
    d_h = 128
    n_tok, n_out = x.shape[0], w.shape[0]
    assert n_out % d_h == 0 and x.shape[1] == w.shape[1]
    y = x @ w.T
    if bias is not None:
        b = bias.to(torch.float64).numpy() if hasattr(bias, "numpy") else np.asarray(bias)
        y = y + b[None, :]
    y = y.reshape(n_tok, n_out // d_h, d_h)
    half = d_h // 2
    inv_freq = np.power(float(theta), -2.0 * np.arange(half, dtype=np.float64) / d_h)
    ang = (pos0 + np.arange(n_tok, dtype=np.float64))[:, None] * inv_freq[None, :]
    cs, sn = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    out = np.empty_like(y)
    out[..., :half] = y[..., :half] * cs - y[..., half:] * sn
    out[..., half:] = y[..., :half] * sn + y[..., half:] * cs
    return out


def chunk_attention(Q, K, V, n_prefix: int) -> np.ndarray:
    """Streaming chunked prefill attention of one chunk (Eq. 2 with the Lambda-shaped mask), fp64.

    Q: bf16 [c, n_q, d] queries of the chunk's tokens; K, V: bf16 [n_prefix + c, n_kv, d], the
    cached sink and sliding-window keys/values (the first n_prefix rows, visible to every query)
    followed by the chunk's own, which are visible causally: query j sees rows
    0 .. n_prefix + j.  Query head h reads kv head h // (n_q // n_kv).  Returns the attention
    output fp64 [c, n_q, d].  Written as plain loops over heads with a library softmax-free
    definition: exp, sum, divide."""
    import torch
    q = Q.to(torch.float64).numpy()
    k = K.to(torch.float64).numpy()
    v = V.to(torch.float64).numpy()
    c, n_q, d = q.shape
    n_kv = k.shape[1]
    group = n_q // n_kv
    assert k.shape[0] == n_prefix + c and v.shape == k.shape
    out = np.empty((c, n_q, d), dtype=np.float64)
    for h in range(n_q):
        g = h // group
        s = (q[:, h, :] @ k[:, g, :].T) / np.sqrt(d)                     # [c, n_prefix + c]
        for j in range(c):
            row = s[j, : n_prefix + j + 1]
            p = np.exp(row - row.max())
            p /= p.sum()
            out[j, h, :] = p @ v[: n_prefix + j + 1, g, :]
    return out


def span_hits(idx: Sequence[int], spans: Sequence[Sequence[int]]) -> np.ndarray:
    """How many positions of every planted key phrase (begin, length) the recalled index list
    contains (retrieval task of Appendix A.1).  Plain set membership, position by position."""
    have = set(int(i) for i in idx)
    return np.array([sum(1 for p in range(int(b), int(b) + int(n)) if p in have)
                     for b, n in spans], dtype=np.int64)


def layer_choice(idx_per_layer: Sequence[Sequence[int]], spans: Sequence[Sequence[int]]):
    """Offline choice of the retrieval layer (Section 3.3, first paragraph; Appendix A.1).

    A phrase counts as retrieved only if every one of its positions was recalled (exact match);
    a layer's recall rate is the fraction of phrases retrieved; l_R is the layer with the
    smallest index among those with the highest recall rate.  Returns
    (hits [n_layers, n_spans], retrieved phrases per layer [n_layers], l_R)."""
    lens = np.array([int(n) for _, n in spans], dtype=np.int64)
    hits = np.stack([span_hits(idx, spans) for idx in idx_per_layer]) if len(spans) else \
        np.zeros((len(idx_per_layer), 0), dtype=np.int64)
    full = (hits == lens[None, :]).sum(axis=1)
    rates = [f / max(len(spans), 1) for f in full]
    best = max(rates)
    l_r = next(l for l, r in enumerate(rates) if r == best)
    return hits, full, l_r
