"""Python binding of the C ABI in ``include/ilre_recall.h`` (argument marshalling only).

Every step of the recall path runs inside ``libilre_recall.so``; this module only turns torch
tensors into pointers and sizes.  There is no CPU fallback: a missing library or a non-sm_100
device raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libilre_recall.so")

STAGE_NAMES = ("prepare", "row_stats", "scores", "select")

EXPORTED_SYMBOLS = (
    "ilre_recall_create", "ilre_recall_run", "ilre_recall_run_host", "ilre_recall_fill_keys",
    "ilre_recall_shard_stats", "ilre_recall_shard_scores", "ilre_recall_allocate",
    "ilre_recall_chunk_attention", "ilre_recall_rerope_keys", "ilre_recall_rerope_sinks",
    "ilre_gather_input_ids",
    "ilre_layer_recall",
    "ilre_recall_copy_row_lse",
    "ilre_recall_status", "ilre_recall_selftest_wait", "ilre_recall_set_profiling", "ilre_recall_stage_times",
    "ilre_recall_sm_clock",
    "ilre_recall_last_launch_count", "ilre_recall_check_guards", "ilre_recall_destroy", "ilre_strerror",
    "ilre_topk_positions_noalloc",
)

NOALLOC_MAX_L = 1048576


class IlreConfig(ctypes.Structure):
    _fields_ = [("n_kv_heads", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("max_L", ctypes.c_int64),
                ("max_q_len", ctypes.c_int32), ("max_budget", ctypes.c_int32),
                ("max_combinations", ctypes.c_int32), ("device", ctypes.c_int32),
                ("host_staging", ctypes.c_int32)]


class IlrePoolSpec(ctypes.Structure):
    _fields_ = [("n_max", ctypes.c_int32), ("max_sizes", ctypes.POINTER(ctypes.c_int32)),
                ("n_win", ctypes.c_int32), ("win_sizes", ctypes.POINTER(ctypes.c_int32)),
                ("win_op", ctypes.c_int32), ("reduce_op", ctypes.c_int32),
                ("n_sink", ctypes.c_int32)]


class IlreError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {code} ({strerror(code)})")
        self.code = code


_lib = None


def load_library() -> ctypes.CDLL:
    """dlopen the in-tree shared library and declare the prototypes.  Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            f"{LIB_PATH} not found: build it with `python -m paper_2508_17892_b200.build`")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    lib.ilre_recall_create.argtypes = [ctypes.POINTER(IlreConfig), ctypes.POINTER(vp)]
    lib.ilre_recall_run.argtypes = [vp, vp, i64, vp, i32, i32, ctypes.POINTER(IlrePoolSpec), vp, vp, vp]
    lib.ilre_recall_run_host.argtypes = lib.ilre_recall_run.argtypes
    lib.ilre_recall_shard_stats.argtypes = [vp, vp, i64, vp, i32, vp, vp]
    lib.ilre_recall_shard_scores.argtypes = [vp, vp, i64, vp, i32, vp, i32, vp, vp]
    lib.ilre_recall_allocate.argtypes = [vp, vp, i64, i32, ctypes.POINTER(IlrePoolSpec), vp, vp]
    lib.ilre_recall_chunk_attention.argtypes = [vp, vp, vp, vp, i32, i32, vp, vp]
    lib.ilre_recall_fill_keys.argtypes = [vp, vp, i64, i32, vp, vp, i64, ctypes.c_double, vp, i64, vp]
    lib.ilre_recall_rerope_keys.argtypes = [vp, vp, vp, i64, i32, i32, ctypes.c_double, vp]
    lib.ilre_recall_rerope_sinks.argtypes = [vp, vp, vp, i32, i32, i32, ctypes.c_double, vp]
    lib.ilre_gather_input_ids.argtypes = [vp, i64, vp, i32, vp, i32, vp, vp]
    lib.ilre_layer_recall.argtypes = [vp, i32, i32, vp, vp, i32, vp, vp, vp, vp]
    lib.ilre_recall_copy_row_lse.argtypes = [vp, vp, i32, vp]
    lib.ilre_recall_status.argtypes = [vp]
    lib.ilre_recall_sm_clock.argtypes = [vp, ctypes.POINTER(ctypes.c_float)]
    lib.ilre_recall_set_profiling.argtypes = [vp, i32]
    lib.ilre_recall_selftest_wait.argtypes = [vp, i64, i32]
    lib.ilre_recall_stage_times.argtypes = [vp, ctypes.POINTER(ctypes.c_float), i32]
    lib.ilre_recall_last_launch_count.argtypes = [vp]
    lib.ilre_recall_check_guards.argtypes = [vp]
    lib.ilre_recall_destroy.argtypes = [vp]
    lib.ilre_strerror.argtypes = [ctypes.c_int]
    lib.ilre_topk_positions_noalloc.argtypes = [vp, i64, i32, vp, vp]
    lib.ilre_strerror.restype = ctypes.c_char_p
    for name in EXPORTED_SYMBOLS:
        if name != "ilre_strerror":
            getattr(lib, name).restype = ctypes.c_int
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load_library().ilre_strerror(code).decode()


def _spec(max_sizes: Sequence[int], win_sizes: Sequence[int], win_op: int, n_sink: int):
    ms = (ctypes.c_int32 * len(max_sizes))(*max_sizes)
    ws = (ctypes.c_int32 * len(win_sizes))(*win_sizes)
    spec = IlrePoolSpec(len(max_sizes), ms, len(win_sizes), ws, win_op, 0, n_sink)
    return spec, (ms, ws)


def gather_input_ids(input_ids: torch.Tensor, idx: torch.Tensor, query_ids: torch.Tensor,
                     stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """Compressed prompt: input_ids at the recalled positions, then the query's ids (int32)."""
    for t in (input_ids, idx, query_ids):
        assert t.is_cuda and t.dtype == torch.int32 and t.is_contiguous() and t.dim() == 1
    out = torch.empty(idx.numel() + query_ids.numel(), dtype=torch.int32, device=input_ids.device)
    st = stream if stream is not None else torch.cuda.current_stream(input_ids.device)
    with torch.cuda.device(input_ids.device):
        rc = load_library().ilre_gather_input_ids(input_ids.data_ptr(), input_ids.numel(),
                                                  idx.data_ptr(), idx.numel(), query_ids.data_ptr(),
                                                  query_ids.numel(), out.data_ptr(), st.cuda_stream)
    if rc != 0:
        raise IlreError(rc, "ilre_gather_input_ids")
    return out


def layer_recall(idx: torch.Tensor, span_begin: torch.Tensor, span_len: torch.Tensor,
                 stream: Optional[torch.cuda.Stream] = None):
    """Offline retrieval-layer choice from the recalled lists of the candidate layers.

    idx: int32 [n_layers, n_idx] (ascending rows); span_begin / span_len: int32 [n_spans], the
    planted key phrases.  Returns (hits int32 [n_layers, n_spans], phrases retrieved completely
    int32 [n_layers], chosen layer int32 [1]) on the device."""
    for t in (idx, span_begin, span_len):
        assert t.is_cuda and t.dtype == torch.int32 and t.is_contiguous()
    assert idx.dim() == 2 and span_begin.dim() == 1 and span_begin.shape == span_len.shape
    n_layers, n_idx = idx.shape
    n_spans = span_begin.numel()
    hits = torch.empty(n_layers, n_spans, dtype=torch.int32, device=idx.device)
    full = torch.empty(n_layers, dtype=torch.int32, device=idx.device)
    layer = torch.empty(1, dtype=torch.int32, device=idx.device)
    st = stream if stream is not None else torch.cuda.current_stream(idx.device)
    with torch.cuda.device(idx.device):
        rc = load_library().ilre_layer_recall(idx.data_ptr(), n_layers, n_idx, span_begin.data_ptr(),
                                              span_len.data_ptr(), n_spans, hits.data_ptr(),
                                              full.data_ptr(), layer.data_ptr(), st.cuda_stream)
    if rc != 0:
        raise IlreError(rc, "ilre_layer_recall")
    return hits, full, layer


def topk_positions_noalloc(scores: torch.Tensor, k: int,
                           out_idx: Optional[torch.Tensor] = None,
                           stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """Ascending positions of the k highest scores (ties: lower position first).

    For callers that may not allocate device memory: the library call behind this function
    needs no handle and allocates nothing (its scratch is a fixed array inside the library,
    shared by all calls -- do not overlap two calls on one GPU).  Pass ``out_idx`` (int32 [k]
    on the same device) to keep this wrapper allocation-free too.  ``len(scores)`` must not
    exceed ``NOALLOC_MAX_L``.
    """
    assert scores.is_cuda and scores.dtype == torch.float32 and scores.is_contiguous()
    if out_idx is None:
        out_idx = torch.empty(k, dtype=torch.int32, device=scores.device)
    st = stream if stream is not None else torch.cuda.current_stream(scores.device)
    with torch.cuda.device(scores.device):
        rc = load_library().ilre_topk_positions_noalloc(scores.data_ptr(), scores.numel(), k,
                                                        out_idx.data_ptr(), st.cuda_stream)
    if rc != 0:
        raise IlreError(rc, "ilre_topk_positions_noalloc")
    return out_idx


class IlreRecall:
    """Owns one ``ilre_recall_t`` handle (device workspace sized at construction)."""

    def __init__(self, max_L: int, max_q_len: int, max_budget: int = 4096,
                 max_combinations: int = 48, n_kv_heads: int = 8, n_q_heads: int = 32,
                 head_dim: int = 128, device: int = 0, host_staging: bool = False):
        self._lib = load_library()
        self.cfg = IlreConfig(n_kv_heads, n_q_heads, head_dim, max_L, max_q_len, max_budget,
                              max_combinations, device, int(host_staging))
        self._h = ctypes.c_void_p()
        rc = self._lib.ilre_recall_create(ctypes.byref(self.cfg), ctypes.byref(self._h))
        if rc != 0:
            self._h = ctypes.c_void_p()
            raise IlreError(rc, "ilre_recall_create")
        self.device = torch.device("cuda", device)

    # -- the recall --------------------------------------------------------------------
    def run(self, K: torch.Tensor, Q: torch.Tensor, budget: int, max_sizes: Sequence[int],
            win_sizes: Sequence[int], win_op: int = 0, n_sink: int = 0,
            out_idx: Optional[torch.Tensor] = None, out_scores: Optional[torch.Tensor] = None,
            want_scores: bool = False, stream: Optional[torch.cuda.Stream] = None):
        """Asynchronous recall on ``stream`` (default: torch's current stream).

        K: bf16 [L, n_kv_heads, 128] on the device; Q: bf16 [q_len, n_q_heads, 128].
        Returns (indices int32 [n_sink + budget], scores fp32 [L] or None).
        """
        assert K.is_cuda and Q.is_cuda and K.dtype == torch.bfloat16 and Q.dtype == torch.bfloat16
        assert K.is_contiguous() and Q.is_contiguous()
        L, q_len = K.shape[0], Q.shape[0]
        assert K.shape[1:] == (self.cfg.n_kv_heads, self.cfg.head_dim)
        assert Q.shape[1:] == (self.cfg.n_q_heads, self.cfg.head_dim)
        if out_idx is None:
            out_idx = torch.empty(n_sink + budget, dtype=torch.int32, device=K.device)
        if out_scores is None and want_scores:
            out_scores = torch.empty(L, dtype=torch.float32, device=K.device)
        spec, _keep = _spec(max_sizes, win_sizes, win_op, n_sink)
        st = stream if stream is not None else torch.cuda.current_stream(K.device)
        rc = self._lib.ilre_recall_run(self._h, K.data_ptr(), L, Q.data_ptr(), q_len, budget,
                                       ctypes.byref(spec), out_idx.data_ptr(),
                                       out_scores.data_ptr() if out_scores is not None else None,
                                       st.cuda_stream)
        if rc != 0:
            raise IlreError(rc, "ilre_recall_run")
        return out_idx, out_scores

    # -- key-range sharded recall: the per-rank steps -----------------------------------
    def _check_kq(self, K: torch.Tensor, Q: torch.Tensor):
        assert K.is_cuda and Q.is_cuda and K.dtype == torch.bfloat16 and Q.dtype == torch.bfloat16
        assert K.is_contiguous() and Q.is_contiguous()
        assert K.shape[1:] == (self.cfg.n_kv_heads, self.cfg.head_dim)
        assert Q.shape[1:] == (self.cfg.n_q_heads, self.cfg.head_dim)

    def shard_stats(self, K_shard: torch.Tensor, Q: torch.Tensor,
                    out: Optional[torch.Tensor] = None,
                    stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        """(max in log2 units, sum of exponentials) of every query row over this shard's keys:
        fp32 [q_len * n_q_heads, 2], to be all-gathered over the shards."""
        self._check_kq(K_shard, Q)
        n_rows = Q.shape[0] * self.cfg.n_q_heads
        if out is None:
            out = torch.empty(n_rows, 2, dtype=torch.float32, device=K_shard.device)
        assert out.is_cuda and out.dtype == torch.float32 and out.is_contiguous()
        assert out.numel() == 2 * n_rows
        st = stream if stream is not None else torch.cuda.current_stream(K_shard.device)
        with torch.cuda.device(K_shard.device):
            rc = self._lib.ilre_recall_shard_stats(self._h, K_shard.data_ptr(), K_shard.shape[0],
                                                   Q.data_ptr(), Q.shape[0], out.data_ptr(),
                                                   st.cuda_stream)
        if rc != 0:
            raise IlreError(rc, "ilre_recall_shard_stats")
        return out

    def shard_scores(self, K_shard: torch.Tensor, Q: torch.Tensor, stats_all: torch.Tensor,
                     out: Optional[torch.Tensor] = None,
                     stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        """A^C of this shard's positions given every shard's statistics
        (fp32 [n_shards, q_len * n_q_heads, 2]); fp32 [L_shard], to be all-gathered in
        position order."""
        self._check_kq(K_shard, Q)
        n_rows = Q.shape[0] * self.cfg.n_q_heads
        assert stats_all.is_cuda and stats_all.dtype == torch.float32 and stats_all.is_contiguous()
        assert stats_all.dim() == 3 and stats_all.shape[1:] == (n_rows, 2)
        if out is None:
            out = torch.empty(K_shard.shape[0], dtype=torch.float32, device=K_shard.device)
        assert out.is_cuda and out.dtype == torch.float32 and out.is_contiguous()
        assert out.numel() == K_shard.shape[0]
        st = stream if stream is not None else torch.cuda.current_stream(K_shard.device)
        with torch.cuda.device(K_shard.device):
            rc = self._lib.ilre_recall_shard_scores(self._h, K_shard.data_ptr(), K_shard.shape[0],
                                                    Q.data_ptr(), Q.shape[0], stats_all.data_ptr(),
                                                    stats_all.shape[0], out.data_ptr(),
                                                    st.cuda_stream)
        if rc != 0:
            raise IlreError(rc, "ilre_recall_shard_scores")
        return out

    def allocate(self, scores: torch.Tensor, budget: int, max_sizes: Sequence[int],
                 win_sizes: Sequence[int], win_op: int = 0, n_sink: int = 0,
                 out_idx: Optional[torch.Tensor] = None,
                 stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        """Algorithm 1 on given scores (fp32 [L], finite, >= 0): ascending int32 indices."""
        assert scores.is_cuda and scores.dtype == torch.float32 and scores.is_contiguous()
        assert scores.dim() == 1
        if out_idx is None:
            out_idx = torch.empty(n_sink + budget, dtype=torch.int32, device=scores.device)
        spec, _keep = _spec(max_sizes, win_sizes, win_op, n_sink)
        st = stream if stream is not None else torch.cuda.current_stream(scores.device)
        with torch.cuda.device(scores.device):
            rc = self._lib.ilre_recall_allocate(self._h, scores.data_ptr(), scores.numel(), budget,
                                                ctypes.byref(spec), out_idx.data_ptr(),
                                                st.cuda_stream)
        if rc != 0:
            raise IlreError(rc, "ilre_recall_allocate")
        return out_idx

    def run_host(self, K: torch.Tensor, Q: torch.Tensor, budget: int, max_sizes: Sequence[int],
                 win_sizes: Sequence[int], win_op: int = 0, n_sink: int = 0,
                 out_idx: Optional[torch.Tensor] = None, out_scores: Optional[torch.Tensor] = None,
                 stream: Optional[torch.cuda.Stream] = None):
        """Recall from HOST tensors (pinned for speed); synchronises before returning."""
        assert not K.is_cuda and not Q.is_cuda
        assert K.dtype == torch.bfloat16 and Q.dtype == torch.bfloat16
        assert K.is_contiguous() and Q.is_contiguous()
        L, q_len = K.shape[0], Q.shape[0]
        if out_idx is None:
            out_idx = torch.empty(n_sink + budget, dtype=torch.int32)
        spec, _keep = _spec(max_sizes, win_sizes, win_op, n_sink)
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        rc = self._lib.ilre_recall_run_host(self._h, K.data_ptr(), L, Q.data_ptr(), q_len, budget,
                                            ctypes.byref(spec), out_idx.data_ptr(),
                                            out_scores.data_ptr() if out_scores is not None else None,
                                            st.cuda_stream)
        if rc != 0:
            raise IlreError(rc, "ilre_recall_run_host")
        return out_idx, out_scores

    def chunk_attention(self, Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, n_prefix: int,
                        out: Optional[torch.Tensor] = None,
                        stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        """Attention of one prefill chunk over n_prefix cached rows plus, causally, its own.
        Writes into ``out`` (bf16, Q's shape) when given."""
        for t in (Q, K, V):
            assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous() and t.dim() == 3
        c = Q.shape[0]
        assert Q.shape[1:] == (self.cfg.n_q_heads, self.cfg.head_dim)
        assert K.shape == (n_prefix + c, self.cfg.n_kv_heads, self.cfg.head_dim) and V.shape == K.shape
        if out is None:
            out = torch.empty_like(Q)
        assert out.is_cuda and out.dtype == torch.bfloat16 and out.is_contiguous() and out.shape == Q.shape
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        rc = self._lib.ilre_recall_chunk_attention(self._h, Q.data_ptr(), K.data_ptr(), V.data_ptr(),
                                                   c, n_prefix, out.data_ptr(), st.cuda_stream)
        if rc != 0:
            raise IlreError(rc, "ilre_recall_chunk_attention")
        return out

    def fill_keys(self, X: torch.Tensor, W_k: torch.Tensor, K_cache: torch.Tensor, pos0: int,
                  bias: Optional[torch.Tensor] = None, rope_theta: float = 500000.0,
                  stream: Optional[torch.cuda.Stream] = None) -> None:
        """Key projection + RoPE of the tokens X (positions pos0 ..) written into K_cache."""
        for t in (X, W_k, K_cache) + ((bias,) if bias is not None else ()):
            assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()
        assert X.dim() == 2 and W_k.shape == (self.cfg.n_kv_heads * self.cfg.head_dim, X.shape[1])
        assert K_cache.shape[1:] == (self.cfg.n_kv_heads, self.cfg.head_dim)
        assert bias is None or bias.shape == (W_k.shape[0],)
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        rc = self._lib.ilre_recall_fill_keys(
            self._h, X.data_ptr(), X.shape[0], X.shape[1], W_k.data_ptr(),
            bias.data_ptr() if bias is not None else None, pos0, float(rope_theta),
            K_cache.data_ptr(), K_cache.shape[0], st.cuda_stream)
        if rc != 0:
            raise IlreError(rc, "ilre_recall_fill_keys")

    def rerope_keys(self, K: torch.Tensor, chunk_size: int, n_sink: int = 0,
                    rope_theta: float = 500000.0, out: Optional[torch.Tensor] = None,
                    stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        """Eq. 7 (Dual Chunk Attention): re-rotate the cached keys chunk by chunk.  In place
        unless ``out`` is given.  Returns the tensor that holds the result."""
        dst = K if out is None else out
        for t in (K, dst):
            assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()
            assert t.shape[1:] == (self.cfg.n_kv_heads, self.cfg.head_dim)
        assert dst.shape == K.shape
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        rc = self._lib.ilre_recall_rerope_keys(self._h, K.data_ptr(), dst.data_ptr(), K.shape[0],
                                               chunk_size, n_sink, float(rope_theta),
                                               st.cuda_stream)
        if rc != 0:
            raise IlreError(rc, "ilre_recall_rerope_keys")
        return dst

    def rerope_sinks(self, K_sink: torch.Tensor, chunk_size: int, chunk_index: int,
                     rope_theta: float = 500000.0, out: Optional[torch.Tensor] = None,
                     stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        """Eq. 6: the cached sink keys [n_sink, n_kv_heads, 128] as the prefill of chunk
        ``chunk_index`` (1-based) sees them.  Pass the cached keys every time, not an earlier
        result.  Returns a new tensor unless ``out`` is given (``out`` may be ``K_sink``)."""
        dst = torch.empty_like(K_sink) if out is None else out
        for t in (K_sink, dst):
            assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()
            assert t.shape[1:] == (self.cfg.n_kv_heads, self.cfg.head_dim)
        assert dst.shape == K_sink.shape
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        rc = self._lib.ilre_recall_rerope_sinks(self._h, K_sink.data_ptr(), dst.data_ptr(),
                                                K_sink.shape[0], chunk_size, chunk_index,
                                                float(rope_theta), st.cuda_stream)
        if rc != 0:
            raise IlreError(rc, "ilre_recall_rerope_sinks")
        return dst

    # -- diagnostics -------------------------------------------------------------------
    def row_lse(self, q_len: int, stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        out = torch.empty(q_len, self.cfg.n_q_heads, dtype=torch.float32, device=self.device)
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        rc = self._lib.ilre_recall_copy_row_lse(self._h, out.data_ptr(), q_len, st.cuda_stream)
        if rc != 0:
            raise IlreError(rc, "ilre_recall_copy_row_lse")
        return out

    def status(self) -> int:
        return self._lib.ilre_recall_status(self._h)

    def check_status(self) -> None:
        rc = self.status()
        if rc != 0:
            raise IlreError(rc, "ilre_recall_status")

    def selftest_wait(self, wait_cycle_limit: int = 0, what: int = 0) -> None:
        """Failure-detection self test: spin budget (SM cycles, 0 = default) of the kernels'
        bounded waits for the following runs, and which wait is made impossible to complete
        (0 none, 1 the Algorithm 1 kernel's grid barrier, 2 a key tile that never arrives)."""
        rc = self._lib.ilre_recall_selftest_wait(self._h, int(wait_cycle_limit), int(what))
        if rc != 0:
            raise IlreError(rc, "ilre_recall_selftest_wait")

    def set_profiling(self, on: bool) -> None:
        self._lib.ilre_recall_set_profiling(self._h, int(on))

    def stage_times(self) -> dict:
        buf = (ctypes.c_float * len(STAGE_NAMES))()
        n = self._lib.ilre_recall_stage_times(self._h, buf, len(STAGE_NAMES))
        if n < 0:
            raise IlreError(n, "ilre_recall_stage_times")
        return {STAGE_NAMES[i]: float(buf[i]) for i in range(n)}

    def sm_clock_mhz(self) -> float:
        """SM clock the row-statistics kernel of the last profiled run really ran at (0 = none)."""
        mhz = ctypes.c_float(0.0)
        rc = self._lib.ilre_recall_sm_clock(self._h, ctypes.byref(mhz))
        if rc != 0:
            raise IlreError(rc, "ilre_recall_sm_clock")
        return float(mhz.value)

    def check_guards(self) -> int:
        """Number of workspace buffers whose guard zone was written to (0 = none); synchronises."""
        rc = self._lib.ilre_recall_check_guards(self._h)
        if rc < 0:
            raise IlreError(rc, "ilre_recall_check_guards")
        return rc

    def last_launch_count(self) -> int:
        return self._lib.ilre_recall_last_launch_count(self._h)

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h.value:
            self._lib.ilre_recall_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
